"""The C-ABI boundary without a GPU: the library loads, exports what the header declares,
rejects bad arguments on the host before any CUDA call, and agrees with the oracle's
independent statement of the pool layout."""
import ctypes
import os
import re

import pytest

import oracle
from paper_2609_14237_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    B.build()


def declared_functions():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(inc, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(opw_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol():
    L = B.lib()
    names = declared_functions()
    assert set(B.EXPORTS) <= set(names) and len(names) >= 11
    for n in names:
        assert hasattr(L, n), n


def test_status_strings():
    assert B.status_string(B.OPW_OK) == "ok"
    for s in range(1, 7):
        assert B.status_string(s) not in ("", "ok", "unknown status")
    assert B.status_string(99) == "unknown status"


def test_pool_index_agrees_with_the_oracles_own_formula():
    for Hkv, D in [(2, 64), (8, 128), (2, 256)]:
        for p in (0, 3):
            for g in range(Hkv):
                for kv in range(2):
                    for t in range(16):
                        for d in range(D):
                            assert B.opw_kv_pool_index(Hkv, 16, D, p, g, kv, t, d) == oracle.pool_index(Hkv, 16, D, p, g, kv, t, d)
    assert B.opw_kv_pool_bytes(8, 16, 128, 10) == 10 * 8 * 2 * 16 * 128 * 2
    assert B.opw_kv_pool_bytes(0, 16, 128, 10) == 0


def good_cfg(**over):
    kw = dict(device=0, num_q_heads=8, num_kv_heads=2, head_dim=64, max_batch=4, max_pages_per_seq=17,
              layer_window=[0], layer_num_pages=[40], layer_kv_pool=[0x10000], workspace=0x100000,
              workspace_bytes=1 << 30)
    kw.update(over)
    return B.make_config(**kw)


def create_rc(cfg):
    h = ctypes.c_void_p()
    rc = B.lib().opw_attn_stage_create(ctypes.byref(cfg), ctypes.byref(h))
    assert rc != B.OPW_OK and h.value is None
    return rc


def test_workspace_bytes_needs_a_valid_shape():
    cfg, keep = good_cfg()
    n = B.opw_attn_stage_workspace_bytes(cfg)
    assert n > 0 and n % 256 == 0
    big, keep2 = good_cfg(max_batch=64)
    assert B.opw_attn_stage_workspace_bytes(big) > n
    bad, keep3 = good_cfg(num_q_heads=7)
    assert B.opw_attn_stage_workspace_bytes(bad) == 0
    assert B.lib().opw_attn_stage_workspace_bytes(None) == 0


@pytest.mark.parametrize("over,want", [
    (dict(num_q_heads=7), B.OPW_ERR_INVALID_ARG),
    (dict(head_dim=96), B.OPW_ERR_UNSUPPORTED),
    (dict(page_size=32), B.OPW_ERR_UNSUPPORTED),
    (dict(head_dim=256, num_q_heads=32, num_kv_heads=2), B.OPW_ERR_UNSUPPORTED),
    (dict(head_dim=256, tune_warps=8), B.OPW_ERR_CAPACITY),
    (dict(num_q_heads=34, num_kv_heads=2), B.OPW_ERR_UNSUPPORTED),
    (dict(workspace=0), B.OPW_ERR_INVALID_ARG),
    (dict(workspace=0x100010), B.OPW_ERR_INVALID_ARG),
    (dict(layer_kv_pool=[0x10010]), B.OPW_ERR_INVALID_ARG),
    (dict(layer_num_pages=[0]), B.OPW_ERR_INVALID_ARG),
    (dict(layer_window=[-1]), B.OPW_ERR_INVALID_ARG),
    (dict(tune_warps=17), B.OPW_ERR_INVALID_ARG),
    (dict(tune_stages=1), B.OPW_ERR_INVALID_ARG),
    (dict(softmax_scale=-1.0), B.OPW_ERR_INVALID_ARG),
    (dict(head_dim=128, tune_warps=8, tune_stages=4), B.OPW_ERR_CAPACITY),
    (dict(max_batch=0), B.OPW_ERR_INVALID_ARG),
    (dict(flags=4), B.OPW_ERR_INVALID_ARG),                      # only OPW_FLAG_NO_PDL and OPW_FLAG_COPY_STREAMS are defined
])
def test_create_rejects_bad_configs_before_touching_cuda(over, want):
    cfg, keep = good_cfg(**over)
    assert create_rc(cfg) == want


def test_create_checks_struct_size_and_null():
    cfg, keep = good_cfg()
    cfg.struct_size = 8
    assert create_rc(cfg) == B.OPW_ERR_INVALID_ARG
    assert B.lib().opw_attn_stage_create(None, None) == B.OPW_ERR_INVALID_ARG
    cfg2, keep2 = good_cfg()
    cfg2.reserved = 1
    assert create_rc(cfg2) == B.OPW_ERR_INVALID_ARG


def test_step_calls_reject_a_null_handle_and_destroy_accepts_it():
    L = B.lib()
    assert L.opw_kv_append(None, 0, 1, 16, 16, 16, 16, None) == B.OPW_ERR_INVALID_ARG
    assert L.opw_decode_attention(None, 0, 1, 16, 16, 16, 16, None, None) == B.OPW_ERR_INVALID_ARG
    assert L.opw_decode_step_host(None, 0, 1, 16, 16, 16, 16, None, 16, None, None) == B.OPW_ERR_INVALID_ARG
    assert L.opw_attn_stage_poll_error(None, None) == B.OPW_ERR_INVALID_ARG
    assert L.opw_attn_stage_page_table_delta_host(None, 0, 16, 1, None) == B.OPW_ERR_INVALID_ARG
    assert L.opw_attn_stage_launch_count(None) == 0
    assert L.opw_attn_stage_destroy(None) == B.OPW_OK


def test_plan_calls_reject_null_arguments():
    L = B.lib()
    h = ctypes.c_void_p()
    assert L.opw_attn_plan_create(None, None, 1, 0, ctypes.byref(h)) == B.OPW_ERR_INVALID_ARG and h.value is None
    assert L.opw_attn_plan_submit(None, None) == B.OPW_ERR_INVALID_ARG
    assert L.opw_attn_plan_destroy(None) == B.OPW_OK
    assert ctypes.sizeof(B.StepItem) == 72


def test_without_a_device_create_fails_loudly_instead_of_falling_back():
    import torch

    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    cfg, keep = good_cfg()
    assert create_rc(cfg) == B.OPW_ERR_CUDA
    with pytest.raises(RuntimeError):
        B.Stage(pools=[torch.zeros(2 * 2 * 16 * 64 * 4, dtype=torch.bfloat16)], layer_window=[0], num_q_heads=8,
                num_kv_heads=2, head_dim=64, max_batch=4, max_pages_per_seq=4)


def test_attention_module_workspace_and_null_arguments_need_no_device():
    """Host-only parts of the attention-module ABI: the workspace formula and the argument checks
    that come before any CUDA call."""
    base = B.opw_afd_module_workspace_bytes(32, 8, 128, 64, 4096)
    # qkv + q + k + v + attention output buffers, split-K partial tiles, 32 MiB for the library GEMM
    acts = 64 * (48 + 32 + 8 + 8 + 32) * 128 * 2
    assert base >= acts + (32 << 20) and base % 256 == 0
    assert B.opw_afd_module_workspace_bytes(32, 8, 128, 128, 4096) > base          # grows with the batch
    # from 2048 to 4096 rows: the activation buffers, eight more batch tiles of unsplit partial sums for the wider
    # projection (48 weight tiles x 256 columns x 128 rows of fp32), the angle table, two counters per (weight, batch) tile
    grow = B.opw_afd_module_workspace_bytes(32, 8, 128, 4096, 4096) - B.opw_afd_module_workspace_bytes(32, 8, 128, 2048, 4096)
    assert grow == 2048 * (48 + 32 + 8 + 8 + 32) * 128 * 2 + 8 * 48 * 256 * 128 * 4 + 2048 * 64 * 8 + 8 * 48 * 2 * 4
    for bad in ((32, 7, 128, 64, 4096), (32, 8, 96, 64, 4096), (32, 8, 128, 0, 4096), (32, 8, 128, 64, 4100), (0, 8, 128, 64, 4096)):
        assert B.opw_afd_module_workspace_bytes(*bad) == 0
    L = B.lib()
    h = ctypes.c_void_p()
    assert L.opw_afd_module_create(None, 0, 4096, 16, 16, 1e4, 0, 256, 1 << 30, ctypes.byref(h)) == B.OPW_ERR_INVALID_ARG
    assert L.opw_afd_module_step(None, 1, 16, 16, 16, 16, None) == B.OPW_ERR_INVALID_ARG
    assert L.opw_afd_module_poll_error(None, None) == B.OPW_ERR_INVALID_ARG
    assert L.opw_afd_module_set_trace(None, None, 0) == B.OPW_ERR_INVALID_ARG
    assert L.opw_afd_module_launch_count(None) == 0
    assert L.opw_afd_module_destroy(None) == B.OPW_OK
    assert L.opw_attn_stage_shape(None, None, None, None, None, None, None) == B.OPW_ERR_INVALID_ARG
    for buf, n in ((0, 1024), (4096, 0), (4096, 1000), (4104, 1024)):             # null, empty, ragged, misaligned
        assert L.opw_hbm_read_probe(buf, n, 4096, None) == B.OPW_ERR_INVALID_ARG

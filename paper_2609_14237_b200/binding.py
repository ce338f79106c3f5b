"""ctypes binding of the C-ABI library (argument marshalling only).

Every function here has the name and the meaning of the entry point it wraps (see
``include/opw_attn.h``).  Tensors are passed as raw device (or host) addresses; torch is
used by callers for memory and streams only.  There is no fallback: if the shared
library is missing, or was built without the kernels, importing ``lib()`` raises.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
LIB_PATH = os.path.join(_HERE, "libopw_attn.so")
SOURCES = [os.path.join(_HERE, "csrc", "opw_attn.cu"), os.path.join(_HERE, "csrc", "opw_noalloc.cu"),
           os.path.join(_HERE, "csrc", "opw_linear_attn.cu"), os.path.join(_HERE, "csrc", "opw_afd.cu")]
HEADERS = [os.path.join(_HERE, "csrc", "opw_kernels.cuh"), os.path.join(_HERE, "csrc", "opw_afd_gemm.cuh"), os.path.join(_ROOT, "include", "opw_attn.h"),
           os.path.join(_ROOT, "include", "opw_linear_attn.h"), os.path.join(_ROOT, "include", "opw_afd.h")]

OPW_FLAG_NO_PDL = 1
OPW_FLAG_COPY_STREAMS = 2
OPW_OK, OPW_ERR_INVALID_ARG, OPW_ERR_UNSUPPORTED, OPW_ERR_CAPACITY, OPW_ERR_CUDA, OPW_ERR_BAD_PAGE, OPW_ERR_TIMEOUT = range(7)

EXPORTS = [
    "opw_kv_pool_index", "opw_kv_pool_bytes", "opw_attn_stage_workspace_bytes", "opw_attn_stage_create",
    "opw_kv_append", "opw_decode_attention", "opw_decode_step_host", "opw_attn_stage_poll_error",
    "opw_attn_stage_launch_count", "opw_attn_stage_destroy", "opw_status_string", "opw_attn_stage_set_trace",
    "opw_decode_attention_noalloc", "opw_attn_plan_create", "opw_attn_plan_submit", "opw_attn_plan_destroy",
    "opw_decode_step", "opw_attn_stage_host_layout", "opw_attn_stage_probe_timeout",
    "opw_linear_attn_decode_step", "opw_linear_attn_state_bytes", "opw_attn_plan_create_mixed",
    "opw_attn_stage_page_table_delta_host", "opw_attn_stage_wait_host_output",
    "opw_attn_stage_shape", "opw_afd_module_workspace_bytes", "opw_afd_module_create", "opw_afd_module_step",
    "opw_afd_module_intermediates", "opw_afd_module_destroy", "opw_afd_module_poll_error",
    "opw_afd_module_launch_count", "opw_afd_module_set_trace", "opw_hbm_read_probe",
]


class StageConfig(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("device", ctypes.c_int32),
        ("num_layers", ctypes.c_int32),
        ("num_q_heads", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("page_size", ctypes.c_int32),
        ("max_batch", ctypes.c_int32),
        ("max_pages_per_seq", ctypes.c_int32),
        ("layer_window", ctypes.POINTER(ctypes.c_int32)),
        ("layer_num_pages", ctypes.POINTER(ctypes.c_int64)),
        ("layer_kv_pool", ctypes.POINTER(ctypes.c_void_p)),
        ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t),
        ("softmax_scale", ctypes.c_float),
        ("flags", ctypes.c_uint32),
        ("tune_warps", ctypes.c_int32),
        ("tune_stages", ctypes.c_int32),
        ("tune_ctas_per_sm", ctypes.c_int32),
        ("reserved", ctypes.c_int32),
    ]


class StepItem(ctypes.Structure):
    _fields_ = [
        ("layer", ctypes.c_int32),
        ("batch", ctypes.c_int32),
        ("q", ctypes.c_void_p),
        ("k_new", ctypes.c_void_p),
        ("v_new", ctypes.c_void_p),
        ("positions", ctypes.c_void_p),
        ("kv_lens", ctypes.c_void_p),
        ("page_table", ctypes.c_void_p),
        ("out", ctypes.c_void_p),
        ("lse", ctypes.c_void_p),
    ]


class LinearItem(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("num_k_heads", ctypes.c_int32), ("num_v_heads", ctypes.c_int32),
        ("dk", ctypes.c_int32), ("dv", ctypes.c_int32),
        ("state", ctypes.c_void_p), ("num_slots", ctypes.c_int64), ("slot", ctypes.c_void_p),
        ("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p),
        ("a", ctypes.c_void_p), ("beta", ctypes.c_void_p), ("scale", ctypes.c_float), ("out", ctypes.c_void_p),
    ]


class AfdItem(ctypes.Structure):
    _fields_ = [("module", ctypes.c_void_p), ("batch", ctypes.c_int32), ("x", ctypes.c_void_p),
                ("positions", ctypes.c_void_p), ("page_table", ctypes.c_void_p), ("y", ctypes.c_void_p)]


class PlanOp(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("attention", StepItem), ("linear", LinearItem), ("afd", AfdItem)]


OPW_OP_ATTENTION, OPW_OP_LINEAR, OPW_OP_AFD_MODULE = 0, 1, 2
OPW_PLAN_GRAPH, OPW_PLAN_ADVANCE, OPW_PLAN_OVERLAP = 1, 2, 4
OPW_AFD_LIBRARY_GEMM, OPW_AFD_NO_PDL, OPW_AFD_NO_CLUSTER = 1, 2, 4


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the library in-tree for sm_100a with nvcc (cross-compiles without a GPU)."""
    srcs = [s for s in SOURCES if os.path.exists(s)]
    deps = srcs + HEADERS
    if not force and os.path.exists(LIB_PATH) and all(os.path.getmtime(LIB_PATH) >= os.path.getmtime(d) for d in deps):
        return LIB_PATH
    tmp = LIB_PATH + f".tmp{os.getpid()}"
    cmd = [
        "nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
        "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(_ROOT, "include"), "-o", tmp, *srcs,
        "-lcublasLt",
    ]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


class OpwError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load the C-ABI library; raises if it has not been built (no CPU fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -c 'import __graft_entry__ as g; g.build()'` first")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    L.opw_kv_pool_index.restype = i64
    L.opw_kv_pool_index.argtypes = [i64] * 8
    L.opw_kv_pool_bytes.restype = ctypes.c_size_t
    L.opw_kv_pool_bytes.argtypes = [i32, i32, i32, i64]
    L.opw_attn_stage_workspace_bytes.restype = ctypes.c_size_t
    L.opw_attn_stage_workspace_bytes.argtypes = [ctypes.POINTER(StageConfig)]
    L.opw_attn_stage_create.restype = ctypes.c_int
    L.opw_attn_stage_create.argtypes = [ctypes.POINTER(StageConfig), ctypes.POINTER(vp)]
    L.opw_kv_append.restype = ctypes.c_int
    L.opw_kv_append.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
    L.opw_decode_attention.restype = ctypes.c_int
    L.opw_decode_attention.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp]
    L.opw_decode_step.restype = ctypes.c_int
    L.opw_decode_step.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    L.opw_attn_stage_host_layout.restype = ctypes.c_int
    L.opw_attn_stage_host_layout.argtypes = [vp] + [ctypes.POINTER(ctypes.c_size_t)] * 5
    L.opw_decode_step_host.restype = ctypes.c_int
    L.opw_decode_step_host.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    L.opw_attn_stage_wait_host_output.restype = ctypes.c_int
    L.opw_attn_stage_wait_host_output.argtypes = [vp]
    L.opw_attn_stage_page_table_delta_host.restype = ctypes.c_int
    L.opw_attn_stage_page_table_delta_host.argtypes = [vp, i32, vp, i32, vp]
    L.opw_linear_attn_decode_step.restype = ctypes.c_int
    L.opw_linear_attn_decode_step.argtypes = [i32, i32, i32, i32, i32, vp, i64, vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp]
    L.opw_linear_attn_state_bytes.restype = ctypes.c_size_t
    L.opw_linear_attn_state_bytes.argtypes = [i32, i32, i32, i64]
    L.opw_attn_stage_probe_timeout.restype = ctypes.c_int
    L.opw_attn_stage_probe_timeout.argtypes = [vp, vp]
    L.opw_attn_stage_poll_error.restype = ctypes.c_int
    L.opw_attn_stage_poll_error.argtypes = [vp, vp]
    L.opw_attn_stage_set_trace.restype = ctypes.c_int
    L.opw_attn_stage_set_trace.argtypes = [vp, vp, ctypes.c_size_t, ctypes.POINTER(i32)]
    L.opw_decode_attention_noalloc.restype = ctypes.c_int
    L.opw_decode_attention_noalloc.argtypes = [i32, i32, i32, i32, i32, ctypes.c_float, vp, i64, i32, i32, vp, vp, vp, vp,
                                               vp, vp]
    L.opw_attn_plan_create.restype = ctypes.c_int
    L.opw_attn_plan_create.argtypes = [vp, ctypes.POINTER(StepItem), i32, ctypes.c_uint32, ctypes.POINTER(vp)]
    L.opw_attn_plan_create_mixed.restype = ctypes.c_int
    L.opw_attn_plan_create_mixed.argtypes = [vp, ctypes.POINTER(PlanOp), i32, ctypes.c_uint32, ctypes.POINTER(vp)]
    L.opw_attn_plan_submit.restype = ctypes.c_int
    L.opw_attn_plan_submit.argtypes = [vp, vp]
    L.opw_attn_plan_destroy.restype = ctypes.c_int
    L.opw_attn_plan_destroy.argtypes = [vp]
    L.opw_hbm_read_probe.restype = ctypes.c_int
    L.opw_hbm_read_probe.argtypes = [vp, ctypes.c_size_t, vp, vp]
    L.opw_attn_stage_shape.restype = ctypes.c_int
    L.opw_attn_stage_shape.argtypes = [vp] + [ctypes.POINTER(i32)] * 6
    L.opw_afd_module_workspace_bytes.restype = ctypes.c_size_t
    L.opw_afd_module_workspace_bytes.argtypes = [i32, i32, i32, i32, i32]
    L.opw_afd_module_create.restype = ctypes.c_int
    L.opw_afd_module_create.argtypes = [vp, i32, i32, vp, vp, ctypes.c_float, ctypes.c_uint32, vp, ctypes.c_size_t,
                                        ctypes.POINTER(vp)]
    L.opw_afd_module_poll_error.restype = ctypes.c_int
    L.opw_afd_module_poll_error.argtypes = [vp, vp]
    L.opw_afd_module_set_trace.restype = ctypes.c_int
    L.opw_afd_module_set_trace.argtypes = [vp, vp, ctypes.c_size_t]
    L.opw_afd_module_launch_count.restype = i64
    L.opw_afd_module_launch_count.argtypes = [vp]
    L.opw_afd_module_step.restype = ctypes.c_int
    L.opw_afd_module_step.argtypes = [vp, i32, vp, vp, vp, vp, vp]
    L.opw_afd_module_intermediates.restype = ctypes.c_int
    L.opw_afd_module_intermediates.argtypes = [vp] + [ctypes.POINTER(vp)] * 4
    L.opw_afd_module_destroy.restype = ctypes.c_int
    L.opw_afd_module_destroy.argtypes = [vp]
    L.opw_attn_stage_launch_count.restype = i64
    L.opw_attn_stage_launch_count.argtypes = [vp]
    L.opw_attn_stage_destroy.restype = ctypes.c_int
    L.opw_attn_stage_destroy.argtypes = [vp]
    L.opw_status_string.restype = ctypes.c_char_p
    L.opw_status_string.argtypes = [ctypes.c_int]
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().opw_status_string(int(status)).decode()


def opw_kv_pool_index(Hkv: int, P: int, D: int, page: int, g: int, kv: int, t: int, d: int) -> int:
    return int(lib().opw_kv_pool_index(Hkv, P, D, page, g, kv, t, d))


def opw_kv_pool_bytes(Hkv: int, P: int, D: int, num_pages: int) -> int:
    return int(lib().opw_kv_pool_bytes(Hkv, P, D, num_pages))


def make_config(*, device: int, num_q_heads: int, num_kv_heads: int, head_dim: int, max_batch: int,
                max_pages_per_seq: int, layer_window: Sequence[int], layer_num_pages: Sequence[int],
                layer_kv_pool: Sequence[int], workspace: int = 0, workspace_bytes: int = 0, page_size: int = 16,
                softmax_scale: float = 0.0, flags: int = 0, tune_warps: int = 0, tune_stages: int = 0,
                tune_ctas_per_sm: int = 0):
    """Fill a StageConfig; returns (cfg, keepalive) -- keep `keepalive` until create returns."""
    L = len(layer_window)
    win = (ctypes.c_int32 * L)(*[int(w) for w in layer_window])
    npg = (ctypes.c_int64 * L)(*[int(n) for n in layer_num_pages])
    pools = (ctypes.c_void_p * L)(*[int(p) for p in layer_kv_pool])
    cfg = StageConfig()
    cfg.struct_size = ctypes.sizeof(StageConfig)
    cfg.device = device
    cfg.num_layers = L
    cfg.num_q_heads = num_q_heads
    cfg.num_kv_heads = num_kv_heads
    cfg.head_dim = head_dim
    cfg.page_size = page_size
    cfg.max_batch = max_batch
    cfg.max_pages_per_seq = max_pages_per_seq
    cfg.layer_window = ctypes.cast(win, ctypes.POINTER(ctypes.c_int32))
    cfg.layer_num_pages = ctypes.cast(npg, ctypes.POINTER(ctypes.c_int64))
    cfg.layer_kv_pool = ctypes.cast(pools, ctypes.POINTER(ctypes.c_void_p))
    cfg.workspace = workspace
    cfg.workspace_bytes = workspace_bytes
    cfg.softmax_scale = softmax_scale
    cfg.flags = flags
    cfg.tune_warps = tune_warps
    cfg.tune_stages = tune_stages
    cfg.tune_ctas_per_sm = tune_ctas_per_sm
    cfg.reserved = 0
    return cfg, (win, npg, pools)


def opw_attn_stage_workspace_bytes(cfg: StageConfig) -> int:
    return int(lib().opw_attn_stage_workspace_bytes(ctypes.byref(cfg)))


def opw_attn_stage_create(cfg: StageConfig) -> int:
    """Returns the opaque handle (an integer address); raises OpwError on failure."""
    h = ctypes.c_void_p()
    rc = lib().opw_attn_stage_create(ctypes.byref(cfg), ctypes.byref(h))
    if rc != OPW_OK:
        raise OpwError(rc, "opw_attn_stage_create")
    return h.value


def _check(rc: int, where: str) -> None:
    if rc != OPW_OK:
        raise OpwError(rc, where)


def opw_kv_append(stage: int, layer: int, batch: int, k_new: int, v_new: int, positions: int, page_table: int,
                  stream: Optional[int] = None) -> None:
    _check(lib().opw_kv_append(stage, layer, batch, k_new, v_new, positions, page_table, stream), "opw_kv_append")


def opw_decode_attention(stage: int, layer: int, batch: int, q: int, kv_lens: int, page_table: int, out: int,
                         lse: Optional[int] = None, stream: Optional[int] = None) -> None:
    _check(lib().opw_decode_attention(stage, layer, batch, q, kv_lens, page_table, out, lse, stream),
           "opw_decode_attention")


def opw_decode_step(stage: int, layer: int, batch: int, q: int, k_new: int, v_new: int, positions: int,
                    page_table: int, out: int, lse: Optional[int] = None, stream: Optional[int] = None) -> None:
    _check(lib().opw_decode_step(stage, layer, batch, q, k_new, v_new, positions, page_table, out, lse, stream),
           "opw_decode_step")


def opw_attn_stage_host_layout(stage: int):
    """Returns (q_off, k_off, v_off, pos_off, total_bytes) of the packed host buffer."""
    v = [ctypes.c_size_t(0) for _ in range(5)]
    _check(lib().opw_attn_stage_host_layout(stage, *[ctypes.byref(x) for x in v]), "opw_attn_stage_host_layout")
    return tuple(int(x.value) for x in v)


def opw_decode_step_host(stage: int, layer: int, batch: int, q_host: int, k_new_host: int, v_new_host: int,
                         positions_host: int, page_table_host: Optional[int], out_host: int,
                         lse_host: Optional[int] = None, stream: Optional[int] = None) -> None:
    _check(lib().opw_decode_step_host(stage, layer, batch, q_host, k_new_host, v_new_host, positions_host,
                                      page_table_host, out_host, lse_host, stream), "opw_decode_step_host")


def opw_attn_stage_page_table_delta_host(stage: int, layer: int, triples_host: int, n: int,
                                         stream: Optional[int] = None) -> None:
    """triples_host: host address of int32 [n][3] = (batch row, logical page, physical page)."""
    _check(lib().opw_attn_stage_page_table_delta_host(stage, layer, triples_host, n, stream),
           "opw_attn_stage_page_table_delta_host")


def opw_decode_attention_noalloc(*, num_q_heads: int, num_kv_heads: int, head_dim: int, kv_pool: int, num_pages: int,
                                 batch: int, max_pages_per_seq: int, q: int, kv_lens: int, page_table: int, out: int,
                                 lse: Optional[int] = None, window: int = 0, softmax_scale: float = 0.0,
                                 page_size: int = 16, stream: Optional[int] = None) -> None:
    """Decode attention for callers that cannot allocate: no stage, no workspace (the scratch is a
    fixed array inside the library).  The buffers' device must be current; calls sharing a device
    must not overlap."""
    _check(lib().opw_decode_attention_noalloc(num_q_heads, num_kv_heads, head_dim, page_size, window, softmax_scale,
                                              kv_pool, num_pages, batch, max_pages_per_seq, q, kv_lens, page_table,
                                              out, lse, stream), "opw_decode_attention_noalloc")


def opw_attn_plan_create(stage: int, items: Sequence[dict], flags: int = 0) -> int:
    """items: dicts with layer, batch and the device addresses q, k_new, v_new, positions, kv_lens,
    page_table, out, lse (missing / None = NULL).  Returns the plan handle."""
    arr = (StepItem * len(items))()
    for a, it in zip(arr, items):
        a.layer, a.batch = it["layer"], it["batch"]
        for k in ("q", "k_new", "v_new", "positions", "kv_lens", "page_table", "out", "lse"):
            setattr(a, k, it.get(k))
    h = ctypes.c_void_p()
    _check(lib().opw_attn_plan_create(stage, arr, len(items), flags, ctypes.byref(h)), "opw_attn_plan_create")
    return h.value


def opw_attn_plan_create_mixed(stage: int, ops: Sequence[dict], flags: int = 0) -> int:
    """ops: dicts with kind "attention" (fields of an attention item), "linear" (batch, num_k_heads,
    num_v_heads, dk, dv, state, num_slots, slot, q, k, v, a, beta, out and optionally scale) or
    "afd_module" (module, batch, x, positions, page_table, y)."""
    arr = (PlanOp * len(ops))()
    for a, op in zip(arr, ops):
        if op["kind"] == "attention":
            a.kind = OPW_OP_ATTENTION
            a.attention.layer, a.attention.batch = op["layer"], op["batch"]
            for k in ("q", "k_new", "v_new", "positions", "kv_lens", "page_table", "out", "lse"):
                setattr(a.attention, k, op.get(k))
        elif op["kind"] == "afd_module":
            a.kind = OPW_OP_AFD_MODULE
            a.afd.batch = int(op["batch"])
            for k in ("module", "x", "positions", "page_table", "y"):
                setattr(a.afd, k, op[k])
        else:
            a.kind = OPW_OP_LINEAR
            for k in ("batch", "num_k_heads", "num_v_heads", "dk", "dv", "num_slots"):
                setattr(a.linear, k, int(op[k]))
            for k in ("state", "slot", "q", "k", "v", "a", "beta", "out"):
                setattr(a.linear, k, op[k])
            a.linear.scale = float(op.get("scale", 0.0))
    h = ctypes.c_void_p()
    _check(lib().opw_attn_plan_create_mixed(stage, arr, len(ops), flags, ctypes.byref(h)), "opw_attn_plan_create_mixed")
    return h.value


def opw_attn_plan_submit(plan: int, stream: Optional[int] = None) -> None:
    _check(lib().opw_attn_plan_submit(plan, stream), "opw_attn_plan_submit")


def opw_attn_plan_destroy(plan: Optional[int]) -> None:
    _check(lib().opw_attn_plan_destroy(plan), "opw_attn_plan_destroy")


def opw_linear_attn_decode_step(*, batch: int, num_k_heads: int, num_v_heads: int, dk: int, dv: int, state: int,
                                num_slots: int, slot: int, q: int, k: int, v: int, a: int, beta: int, out: int,
                                scale: float = 0.0, stream: Optional[int] = None) -> None:
    """One in-place decode step of a recurrent-state layer (all arguments are device addresses)."""
    _check(lib().opw_linear_attn_decode_step(batch, num_k_heads, num_v_heads, dk, dv, state, num_slots, slot, q, k, v,
                                             a, beta, scale, out, stream), "opw_linear_attn_decode_step")


def opw_linear_attn_state_bytes(num_v_heads: int, dk: int, dv: int, num_slots: int) -> int:
    return int(lib().opw_linear_attn_state_bytes(num_v_heads, dk, dv, num_slots))


def opw_attn_stage_probe_timeout(stage: int, stream: Optional[int] = None) -> None:
    _check(lib().opw_attn_stage_probe_timeout(stage, stream), "opw_attn_stage_probe_timeout")


def opw_attn_stage_poll_error(stage: int, stream: Optional[int] = None) -> int:
    return int(lib().opw_attn_stage_poll_error(stage, stream))


def opw_attn_stage_set_trace(stage: int, trace: Optional[int], trace_bytes: int = 0) -> int:
    """Returns the worker count; raises OpwError if the buffer is too small or misaligned."""
    n = ctypes.c_int32(0)
    _check(lib().opw_attn_stage_set_trace(stage, trace, trace_bytes, ctypes.byref(n)), "opw_attn_stage_set_trace")
    return int(n.value)


def opw_attn_stage_launch_count(stage: int) -> int:
    return int(lib().opw_attn_stage_launch_count(stage))


def opw_hbm_read_probe(buffer: int, nbytes: int, sink: int, stream: Optional[int] = None) -> None:
    """Enqueue one pass of 16-byte evict-first loads over [buffer, buffer + nbytes) (device addresses)."""
    _check(lib().opw_hbm_read_probe(buffer, nbytes, sink, stream), "opw_hbm_read_probe")


def opw_attn_stage_shape(stage: int) -> dict:
    """The static shape the stage was bound with."""
    names = ("device", "num_layers", "num_q_heads", "num_kv_heads", "head_dim", "max_batch")
    vals = [ctypes.c_int32(0) for _ in names]
    _check(lib().opw_attn_stage_shape(stage, *[ctypes.byref(v) for v in vals]), "opw_attn_stage_shape")
    return {n: int(v.value) for n, v in zip(names, vals)}


def opw_afd_module_workspace_bytes(num_q_heads: int, num_kv_heads: int, head_dim: int, max_batch: int,
                                   hidden: int) -> int:
    return int(lib().opw_afd_module_workspace_bytes(num_q_heads, num_kv_heads, head_dim, max_batch, hidden))


def opw_afd_module_create(stage: int, layer: int, hidden: int, w_qkv: int, w_o: int, rope_theta: float,
                          workspace: int, workspace_bytes: int, flags: int = 0) -> int:
    h = ctypes.c_void_p()
    _check(lib().opw_afd_module_create(stage, layer, hidden, w_qkv, w_o, rope_theta, flags, workspace,
                                       workspace_bytes, ctypes.byref(h)), "opw_afd_module_create")
    return h.value


def opw_afd_module_poll_error(module: int, stream: Optional[int] = None) -> int:
    return int(lib().opw_afd_module_poll_error(module, stream))


def opw_afd_module_set_trace(module: int, trace: Optional[int], trace_bytes: int = 0) -> None:
    _check(lib().opw_afd_module_set_trace(module, trace, trace_bytes), "opw_afd_module_set_trace")


def opw_afd_module_launch_count(module: int) -> int:
    return int(lib().opw_afd_module_launch_count(module))


def opw_afd_module_step(module: int, batch: int, x: int, positions: int, page_table: int, y: int,
                        stream: Optional[int] = None) -> None:
    _check(lib().opw_afd_module_step(module, batch, x, positions, page_table, y, stream), "opw_afd_module_step")


def opw_afd_module_intermediates(module: int):
    """Device addresses (q, k_new, v_new, attn_out) of the last step's intermediates."""
    ptrs = [ctypes.c_void_p() for _ in range(4)]
    _check(lib().opw_afd_module_intermediates(module, *[ctypes.byref(p) for p in ptrs]), "opw_afd_module_intermediates")
    return tuple(p.value for p in ptrs)


def opw_afd_module_destroy(module: Optional[int]) -> None:
    _check(lib().opw_afd_module_destroy(module), "opw_afd_module_destroy")


def opw_attn_stage_destroy(stage: Optional[int]) -> None:
    _check(lib().opw_attn_stage_destroy(stage), "opw_attn_stage_destroy")


class Stage:
    """Convenience owner of one stage handle over caller-provided torch tensors.

    Holds references to the pools and the workspace so they outlive the handle.  All
    methods forward to the C entry points of the same name.
    """

    def __init__(self, *, pools, layer_window, num_q_heads, num_kv_heads, head_dim, max_batch, max_pages_per_seq,
                 layer_num_pages=None, device=None, softmax_scale=0.0, tune_warps=0, tune_stages=0,
                 tune_ctas_per_sm=0, flags=0):
        import torch

        dev = pools[0].device if device is None else torch.device(device)
        if dev.type != "cuda":
            raise RuntimeError("the attention stage runs on a CUDA device only")
        self.device = dev
        self.pools = list(pools)
        page_elems = num_kv_heads * 2 * 16 * head_dim
        if layer_num_pages is None:
            layer_num_pages = [p.numel() // page_elems for p in pools]
        kw = dict(device=dev.index or 0, num_q_heads=num_q_heads, num_kv_heads=num_kv_heads, head_dim=head_dim,
                  max_batch=max_batch, max_pages_per_seq=max_pages_per_seq, layer_window=layer_window,
                  layer_num_pages=layer_num_pages, layer_kv_pool=[p.data_ptr() for p in pools],
                  softmax_scale=softmax_scale, tune_warps=tune_warps, tune_stages=tune_stages,
                  tune_ctas_per_sm=tune_ctas_per_sm, flags=flags)
        cfg, _keep = make_config(**kw)
        nbytes = opw_attn_stage_workspace_bytes(cfg)
        if nbytes == 0:
            raise OpwError(OPW_ERR_INVALID_ARG, "opw_attn_stage_workspace_bytes")
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=dev)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        cfg.workspace = base
        cfg.workspace_bytes = nbytes
        self.num_q_heads, self.num_kv_heads, self.head_dim = num_q_heads, num_kv_heads, head_dim
        self.handle = opw_attn_stage_create(cfg)

    @staticmethod
    def _stream():
        import torch

        return torch.cuda.current_stream().cuda_stream

    def kv_append(self, layer, k_new, v_new, positions, page_table):
        opw_kv_append(self.handle, layer, positions.shape[0], k_new.data_ptr(), v_new.data_ptr(),
                      positions.data_ptr(), page_table.data_ptr(), self._stream())

    def decode_attention(self, layer, q, kv_lens, page_table, out, lse=None):
        opw_decode_attention(self.handle, layer, kv_lens.shape[0], q.data_ptr(), kv_lens.data_ptr(),
                             page_table.data_ptr(), out.data_ptr(), None if lse is None else lse.data_ptr(),
                             self._stream())

    def decode_step(self, layer, q, k_new, v_new, positions, page_table, out, lse=None):
        opw_decode_step(self.handle, layer, positions.shape[0], q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(),
                        positions.data_ptr(), page_table.data_ptr(), out.data_ptr(),
                        None if lse is None else lse.data_ptr(), self._stream())

    def decode_step_host(self, layer, q, k_new, v_new, positions, page_table, out, lse=None):
        opw_decode_step_host(self.handle, layer, positions.shape[0], q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(),
                             positions.data_ptr(), None if page_table is None else page_table.data_ptr(),
                             out.data_ptr(), None if lse is None else lse.data_ptr(), self._stream())

    def wait_host_output(self):
        _check(lib().opw_attn_stage_wait_host_output(self.handle), "opw_attn_stage_wait_host_output")

    def page_table_delta_host(self, layer, triples):
        """triples: int32 host tensor [n, 3] of (batch row, logical page, physical page), pinned for an asynchronous copy."""
        opw_attn_stage_page_table_delta_host(self.handle, layer, triples.data_ptr(), int(triples.shape[0]), self._stream())

    def enable_trace(self):
        """Allocate a trace buffer (torch) and switch per-worker tracing on; returns the int64 tensor [workers, 4]."""
        import torch

        n = opw_attn_stage_set_trace(self.handle, None)
        self.trace = torch.zeros(n, 4, dtype=torch.int64, device=self.device)
        opw_attn_stage_set_trace(self.handle, self.trace.data_ptr(), self.trace.numel() * 8)
        return self.trace

    def packed_host_buffers(self, batch):
        """One pinned host buffer holding q, k_new, v_new, positions at the packed offsets;
        returns (buffer, q, k_new, v_new, positions) -- the last four are views into it."""
        import torch

        qo, ko, vo, po, total = opw_attn_stage_host_layout(self.handle)
        buf = torch.empty(total, dtype=torch.uint8).pin_memory()
        Hq, Hkv, D = self.num_q_heads, self.num_kv_heads, self.head_dim
        q = buf[qo:qo + batch * Hq * D * 2].view(torch.bfloat16).view(batch, Hq, D)
        k = buf[ko:ko + batch * Hkv * D * 2].view(torch.bfloat16).view(batch, Hkv, D)
        v = buf[vo:vo + batch * Hkv * D * 2].view(torch.bfloat16).view(batch, Hkv, D)
        pos = buf[po:po + batch * 4].view(torch.int32)
        return buf, q, k, v, pos

    def poll_error(self) -> int:
        return opw_attn_stage_poll_error(self.handle, self._stream())

    def launch_count(self) -> int:
        return opw_attn_stage_launch_count(self.handle)

    def close(self):
        if getattr(self, "handle", None):
            opw_attn_stage_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class AfdModule:
    """Owner of one complete-attention-module handle (projections + rotary encoding + the stage's
    core attention) over torch tensors; forwards to the opw_afd_module_* entry points."""

    def __init__(self, stage: Stage, layer: int, w_qkv, w_o, rope_theta: float = 10000.0, flags: int = 0):
        import torch

        shp = opw_attn_stage_shape(stage.handle)
        self.stage, self.w_qkv, self.w_o = stage, w_qkv, w_o
        self.hidden = int(w_qkv.shape[1])
        n_qkv = (shp["num_q_heads"] + 2 * shp["num_kv_heads"]) * shp["head_dim"]
        if tuple(w_qkv.shape) != (n_qkv, self.hidden) or tuple(w_o.shape) != (self.hidden, shp["num_q_heads"] * shp["head_dim"]):
            raise ValueError("weight shapes do not match the stage")
        if w_qkv.dtype != torch.bfloat16 or w_o.dtype != torch.bfloat16 or not (w_qkv.is_contiguous() and w_o.is_contiguous()):
            raise ValueError("weights must be contiguous bf16")
        nbytes = opw_afd_module_workspace_bytes(shp["num_q_heads"], shp["num_kv_heads"], shp["head_dim"], shp["max_batch"],
                                                self.hidden)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=stage.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        self.shape = shp
        self.handle = opw_afd_module_create(stage.handle, layer, self.hidden, w_qkv.data_ptr(), w_o.data_ptr(),
                                            rope_theta, base, nbytes, flags)

    def poll_error(self) -> int:
        return opw_afd_module_poll_error(self.handle, Stage._stream())

    def launch_count(self) -> int:
        return opw_afd_module_launch_count(self.handle)

    def enable_trace(self):
        """Allocate the trace buffer and switch tracing on; returns the int64 tensor [2, 1024, 8]
        (region 0: output projection, region 1: QKV projection)."""
        import torch

        self.trace = torch.zeros(2, 1024, 8, dtype=torch.int64, device=self.stage.device)
        opw_afd_module_set_trace(self.handle, self.trace.data_ptr(), self.trace.numel() * 8)
        return self.trace

    def step(self, x, positions, page_table, y):
        opw_afd_module_step(self.handle, positions.shape[0], x.data_ptr(), positions.data_ptr(), page_table.data_ptr(),
                            y.data_ptr(), Stage._stream())

    def intermediates(self, batch: int):
        """Copies of the last step's q, k_new, v_new and attention output as torch tensors."""
        import torch

        Hq, Hkv, D = self.shape["num_q_heads"], self.shape["num_kv_heads"], self.shape["head_dim"]
        base = self.workspace.data_ptr()
        out = []
        for ptr, heads in zip(opw_afd_module_intermediates(self.handle), (Hq, Hkv, Hkv, Hq)):
            off = ptr - base
            out.append(self.workspace[off:off + batch * heads * D * 2].view(torch.bfloat16).view(batch, heads, D).clone())
        return tuple(out)

    def close(self):
        if getattr(self, "handle", None):
            opw_afd_module_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

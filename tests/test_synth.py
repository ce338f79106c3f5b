"""Host-side checks of the seeded input generator (no GPU)."""
import numpy as np
import torch

from paper_2609_14237_b200 import synth


def test_lengths_follow_the_recipes_and_are_seeded():
    a = synth.draw_lengths("tiny", 4, 1)
    assert a.tolist() == [17, 64, 100, 255]
    u = synth.draw_lengths("uniform_1024_4096", 64, 1002)
    assert u.min() >= 1024 and u.max() <= 4096
    assert (u == synth.draw_lengths("uniform_1024_4096", 64, 1002)).all()
    ln = synth.draw_lengths("lognormal_2048", 256, 1004)
    assert ln.min() >= 16 and ln.max() <= 16384 and 1200 < np.median(ln) < 3500
    assert (synth.draw_lengths("const_32768", 16, 3) == 32768).all()


def test_page_tables_are_disjoint_permutations_and_cover_growth():
    wl = synth.WORKLOADS["c1_tiny"]
    inp = synth.make_inputs(wl, growth=3, steps=3)
    tab = inp.page_tables[0].numpy()
    used = tab[tab >= 0]
    assert len(set(used.tolist())) == used.size and used.max() < inp.num_pages[0]
    for b, n in enumerate(inp.lengths):
        need = (n + 3 - 1) // 16 + 1
        assert (tab[b, :need] >= 0).all() and (tab[b, need:] == -1).all()
    assert inp.pools[0].numel() == inp.num_pages[0] * wl.num_kv_heads * 2 * 16 * wl.head_dim
    assert inp.q.shape == (3, 1, 4, 8, 64) and inp.q.dtype == torch.bfloat16
    assert inp.kv_bytes(0) == (18 + 65 + 101 + 256) * 512


def test_window_layers_map_only_the_pages_a_step_can_touch():
    wl = synth.Workload("w", 3, 8, 2, 64, [32, 0], "tiny", 5)
    inp = synth.make_inputs(wl, growth=2, lengths=np.array([10, 100, 255], np.int32))
    swa, full = inp.page_tables[0].numpy(), inp.page_tables[1].numpy()
    for b, n in enumerate([10, 100, 255]):
        first = max(0, n + 1 - 32) // 16
        assert (swa[b, :first] == -1).all() and swa[b, first] >= 0
        assert (full[b, : (n + 1) // 16 + 1] >= 0).all()
    assert inp.visible_tokens(0) == 11 + 32 + 32 and inp.visible_tokens(1) == 11 + 101 + 256


def test_shard_rows_partition_the_batch():
    for batch, world in [(256, 8), (5, 2), (3, 4)]:
        got = [r for k in range(world) for r in synth.shard_rows(batch, k, world)]
        assert got == list(range(batch))

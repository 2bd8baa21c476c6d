"""Seeded input generators: determinism, block-wise regeneration, distributions."""
import torch

from paper_2603_08343_b200 import workloads as wl


def test_configs_table():
    assert set(wl.CONFIGS) == {"tiny", "prefill", "decode", "training", "large"}
    assert (wl.CONFIGS["prefill"].T, wl.CONFIGS["prefill"].d) == (16384, 1024)
    assert (wl.CONFIGS["training"].T, wl.CONFIGS["training"].d) == (65536, 2048)
    assert (wl.CONFIGS["large"].T, wl.CONFIGS["large"].d) == (131072, 8192)
    assert wl.CONFIGS["tiny"].io_torch_dtype == torch.float32
    assert wl.CONFIGS["training"].param_torch_dtype == torch.float32
    assert wl.CONFIGS["prefill"].param_torch_dtype == torch.bfloat16


def test_row_ranges_regenerate_identically():
    w = wl.CONFIGS["prefill"].with_rows(3000)
    full = wl.gen_full(w, "x", threads=4)
    assert full.shape == (3000, 1024) and full.dtype == torch.bfloat16
    assert torch.equal(wl.gen_rows(w, "x", 1000, 2100), full[1000:2100])
    assert torch.equal(wl.gen_full(w, "x", threads=1), full)
    assert not torch.equal(wl.gen_rows(w, "dy", 0, 8), full[0:8])


def test_distributions():
    w = wl.CONFIGS["training"].with_rows(1024)
    x = wl.gen_full(w, "x").float()
    assert abs(x.mean().item()) < 0.01 and abs(x.std().item() - 1.0) < 0.01
    a, b = wl.gen_params(w)
    assert a.dtype == torch.float32 and 0.5 <= a.min().item() and a.max().item() <= 1.5
    assert abs(b.std().item() - 0.1) < 0.02
    t = wl.CONFIGS["large"].with_rows(256)
    h = wl.gen_full(t, "x").float()
    # 0.5 * t_3 has variance 0.25 * 3 = 0.75 and far heavier tails than a normal
    assert h.abs().max().item() > 8.0
    assert 0.4 < h.median().abs().item() + 0.4 < 0.45


def test_shard_rows_partition():
    from paper_2603_08343_b200 import dp
    for T, n in [(10, 3), (65536, 8), (7, 8), (0, 2)]:
        spans = [dp.shard_rows(T, n, r) for r in range(n)]
        assert spans[0][0] == 0 and spans[-1][1] == T
        assert all(spans[i][1] == spans[i + 1][0] for i in range(n - 1))
        sizes = [b - a for a, b in spans]
        assert max(sizes) - min(sizes) <= 1

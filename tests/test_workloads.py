"""Seeded input generators: reproducible, bf16-representable, shaped as stated (CPU only)."""
import numpy as np

from paper_2604_03815_b200 import workloads as wl


def _is_bf16(x):
    return np.all((x.view(np.uint32) & 0xFFFF) == 0)


def test_counter_based_and_chunk_independent():
    key = wl.stream_key(7, 3)
    a = wl.normal(key, 1000, chunk=1000)
    b = wl.normal(key, 1000, chunk=64)
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(wl.normal(key, 10), a[:10])
    assert wl.stream_key(7, 3) != wl.stream_key(7, 4) != wl.stream_key(8, 3)


def test_normal_moments():
    z = wl.normal(wl.stream_key(1, 1), 400_000)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1) < 0.01
    assert abs(np.mean(z ** 3)) < 0.03 and abs(np.mean(z ** 4) - 3) < 0.08


def test_round_to_bf16_ties_to_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -7, -1.0 - 2 ** -8, 0.0], dtype=np.float32)
    y = wl.round_to_bf16(x)
    np.testing.assert_array_equal(y, np.array([1.0, 1.0, 1.0 + 2 ** -6, 1.0 + 2 ** -7, -1.0, 0.0], dtype=np.float32))
    assert _is_bf16(y)


def test_config_shapes():
    c1 = wl.make_config(1)
    assert (c1.N, c1.H, c1.d, c1.k, c1.G, c1.mode) == (1024, 1, 32, 16, 1, wl.MODE_FP32_EXACT)
    assert _is_bf16(c1.Q) and _is_bf16(c1.K) and _is_bf16(c1.V)
    assert abs(c1.Q.std() - 1 / np.sqrt(32)) < 0.01
    c2 = wl.make_config(2)
    n = np.diff(c2.graph_offsets)
    assert c2.G == 128 and n.min() >= 50 and n.max() <= 300 and (c2.H, c2.d, c2.k) == (4, 16, 8)
    assert c2.n_scores == 4 * int(np.sum(n.astype(np.int64) ** 2))
    c4 = wl.make_config(4, N=4096)
    assert c4.Q.shape == (4096, 4, 32) and c4.k == 32 and _is_bf16(c4.Q)
    lab = c4.meta["labels"]
    assert lab.min() == 0 and lab.max() == 63
    # a node's query is closest (in inner product) to keys of its own cluster
    same = lab[:, None] == lab[None, :]
    S = c4.Q[:256, 0].astype(np.float64) @ c4.K[:, 0].astype(np.float64).T
    assert S[same[:256]].mean() > S[~same[:256]].mean() + 10
    c5 = wl.make_config(5, n_per_graph=1000)
    hubs = c5.meta["hubs"]
    assert c5.G == 4 and hubs.reshape(4, 1000).sum(axis=1).tolist() == [10, 10, 10, 10]
    assert np.abs(c5.K[hubs]).mean() > 4 * np.abs(c5.K[~hubs]).mean()


def test_sample_rows_in_range_and_cover_edges():
    w = wl.make_config(2)
    rows = wl.sample_rows(w, 300)
    assert rows.min() == 0 and rows.max() == w.N - 1 and len(np.unique(rows)) == len(rows)

"""Seeded synthetic inputs for k-MIP attention (numpy only, no attention arithmetic).

This module is the one piece shared by the CUDA path's tests, the CPU oracle's
tests and the benchmark: it only *draws inputs*.  Nothing here computes a
score, a top-k, a softmax or a gradient.

Random numbers come from a counter-based generator so that any element of any
array can be reproduced independently of array size, chunking or platform:

    u64(stream, i) = splitmix64_mix(stream_key + (i + 1) * GOLDEN)
    uniform(i)     = (u64 >> 11 + 0.5) * 2^-53                      in (0, 1)
    normal(i)      = sqrt(-2 ln uniform(2i)) * cos(2 pi uniform(2i+1))   (Box-Muller, fp64)

Every value is rounded to the nearest bf16 (ties to even) before it is handed
out, and returned as float32 (a bf16 value is exactly representable in float32),
so the fp32 path, the bf16 path and the fp64 oracle all see the same real numbers.

The five workloads mirror the shapes of the paper's experiments (Sec. 5,
App. H: batched small graphs of a few hundred nodes, single city-scale graphs
of 1e5..5e5 nodes, 4-8 heads, k between 5 and 45) with synthetic values.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

MODE_BF16_TC = 0
MODE_FP32_EXACT = 1


def _mix(z: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on a uint64 array (wrap-around arithmetic)."""
    z = z.copy()
    z ^= z >> np.uint64(30)
    z *= _M1
    z ^= z >> np.uint64(27)
    z *= _M2
    z ^= z >> np.uint64(31)
    return z


def stream_key(seed: int, stream: int) -> np.uint64:
    """A 64-bit key for (seed, stream); distinct arrays use distinct streams."""
    with np.errstate(over="ignore"):
        a = _mix(np.array([np.uint64(seed) * _GOLDEN + np.uint64(0x1234567)], dtype=np.uint64))
        b = _mix(a + np.uint64(stream + 1) * _M1)
    return b[0]


def raw_u64(key: np.uint64, start: int, count: int) -> np.ndarray:
    """u64(key, i) for i in [start, start+count)."""
    with np.errstate(over="ignore"):
        ctr = np.arange(start + 1, start + 1 + count, dtype=np.uint64)
        return _mix(np.uint64(key) + ctr * _GOLDEN)


def uniform(key: np.uint64, start: int, count: int) -> np.ndarray:
    """fp64 uniforms strictly inside (0, 1)."""
    r = raw_u64(key, start, count) >> np.uint64(11)
    return (r.astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(key: np.uint64, count: int, chunk: int = 1 << 22) -> np.ndarray:
    """fp64 standard normals; element i depends only on (key, i)."""
    out = np.empty(count, dtype=np.float64)
    for s in range(0, count, chunk):
        n = min(chunk, count - s)
        u = uniform(key, 2 * s, 2 * n)
        out[s:s + n] = np.sqrt(-2.0 * np.log(u[0::2])) * np.cos((2.0 * np.pi) * u[1::2])
    return out


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float values to the nearest bf16 (ties to even); result is float32."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    b = f.view(np.uint32).astype(np.uint64)
    lsb = (b >> np.uint64(16)) & np.uint64(1)
    b = (b + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return b.astype(np.uint32).view(np.float32).reshape(f.shape)


@dataclass
class Workload:
    """One problem instance.  Arrays are float32 holding bf16-representable values."""
    name: str
    mode: int                 # MODE_BF16_TC or MODE_FP32_EXACT
    H: int
    d: int
    k: int
    graph_offsets: np.ndarray  # int32 [G+1]
    Q: np.ndarray              # float32 [N, H, d]
    K: np.ndarray
    V: np.ndarray
    dOut: np.ndarray           # float32 [N, H, d] upstream gradient (seed + 100)
    backward: bool = True
    meta: dict = field(default_factory=dict)

    @property
    def N(self) -> int:
        return int(self.Q.shape[0])

    @property
    def G(self) -> int:
        return int(self.graph_offsets.shape[0] - 1)

    @property
    def n_scores(self) -> int:
        """Query-key pairs the method evaluates: H * sum_g n_g^2."""
        n = np.diff(self.graph_offsets.astype(np.int64))
        return int(self.H * np.sum(n * n))


def _normal_array(seed: int, stream: int, shape, scale: float = 1.0) -> np.ndarray:
    n = int(np.prod(shape))
    z = normal(stream_key(seed, stream), n)
    if scale != 1.0:
        z *= scale
    return round_to_bf16(z.astype(np.float32)).reshape(shape)


def iid_workload(name, seed, sizes, H, d, k, mode, input_scale=1.0, backward=True) -> Workload:
    """Q, K, V iid N(0,1)*input_scale over graphs with the given node counts."""
    sizes = np.asarray(sizes, dtype=np.int64)
    offs = np.zeros(len(sizes) + 1, dtype=np.int64)
    np.cumsum(sizes, out=offs[1:])
    N = int(offs[-1])
    shape = (N, H, d)
    return Workload(
        name=name, mode=mode, H=H, d=d, k=k,
        graph_offsets=offs.astype(np.int32),
        Q=_normal_array(seed, 0, shape, input_scale),
        K=_normal_array(seed, 1, shape, input_scale),
        V=_normal_array(seed, 2, shape, input_scale),
        dOut=_normal_array(seed + 100, 3, shape),
        backward=backward,
        meta={"seed": seed},
    )


def padded_workload(name, seed, N, H, d_model, d_pad, k, mode, backward=True) -> Workload:
    """One graph of N nodes with d_model-wide heads stored zero-padded to d_pad columns (the
    library takes head widths 16, 32, 64, 128; zero columns leave every inner product and every
    output column of the first d_model unchanged).  The softmax scale follows the stored width,
    so a caller who wants 1/sqrt(d_model) multiplies Q by sqrt(d_pad / d_model) first."""
    w = iid_workload(name, seed, [N], H, d_pad, k, mode, backward=backward)
    for a in (w.Q, w.K, w.V, w.dOut):
        a[:, :, d_model:] = 0.0
    w.meta["d_model"] = d_model
    return w


def config1() -> Workload:
    """One graph, N=1024, H=1, d=32, k=16, fp32 exact mode, values N(0,1)/sqrt(d), seed 0."""
    return iid_workload("c1_single_1k_fp32", 0, [1024], 1, 32, 16, MODE_FP32_EXACT,
                        input_scale=1.0 / np.sqrt(32.0), backward=False)


def config2() -> Workload:
    """128 graphs with node counts uniform in [50, 300], H=4, d=16, k=8, bf16, seed 1."""
    seed = 1
    r = raw_u64(stream_key(seed, 10), 0, 128)
    sizes = 50 + (r % np.uint64(251)).astype(np.int64)
    return iid_workload("c2_batched_small_graphs", seed, sizes, 4, 16, 8, MODE_BF16_TC)


def config3(N: int = 100_000) -> Workload:
    """One graph of 100k nodes, H=4, d=32, k=16, bf16, values N(0,1)/sqrt(d), seed 2."""
    return iid_workload("c3_single_100k", 2, [N], 4, 32, 16, MODE_BF16_TC,
                        input_scale=1.0 / np.sqrt(32.0))


def config4(N: int = 500_000, H: int = 4, d: int = 32, k: int = 32) -> Workload:
    """Point-cloud-like graph: Q and K from a mixture of 64 Gaussian clusters.

    Centres are N(0,1) in R^{H*d}; every node draws one cluster label shared by its
    query and key rows; Q_i = c_z + 0.2 eps, K_i = c_z + 0.2 eps'; V iid N(0,1); seed 3.
    """
    seed = 3
    shape = (N, H, d)
    centres = normal(stream_key(seed, 20), 64 * H * d).reshape(64, H, d)
    labels = (raw_u64(stream_key(seed, 21), 0, N) % np.uint64(64)).astype(np.int64)
    Q = centres[labels] + 0.2 * normal(stream_key(seed, 0), N * H * d).reshape(shape)
    K = centres[labels] + 0.2 * normal(stream_key(seed, 1), N * H * d).reshape(shape)
    return Workload(
        name="c4_pointcloud_500k" if N == 500_000 else f"c4_pointcloud_{N}",
        mode=MODE_BF16_TC, H=H, d=d, k=k,
        graph_offsets=np.array([0, N], dtype=np.int32),
        Q=round_to_bf16(Q.astype(np.float32)), K=round_to_bf16(K.astype(np.float32)),
        V=_normal_array(seed, 2, shape), dOut=_normal_array(seed + 100, 3, shape),
        meta={"seed": seed, "labels": labels},
    )


def config5(n_per_graph: int = 200_000, G: int = 4, H: int = 8, d: int = 16, k: int = 16) -> Workload:
    """G graphs of equal size; per graph 1% of the nodes are hubs whose K rows are x5; seed 4."""
    seed = 4
    w = iid_workload("c5_hub_batch" if n_per_graph == 200_000 else f"c5_hub_batch_{n_per_graph}",
                     seed, [n_per_graph] * G, H, d, k, MODE_BF16_TC)
    u = uniform(stream_key(seed, 30), 0, w.N).reshape(G, n_per_graph)
    n_hub = max(1, int(round(0.01 * n_per_graph)))
    hubs = np.zeros((G, n_per_graph), dtype=bool)
    pick = np.argpartition(u, n_hub - 1, axis=1)[:, :n_hub]
    np.put_along_axis(hubs, pick, True, axis=1)
    hubs = hubs.reshape(-1)
    w.K[hubs] = round_to_bf16(w.K[hubs] * np.float32(5.0))
    w.meta["hubs"] = hubs
    return w


CONFIGS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5}


def make_config(i: int, **kw) -> Workload:
    """Workload number i (1-based, the order of the benchmark's config list)."""
    return CONFIGS[i](**kw)


def sample_rows(w: Workload, n: int, seed: int = 12345) -> np.ndarray:
    """A stratified, seeded sample of query rows: first/last rows of each graph and of its
    128-, 256- and 384-row blocks, plus uniform picks; sorted, unique, int64."""
    offs = w.graph_offsets.astype(np.int64)
    picks = []
    for g in range(w.G):
        lo, hi = offs[g], offs[g + 1]
        if hi > lo:
            picks += [lo, hi - 1, min(lo + 127, hi - 1), min(lo + 128, hi - 1),
                      min(lo + 255, hi - 1), min(lo + 256, hi - 1),
                      min(lo + 383, hi - 1), min(lo + 384, hi - 1)]
            for blk in (256, 384):
                last_block = lo + ((hi - lo - 1) // blk) * blk
                picks += [last_block, max(lo, last_block - 1)]
    r = raw_u64(stream_key(seed, 40), 0, max(n, 1))
    picks += list((r % np.uint64(max(w.N, 1))).astype(np.int64))
    rows = np.unique(np.asarray(picks, dtype=np.int64))
    if len(rows) > n:
        keep = np.unique(np.concatenate([rows[:: max(1, len(rows) // n)][:n], rows[:1], rows[-1:]]))
        rows = keep
    return rows

"""Seeded synthetic workloads with the shapes and skew of the paper's experiments.

The paper evaluates MTTKRP and TTMc on FROSTT tensors (Table 2, Secs. 5.2-5.3) and a
sparse-dense-sparse network with locality structure (Sec. 5.1, intro example
Z_im = U_ijk V_jl W_klm).  Neither data set ships with this repository, so every
input here is drawn from a seeded generator that mimics the published shapes:
power-law slice sizes along the root mode, optional power-law coordinates inside a
slice, banded locality for the network.

Nothing in this module contracts tensors or builds CSF arrays.  It returns COO
coordinates, values, dense factors and the textual schedule descriptor (expression,
contraction tree, CSF mode orders, loop orders) that both the CUDA library and the
CPU oracle consume as inputs.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, List, Sequence, Tuple

import numpy as np


def _rng(seed: int, config_id: int, tensor_id: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, config_id, tensor_id])))


@dataclass
class SparseOperand:
    """COO tensor. coords[m] holds the coordinates of mode m (the m-th index of the reference)."""
    coords: List[np.ndarray]
    vals: np.ndarray
    dims: Tuple[int, ...]

    @property
    def nnz(self) -> int:
        return int(self.vals.shape[0])


@dataclass
class Workload:
    name: str
    family: str                       # "ttmc3" | "ttmc4" | "mttkrp" | "network"
    dtype: np.dtype
    extents: Dict[str, int]           # iteration index -> extent
    sparse: Dict[str, SparseOperand]
    dense: Dict[str, np.ndarray]      # row-major factors
    expression: str
    tree: List[str]                   # binary contractions in execution order
    mode_orders: Dict[str, Tuple[int, ...]]   # per sparse tensor: mode stored at each CSF level
    loop_orders: List[str]            # one index string per contraction, outermost first
    out_shape: Tuple[int, ...]
    notes: Dict[str, object] = field(default_factory=dict)


# --------------------------------------------------------------------------------------
# power-law helpers
# --------------------------------------------------------------------------------------

def zipf_slice_sizes(total: int, n: int, s: float, rng: np.random.Generator) -> np.ndarray:
    """Deterministic rank-size law n_rank ~ rank^-s summing exactly to `total`.

    Largest-remainder rounding; every slice keeps at least one nonzero; the rank -> coordinate
    map is a seeded random permutation.  Returns sizes indexed by coordinate.
    """
    if total < n:
        raise ValueError("need at least one nonzero per slice")
    w = np.arange(1, n + 1, dtype=np.float64) ** (-s)
    ideal = (total - n) * w / w.sum()          # one nonzero per slice is reserved up front
    base = np.floor(ideal).astype(np.int64)
    rem = int(total - n - base.sum())
    if rem > 0:
        frac = ideal - base
        top = np.argsort(-frac, kind="stable")[:rem]
        base[top] += 1
    sizes_by_rank = base + 1
    perm = rng.permutation(n)
    sizes = np.empty(n, dtype=np.int64)
    sizes[perm] = sizes_by_rank
    return sizes


def _zipf_cdf(n: int, s: float) -> np.ndarray:
    w = np.arange(1, n + 1, dtype=np.float64) ** (-s)
    c = np.cumsum(w)
    return c / c[-1]


def _bits(extent: int) -> int:
    return max(1, int(extent - 1).bit_length())


def _unique_fill(sizes: np.ndarray, rest_dims: Sequence[int],
                 draw_rest: Callable[[np.ndarray, np.random.Generator], List[np.ndarray]],
                 rng: np.random.Generator, max_rounds: int = 60) -> np.ndarray:
    """Draw, for every slice s, sizes[s] distinct coordinate tuples of the remaining modes.

    Tuples are packed into one 64-bit key (slice in the top bits), duplicates are discarded
    and slices are topped up with fresh draws until each holds exactly sizes[s] tuples.
    Returns the sorted packed keys.
    """
    n = len(sizes)
    bits = [_bits(d) for d in rest_dims]
    rest_bits = sum(bits)
    if _bits(n) + rest_bits > 63:
        raise ValueError("coordinate tuple does not fit one 64-bit key")
    cap = np.ones(n, dtype=np.float64)
    for d in rest_dims:
        cap *= float(d)
    if np.any(sizes > cap):
        raise ValueError("slice size exceeds the number of cells in the slice")

    need = sizes.astype(np.int64).copy()
    have = np.empty(0, dtype=np.uint64)        # sorted unique keys accepted so far
    accept = np.ones(n, dtype=np.float64)      # running estimate of the acceptance rate
    for _ in range(max_rounds):
        active = np.nonzero(need > 0)[0]
        if active.size == 0:
            break
        m = np.ceil(need[active] / np.clip(accept[active], 0.02, 1.0) * 1.05).astype(np.int64) + 4
        sl = np.repeat(active, m)
        rest = draw_rest(sl, rng)
        key = sl.astype(np.uint64)
        for c, b in zip(rest, bits):
            key = (key << np.uint64(b)) | c.astype(np.uint64)
        uniq, first = np.unique(key, return_index=True)
        if have.size:
            idx = np.searchsorted(have, uniq)
            idx[idx == have.size] = have.size - 1
            fresh = have[idx] != uniq
            uniq, first = uniq[fresh], first[fresh]
        order = np.argsort(first, kind="stable")      # back to draw order: grouped by slice
        uniq = uniq[order]
        usl = (uniq >> np.uint64(rest_bits)).astype(np.int64)
        cnt = np.bincount(usl, minlength=n)
        start = np.concatenate(([0], np.cumsum(cnt)[:-1]))
        rank = np.arange(uniq.size, dtype=np.int64) - start[usl]
        keep = rank < need[usl]
        kept = uniq[keep]
        got = np.bincount(usl[keep], minlength=n)
        accept[active] = np.maximum(cnt[active] / m, 1e-3)
        need -= got
        have = np.sort(np.concatenate([have, kept]))
    if np.any(need > 0):
        raise RuntimeError("could not reach the requested number of distinct coordinates")
    return have


def _unpack(keys: np.ndarray, dims: Sequence[int]) -> List[np.ndarray]:
    bits = [_bits(d) for d in dims[1:]]
    out = []
    k = keys.copy()
    for b in reversed(bits):
        out.append((k & np.uint64((1 << b) - 1)).astype(np.int32))
        k >>= np.uint64(b)
    out.append(k.astype(np.int32))
    return out[::-1]


def _skewed_tensor(dims: Sequence[int], nnz: int, slice_s: float, inner_s, rng: np.random.Generator,
                   value: str, dtype) -> SparseOperand:
    """Sparse tensor with Zipf(slice_s) slice sizes along mode 0.

    inner_s = None draws the remaining coordinates uniformly; a float draws each of them from
    Zipf(inner_s) over one global random permutation per mode, so hot rows are shared by all slices.
    Nonzeros are returned in a random order (COO has no order).
    """
    n0 = dims[0]
    sizes = zipf_slice_sizes(nnz, n0, slice_s, rng)
    rest_dims = list(dims[1:])
    if inner_s is None:
        def draw(sl, g):
            return [g.integers(0, d, size=sl.size, dtype=np.int64) for d in rest_dims]
    else:
        cdfs = [_zipf_cdf(d, inner_s) for d in rest_dims]
        perms = [rng.permutation(d) for d in rest_dims]

        def draw(sl, g):
            out = []
            for cdf, perm in zip(cdfs, perms):
                r = np.searchsorted(cdf, g.random(sl.size), side="left")
                np.minimum(r, len(perm) - 1, out=r)
                out.append(perm[r])
            return out
    keys = _unique_fill(sizes, rest_dims, draw, rng)
    coords = _unpack(keys, dims)
    shuffle = rng.permutation(keys.size)
    coords = [np.ascontiguousarray(c[shuffle]) for c in coords]
    if value == "pm1":          # U[-1, 1]
        vals = 2.0 * rng.random(keys.size) - 1.0
    elif value == "unit":       # U(0, 1]
        vals = 1.0 - rng.random(keys.size)
    elif value == "normal":
        vals = rng.standard_normal(keys.size)
    else:
        raise ValueError(value)
    return SparseOperand(coords, vals.astype(dtype), tuple(int(d) for d in dims))


def _factor(rows: int, rank: int, rng: np.random.Generator, dtype) -> np.ndarray:
    return np.ascontiguousarray(rng.standard_normal((rows, rank)).astype(dtype))


# --------------------------------------------------------------------------------------
# workload families
# --------------------------------------------------------------------------------------

def ttmc3_workload(dims, nnz, rank, *, slice_s=None, inner_s=None, value="pm1", seed=0, config_id=1,
                   name="ttmc3") -> Workload:
    """Y[i,a,b] = sum_{j,k} X[i,j,k] U[j,a] V[k,b]  (Sec. 5.3, first TTMc), fused i->j->k with t[b] per (i,j)."""
    g = _rng(seed, config_id, 0)
    if slice_s is None:
        X = _uniform_tensor(dims, nnz, g, value, np.float32)
    else:
        X = _skewed_tensor(dims, nnz, slice_s, inner_s, g, value, np.float32)
    r2, r3 = (rank, rank) if np.isscalar(rank) else rank
    U = _factor(dims[1], r2, _rng(seed, config_id, 1), np.float32)
    V = _factor(dims[2], r3, _rng(seed, config_id, 2), np.float32)
    return Workload(
        name=name, family="ttmc3", dtype=np.dtype(np.float32),
        extents={"i": dims[0], "j": dims[1], "k": dims[2], "a": r2, "b": r3},
        sparse={"X": X}, dense={"U": U, "V": V},
        expression="Y[i,a,b] = X[i,j,k] * U[j,a] * V[k,b]",
        tree=["T[i,j,b] = X[i,j,k] * V[k,b]", "Y[i,a,b] = T[i,j,b] * U[j,a]"],
        mode_orders={"X": (0, 1, 2)}, loop_orders=["ijkb", "ijab"],
        out_shape=(dims[0], r2, r3))


def ttmc4_workload(dims, nnz, rank, *, slice_s=None, value="pm1", seed=0, config_id=3,
                   name="ttmc4") -> Workload:
    """Y[i,a,b,c] = sum_{j,k,l} X[i,j,k,l] U[j,a] V[k,b] W[l,c]; intermediates of order 1 and 2."""
    g = _rng(seed, config_id, 0)
    if slice_s is None:
        X = _uniform_tensor(dims, nnz, g, value, np.float32)
    else:
        X = _skewed_tensor(dims, nnz, slice_s, None, g, value, np.float32)
    U = _factor(dims[1], rank, _rng(seed, config_id, 1), np.float32)
    V = _factor(dims[2], rank, _rng(seed, config_id, 2), np.float32)
    W = _factor(dims[3], rank, _rng(seed, config_id, 3), np.float32)
    return Workload(
        name=name, family="ttmc4", dtype=np.dtype(np.float32),
        extents={"i": dims[0], "j": dims[1], "k": dims[2], "l": dims[3], "a": rank, "b": rank, "c": rank},
        sparse={"X": X}, dense={"U": U, "V": V, "W": W},
        expression="Y[i,a,b,c] = X[i,j,k,l] * U[j,a] * V[k,b] * W[l,c]",
        tree=["P[i,j,k,c] = X[i,j,k,l] * W[l,c]",
              "Q[i,j,b,c] = P[i,j,k,c] * V[k,b]",
              "Y[i,a,b,c] = Q[i,j,b,c] * U[j,a]"],
        mode_orders={"X": (0, 1, 2, 3)}, loop_orders=["ijklc", "ijkbc", "ijabc"],
        out_shape=(dims[0], rank, rank, rank))


def mttkrp_workload(dims, nnz, rank, *, slice_s=None, value="unit", seed=0, config_id=4,
                    name="mttkrp") -> Workload:
    """A[i,r] = sum_{j,k} X[i,j,k] B[j,r] C[k,r]  (Sec. 5.2, first MTTKRP); r is a batch index of the 2nd contraction."""
    g = _rng(seed, config_id, 0)
    if slice_s is None:
        X = _uniform_tensor(dims, nnz, g, value, np.float32)
    else:
        X = _skewed_tensor(dims, nnz, slice_s, None, g, value, np.float32)
    B = _factor(dims[1], rank, _rng(seed, config_id, 1), np.float32)
    C = _factor(dims[2], rank, _rng(seed, config_id, 2), np.float32)
    return Workload(
        name=name, family="mttkrp", dtype=np.dtype(np.float32),
        extents={"i": dims[0], "j": dims[1], "k": dims[2], "r": rank},
        sparse={"X": X}, dense={"B": B, "C": C},
        expression="A[i,r] = X[i,j,k] * B[j,r] * C[k,r]",
        tree=["T[i,j,r] = X[i,j,k] * C[k,r]", "A[i,r] = T[i,j,r] * B[j,r]"],
        mode_orders={"X": (0, 1, 2)}, loop_orders=["ijkr", "ijr"],
        out_shape=(dims[0], rank))


def _uniform_tensor(dims, nnz, rng, value, dtype) -> SparseOperand:
    """nnz distinct coordinates drawn uniformly from the whole index space."""
    total_cells = 1
    for d in dims:
        total_cells *= int(d)
    if nnz > total_cells:
        raise ValueError("more nonzeros than cells")
    bits = [_bits(d) for d in dims]
    have = np.empty(0, dtype=np.uint64)
    while have.size < nnz:
        m = int((nnz - have.size) * 1.1) + 16
        key = np.zeros(m, dtype=np.uint64)
        for d, b in zip(dims, bits):
            key = (key << np.uint64(b)) | rng.integers(0, d, size=m, dtype=np.int64).astype(np.uint64)
        uniq, first = np.unique(key, return_index=True)
        if have.size:
            fresh = ~np.isin(uniq, have)
            uniq, first = uniq[fresh], first[fresh]
        uniq = uniq[np.argsort(first, kind="stable")][: nnz - have.size]
        have = np.concatenate([have, uniq])
    coords = []
    k = have.copy()
    for b in reversed(bits):
        coords.append((k & np.uint64((1 << b) - 1)).astype(np.int32))
        k >>= np.uint64(b)
    coords = coords[::-1]
    if value == "pm1":
        vals = 2.0 * rng.random(nnz) - 1.0
    elif value == "unit":
        vals = 1.0 - rng.random(nnz)
    else:
        vals = rng.standard_normal(nnz)
    return SparseOperand([np.ascontiguousarray(c) for c in coords], vals.astype(dtype),
                         tuple(int(d) for d in dims))


def _banded(n_a: int, n_b: int, n_k: int, band: int, keep: float, rng) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """All (a, b, k) with |a-b| < band, each kept independently with probability `keep`."""
    a = np.repeat(np.arange(n_a, dtype=np.int64), n_b)
    b = np.tile(np.arange(n_b, dtype=np.int64), n_a)
    near = np.abs(a - b) < band
    a, b = a[near], b[near]
    mask = rng.random((a.size, n_k)) < keep
    pair, k = np.nonzero(mask)
    return a[pair].astype(np.int32), b[pair].astype(np.int32), k.astype(np.int32)


def network_workload(n=1024, n_k=128, band=32, keep=0.25, *, seed=0, config_id=5,
                     name="network") -> Workload:
    """Z[i,m] = sum_{j,k,l} U[i,j,k] V[j,l] W[k,l,m]  (intro example), fused over i with T_i[k,l] dense."""
    gu, gv, gw = _rng(seed, config_id, 0), _rng(seed, config_id, 1), _rng(seed, config_id, 2)
    ui, uj, uk = _banded(n, n, n_k, band, keep, gu)
    uvals = gu.standard_normal(ui.size)
    pu = gu.permutation(ui.size)
    U = SparseOperand([ui[pu], uj[pu], uk[pu]], uvals[pu].astype(np.float64), (n, n, n_k))
    V = np.ascontiguousarray(gv.standard_normal((n, n)))
    wl, wm, wk = _banded(n, n, n_k, band, keep, gw)
    wvals = gw.standard_normal(wl.size)
    pw = gw.permutation(wl.size)
    W = SparseOperand([wk[pw], wl[pw], wm[pw]], wvals[pw].astype(np.float64), (n_k, n, n))
    return Workload(
        name=name, family="network", dtype=np.dtype(np.float64),
        extents={"i": n, "j": n, "k": n_k, "l": n, "m": n},
        sparse={"U": U, "W": W}, dense={"V": V},
        expression="Z[i,m] = U[i,j,k] * V[j,l] * W[k,l,m]",
        tree=["T[i,k,l] = U[i,j,k] * V[j,l]", "Z[i,m] = T[i,k,l] * W[k,l,m]"],
        mode_orders={"U": (0, 2, 1), "W": (1, 2, 0)}, loop_orders=["ikjl", "ilmk"],
        out_shape=(n, n))


# --------------------------------------------------------------------------------------
# the five named configurations
# --------------------------------------------------------------------------------------

CONFIG_NAMES = {
    1: "ttmc3_small_200x200x200_nnz20k_r8",
    2: "ttmc3_skewed_12000x9000x29000_nnz77M_r16",
    3: "ttmc4_20000^4_nnz50M_r8",
    4: "mttkrp3_50000^3_nnz100M_r32",
    5: "network_fp64_1024_k128_band32",
}


def make_config(config_id: int, scale: float = 1.0, seed: int = 0) -> Workload:
    """The five benchmark configurations; scale < 1 shrinks the nonzero count (and, for the
    network, the extents) while keeping the distribution, for cases a CPU can check in full."""
    if config_id == 1:
        return ttmc3_workload((200, 200, 200), 20_000, 8, value="pm1", seed=seed, config_id=1,
                              name=CONFIG_NAMES[1])
    if config_id == 2:
        nnz = max(12_000, int(77_000_000 * scale))
        return ttmc3_workload((12_000, 9_000, 29_000), nnz, 16, slice_s=1.1, inner_s=0.9, value="unit",
                              seed=seed, config_id=2, name=CONFIG_NAMES[2])
    if config_id == 3:
        nnz = max(20_000, int(50_000_000 * scale))
        return ttmc4_workload((20_000,) * 4, nnz, 8, slice_s=1.0, value="pm1", seed=seed, config_id=3,
                              name=CONFIG_NAMES[3])
    if config_id == 4:
        nnz = max(50_000, int(100_000_000 * scale))
        return mttkrp_workload((50_000,) * 3, nnz, 32, slice_s=1.2, value="unit", seed=seed, config_id=4,
                               name=CONFIG_NAMES[4])
    if config_id == 5:
        if scale >= 1.0:
            return network_workload(1024, 128, 32, 0.25, seed=seed, config_id=5, name=CONFIG_NAMES[5])
        n = max(64, int(1024 * scale) // 8 * 8)
        return network_workload(n, max(8, int(128 * scale)), max(4, int(32 * scale)), 0.25, seed=seed,
                                config_id=5, name=CONFIG_NAMES[5] + f"_scale{scale}")
    raise ValueError(f"unknown config {config_id}")


def row_sample(op: SparseOperand, rows: np.ndarray, mode: int = 0) -> SparseOperand:
    """The nonzeros of `op` whose coordinate along `mode` lies in `rows` (pure filtering)."""
    sel = np.isin(op.coords[mode], np.asarray(rows))
    return SparseOperand([np.ascontiguousarray(c[sel]) for c in op.coords],
                         np.ascontiguousarray(op.vals[sel]), op.dims)

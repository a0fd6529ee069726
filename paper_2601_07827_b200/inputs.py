"""Seeded synthetic inputs for the contraction workloads.

This module only *creates tensors*: it holds none of the contraction's arithmetic and is the one
piece of code that both the GPU tests/benchmark and the CPU checker read.  Values come from a
counter-based generator (SplitMix64 finaliser applied to key + counter), so an element's value
depends only on (seed, logical index, component) and never on the memory layout: permuting a
tensor's strides regenerates the same logical tensor.

The workloads are synthetic stand-ins for the application shapes the paper names (coupled-cluster
ladder terms, tensor-network contractions, batched and complex contractions); no external data
set is involved.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Sequence, Tuple

import torch

_MASK64 = (1 << 64) - 1
_GAMMA = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB


def _s64(x: int) -> int:
    """Two's-complement view of an unsigned 64-bit constant (torch has no uint64 arithmetic)."""
    x &= _MASK64
    return x - (1 << 64) if x >> 63 else x


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right on int64 tensors."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def splitmix64(x: torch.Tensor) -> torch.Tensor:
    """SplitMix64 output function (Steele, Lea, Flood 2014) on wrapped int64 lanes."""
    z = x + _s64(_GAMMA)
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


def splitmix64_int(x: int) -> int:
    """The same function on Python integers (used to pin the tensor version)."""
    z = (x + _GAMMA) & _MASK64
    z = ((z ^ (z >> 30)) * _M1) & _MASK64
    z = ((z ^ (z >> 27)) * _M2) & _MASK64
    return z ^ (z >> 31)


def _unit(h: torch.Tensor) -> torch.Tensor:
    """53 high bits -> double in [0, 1)."""
    return _lsr(h, 11).to(torch.float64) * (2.0 ** -53)


def draw(seed: int, index: torch.Tensor, component: int, dist: str, scale: float) -> torch.Tensor:
    """float64 values for the given logical linear indices.

    dist = "uniform": scale * (2u - 1); dist = "normal": scale * Box-Muller(u1, u2);
    dist = "smallint": integers in [-scale, scale] (exactly representable, for bit-exact tests).
    """
    key = splitmix64_int((seed * 0x100000001B3 + 0x7F4A7C15) & _MASK64)
    ctr = index * 4 + (2 * component)
    h0 = splitmix64(ctr + _s64(key))
    if dist == "uniform":
        return (2.0 * _unit(h0) - 1.0) * scale
    if dist == "smallint":
        span = 2 * int(scale) + 1
        return (torch.floor(_unit(h0) * span) - int(scale)).clamp_(-int(scale), int(scale))
    if dist == "normal":
        h1 = splitmix64(ctr + 1 + _s64(key))
        u1 = 1.0 - _unit(h0)  # (0, 1]
        u2 = _unit(h1)
        return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2) * scale
    raise ValueError(dist)


DTYPES = {
    "f32": torch.float32,
    "f64": torch.float64,
    "c32": torch.complex64,   # two 32-bit parts
    "c64": torch.complex128,  # two 64-bit parts
}


def col_major_strides(extents: Sequence[int]) -> List[int]:
    s, out = 1, []
    for e in extents:
        out.append(s)
        s *= e
    return out


def span_elements(extents: Sequence[int], strides: Sequence[int]) -> Tuple[int, int]:
    """(lowest, highest) element offset a non-empty strided tensor touches."""
    lo = hi = 0
    for e, s in zip(extents, strides):
        if s < 0:
            lo += s * (e - 1)
        else:
            hi += s * (e - 1)
    return lo, hi


def logical_values(seed: int, extents: Sequence[int], dtype: torch.dtype, dist: str, scale: float,
                   device="cpu", canonical=None, chunk: int = 1 << 24) -> torch.Tensor:
    """Flat tensor of the logical values in column-major order over `extents`.

    `canonical(index) -> index` may fold indices onto representatives (imposes symmetries).
    """
    n = 1
    for e in extents:
        n *= e
    out = torch.empty(n, dtype=dtype, device=device)
    cplx = dtype.is_complex
    real_view = torch.view_as_real(out) if cplx else None
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        idx = torch.arange(lo, hi, dtype=torch.int64, device=device)
        if canonical is not None:
            idx = canonical(idx)
        if cplx:
            real_view[lo:hi, 0] = draw(seed, idx, 0, dist, scale).to(real_view.dtype)
            real_view[lo:hi, 1] = draw(seed, idx, 1, dist, scale).to(real_view.dtype)
        else:
            out[lo:hi] = draw(seed, idx, 0, dist, scale).to(dtype)
    return out


@dataclasses.dataclass
class StridedTensor:
    """A logical tensor placed in a flat buffer: element (i0, i1, ...) sits at
    buffer[origin + sum_k i_k * strides[k]]."""
    buffer: torch.Tensor          # 1-D storage, includes padding
    extents: Tuple[int, ...]
    strides: Tuple[int, ...]      # in elements, signed
    origin: int                   # element offset of logical (0,...,0) inside `buffer`

    @property
    def dtype(self):
        return self.buffer.dtype

    def data_ptr(self) -> int:
        return self.buffer.data_ptr() + self.origin * self.buffer.element_size()

    def numel(self) -> int:
        n = 1
        for e in self.extents:
            n *= e
        return n

    def offsets(self) -> torch.Tensor:
        """Buffer positions of all elements, flat, column-major over the extents."""
        dev = self.buffer.device
        off = torch.full((1,), self.origin, dtype=torch.int64, device=dev)
        for e, s in zip(self.extents, self.strides):
            step = torch.arange(e, dtype=torch.int64, device=dev) * s
            off = (off.view(1, -1) + step.view(-1, 1)).reshape(-1)
        return off

    def is_dense_col_major(self) -> bool:
        return self.origin == 0 and list(self.strides) == col_major_strides(self.extents)

    def set_logical(self, flat: torch.Tensor) -> None:
        """Store values given flat in column-major logical order."""
        if self.is_dense_col_major():
            self.buffer[: flat.numel()].copy_(flat)
        else:
            self.buffer[self.offsets()] = flat.to(self.buffer.device)

    def get_logical(self) -> torch.Tensor:
        """Values flat in column-major logical order (a copy)."""
        if self.is_dense_col_major():
            return self.buffer[: self.numel()].clone()
        return self.buffer[self.offsets()]

    def to(self, device) -> "StridedTensor":
        return StridedTensor(self.buffer.to(device), self.extents, self.strides, self.origin)

    def clone(self) -> "StridedTensor":
        return StridedTensor(self.buffer.clone(), self.extents, self.strides, self.origin)

    def numpy(self):
        """numpy view with the same extents and strides (CPU tensors only)."""
        import numpy as np
        base = self.buffer.numpy()
        item = base.itemsize
        return np.lib.stride_tricks.as_strided(
            base[self.origin:], shape=self.extents,
            strides=tuple(s * item for s in self.strides), writeable=True)


CANARY = float("nan")


def place(flat: Optional[torch.Tensor], extents: Sequence[int], strides: Optional[Sequence[int]],
          dtype: torch.dtype, device="cpu", fill=CANARY) -> StridedTensor:
    """Allocate storage for the layout (padding pre-filled with `fill`) and store `flat` in it."""
    extents = tuple(int(e) for e in extents)
    strides = tuple(col_major_strides(extents)) if strides is None else tuple(int(s) for s in strides)
    lo, hi = span_elements(extents, strides)
    buf = torch.full((hi - lo + 1,), fill, dtype=dtype, device=device)
    t = StridedTensor(buf, extents, strides, -lo)
    if flat is not None:
        t.set_logical(flat)
    return t


@dataclasses.dataclass
class Workload:
    name: str
    dtype: str
    labelsA: str
    labelsB: str
    labelsD: str
    extents: Dict[str, int]
    alpha: complex = 1.0
    beta: complex = 0.0
    conjA: bool = False
    conjB: bool = False
    conjC: bool = False
    in_place: bool = False                      # C and D are the same buffer
    stridesA: Optional[Tuple[int, ...]] = None  # None = dense column-major in label order
    stridesB: Optional[Tuple[int, ...]] = None
    stridesD: Optional[Tuple[int, ...]] = None
    distA: Tuple[str, float] = ("uniform", 1.0)
    distB: Tuple[str, float] = ("uniform", 1.0)
    distC: Tuple[str, float] = ("uniform", 1.0)
    seed: int = 0
    symmetryA: Optional[str] = None             # "pair_swap": A[a,b,c,d] = A[b,a,d,c]

    def ext(self, labels: str) -> Tuple[int, ...]:
        return tuple(self.extents[l] for l in labels)

    def groups(self):
        """(batch, M, N, K) sizes: products of the extents of each label class."""
        a, b, d = set(self.labelsA), set(self.labelsB), set(self.labelsD)
        size = lambda ls: math.prod(self.extents[l] for l in ls)
        return size(a & b & d), size((a & d) - b), size((b & d) - a), size((a & b) - d)

    def flops(self) -> float:
        h, m, n, k = self.groups()
        return (8.0 if self.dtype in ("c32", "c64") else 2.0) * h * m * n * k

    def algorithmic_bytes(self) -> float:
        """A and B read once, C read once when beta != 0, D written once."""
        item = {"f32": 4, "f64": 8, "c32": 8, "c64": 16}[self.dtype]
        size = lambda ls: math.prod(self.extents[l] for l in ls)
        n = size(self.labelsA) + size(self.labelsB) + size(self.labelsD)
        if self.beta != 0:
            n += size(self.labelsD)
        return float(n * item)


def _pair_swap_canonical(extents):
    e0, e1, e2, e3 = extents

    def canon(idx):
        a = idx % e0
        b = (idx // e0) % e1
        c = (idx // (e0 * e1)) % e2
        d = idx // (e0 * e1 * e2)
        partner = b + e0 * (a + e1 * (d + e2 * c))
        return torch.minimum(idx, partner)
    return canon


def make_workload_tensors(w: Workload, device="cpu"):
    """(A, B, C, D) as StridedTensor; C is None when beta == 0, C is D when w.in_place.

    D starts as canary NaNs (or, in place, as the seeded C values)."""
    dt = DTYPES[w.dtype]
    eA, eB, eD = w.ext(w.labelsA), w.ext(w.labelsB), w.ext(w.labelsD)
    canon = None
    if w.symmetryA == "pair_swap":
        assert eA[0] == eA[1] and eA[2] == eA[3]
        canon = _pair_swap_canonical(eA)
    A = place(logical_values(w.seed + 1, eA, dt, *w.distA, device=device, canonical=canon),
              eA, w.stridesA, dt, device)
    B = place(logical_values(w.seed + 2, eB, dt, *w.distB, device=device), eB, w.stridesB, dt, device)
    C = None
    if w.beta != 0:
        C = place(logical_values(w.seed + 3, eD, dt, *w.distC, device=device), eD, w.stridesD, dt, device)
    if w.in_place:
        assert C is not None
        D = C
    else:
        D = place(None, eD, w.stridesD, dt, device)
    return A, B, C, D


def _all(extent, labels):
    return {l: extent for l in labels}


def workloads() -> Dict[str, Workload]:
    """The five fixed workloads (1-based names follow their order)."""
    w = {}
    # 1: small fp64 contraction with interleaved free / contracted modes; oracle runs it in seconds
    w["cfg1_f64_small"] = Workload(
        "cfg1_f64_small", "f64", "acid", "dbcj", "abij", _all(16, "abcdij"),
        alpha=1.0, beta=0.5, seed=1000)
    # 2: coupled-cluster ladder term R[a,b,i,j] += sum_cd V[a,b,c,d] T[c,d,i,j]
    w["cfg2_f64_ccsd_ladder"] = Workload(
        "cfg2_f64_ccsd_ladder", "f64", "abcd", "cdij", "abij",
        {**_all(128, "abcd"), **_all(32, "ij")},
        alpha=1.0, beta=1.0, in_place=True, seed=2000,
        distA=("normal", 0.1), distB=("uniform", 0.01), distC=("uniform", 0.01),
        symmetryA="pair_swap")
    # 2p: the same ladder term with c,d = 64 (0.5 GiB of V): the case profiler captures use
    w["cfg2p_f64_ccsd_ladder_profile"] = dataclasses.replace(
        w["cfg2_f64_ccsd_ladder"], name="cfg2p_f64_ccsd_ladder_profile",
        extents={**_all(128, "ab"), **_all(64, "cd"), **_all(32, "ij")})
    # 3: fp32, batch label z, permuted output with a padded leading stride
    e3 = {"z": 64, "a": 96, "b": 96, "j": 96, "k": 24, "l": 24}
    w["cfg3_f32_batched_permuted"] = Workload(
        "cfg3_f32_batched_permuted", "f32", "akzl", "lbkjz", "jbza", e3,
        alpha=1.0, beta=0.0, seed=3000, distA=("normal", 1.0), distB=("normal", 1.0),
        stridesD=(1, 104, 104 * 96, 104 * 96 * 64))
    # 3p: workload 3 with 16 batch entries (0.4 GB on the device): the case profiler captures use
    w["cfg3p_f32_batched_permuted_profile"] = dataclasses.replace(
        w["cfg3_f32_batched_permuted"], name="cfg3p_f32_batched_permuted_profile", extents={**e3, "z": 16},
        stridesD=(1, 104, 104 * 96, 104 * 96 * 16))
    # 4: complex128 with conj(A) and complex alpha
    e4 = {"p": 256, "q": 256, "r": 64, "s": 48, "t": 48}
    w["cfg4_c64_conj"] = Workload(
        "cfg4_c64_conj", "c64", "spt", "tqsr", "pqr", e4,
        alpha=complex(0.5, -0.25), beta=0.0, conjA=True, seed=4000)
    # 4c: the same contraction in complex64 (the element type the five fixed workloads leave out)
    w["cfg4c_c32_conj"] = dataclasses.replace(w["cfg4_c64_conj"], name="cfg4c_c32_conj", dtype="c32", seed=4500)
    # 5: memory-bound tensor-network case, rank-8 inputs of extent 4, rank-10 output
    w["cfg5_f32_tensor_network"] = Workload(
        "cfg5_f32_tensor_network", "f32", "axbycwde", "wfygxhij", "afbgchdiej",
        _all(4, "abcdefghijxyw"), alpha=1.0, beta=0.0, seed=5000)
    # 5b: same with D's fastest label being B's slowest (adversarial output order)
    w["cfg5b_f32_tensor_network_rev"] = dataclasses.replace(
        w["cfg5_f32_tensor_network"], name="cfg5b_f32_tensor_network_rev", labelsD="jeidhcgbfa")
    # 7: outer product with interleaved output labels (no contracted label): 1 GiB of D from two 64 KiB inputs
    w["cfg7_f32_outer_product"] = Workload(
        "cfg7_f32_outer_product", "f32", "ab", "cd", "acbd", _all(128, "abcd"), alpha=1.0, beta=0.0, seed=7000)
    # 6: Case 4, the ladder term with an extra label x that only A carries (summed over first):
    #    D[a,b,i,j] = sum_cd (sum_x A[a,b,c,d,x]) T[c,d,i,j];  A is 1 GiB, the sum over x is HBM-bound
    e6 = {**_all(64, "abcd"), **_all(32, "ij"), "x": 8}
    w["cfg6_f64_case4_isolated"] = Workload(
        "cfg6_f64_case4_isolated", "f64", "abcdx", "cdij", "abij", e6, alpha=1.0, beta=0.0, seed=6000,
        distA=("normal", 0.1), distB=("uniform", 0.01))
    # 6b: the isolated label is A's fastest one (one warp per summed element)
    w["cfg6b_f64_case4_isolated_fast"] = dataclasses.replace(
        w["cfg6_f64_case4_isolated"], name="cfg6b_f64_case4_isolated_fast", labelsA="xabcd",
        extents={**e6, "x": 32, **_all(32, "ab")})
    return w


@dataclasses.dataclass(frozen=True)
class ElementwiseWorkload:
    """C[labelsC] := alpha * op(A[labelsA]) + beta * op(B[labelsC]) with dense column-major tensors."""
    name: str
    dtype: str
    labelsA: str
    labelsC: str
    extents: Dict[str, int]
    alpha: complex = 1.0
    beta: complex = 0.0          # != 0: B is present
    seed: int = 0

    def ext(self, labels: str) -> Tuple[int, ...]:
        return tuple(self.extents[l] for l in labels)

    def algorithmic_bytes(self) -> float:
        """A read once, B read once when beta != 0, C written once."""
        item = {"f32": 4, "f64": 8, "c32": 8, "c64": 16}[self.dtype]
        size = lambda ls: math.prod(self.extents[l] for l in ls)
        return float(item * (size(set(self.labelsA)) + size(self.labelsC) * (2 if self.beta != 0 else 1)))


def elementwise_workloads() -> Dict[str, ElementwiseWorkload]:
    """Bandwidth-bound cases of the binary / unary operation, each about 1-2 GB of traffic."""
    w = {}
    # full reversal of a rank-4 tensor: input and output contiguous along different labels
    w["ew1_f32_permute_reverse"] = ElementwiseWorkload(
        "ew1_f32_permute_reverse", "f32", "abcd", "dcba", {"a": 256, "b": 64, "c": 64, "d": 256}, seed=7100)
    # the fast label stays, the others rotate (no transposition needed)
    w["ew2_f64_permute_keep_fast"] = ElementwiseWorkload(
        "ew2_f64_permute_keep_fast", "f64", "abcd", "acdb", {"a": 128, "b": 64, "c": 128, "d": 128}, seed=7200)
    # C = alpha A + beta B, same layout
    w["ew3_f64_axpby"] = ElementwiseWorkload(
        "ew3_f64_axpby", "f64", "ab", "ab", {"a": 8192, "b": 8192}, alpha=0.75, beta=-0.5, seed=7300)
    # reduction over a slow label with a transposition: C[j,i] = sum_x A[i,x,j]
    w["ew4_f32_reduce_transpose"] = ElementwiseWorkload(
        "ew4_f32_reduce_transpose", "f32", "ixj", "ji", {"i": 4096, "x": 16, "j": 4096}, seed=7400)
    return w


def make_elementwise_tensors(w: ElementwiseWorkload, device="cpu"):
    """(A, B, C) as StridedTensor; B is None when beta == 0; C starts as canary NaNs."""
    dt = DTYPES[w.dtype]
    eA, eC = w.ext(w.labelsA), w.ext(w.labelsC)
    A = place(logical_values(w.seed + 1, eA, dt, "uniform", 1.0, device=device), eA, None, dt, device)
    B = place(logical_values(w.seed + 2, eC, dt, "uniform", 1.0, device=device), eC, None, dt, device) if w.beta != 0 else None
    C = place(None, eC, None, dt, device)
    return A, B, C


def scaled_down(w: Workload, factors: Dict[str, int], name: Optional[str] = None) -> Workload:
    """Same structure with some extents replaced (parity cases the oracle finishes quickly).
    Explicit strides are rebuilt as column-major with the same relative padding on mode 0."""
    ext = {**w.extents, **factors}
    out = dataclasses.replace(w, name=name or (w.name + "_small"), extents=ext)
    if w.stridesD is not None:
        eD = out.ext(out.labelsD)
        pad = w.stridesD[1] - w.extents[w.labelsD[0]]
        lead = eD[0] + pad
        s, strides = 1, []
        for i, e in enumerate(eD):
            strides.append(s)
            s *= lead if i == 0 else e
        out = dataclasses.replace(out, stridesD=tuple(strides))
    return out


def random_contraction(seed: int, max_work: int = 1 << 21):
    """A seeded random contraction in the spirit of a randomized benchmark set: 0-1 batch labels,
    0-3 free labels per input, 0-3 contracted labels, extents from a mixed list, every tensor in its
    own random memory order with padding on one mode, negative strides on some modes of A and B.
    Returns (labelsA, labelsB, labelsD, extents, stridesA, stridesB, stridesD); no arithmetic of the
    method happens here."""
    import numpy as np
    rng = np.random.default_rng(seed)
    pool = [1, 2, 3, 4, 5, 7, 8, 12, 16, 24, 33]
    while True:
        counts = [int(rng.integers(0, 2)), int(rng.integers(0, 4)), int(rng.integers(0, 4)), int(rng.integers(0, 4))]
        if counts[0] + counts[1] + counts[3] > 8 or counts[0] + counts[2] + counts[3] > 8:
            continue
        names = iter("abcdefghijklmnopqrstuvwxyz")
        groups = [[next(names) for _ in range(c)] for c in counts]          # H, M, N, K
        extents = {l: int(rng.choice(pool)) for g in groups for l in g}
        work = math.prod(extents.values()) if extents else 1
        if work <= max_work:
            break
    H, M, N, K = groups

    def shuffled(ls):
        ls = list(ls)
        rng.shuffle(ls)
        return "".join(ls)
    la, lb, ld = shuffled(H + M + K), shuffled(H + N + K), shuffled(H + M + N)

    def strides_for(labels, allow_negative):
        order = list(range(len(labels)))
        rng.shuffle(order)                                   # memory order: order[0] is the fastest mode
        st, run = [0] * len(labels), 1
        padded = int(rng.integers(0, len(labels))) if labels else -1
        for pos, mode in enumerate(order):
            st[mode] = run
            run *= extents[labels[mode]] + (int(rng.integers(0, 4)) if pos == padded else 0)
        if allow_negative:
            st = [-x if rng.random() < 0.25 else x for x in st]
        return tuple(st)
    return la, lb, ld, extents, strides_for(la, True), strides_for(lb, True), strides_for(ld, False)

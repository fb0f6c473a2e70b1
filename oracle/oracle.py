"""ctypes front end of the fp64 CPU oracle (``rtprune_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's CPU-baseline
leg, never by the product package.  It marshals numpy arrays into the C functions and strings the
per-image driver (Algorithm 1) over a ragged batch.  No arithmetic of the method lives here except
the final rounding of the merged features to the output dtype, which is a library cast.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rtprune_oracle.c")
_LIB = os.path.join(_HERE, "librtprune_oracle.so")

_c_double_p = ctypes.POINTER(ctypes.c_double)
_c_int32_p = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no fast-math) if the library is missing or stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.rtp_oracle_phi.restype = ctypes.c_double
        _lib.rtp_oracle_image.restype = ctypes.c_int
    return _lib


def _dp(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_c_double_p)


def _ip(a: np.ndarray):
    return a.ctypes.data_as(_c_int32_p)


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


# ----------------------------------------------------------------------------------------------
# step functions (one per passage of the paper)
# ----------------------------------------------------------------------------------------------
def norms(T) -> np.ndarray:
    """Eq. 1."""
    T = _f64(T)
    C = np.empty(T.shape[0], dtype=np.float64)
    lib().rtp_oracle_norms(_dp(T), ctypes.c_int(T.shape[0]), ctypes.c_int(T.shape[1]), _dp(C))
    return C


def variance(T) -> np.ndarray:
    """Selection-metric ablation: population variance of each token over its D features."""
    T = _f64(T)
    C = np.empty(T.shape[0])
    lib().rtp_oracle_variance(_dp(T), ctypes.c_int(T.shape[0]), ctypes.c_int(T.shape[1]), _dp(C))
    return C


def entropy(T) -> np.ndarray:
    """Selection-metric ablation: entropy of the softmax of each token's features (a reading: the
    paper names the metric without a formula)."""
    T = _f64(T)
    C = np.empty(T.shape[0])
    lib().rtp_oracle_entropy(_dp(T), ctypes.c_int(T.shape[0]), ctypes.c_int(T.shape[1]), _dp(C))
    return C


def criterion(T, which: int) -> np.ndarray:
    return (norms, variance, entropy)[which](T)


def phi(T, C=None) -> float:
    """Eq. 8, by the i<j double loop."""
    T = _f64(T)
    C = norms(T) if C is None else _f64(C)
    return float(lib().rtp_oracle_phi(_dp(T), _dp(C), ctypes.c_int(T.shape[0]),
                                      ctypes.c_int(T.shape[1])))


def ratio(phi_value: float, rho: float, N: int, *, dynamic: bool, r_fixed: float = 0.25,
          phi_lo: float = 0.0, phi_hi: float = 1.0, r_max: float = 1.0):
    """Eq. 10 and M = N (1 - r).  Returns (r, B, M)."""
    r = ctypes.c_double()
    B = ctypes.c_int()
    M = ctypes.c_int()
    lib().rtp_oracle_ratio(ctypes.c_double(phi_value), ctypes.c_double(rho),
                           ctypes.c_int(int(dynamic)), ctypes.c_double(r_fixed),
                           ctypes.c_double(phi_lo), ctypes.c_double(phi_hi),
                           ctypes.c_double(r_max), ctypes.c_int(N), ctypes.byref(r),
                           ctypes.byref(B), ctypes.byref(M))
    return r.value, B.value, M.value


def select(C, M: int):
    """Stage 1: (kept, prop), image-local indices, ascending."""
    C = _f64(C)
    N = C.shape[0]
    kept = np.empty(max(N, 1), dtype=np.int32)
    prop = np.empty(max(N, 1), dtype=np.int32)
    lib().rtp_oracle_select(_dp(C), ctypes.c_int(N), ctypes.c_int(M), _ip(kept), _ip(prop))
    return kept[:M].copy(), prop[:N - M].copy()


def scores(T, C, kept, prop) -> np.ndarray:
    """Cosine score matrix S [M x B]."""
    T = _f64(T)
    C = _f64(C)
    kept = np.ascontiguousarray(kept, dtype=np.int32)
    prop = np.ascontiguousarray(prop, dtype=np.int32)
    S = np.empty((len(kept), len(prop)), dtype=np.float64)
    lib().rtp_oracle_scores(_dp(T), _dp(C), ctypes.c_int(T.shape[1]), _ip(kept),
                            ctypes.c_int(len(kept)), _ip(prop), ctypes.c_int(len(prop)), _dp(S))
    return S


def sinkhorn(S, *, z: float = 0.2, eps: float = 1.0, iters: int = 100):
    """Eq. 5 + Appendix C.  Returns (u [M+1], v [B+1], Pbar [(M+1) x (B+1)])."""
    S = _f64(S)
    M, B = S.shape
    u = np.empty(M + 1)
    v = np.empty(B + 1)
    Pbar = np.empty((M + 1, B + 1))
    lib().rtp_oracle_sinkhorn(_dp(S), ctypes.c_int(M), ctypes.c_int(B), ctypes.c_double(z),
                              ctypes.c_double(eps), ctypes.c_int(iters), _dp(u), _dp(v), _dp(Pbar))
    return u, v, Pbar


def exact_matching(S, *, z: float = 0.2):
    """Eq. 2-6 solved exactly: the maximum-weight partial matching with gains S_ij - z.
    Returns (match_prop [B] kept position or -1, objective, dual_kept [M], dual_prop [B])."""
    S = _f64(S)
    M, B = S.shape
    match = np.empty(max(B, 1), dtype=np.int32)
    obj = ctypes.c_double()
    du = np.empty(max(M, 1))
    dv = np.empty(max(B, 1))
    lib().rtp_oracle_exact_matching(_dp(S), ctypes.c_int(M), ctypes.c_int(B), ctypes.c_double(z), _ip(match),
                                    ctypes.byref(obj), _dp(du), _dp(dv))
    return match[:B].copy(), obj.value, du[:M].copy(), dv[:B].copy()


def matching_plan(match_prop, M: int) -> np.ndarray:
    """The vertex of the LP that a matching stands for: P-bar [(M+1) x (B+1)] of zeros and ones plus the
    dustbin cells (marginals a = [1_M, B], b = [1_B, M])."""
    B = len(match_prop)
    Pbar = np.zeros((M + 1, B + 1))
    pairs = 0
    for j, i in enumerate(match_prop):
        if i >= 0:
            Pbar[i, j] = 1.0
            pairs += 1
        else:
            Pbar[M, j] = 1.0           # pruned token j goes to the dustbin row
    for i in range(M):
        if Pbar[i, :B].sum() == 0:
            Pbar[i, B] = 1.0           # kept token i goes to the dustbin column
    Pbar[M, B] = pairs
    return Pbar


def merge(T, kept, prop, Pbar, *, alpha: float = 0.1) -> np.ndarray:
    """Eq. 7.  Returns Y [M x D] fp64 (not rounded)."""
    T = _f64(T)
    Pbar = _f64(Pbar)
    kept = np.ascontiguousarray(kept, dtype=np.int32)
    prop = np.ascontiguousarray(prop, dtype=np.int32)
    Y = np.empty((len(kept), T.shape[1]))
    lib().rtp_oracle_merge(_dp(T), ctypes.c_int(T.shape[1]), _ip(kept), ctypes.c_int(len(kept)),
                           _ip(prop), ctypes.c_int(len(prop)), _dp(Pbar), ctypes.c_double(alpha),
                           _dp(Y))
    return Y


def partners(Pbar):
    """argmax_i P_ij per proposed token j.  Returns (partner, weight, log-gap)."""
    Pbar = _f64(Pbar)
    M, B = Pbar.shape[0] - 1, Pbar.shape[1] - 1
    partner = np.empty(max(B, 1), dtype=np.int32)
    weight = np.empty(max(B, 1))
    gap = np.empty(max(B, 1))
    lib().rtp_oracle_partners(_dp(Pbar), ctypes.c_int(M), ctypes.c_int(B), _ip(partner),
                              _dp(weight), _dp(gap))
    return partner[:B].copy(), weight[:B].copy(), gap[:B].copy()


# ----------------------------------------------------------------------------------------------
# Algorithm 1 over one image / a ragged batch
# ----------------------------------------------------------------------------------------------
@dataclass
class Params:
    """The paper's knobs (Algorithm 1 inputs; Appendix C for iters) plus the readings of Eq. 10."""
    dynamic: bool = False
    r_fixed: float = 0.25
    phi_lo: float = 0.0
    phi_hi: float = 1.0
    r_max: float = 1.0
    z: float = 0.2
    alpha: float = 0.1
    eps: float = 1.0
    iters: int = 100
    criterion: int = 0      # ranking of stage 1: 0 l2 norm (Eq. 1), 1 variance, 2 entropy (selection-metric ablation)
    exact: bool = False     # solve the linear program of Eq. 2-6 exactly instead of running Sinkhorn iterations


@dataclass
class ImageResult:
    N: int
    M: int
    B: int
    C: np.ndarray          # [N] norms
    phi: float
    rho: float
    r: float
    kept: np.ndarray       # [M] int32, ascending
    prop: np.ndarray       # [B] int32, ascending
    partner: np.ndarray    # [B] int32 (position in `kept`)
    weight: np.ndarray     # [B]
    gap: np.ndarray        # [B] log-gap of the partner argmax
    Y: np.ndarray          # [M x D] fp64
    u: Optional[np.ndarray] = None
    v: Optional[np.ndarray] = None
    Pbar: Optional[np.ndarray] = None
    S: Optional[np.ndarray] = None          # exact mode: the score matrix the matching was solved on
    objective: Optional[float] = None       # exact mode: value of the linear program


def run_image_exact(T, p: Params, rho: float = 0.0) -> ImageResult:
    """Algorithm 1 with the transport problem of Eq. 2-6 solved exactly: the steps of run_image strung
    together from the step functions, the matching in place of the Sinkhorn iterations, hard pairs in Eq. 7."""
    T = _f64(T)
    N = T.shape[0]
    C = norms(T)
    ph = phi(T, C) if N >= 2 else 0.0
    r, B, M = ratio(ph, rho, N, dynamic=p.dynamic, r_fixed=p.r_fixed, phi_lo=p.phi_lo, phi_hi=p.phi_hi,
                    r_max=p.r_max)
    kept, prop = select(criterion(T, p.criterion) if p.criterion else C, M)
    if B == 0:
        return ImageResult(N=N, M=M, B=0, C=C, phi=ph, rho=rho, r=r, kept=kept, prop=prop,
                           partner=np.zeros(0, np.int32), weight=np.zeros(0), gap=np.zeros(0), Y=T[kept].copy())
    S = scores(T, C, kept, prop)
    match, obj, _, _ = exact_matching(S, z=p.z)
    Pbar = matching_plan(match, M)
    Y = merge(T, kept, prop, Pbar, alpha=p.alpha)
    res = ImageResult(N=N, M=M, B=B, C=C, phi=ph, rho=rho, r=r, kept=kept, prop=prop, partner=match,
                      weight=(match >= 0).astype(np.float64), gap=np.full(B, np.inf), Y=Y, Pbar=Pbar)
    res.S = S
    res.objective = obj
    return res


def run_image(T, p: Params, rho: float = 0.0, *, want_plan: bool = False,
              compute_phi: bool = True) -> ImageResult:
    if p.exact:
        return run_image_exact(T, p, rho)
    T = _f64(T)
    N, D = T.shape
    C = np.empty(N)
    stats = np.empty(4)
    kept = np.empty(N, dtype=np.int32)
    prop = np.empty(N, dtype=np.int32)
    partner = np.empty(N, dtype=np.int32)
    weight = np.empty(N)
    gap = np.empty(N)
    Y = np.empty((N, D))
    u = v = Pbar = None
    if want_plan:
        u = np.empty(N + 1)
        v = np.empty(N + 1)
        Pbar = np.empty((N // 2 + 2) ** 2)
    M = lib().rtp_oracle_image(
        _dp(T), ctypes.c_int(N), ctypes.c_int(D), ctypes.c_double(rho),
        ctypes.c_int(int(p.dynamic)), ctypes.c_double(p.r_fixed), ctypes.c_double(p.phi_lo),
        ctypes.c_double(p.phi_hi), ctypes.c_double(p.r_max), ctypes.c_double(p.z),
        ctypes.c_double(p.alpha), ctypes.c_double(p.eps), ctypes.c_int(p.iters),
        ctypes.c_int(int(compute_phi)), ctypes.c_int(int(p.criterion)), _dp(C), _dp(stats), _ip(kept), _ip(prop), _ip(partner),
        _dp(weight), _dp(gap), _dp(Y), _dp(u), _dp(v), _dp(Pbar))
    B = N - M
    res = ImageResult(N=N, M=M, B=B, C=C, phi=float(stats[0]), rho=float(stats[1]),
                      r=float(stats[2]), kept=kept[:M].copy(), prop=prop[:B].copy(),
                      partner=partner[:B].copy(), weight=weight[:B].copy(), gap=gap[:B].copy(),
                      Y=Y[:M].copy())
    if want_plan and B > 0:
        res.u = u[:M + 1].copy()
        res.v = v[:B + 1].copy()
        res.Pbar = Pbar[:(M + 1) * (B + 1)].reshape(M + 1, B + 1).copy()
    return res


@dataclass
class BatchResult:
    images: List[ImageResult] = field(default_factory=list)

    @property
    def counts(self) -> np.ndarray:
        return np.array([im.M for im in self.images], dtype=np.int32)

    @property
    def out_offsets(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.counts)]).astype(np.int32)


def run_batch(X, offsets: Sequence[int], p: Params, rho: Optional[Sequence[float]] = None, *,
              images: Optional[Sequence[int]] = None, threads: int = 1,
              want_plan: bool = False, compute_phi: bool = True) -> BatchResult:
    """Algorithm 1 on every image (or on the listed ones) of a ragged batch.

    ``X`` is [sum N_i, D] (any float dtype numpy can hold exactly in fp64), ``offsets`` has
    batch+1 entries.  ``threads`` > 1 runs images concurrently (the C code holds no global state
    and ctypes releases the GIL); the arithmetic per image is unchanged.
    """
    offsets = np.asarray(offsets, dtype=np.int64)
    batch = len(offsets) - 1
    todo = list(range(batch)) if images is None else list(images)

    def one(i: int) -> ImageResult:
        T = np.asarray(X[offsets[i]:offsets[i + 1]], dtype=np.float64)
        return run_image(T, p, 0.0 if rho is None else float(rho[i]), want_plan=want_plan,
                         compute_phi=compute_phi)

    if threads <= 1:
        out = [one(i) for i in todo]
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            out = list(ex.map(one, todo))
    return BatchResult(images=out)

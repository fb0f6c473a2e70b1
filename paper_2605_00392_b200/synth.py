"""Seeded synthetic token batches (and page images) with the shapes of the paper's workloads.

This module is the ONLY code shared by the CUDA path's tests/benchmark and the CPU oracle.  It
draws random inputs and nothing else: none of the pruning method's arithmetic lives here.  (The one
computation it does on the data is measuring row lengths so that it can space them apart, see
``_space_norms``; that is input conditioning, not a step of the method.)

The paper evaluates on document-OCR benchmarks with DeepSeek-OCR weights; neither exists here, so
the batches take only the token-count / width shapes of the DeepSeek-OCR resolution modes (64, 100,
256, 400 tokens of width 1280; multi-view pages with a 256-token global view plus 100-token tiles)
and the structure the paper describes: text-bearing tokens with large norms and many distinct
directions, background tokens that are near-duplicates of one another with small norms.

All randomness is counter-based (Philox) keyed by (config seed, image index), so any single image
of any configuration can be regenerated on its own.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np
import torch

D_MODEL = 1280          # DeepSeek-OCR hidden width
SEED_BASE = 0x5EED0000
NORM_GAP = 1.5e-3       # relative spacing enforced between neighbouring sorted row norms


@dataclass
class Workload:
    """A ragged batch: X[sum N_i, d], offsets[batch+1], per-image textual density rho[batch]."""
    name: str
    X: torch.Tensor                     # CPU, bf16 or fp32, contiguous
    offsets: np.ndarray                 # int32 [batch+1]
    rho: np.ndarray                     # float32 [batch]
    params: Dict[str, float] = field(default_factory=dict)   # ratio / OT parameters to run with

    @property
    def batch(self) -> int:
        return len(self.offsets) - 1

    @property
    def total_tokens(self) -> int:
        return int(self.offsets[-1])

    @property
    def d(self) -> int:
        return int(self.X.shape[1])

    @property
    def max_tokens(self) -> int:
        return int(np.diff(self.offsets).max()) if self.batch else 0

    def image_f64(self, i: int) -> np.ndarray:
        """Exact fp64 copy of image i's tokens (bf16/fp32 -> fp64 is lossless)."""
        a, b = int(self.offsets[i]), int(self.offsets[i + 1])
        return self.X[a:b].to(torch.float64).numpy()

    def X_f64(self) -> np.ndarray:
        return self.X.to(torch.float64).numpy()


def _rng(seed: int, image: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed ^ image) & 0xFFFFFFFFFFFFFFFF, image]))


def _round_to(x: np.ndarray, dtype: torch.dtype) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(dtype)


def _space_norms(rows: np.ndarray, dtype: torch.dtype, gap: float = NORM_GAP) -> torch.Tensor:
    """Rescale rows so that neighbouring sorted row lengths differ by a relative `gap` at least.

    A selection by length is then unambiguous in any arithmetic that measures lengths to better
    than `gap`.  Rescaling a row changes none of its angles to other rows.  The rows are re-rounded
    to the storage dtype and the spacing is re-measured on the rounded values.
    """
    master = np.array(rows, dtype=np.float64)   # unrounded rows: a rescale smaller than half an
    for _ in range(16):                          # ulp would be lost if applied to rounded values
        x = _round_to(master, dtype)
        n = np.linalg.norm(x.to(torch.float64).numpy(), axis=1)
        order = np.argsort(n, kind="stable")
        logn = np.log(n[order])
        if len(n) < 2 or np.min(np.diff(logn)) >= np.log1p(0.8 * gap):
            return x
        k = np.arange(len(n)) * np.log1p(gap)
        spaced = np.maximum.accumulate(logn - k) + k
        scale = np.ones(len(n))
        scale[order] = np.exp(spaced - logn)
        master *= scale[:, None]
    raise RuntimeError("could not space the row norms")


def _lognormal_norms(rng: np.random.Generator, n: int, median: float, sigma: float) -> np.ndarray:
    return median * np.exp(sigma * rng.standard_normal(n))


def _unit(rows: np.ndarray) -> np.ndarray:
    return rows / np.linalg.norm(rows, axis=1, keepdims=True)


def gaussian_image(rng: np.random.Generator, n: int, d: int, sigma: float = 0.5,
                   outlier_frac: float = 0.10, outlier_scale: float = 4.0) -> np.ndarray:
    """Gaussian directions, log-normal lengths, a fraction of tokens blown up by `outlier_scale`."""
    dirs = _unit(rng.standard_normal((n, d)))
    norms = _lognormal_norms(rng, n, np.sqrt(d), sigma)
    n_out = int(round(outlier_frac * n))
    if n_out:
        norms[rng.choice(n, size=n_out, replace=False)] *= outlier_scale
    return dirs * norms[:, None]


def document_image(rng: np.random.Generator, n: int, d: int, text_density: float,
                   clusters: int = 16, sigma: float = 0.5) -> np.ndarray:
    """Text-like tokens from `clusters` Gaussian clusters plus near-duplicate background tokens.

    A fraction `1 - text_density` of the tokens are background: one centre per image plus 0.01
    noise, with a median length half that of the text tokens.  Positions are shuffled.
    """
    n_blank = int(round((1.0 - text_density) * n))
    n_blank = min(max(n_blank, 0), n)
    n_text = n - n_blank
    centres = rng.standard_normal((clusters, d))
    which = rng.integers(0, clusters, size=n_text)
    text = centres[which] + 0.5 * rng.standard_normal((n_text, d))
    blank_centre = rng.standard_normal(d)
    blank = blank_centre[None, :] + 0.01 * rng.standard_normal((n_blank, d))
    rows = np.concatenate([_unit(text) * _lognormal_norms(rng, n_text, np.sqrt(d), sigma)[:, None],
                           _unit(blank) * _lognormal_norms(rng, n_blank, 0.5 * np.sqrt(d),
                                                           sigma)[:, None]])
    return rows[rng.permutation(n)]


def paired_image(rng: np.random.Generator, n: int, d: int, r: float, noise: float = 0.3):
    """An image whose pruning has a known answer: n - B "anchor" tokens with Gaussian directions and lengths in
    [1.5, 3] sqrt(d), and B = round(r n) "echo" tokens, each a noisy copy of a random anchor's direction with a
    length in [0.3, 0.8] sqrt(d).  Ranked by norm at ratio r the anchors are kept and the echoes pruned, and every
    echo's look-alike among the kept tokens is its anchor by a wide margin (cosine about 0.95 against about 0).
    Returns (rows, echo_of): echo_of[k] = token index of the anchor that token k echoes, -1 for an anchor."""
    n_echo = int(np.floor(r * n + 0.5))
    n_anchor = n - n_echo
    anchors = _unit(rng.standard_normal((n_anchor, d)))
    src = rng.integers(0, n_anchor, size=n_echo)
    echoes = _unit(anchors[src] + noise * _unit(rng.standard_normal((n_echo, d))))
    rows = np.concatenate([anchors * (np.sqrt(d) * rng.uniform(1.5, 3.0, n_anchor))[:, None],
                           echoes * (np.sqrt(d) * rng.uniform(0.3, 0.8, n_echo))[:, None]])
    perm = rng.permutation(n)                  # new position p holds old row perm[p]
    where = np.empty(n, dtype=np.int64)
    where[perm] = np.arange(n)                 # old row -> new position
    echo_of = np.full(n, -1, dtype=np.int64)
    echo_of[where[n_anchor + np.arange(n_echo)]] = where[src]
    return rows[perm], echo_of


def paired(lengths: List[int], r: float, *, seed: int = 3, d: int = D_MODEL,
           dtype: torch.dtype = torch.bfloat16):
    """A batch of paired_image images at fixed ratio r.  Returns (workload, [echo_of per image])."""
    ims, truth = [], []
    for i, n in enumerate(lengths):
        rows, echo_of = paired_image(_rng(SEED_BASE + 0x200 + seed, i), n, d, r)
        ims.append(_space_norms(rows, dtype))
        truth.append(echo_of)
    w = _assemble("paired", ims, np.zeros(len(lengths)), dict(dynamic=0, r_fixed=float(r), phi_lo=0.0, phi_hi=1.0, r_max=1.0))
    return w, truth


# Ratio parameters of the dynamic configurations.  phi_hi was chosen so that the Large batch keeps
# about 84 % of its tokens on average, the retention the paper reports for its dynamic mode.
DYNAMIC_PARAMS = dict(dynamic=1, r_fixed=0.0, phi_lo=0.0, phi_hi=0.737, r_max=0.5)
OT_PARAMS = dict(z=0.2, alpha=0.1, eps=1.0, iters=100)

CONFIG_IDS = {"tiny": 0, "base": 1, "large": 2, "gundam": 3, "sweep": 4, "sweep_fp32": 5}


def _assemble(name: str, images: List[torch.Tensor], rho: np.ndarray,
              params: Dict[str, float]) -> Workload:
    lens = np.array([im.shape[0] for im in images], dtype=np.int64)
    offsets = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    X = torch.cat(images, dim=0).contiguous() if images else torch.empty((0, D_MODEL))
    p = dict(OT_PARAMS)
    p.update(params)
    return Workload(name=name, X=X, offsets=offsets, rho=rho.astype(np.float32), params=p)


def make(name: str, *, batch: Optional[int] = None, d: int = D_MODEL,
         dtype: Optional[torch.dtype] = None, r_fixed: Optional[float] = None,
         images: Optional[List[int]] = None, seed_offset: int = 0) -> Workload:
    """Build one of the named configurations.

    tiny        1 x 64, Gaussian directions, log-normal norms (sigma 0.5), 10 % x4 outliers, r = 0.25
    base        32 x 256, 16-cluster documents with 30 % background tokens, dynamic ratio
    large       64 x 400, documents with text density U[0.2, 0.9] per image, dynamic ratio
    gundam      128 ragged images of 256 + 100 n tokens, n U{2..9}, dynamic ratio
    sweep       1024 x 400 documents; fixed r (pass r_fixed) or dynamic (r_fixed None)
    sweep_fp32  256 x 400 documents stored in fp32

    `batch` overrides the number of images (the per-image streams do not change, so a smaller batch
    is a prefix of the full one); `images` picks individual image indices of the full batch.
    """
    cid = CONFIG_IDS[name]
    seed = SEED_BASE + cid + (seed_offset << 8)
    default_batch = {"tiny": 1, "base": 32, "large": 64, "gundam": 128, "sweep": 1024,
                     "sweep_fp32": 256}[name]
    nb = default_batch if batch is None else batch
    idx = list(range(nb)) if images is None else list(images)
    if dtype is None:
        dtype = torch.float32 if name == "sweep_fp32" else torch.bfloat16

    ims: List[torch.Tensor] = []
    rho = np.zeros(len(idx))
    for slot, i in enumerate(idx):
        rng = _rng(seed, i)
        if name == "tiny":
            rows = gaussian_image(rng, 64, d)
            rho[slot] = 0.0
        elif name == "base":
            rho[slot] = 0.7
            rows = document_image(rng, 256, d, text_density=0.7)
        elif name in ("large", "sweep", "sweep_fp32"):
            rho[slot] = rng.uniform(0.2, 0.9)
            rows = document_image(rng, 400, d, text_density=rho[slot])
        elif name == "gundam":
            tiles = int(rng.integers(2, 10))
            rho[slot] = rng.uniform(0.2, 0.9)
            rows = document_image(rng, 256 + 100 * tiles, d, text_density=rho[slot])
        else:  # pragma: no cover
            raise KeyError(name)
        ims.append(_space_norms(rows, dtype))

    if name == "tiny":
        params = dict(dynamic=0, r_fixed=0.25, phi_lo=0.0, phi_hi=1.0, r_max=1.0)
    elif name in ("sweep", "sweep_fp32") and r_fixed is not None:
        params = dict(dynamic=0, r_fixed=float(r_fixed), phi_lo=0.0, phi_hi=1.0, r_max=1.0)
    else:
        params = dict(DYNAMIC_PARAMS)
    return _assemble(name, ims, rho, params)


def ragged(lengths: List[int], *, seed: int = 7, d: int = D_MODEL,
           dtype: torch.dtype = torch.bfloat16, text_density: float = 0.6,
           params: Optional[Dict[str, float]] = None) -> Workload:
    """A batch of document images with the given token counts (edge-case and shape tests)."""
    ims = []
    for i, n in enumerate(lengths):
        rng = _rng(SEED_BASE + 0x100 + seed, i)
        ims.append(_space_norms(document_image(rng, n, d, text_density=text_density), dtype))
    p = dict(dynamic=0, r_fixed=0.25, phi_lo=0.0, phi_hi=1.0, r_max=1.0)
    if params:
        p.update(params)
    return _assemble("ragged", ims, np.full(len(lengths), text_density), p)


# ---------------------------------------------------------------------------------------------
# Page images for the textual-density step (Eq. 9): 8-bit RGB, [batch, H, W, 3].
# ---------------------------------------------------------------------------------------------
PAGE_PATCH = 64          # pixels per token patch side: 1280 x 1280 pixels <-> 20 x 20 = 400 tokens


def page_image(rng: np.random.Generator, height: int, width: int, text_fraction: float) -> np.ndarray:
    """One synthetic document page: a near-white, slightly tinted background with faint sensor noise,
    and text in a `text_fraction` share of the 64 x 64 patches: lines 16 pixels high whose glyph
    cells (8 pixels wide) are inked at random with dark, sharp-edged dots.  Blank patches stay
    uniform up to the noise, whose amplitude (+-2 levels) is far below the edge threshold."""
    ph, pw = height // PAGE_PATCH, width // PAGE_PATCH
    r = rng.integers(0, 256, size=(height, width), dtype=np.uint8)      # one draw serves noise and ink
    text_patch = rng.random((ph, pw)) < text_fraction
    inked_cell = rng.random((height // 16, width // 8)) < 0.55
    rows = np.arange(height) % 16
    line_rows = (rows >= 3) & (rows <= 12)
    mask = np.repeat(np.repeat(text_patch, PAGE_PATCH, axis=0), PAGE_PATCH, axis=1)
    mask &= np.repeat(np.repeat(inked_cell, 16, axis=0), 8, axis=1)
    mask &= line_rows[:, None]
    mask &= (r >> 2) < 22                                               # about a third of the cell's pixels
    base = np.array([rng.integers(244, 253), rng.integers(242, 251), rng.integers(236, 249)], dtype=np.int16)
    ink = np.array([rng.integers(10, 60), rng.integers(10, 60), rng.integers(20, 90)], dtype=np.int16)
    noise = (r & 3).astype(np.int16) - 2                                # -2 .. 1
    img = np.empty((height, width, 3), dtype=np.uint8)
    for ch in range(3):
        plane = np.where(mask, ink[ch], base[ch]) + noise
        img[..., ch] = np.clip(plane, 0, 255).astype(np.uint8)
    return img


def pages(batch: int, height: int = 1280, width: int = 1280, *, seed: int = 11,
          text_fraction: Optional[np.ndarray] = None) -> torch.Tensor:
    """[batch, H, W, 3] uint8 pages; image i's share of text patches is text_fraction[i] (default
    U[0.2, 0.9], the range of the token batches' textual density)."""
    out = np.empty((batch, height, width, 3), dtype=np.uint8)
    for i in range(batch):
        rng = _rng(SEED_BASE + 0x200 + seed, i)
        tf = float(rng.uniform(0.2, 0.9)) if text_fraction is None else float(text_fraction[i])
        out[i] = page_image(rng, height, width, tf)
    return torch.from_numpy(out)

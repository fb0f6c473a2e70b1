"""fp64 CPU oracle of the textual density rho (Eq. 9, Appendix B): plain numpy, written from the paper.

TEST INFRASTRUCTURE ONLY: imported by the tests and the benchmark's CPU-baseline leg, never by the
product package.  It shares no code with the CUDA path.

Steps, in the paper's order (Appendix B, then Eq. 9):
  1. grayscale I = w_R R + w_G G + w_B B with the ITU-R BT.601 weights 0.299, 0.587, 0.114; the
     8-bit channels are taken as intensities in [0, 1] (value / 255): the threshold tau = 0.2 of
     Algorithm 1 only makes sense on that scale.
  2. G_x, G_y = the two 3 x 3 Sobel kernels applied to I.  Only G_x^2 + G_y^2 is used, so the sign
     convention (convolution or correlation) does not matter.
  3. G = sqrt(G_x^2 + G_y^2); E = 1 where G >= tau.
  4. rho_k = mean of E over the h x w pixels of token patch k; rho = average of rho_k over the patches.

Reading where the paper is silent: pixels outside the image take the value of the nearest pixel
inside (replicated border), so that a uniform page has no edge along its border; zero padding would
mark the whole border of a white page as text.  PARITY UNPINNED for this choice alone: nothing in
the paper fixes it.
"""
from __future__ import annotations

import numpy as np

W_R, W_G, W_B = 0.299, 0.587, 0.114


def grayscale(rgb_u8: np.ndarray) -> np.ndarray:
    """[H, W, 3] uint8 -> [H, W] float64 intensities in [0, 1] (Appendix B, first equation)."""
    c = rgb_u8.astype(np.float64) / 255.0
    return W_R * c[..., 0] + W_G * c[..., 1] + W_B * c[..., 2]


def sobel(gray: np.ndarray):
    """G_x and G_y of Appendix B on a replicated border, written out tap by tap."""
    H, W = gray.shape
    P = np.empty((H + 2, W + 2), dtype=np.float64)
    P[1:-1, 1:-1] = gray
    P[0, 1:-1] = gray[0]
    P[-1, 1:-1] = gray[-1]
    P[:, 0] = P[:, 1]
    P[:, -1] = P[:, -2]
    tl, tc, tr = P[:-2, :-2], P[:-2, 1:-1], P[:-2, 2:]
    ml, mr = P[1:-1, :-2], P[1:-1, 2:]
    bl, bc, br = P[2:, :-2], P[2:, 1:-1], P[2:, 2:]
    gx = (tr + 2.0 * mr + br) - (tl + 2.0 * ml + bl)
    gy = (tl + 2.0 * tc + tr) - (bl + 2.0 * bc + br)
    return gx, gy


def edge_map(rgb_u8: np.ndarray, tau: float) -> np.ndarray:
    """E(i, j) = 1 where the gradient magnitude reaches tau (Appendix B, last equation)."""
    gx, gy = sobel(grayscale(rgb_u8))
    return np.sqrt(gx * gx + gy * gy) >= float(tau)


def density(rgb_u8: np.ndarray, patch: int, tau: float = 0.2):
    """(rho, rho_k [H/patch, W/patch], edge counts per patch) of one image (Eq. 9)."""
    H, W, _ = rgb_u8.shape
    if H % patch or W % patch:
        raise ValueError("the patches must tile the image")
    E = edge_map(rgb_u8, tau)
    counts = E.reshape(H // patch, patch, W // patch, patch).sum(axis=(1, 3)).astype(np.int64)
    rho_k = counts / float(patch * patch)
    return float(rho_k.mean()), rho_k, counts


def density_batch(images_u8: np.ndarray, patch: int, tau: float = 0.2):
    """rho [batch] and edge counts [batch, H/patch, W/patch] of a batch of equally sized images."""
    rhos, counts = [], []
    for im in images_u8:
        r, _, c = density(im, patch, tau)
        rhos.append(r)
        counts.append(c)
    return np.array(rhos), np.stack(counts)

"""Seeded synthetic weight generators shared by the tests, the bench and the smoke check.

They stand in for the linear weights of the models the paper compresses (which
are not available offline).  This module holds none of the codec's arithmetic:
it only draws random matrices with numpy's PCG64 generator.
"""
from __future__ import annotations

import numpy as np


def _log_uniform(rng, lo, hi, n):
    return np.exp(rng.uniform(np.log(lo), np.log(hi), size=n)).astype(np.float32)


def gaussian_rows(R, C, seed, lo=0.005, hi=0.05, outlier_p=0.0, outlier_mag=8.0):
    """Rows ~ N(0, sigma_r^2), sigma_r log-uniform in [lo, hi]; optionally a fraction
    outlier_p of entries replaced by +-outlier_mag * sigma_r with a fair sign."""
    rng = np.random.Generator(np.random.PCG64(seed))
    sig = _log_uniform(rng, lo, hi, R)
    W = rng.standard_normal((R, C), dtype=np.float32) * sig[:, None]
    if outlier_p > 0.0:
        mask = rng.random((R, C), dtype=np.float32) < outlier_p
        sign = np.where(rng.random((R, C), dtype=np.float32) < 0.5, -1.0, 1.0).astype(np.float32)
        W = np.where(mask, sign * np.float32(outlier_mag) * sig[:, None], W).astype(np.float32)
    return np.ascontiguousarray(W, np.float32)


def student_t_rows(R, C, seed, nu=5.0, lo=0.01, hi=0.04):
    """Rows ~ sigma_r * t_nu (standard Student-t, not variance-normalised)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    sig = _log_uniform(rng, lo, hi, R)
    W = rng.standard_t(nu, size=(R, C)).astype(np.float32) * sig[:, None]
    return np.ascontiguousarray(W, np.float32)


def laplace_rows(R, C, seed, lo=0.005, hi=0.03):
    """Rows ~ Laplace(0, b_r), b_r log-uniform in [lo, hi]."""
    rng = np.random.Generator(np.random.PCG64(seed))
    b = _log_uniform(rng, lo, hi, R)
    W = rng.laplace(0.0, 1.0, size=(R, C)).astype(np.float32) * b[:, None]
    return np.ascontiguousarray(W, np.float32)


# shapes of one transformer-block bundle: 4 square projections + 3 MLP matrices
BLOCK_SHAPES = [(5120, 5120)] * 4 + [(5120, 17408)] * 3


def config1():
    """512x512 Gaussian rows, seed 0; 4.0 bpp; one tile per 64 rows; BF16."""
    return gaussian_rows(512, 512, 0)


def config2(R=4096, C=4096):
    """Student-t (nu=5) rows scaled by sigma_r in [0.01, 0.04]; 3.0 bpp; BF16."""
    return student_t_rows(R, C, 2)


def config3_tensor(i, shape=None):
    """Tensor i (0..6) of the block bundle: Gaussian rows with 0.1 % +-8 sigma outliers; 2.5 bpp."""
    R, C = shape if shape is not None else BLOCK_SHAPES[i]
    return gaussian_rows(R, C, 30 + i, outlier_p=0.001, outlier_mag=8.0)


def config4(R=8192, C=8192):
    """Laplace rows, b_r in [0.005, 0.03]; targets 2.0 .. 6.0 bpp; FP16."""
    return laplace_rows(R, C, 4)


def config5_tensor(layer, i, shape=None):
    """Tensor i of layer `layer` of the 48-layer stack: Gaussian rows; 3.5 bpp; BF16."""
    R, C = shape if shape is not None else BLOCK_SHAPES[i]
    return gaussian_rows(R, C, 5000 + 7 * layer + i)


def to_container(W, kind):
    """Row-scaled low-precision container used by the FP8 / INT8 routes: returns
    (a_r, W / a_r) with a_r = max_j |W_rj| / 448 (FP8-E4M3) or / 127 (INT8).
    The caller rounds the second array to the container grid with its own cast."""
    amax = np.max(np.abs(W), axis=1).astype(np.float32)
    amax = np.where(amax > 0, amax, np.float32(1.0))
    a = (amax / np.float32(448.0 if kind == "fp8" else 127.0)).astype(np.float32)
    return a, (W / a[:, None]).astype(np.float32)

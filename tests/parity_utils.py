"""Helpers shared by the GPU parity tests: run the float64 oracle on the same bytes the CUDA
path saw and account for code mismatches by their distance to a decision boundary."""
import numpy as np
import torch

from oracle import polarquant_oracle as orc

WINDOW_RAD = 1e-6        # codes may differ only where the oracle's angle is this close to a boundary
MAX_WINDOW_FRACTION = 1e-5
TOL_DECODED = 1e-3       # relative L2 of DeQuant output
TOL_ATTENTION = 2e-3     # relative L2 of attention output (bf16 I/O): asserted on whole outputs or on the sampled units together
TOL_ATTENTION_F32_IO = 1e-3  # the same with float32 I/O: the kernel's arithmetic alone (fp16 operands, measured ~4e-4);
#                              used where a small part of an output is looked at by itself, because rounding a few
#                              hundred values to bf16 costs 1.66e-3 on average and up to 2e-3


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact conversion of a bf16/f16/f32 tensor to float64."""
    return t.detach().float().cpu().double().numpy()


def oracle_codebooks(cache) -> orc.Codebooks:
    """The library's float64 codebooks handed to the oracle as data."""
    return orc.codebooks_from_arrays((4, 2, 2, 2), cache.centroids.numpy(), cache.boundaries.numpy())


def rel_l2(got: np.ndarray, want: np.ndarray) -> float:
    return float(np.linalg.norm(got.ravel() - want.ravel()) / max(np.linalg.norm(want.ravel()), 1e-300))


def code_mismatch_report(gpu_codes: np.ndarray, x: np.ndarray, S: np.ndarray, cb: orc.Codebooks):
    """Encode `x` ([n, d] float64) with the oracle and compare with `gpu_codes` ([n, n_codes]).

    Returns dict(total, inside, outside, radii16) where inside/outside count mismatching codes
    whose oracle angle is within / beyond WINDOW_RAD of a decision boundary."""
    want, radii16, angles = orc.encode(x, S, cb)
    diff = gpu_codes != want
    dist = orc.boundary_distance(angles, cb)
    inside = int(np.count_nonzero(diff & (dist <= WINDOW_RAD)))
    outside = int(np.count_nonzero(diff & (dist > WINDOW_RAD)))
    return dict(total=int(want.size), inside=inside, outside=outside, radii16=radii16, codes=want)


def assert_codes_match(rep):
    assert rep["outside"] == 0, f"{rep['outside']} codes differ outside the {WINDOW_RAD} rad window"
    assert rep["inside"] <= max(1, MAX_WINDOW_FRACTION * rep["total"]), \
        f"{rep['inside']} of {rep['total']} codes differ inside the window"


MAX_RADIUS_ULP_FRACTION = 2.5e-3  # of radii one fp16 ulp off (measured: 0.9e-3 tensor-core encoder, 0.2e-3 the others)


def radii_ulp_report(gpu_radii: np.ndarray, want16: np.ndarray):
    """(radii that differ from the oracle's fp16 value, radii compared); a difference of more than one fp16
    ulp fails at once."""
    g = np.asarray(gpu_radii).astype(np.float16).view(np.uint16).astype(np.int32)
    w = np.asarray(want16).astype(np.float16).view(np.uint16).astype(np.int32)
    delta = np.abs(g - w)
    assert delta.max() <= 1, f"radius differs by {delta.max()} fp16 ulps"
    return int(np.count_nonzero(delta)), int(delta.size)


def assert_radii_match(gpu_radii: np.ndarray = None, want16: np.ndarray = None, counts=None):
    """fp16 radii equal the oracle's single rounding of the float64 block norm, except that the encoder's
    float32-accurate norm (relative error ~2e-7 against an fp16 spacing of 5e-4 .. 1e-3) lands on the neighbouring
    fp16 value for a small fraction of them.  `counts` = (off by one, compared) summed by the caller over many small
    samples (a sample of a few hundred radii cannot be held to a fraction of 1e-3 by itself)."""
    off, n = counts if counts is not None else radii_ulp_report(gpu_radii, want16)
    assert off <= MAX_RADIUS_ULP_FRACTION * n + 3, f"{off} of {n} radii are one fp16 ulp off"

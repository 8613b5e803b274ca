"""Helpers shared by the GPU parity tests: run the float64 oracle on the same bytes the CUDA
path saw and account for code mismatches by their distance to a decision boundary."""
import numpy as np
import torch

from oracle import polarquant_oracle as orc

WINDOW_RAD = 1e-6        # codes may differ only where the oracle's angle is this close to a boundary
MAX_WINDOW_FRACTION = 1e-5
TOL_DECODED = 1e-3       # relative L2 of DeQuant output
TOL_ATTENTION = 2e-3     # relative L2 of attention output


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


def assert_radii_match(gpu_radii: np.ndarray, want16: np.ndarray, max_ulp_fraction=5e-3):
    """fp16 radii: equal, except that the float32-accurate norm of the fast encoder (relative error
    ~1e-6 against an fp16 spacing of ~7e-4) may round to the neighbouring fp16 value on ~0.2 % of radii."""
    g = gpu_radii.astype(np.float16).view(np.uint16).astype(np.int32)
    w = want16.astype(np.float16).view(np.uint16).astype(np.int32)
    delta = np.abs(g - w)
    assert delta.max() <= 1, f"radius differs by {delta.max()} fp16 ulps"
    assert np.count_nonzero(delta) <= max_ulp_fraction * delta.size + 1

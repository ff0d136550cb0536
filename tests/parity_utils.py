"""Tolerance checks shared by the GPU parity tests (no method arithmetic here)."""
import numpy as np

REL_FRO_TOL = 2e-3            # relative Frobenius error of GEMM / GEMV outputs
ABS_SUM_TOL = 1e-4            # per element: 1 bf16 ulp + ABS_SUM_TOL * sum_k |a*w|


def bf16_ulp(y: np.ndarray) -> np.ndarray:
    a = np.abs(y)
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -126)))
    return 2.0 ** (e - 7)


def check_outputs(Y: np.ndarray, Yref: np.ndarray, Sabs: np.ndarray, what: str = ""):
    Y = np.asarray(Y, dtype=np.float64)
    assert Y.shape == Yref.shape, (Y.shape, Yref.shape)
    assert np.all(np.isfinite(Y)), f"{what}: non-finite outputs"
    rel = np.linalg.norm(Y - Yref) / max(np.linalg.norm(Yref), 1e-300)
    assert rel <= REL_FRO_TOL, f"{what}: relative Frobenius error {rel:.3e} > {REL_FRO_TOL}"
    bound = bf16_ulp(Yref) + ABS_SUM_TOL * Sabs
    err = np.abs(Y - Yref)
    worst = np.argmax(err - bound)
    assert np.all(err <= bound), (f"{what}: element {np.unravel_index(worst, err.shape)} off by {err.flat[worst]:.3e}, "
                                  f"bound {bound.flat[worst]:.3e}, ref {Yref.flat[worst]:.6e}")
    return rel

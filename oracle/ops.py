"""Single operations of the forward, as plain definitions (test infrastructure only).

Used to check the projection kernel on its own: y = A @ B^T with the epilogues
the forward applies to it (Section 3.1: attention and feed-forward layers).
"""
import numpy as np

from .transformer import silu


def projection(A, B, epilogue, C0=None):
    """A [M,K], B [N,K] (both K-major) -> epilogue(A @ B^T) in float64.

    "plain": the product; "resid": C0 + product (residual-stream update);
    "swiglu": columns (2j, 2j+1) hold (gate_j, up_j); output column j is
    silu(gate_j) * up_j.
    """
    y = np.asarray(A, dtype=np.float64) @ np.asarray(B, dtype=np.float64).T
    if epilogue == "plain":
        return y
    if epilogue == "resid":
        return np.asarray(C0, dtype=np.float64) + y
    if epilogue == "swiglu":
        return silu(y[:, 0::2]) * y[:, 1::2]
    raise ValueError(epilogue)

"""Helpers for the GPU parity tests: device checks and byte-level comparison with the oracle."""
import numpy as np
import pytest
import torch

from paper_2609_03844_b200 import inputs

KEY = 0x5EED


def require_gpu():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2609_03844_b200 as sbw

    sbw.lib()   # fail loudly if the CUDA library is missing: there is no fallback
    return torch.device("cuda:0")


def host_bits(x: torch.Tensor) -> np.ndarray:
    return inputs.as_oracle_array(x)


def assert_same_bits(got: np.ndarray, want: np.ndarray, allow_nan_payload: bool = False):
    assert got.shape == want.shape and got.dtype == want.dtype
    if got.tobytes() == want.tobytes():
        return
    g = got.view(np.uint32 if got.dtype == np.float32 else got.dtype)
    w = want.view(np.uint32 if want.dtype == np.float32 else want.dtype)
    diff = np.argwhere(g != w)
    if allow_nan_payload:
        if got.dtype == np.uint16:
            isnan = lambda a: ((a & 0x7F80) == 0x7F80) & ((a & 0x007F) != 0)   # noqa: E731
        else:
            isnan = lambda a: ((a & 0x7F800000) == 0x7F800000) & ((a & 0x007FFFFF) != 0)   # noqa: E731
        bad = [tuple(i) for i in diff if not (isnan(g[tuple(i)]) and isnan(w[tuple(i)]))]
        if not bad:
            return
        diff = np.array(bad)
    i = tuple(diff[0])
    raise AssertionError(f"{len(diff)} elements differ; first at {i}: got {g[i]:#x}, want {w[i]:#x}")

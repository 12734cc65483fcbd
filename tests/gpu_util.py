"""Helpers shared by the GPU parity tests."""
import numpy as np
import pytest
import torch


def require_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


# tolerances of the forward pass against the oracle (fp32 accumulation, bf16 K/V)
LOGIT_REL_L2 = 2e-3
LOGIT_MAX_ABS = 5e-2


def to_dev_i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()

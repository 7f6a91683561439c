"""Helpers for the GPU parity tests: numpy <-> device tensors, cached library contexts."""
from functools import lru_cache

import numpy as np
import torch

from paper_2609_12378_b200 import binding
from tests.harness import params


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t: torch.Tensor) -> np.ndarray:
    torch.cuda.synchronize()
    return t.cpu().numpy()


@lru_cache(maxsize=None)
def context(log_n, num_q, num_p, dnum) -> binding.Context:
    P = params(log_n, num_q, num_p, dnum)
    return binding.Context(log_n, P.q, P.p, dnum)


def ct_dev(arr: np.ndarray, scale: float) -> binding.Ciphertext:
    return binding.Ciphertext(dev(arr), scale)


def key_dev(arr: np.ndarray, galois: int) -> binding.SwitchKey:
    return binding.SwitchKey(dev(arr), galois)

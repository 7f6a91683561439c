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


GUARD_BYTES, GUARD_VALUE = 4096, 0xA5
_contexts = []


class GuardedContext(binding.Context):
    """A context whose scratch buffers are exactly as large as the library asks for and sit between two 4 KiB
    blocks of a known byte pattern.  The blocks are checked before the next buffer is handed out and after every
    test (tests/conftest.py), so a kernel that writes outside its workspace fails the test that ran it instead of
    landing silently in a neighbouring allocation.  This stands in for a memory checker, which cannot be run here."""

    _guarded = None

    def workspace(self, nbytes: int) -> torch.Tensor:
        self.check_guards()
        nb = (max(int(nbytes), 256) + 255) // 256 * 256
        buf = torch.empty(nb + 2 * GUARD_BYTES, dtype=torch.uint8, device=self.device)
        buf[:GUARD_BYTES] = GUARD_VALUE
        buf[GUARD_BYTES + nb:] = GUARD_VALUE
        self._guarded = (buf, nb)
        return buf[GUARD_BYTES:GUARD_BYTES + nbytes] if nbytes >= 256 else buf[GUARD_BYTES:GUARD_BYTES + nb]

    def check_guards(self):
        if self._guarded is None:
            return
        buf, nb = self._guarded
        self._guarded = None
        torch.cuda.synchronize()
        lo, hi = buf[:GUARD_BYTES], buf[GUARD_BYTES + nb:]
        assert bool((lo == GUARD_VALUE).all()), "a kernel wrote in front of its workspace"
        assert bool((hi == GUARD_VALUE).all()), "a kernel wrote past the end of its workspace"


def check_all_guards():
    for c in _contexts:
        c.check_guards()


@lru_cache(maxsize=None)
def context(log_n, num_q, num_p, dnum) -> binding.Context:
    P = params(log_n, num_q, num_p, dnum)
    c = GuardedContext(log_n, P.q, P.p, dnum)
    _contexts.append(c)
    return c


def ct_dev(arr: np.ndarray, scale: float) -> binding.Ciphertext:
    return binding.Ciphertext(dev(arr), scale)


def key_dev(arr: np.ndarray, galois: int) -> binding.SwitchKey:
    return binding.SwitchKey(dev(arr), galois)

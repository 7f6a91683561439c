"""ctypes binding of the ckks_b200 C ABI.  Argument marshalling only: every
step of every operation runs in the library's CUDA kernels.  torch provides
device memory and streams."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libckks_b200.so")

OK, ERR_ARG, ERR_LEVEL, ERR_SCALE, ERR_NO_KEY, ERR_WORKSPACE, ERR_RANGE, ERR_UNSUPPORTED, ERR_CUDA, ERR_TIMEOUT = (
    0, -1, -2, -3, -4, -5, -6, -7, -8, -9)
OP_ENCODE, OP_MUL_RELIN, OP_ROTATE, OP_ROTATE_HOISTED, OP_RESCALE, OP_LINEAR_PROJ, OP_POLY_EVAL, OP_POLY_EVAL_TREE, OP_MUL_RELIN_BATCH, OP_ROTATE_BATCH, OP_ROTATE_SUM = 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11
PROJ_LAZY_MODDOWN = 1
OPT_NTT_FP_SHARE, OPT_CONV_KERNEL, OPT_MAC_KERNEL, OPT_WAIT_CYCLES, OPT_STATIC_SCRATCH_BYTES, OPT_NTT_BULK_STORE, OPT_LANES = 1, 2, 3, 4, 5, 6, 7
CONV_FP64, CONV_TENSOR = 0, 1
MAC_MMA, MAC_MMA_ASYNC, MAC_MMA_SPLIT, MAC_MMA_HALF, MAC_TCGEN05 = 82, 83, 81, 42, 100
ATTN_QUERY, ATTN_KEY_VALUE, ATTN_TO_SHARDS = 0, 1, 2

EXPORTS = [
    "ckks_context_create", "ckks_context_destroy", "ckks_context_set_option", "ckks_context_get_option", "ckks_status_string",
    "ckks_last_cuda_error",
    "ckks_workspace_bytes", "ckks_galois_element", "ckks_ntt", "ckks_intt", "ckks_encode",
    "ckks_encode_range_flag", "ckks_mul_plain_acc", "ckks_add", "ckks_mul_relin", "ckks_rotate",
    "ckks_rotate_hoisted", "ckks_rescale", "ckks_linear_proj", "ckks_linear_proj_workspace_bytes",
    "ckks_linear_proj_rotations", "ckks_kernel_launches", "ckks_device_status", "ckks_rescale_static",
    "ckks_poly_eval_bsgs_batch", "ckks_poly_eval_bsgs_batch_workspace_bytes", "ckks_attention_pack_rotations", "ckks_attention_pack", "ckks_attention_pack_workspace_bytes", "ckks_attention_rotations", "ckks_attention_scores", "ckks_attention_scores_workspace_bytes", "ckks_attention_values",
    "ckks_attention_values_workspace_bytes", "ckks_softmax_rows", "ckks_softmax_rows_workspace_bytes", "ckks_attention",
    "ckks_attention_workspace_bytes",
    "ckks_ntt_butterfly_probe", "ckks_mul_relin_sum", "ckks_mul_relin_batch", "ckks_rotate_batch", "ckks_rotate_sum", "ckks_softmax", "ckks_softmax_workspace_bytes", "ckks_poly_eval_bsgs", "ckks_poly_eval_bsgs_workspace_bytes", "ckks_mul_const", "ckks_add_const", "ckks_poly_eval", "ckks_poly_eval_tree", "ckks_linear_proj_multi", "ckks_linear_proj_multi_workspace_bytes",
]


class CParams(C.Structure):
    _fields_ = [("log_n", C.c_uint32), ("num_q", C.c_uint32), ("num_p", C.c_uint32), ("dnum", C.c_uint32),
                ("q", C.POINTER(C.c_uint64)), ("p", C.POINTER(C.c_uint64)), ("device", C.c_int32)]


class CCt(C.Structure):
    _fields_ = [("data", C.c_void_p), ("level", C.c_uint32), ("ncomp", C.c_uint32), ("scale", C.c_double)]


class CPt(C.Structure):
    _fields_ = [("data", C.c_void_p), ("level", C.c_uint32), ("scale", C.c_double)]


class CEvk(C.Structure):
    _fields_ = [("data", C.c_void_p), ("galois", C.c_uint64)]


class CSoftmaxDesc(C.Structure):
    _fields_ = [("shift", C.c_double), ("rounds", C.c_uint32), ("row_len", C.c_uint32), ("exp_degree", C.c_uint32),
                ("rsqrt_degree", C.c_uint32), ("exp_coeffs", C.POINTER(C.c_double)), ("rsqrt_coeffs", C.POINTER(C.c_double)),
                ("exp_m", C.c_uint32), ("rsqrt_m", C.c_uint32)]


class CAttnDesc(C.Structure):
    _fields_ = [("tokens", C.c_uint32), ("heads", C.c_uint32), ("diag_block", C.c_uint32), ("group_baby", C.c_uint32), ("token_inner", C.c_uint32)]


class CProjDesc(C.Structure):
    _fields_ = [("d_in", C.c_uint32), ("d_out", C.c_uint32), ("tokens_per_shard", C.c_uint32),
                ("nshards", C.c_uint32), ("baby", C.c_uint32), ("flags", C.c_uint32), ("pt_scale", C.c_double)]


_lib = None


def load():
    """Load the CUDA library.  There is no fallback: a missing library is an error."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_12378_b200.build`")
    L = C.CDLL(LIB_PATH)
    vp, u32, u64, i32, i64, sz, dbl = C.c_void_p, C.c_uint32, C.c_uint64, C.c_int32, C.c_int64, C.c_size_t, C.c_double
    sig = {
        "ckks_context_create": (i32, [C.POINTER(CParams), C.POINTER(vp)]),
        "ckks_context_destroy": (None, [vp]),
        "ckks_context_set_option": (i32, [vp, i32, i64]),
        "ckks_context_get_option": (i64, [vp, i32]),
        "ckks_status_string": (C.c_char_p, [i32]),
        "ckks_last_cuda_error": (C.c_char_p, [vp]),
        "ckks_workspace_bytes": (sz, [vp, i32, u32, u32]),
        "ckks_kernel_launches": (u64, []),
        "ckks_galois_element": (u64, [vp, i64]),
        "ckks_ntt": (i32, [vp, vp, u32, u32, u32, vp]),
        "ckks_intt": (i32, [vp, vp, u32, u32, u32, vp]),
        "ckks_encode": (i32, [vp, vp, vp, u32, dbl, u32, vp, vp, sz, vp]),
        "ckks_encode_range_flag": (i32, [vp, vp]),
        "ckks_device_status": (i32, [vp, vp]),
        "ckks_mul_plain_acc": (i32, [vp, C.POINTER(CCt), u32, C.POINTER(CPt), C.POINTER(CCt), i32, vp]),
        "ckks_add": (i32, [vp, C.POINTER(CCt), C.POINTER(CCt), C.POINTER(CCt), vp]),
        "ckks_mul_relin": (i32, [vp, C.POINTER(CCt), C.POINTER(CCt), C.POINTER(CEvk), C.POINTER(CCt), vp, sz, vp]),
        "ckks_poly_eval_bsgs": (i32, [vp, C.POINTER(CCt), C.POINTER(C.c_double), u32, u32, C.POINTER(CEvk), C.POINTER(CCt), vp, sz, vp]),
        "ckks_poly_eval_bsgs_workspace_bytes": (sz, [vp, u32, u32, u32]),
        "ckks_softmax": (i32, [vp, C.POINTER(CSoftmaxDesc), C.POINTER(CCt), C.POINTER(CEvk), C.POINTER(CEvk), u32, C.POINTER(CCt), vp, sz, vp]),
        "ckks_softmax_workspace_bytes": (sz, [vp, C.POINTER(CSoftmaxDesc), u32]),
        "ckks_attention_rotations": (i32, [vp, C.POINTER(CAttnDesc), C.POINTER(i64), u32]),
        "ckks_poly_eval_bsgs_batch": (i32, [vp, C.POINTER(CCt), u32, C.POINTER(C.c_double), u32, u32, C.POINTER(CEvk), C.POINTER(CCt), vp, sz, vp]),
        "ckks_poly_eval_bsgs_batch_workspace_bytes": (sz, [vp, u32, u32, u32, u32]),
        "ckks_attention_pack_rotations": (i32, [vp, C.POINTER(CAttnDesc), i32, u32, C.POINTER(i64), u32]),
        "ckks_attention_pack": (i32, [vp, C.POINTER(CAttnDesc), i32, C.POINTER(CCt), u32, C.POINTER(CEvk), u32, C.POINTER(CCt), vp, sz, vp]),
        "ckks_attention_pack_workspace_bytes": (sz, [vp, C.POINTER(CAttnDesc), i32, u32, u32]),
        "ckks_attention_scores": (i32, [vp, C.POINTER(CAttnDesc), C.POINTER(CCt), C.POINTER(CCt), u32, C.POINTER(CEvk), C.POINTER(CEvk), u32,
                                        C.POINTER(CCt), vp, sz, vp]),
        "ckks_attention_scores_workspace_bytes": (sz, [vp, C.POINTER(CAttnDesc), u32, u32]),
        "ckks_attention_values": (i32, [vp, C.POINTER(CAttnDesc), C.POINTER(CCt), C.POINTER(CCt), u32, C.POINTER(CEvk), C.POINTER(CEvk), u32,
                                        C.POINTER(CCt), vp, sz, vp]),
        "ckks_attention_values_workspace_bytes": (sz, [vp, C.POINTER(CAttnDesc), u32]),
        "ckks_softmax_rows": (i32, [vp, C.POINTER(CAttnDesc), C.POINTER(CSoftmaxDesc), C.POINTER(CCt), C.POINTER(CEvk), C.POINTER(CEvk), u32,
                                    C.POINTER(CCt), vp, sz, vp]),
        "ckks_softmax_rows_workspace_bytes": (sz, [vp, C.POINTER(CAttnDesc), C.POINTER(CSoftmaxDesc), u32]),
        "ckks_attention": (i32, [vp, C.POINTER(CAttnDesc), C.POINTER(CSoftmaxDesc), C.POINTER(CCt), C.POINTER(CCt), u32, C.POINTER(CCt), u32,
                                 C.POINTER(CEvk), C.POINTER(CEvk), u32, C.POINTER(CCt), vp, sz, vp]),
        "ckks_attention_workspace_bytes": (sz, [vp, C.POINTER(CAttnDesc), C.POINTER(CSoftmaxDesc), u32, u32]),
        "ckks_rotate_sum": (i32, [vp, C.POINTER(CCt), C.POINTER(CEvk), u32, C.POINTER(CCt), vp, sz, vp]),
        "ckks_rotate_batch": (i32, [vp, C.POINTER(CCt), u32, C.POINTER(CEvk), C.POINTER(CCt), vp, sz, vp]),
        "ckks_mul_relin_batch": (i32, [vp, C.POINTER(CCt), C.POINTER(CCt), u32, C.POINTER(CEvk), C.POINTER(CCt), vp, sz, vp]),
        "ckks_mul_relin_sum": (i32, [vp, C.POINTER(CCt), C.POINTER(CCt), u32, C.POINTER(CEvk), C.POINTER(CCt), vp, sz, vp]),
        "ckks_mul_const": (i32, [vp, C.POINTER(CCt), dbl, dbl, C.POINTER(CCt), vp]),
        "ckks_add_const": (i32, [vp, C.POINTER(CCt), dbl, C.POINTER(CCt), vp]),
        "ckks_poly_eval": (i32, [vp, C.POINTER(CCt), C.POINTER(dbl), u32, C.POINTER(CEvk), C.POINTER(CCt), vp, sz, vp]),
        "ckks_poly_eval_tree": (i32, [vp, C.POINTER(CCt), C.POINTER(dbl), u32, C.POINTER(CEvk), C.POINTER(CCt), vp, sz, vp]),
        "ckks_rotate": (i32, [vp, C.POINTER(CCt), C.POINTER(CEvk), C.POINTER(CCt), vp, sz, vp]),
        "ckks_rotate_hoisted": (i32, [vp, C.POINTER(CCt), C.POINTER(CEvk), u32, C.POINTER(CCt), vp, sz, vp]),
        "ckks_rescale": (i32, [vp, C.POINTER(CCt), C.POINTER(CCt), vp, sz, vp]),
        "ckks_rescale_static": (i32, [vp, C.POINTER(CCt), C.POINTER(CCt), vp]),
        "ckks_linear_proj": (i32, [vp, C.POINTER(CProjDesc), C.POINTER(CCt), vp, C.POINTER(CEvk), u32, C.POINTER(CCt), vp, sz, vp]),
        "ckks_linear_proj_workspace_bytes": (sz, [vp, C.POINTER(CProjDesc), u32]),
        "ckks_linear_proj_rotations": (i32, [vp, C.POINTER(CProjDesc), C.POINTER(i64), u32]),
        "ckks_ntt_butterfly_probe": (i32, [vp, u32, vp, sz, C.POINTER(u64), vp]),
        "ckks_linear_proj_multi": (i32, [vp, C.POINTER(CProjDesc), u32, C.POINTER(CCt), C.POINTER(vp), C.POINTER(CEvk), u32, C.POINTER(CCt), vp, sz, vp]),
        "ckks_linear_proj_multi_workspace_bytes": (sz, [vp, C.POINTER(CProjDesc), u32, u32]),
    }
    for name, (res, args) in sig.items():
        f = getattr(L, name)
        f.restype, f.argtypes = res, args
    _lib = L
    return L


def kernel_launches() -> int:
    """Kernels launched by the library since it was loaded."""
    return int(load().ckks_kernel_launches())


class CkksError(RuntimeError):
    def __init__(self, code: int, detail: str = ""):
        self.code = code
        msg = load().ckks_status_string(code).decode()
        super().__init__(f"ckks_b200 error {code}: {msg}" + (f" ({detail})" if detail else ""))


@dataclass
class Ciphertext:
    data: torch.Tensor      # uint64 [ncomp][level][N] on the device
    scale: float

    @property
    def ncomp(self):
        return self.data.shape[0]

    @property
    def level(self):
        return self.data.shape[1]


@dataclass
class Plaintext:
    data: torch.Tensor      # uint64 [level][N]
    scale: float

    @property
    def level(self):
        return self.data.shape[0]


@dataclass
class SwitchKey:
    data: torch.Tensor      # uint64 [dnum][2][L+K][N]
    galois: int             # 0 for a relinearisation key


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _dev_u64(t: torch.Tensor) -> torch.Tensor:
    if not (t.is_cuda and t.dtype == torch.uint64 and t.is_contiguous()):
        raise TypeError("expected a contiguous CUDA uint64 tensor")
    return t


def _cct(ct: Ciphertext) -> CCt:
    _dev_u64(ct.data)
    return CCt(ct.data.data_ptr(), ct.level, ct.ncomp, ct.scale)


class Context:
    """Owns a library context (device tables) for one parameter set."""

    def __init__(self, log_n: int, q, p, dnum: int, device: int = 0):
        L = load()
        self.q = [int(x) for x in q]
        self.p = [int(x) for x in p]
        self.log_n, self.N, self.n = log_n, 1 << log_n, 1 << (log_n - 1)
        self.L, self.K, self.dnum = len(self.q), len(self.p), dnum
        self.device = torch.device("cuda", device)
        qa = (C.c_uint64 * max(1, self.L))(*self.q)
        pa = (C.c_uint64 * max(1, self.K))(*self.p)
        prm = CParams(log_n, self.L, self.K, dnum, qa, pa, device)
        h = C.c_void_p()
        rc = L.ckks_context_create(C.byref(prm), C.byref(h))
        if rc:
            raise CkksError(rc)
        self._h = h
        self._ws = None

    def close(self):
        if getattr(self, "_h", None):
            load().ckks_context_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -------------------------------------------------------------- helpers
    def _check(self, rc):
        if rc:
            raise CkksError(rc, load().ckks_last_cuda_error(self._h).decode() if rc == ERR_CUDA else "")

    def set_option(self, option: int, value: int):
        self._check(load().ckks_context_set_option(self._h, option, int(value)))

    def get_option(self, option: int) -> int:
        return int(load().ckks_context_get_option(self._h, option))

    def workspace(self, nbytes: int) -> torch.Tensor:
        """A cached device scratch buffer of at least nbytes (grown on demand by torch)."""
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = None
            self._ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=self.device)
        return self._ws

    def workspace_bytes(self, op: int, level: int, count: int = 0) -> int:
        return int(load().ckks_workspace_bytes(self._h, op, level, count))

    def galois_element(self, r: int) -> int:
        return int(load().ckks_galois_element(self._h, r))

    def empty_ct(self, level: int, ncomp: int = 2) -> Ciphertext:
        return Ciphertext(torch.empty((ncomp, level, self.N), dtype=torch.uint64, device=self.device), 0.0)

    # ------------------------------------------------------------------ ops
    def ntt(self, polys: torch.Tensor, first_prime: int = 0, stream=None):
        """In-place forward NTT of [batch][nlimbs][N] (or [nlimbs][N])."""
        _dev_u64(polys)
        nl = polys.shape[-2]
        batch = polys.numel() // (nl * self.N)
        self._check(load().ckks_ntt(self._h, polys.data_ptr(), batch, first_prime, nl, _stream_ptr(stream)))
        return polys

    def intt(self, polys: torch.Tensor, first_prime: int = 0, stream=None):
        _dev_u64(polys)
        nl = polys.shape[-2]
        batch = polys.numel() // (nl * self.N)
        self._check(load().ckks_intt(self._h, polys.data_ptr(), batch, first_prime, nl, _stream_ptr(stream)))
        return polys

    def ntt_butterfly_probe(self, iters: int, scratch: torch.Tensor, stream=None) -> int:
        """Launches the register-resident butterfly kernel; returns the number of butterflies it performs."""
        _dev_u64(scratch)
        n = C.c_uint64(0)
        self._check(load().ckks_ntt_butterfly_probe(self._h, iters, scratch.data_ptr(), scratch.numel(), C.byref(n), _stream_ptr(stream)))
        return int(n.value)

    def encode(self, re: torch.Tensor, im, scale: float, level: int, out: torch.Tensor = None, stream=None):
        """re/im: fp64 [batch][n] on the device -> uint64 [batch][level][N]."""
        if not (re.is_cuda and re.dtype == torch.float64 and re.is_contiguous()):
            raise TypeError("expected a contiguous CUDA float64 tensor")
        batch = re.numel() // self.n
        if out is None:
            out = torch.empty((batch, level, self.N), dtype=torch.uint64, device=self.device)
        nb = self.workspace_bytes(OP_ENCODE, level, batch)
        ws = self.workspace(nb)
        self._check(load().ckks_encode(self._h, re.data_ptr(), im.data_ptr() if im is not None else None, batch,
                                       float(scale), level, _dev_u64(out).data_ptr(), ws.data_ptr(), ws.numel(),
                                       _stream_ptr(stream)))
        return out

    def encode_range_flag(self, stream=None) -> int:
        return int(load().ckks_encode_range_flag(self._h, _stream_ptr(stream)))

    def device_status(self, stream=None) -> int:
        return int(load().ckks_device_status(self._h, _stream_ptr(stream)))

    def mul_plain_acc(self, cts, pt: Plaintext, accs=None, stream=None):
        """accs[s] (+)= cts[s] * pt.  accs None: fresh accumulators are returned."""
        init = accs is None
        if init:
            accs = [self.empty_ct(pt.level) for _ in cts]
        n = len(cts)
        ca = (CCt * n)(*[_cct(c) for c in cts])
        aa = (CCt * n)(*[_cct(a) for a in accs])
        cp = CPt(_dev_u64(pt.data).data_ptr(), pt.level, pt.scale)
        self._check(load().ckks_mul_plain_acc(self._h, ca, n, C.byref(cp), aa, int(init), _stream_ptr(stream)))
        for a, c in zip(accs, aa):
            a.scale = c.scale
        return accs

    def add(self, a: Ciphertext, b: Ciphertext, out: Ciphertext = None, stream=None):
        out = out or self.empty_ct(a.level, a.ncomp)
        co = _cct(out)
        self._check(load().ckks_add(self._h, C.byref(_cct(a)), C.byref(_cct(b)), C.byref(co), _stream_ptr(stream)))
        out.scale = co.scale
        return out

    def mul_relin(self, a: Ciphertext, b: Ciphertext, rlk: SwitchKey, out: Ciphertext = None, stream=None):
        out = out or self.empty_ct(a.level)
        ws = self.workspace(self.workspace_bytes(OP_MUL_RELIN, a.level))
        co, ck = _cct(out), CEvk(_dev_u64(rlk.data).data_ptr(), rlk.galois)
        self._check(load().ckks_mul_relin(self._h, C.byref(_cct(a)), C.byref(_cct(b)), C.byref(ck), C.byref(co),
                                          ws.data_ptr(), ws.numel(), _stream_ptr(stream)))
        out.scale = co.scale
        return out

    def mul_const(self, ct: Ciphertext, c: float, cscale: float = 0.0, out: Ciphertext = None, stream=None):
        """ct times the constant c encoded at cscale (0: the last prime of ct's level)."""
        out = out or Ciphertext(torch.empty_like(ct.data), ct.scale)
        co = _cct(out)
        self._check(load().ckks_mul_const(self._h, C.byref(_cct(ct)), c, cscale, C.byref(co), _stream_ptr(stream)))
        out.scale = co.scale
        return out

    def add_const(self, ct: Ciphertext, c: float, out: Ciphertext = None, stream=None):
        out = out or Ciphertext(torch.empty_like(ct.data), ct.scale)
        co = _cct(out)
        self._check(load().ckks_add_const(self._h, C.byref(_cct(ct)), c, C.byref(co), _stream_ptr(stream)))
        out.scale = co.scale
        return out

    def poly_eval(self, x: Ciphertext, coeffs, rlk: SwitchKey, stream=None):
        """sum_k coeffs[k] x^k by Horner's rule; returns a ciphertext at level x.level - degree."""
        d = len(coeffs) - 1
        out = self.empty_ct(x.level - d) if x.level > d else self.empty_ct(1)
        ws = self.workspace(self.workspace_bytes(OP_POLY_EVAL, x.level))
        ca = (C.c_double * (d + 1))(*[float(v) for v in coeffs])
        co = _cct(out)
        ck = CEvk(_dev_u64(rlk.data).data_ptr() if rlk is not None else None, rlk.galois if rlk is not None else 0)
        self._check(load().ckks_poly_eval(self._h, C.byref(_cct(x)), ca, d, C.byref(ck), C.byref(co), ws.data_ptr(), ws.numel(),
                                          _stream_ptr(stream)))
        out.scale = co.scale
        return out

    def poly_eval_tree(self, x: Ciphertext, coeffs, rlk: SwitchKey, stream=None):
        """sum_k coeffs[k] x^k in depth ceil(log2 degree) + 1; returns a ciphertext at level x.level - depth - 1."""
        d = len(coeffs) - 1
        depth = max(d - 1, 0).bit_length()
        out = self.empty_ct(max(x.level - depth - 1, 1))
        ws = self.workspace(self.workspace_bytes(OP_POLY_EVAL_TREE, x.level, d))
        ca = (C.c_double * (d + 1))(*[float(v) for v in coeffs])
        co = _cct(out)
        ck = CEvk(_dev_u64(rlk.data).data_ptr(), rlk.galois)
        self._check(load().ckks_poly_eval_tree(self._h, C.byref(_cct(x)), ca, d, C.byref(ck), C.byref(co), ws.data_ptr(), ws.numel(),
                                               _stream_ptr(stream)))
        out.scale = co.scale
        return out

    def poly_eval_bsgs(self, x: Ciphertext, coeffs, m: int, rlk: SwitchKey, stream=None):
        """sum_k coeffs[k] x^k by baby steps (blocks of m coefficients) and giant steps with one key switch for their sum."""
        d = len(coeffs) - 1
        need = int(load().ckks_poly_eval_bsgs_workspace_bytes(self._h, x.level, d, m))
        if need == 0:
            raise CkksError(ERR_ARG)
        ws = self.workspace(need)
        out = self.empty_ct(x.level)
        ca = (C.c_double * (d + 1))(*[float(v) for v in coeffs])
        co = _cct(out)
        ck = CEvk(_dev_u64(rlk.data).data_ptr(), rlk.galois)
        self._check(load().ckks_poly_eval_bsgs(self._h, C.byref(_cct(x)), ca, d, m, C.byref(ck), C.byref(co), ws.data_ptr(), ws.numel(),
                                               _stream_ptr(stream)))
        return Ciphertext(out.data.view(-1)[: 2 * co.level * self.N].view(2, co.level, self.N), co.scale)

    def poly_eval_bsgs_batch(self, xs, coeffs, m: int, rlk: SwitchKey, stream=None):
        """[poly_eval_bsgs(x, coeffs, m) for x in xs], the independent evaluations spread over the context's lanes."""
        d, n, level = len(coeffs) - 1, len(xs), xs[0].level
        need = int(load().ckks_poly_eval_bsgs_batch_workspace_bytes(self._h, level, d, m, n))
        if need == 0:
            raise CkksError(ERR_ARG)
        ws = self.workspace(need)
        outs = [self.empty_ct(level) for _ in xs]
        ca = (C.c_double * (d + 1))(*[float(v) for v in coeffs])
        xa = (CCt * n)(*[_cct(x) for x in xs])
        oa = (CCt * n)(*[_cct(o) for o in outs])
        ck = CEvk(_dev_u64(rlk.data).data_ptr(), rlk.galois)
        self._check(load().ckks_poly_eval_bsgs_batch(self._h, xa, n, ca, d, m, C.byref(ck), oa, ws.data_ptr(), ws.numel(), _stream_ptr(stream)))
        return [self._cut(o, c) for o, c in zip(outs, oa)]

    def softmax(self, ct: Ciphertext, shift: float, rounds: int, row_len: int, exp_coeffs, rsqrt_coeffs, rlk: SwitchKey, keys,
                ws: torch.Tensor = None, stream=None, exp_m: int = 0, rsqrt_m: int = 0):
        """Softmax by doubling with a public shift on one ciphertext of score rows (row r in slots i * (n / row_len) + r).
        exp_coeffs: p_exp(z / 2^rounds) as a polynomial in z; rsqrt_coeffs: [rounds][degree + 1]."""
        ec = (C.c_double * len(exp_coeffs))(*[float(v) for v in exp_coeffs])
        flat = [float(v) for row in rsqrt_coeffs for v in row]
        rc = (C.c_double * max(1, len(flat)))(*flat)
        rdeg = (len(rsqrt_coeffs[0]) - 1) if rounds else 0
        d = CSoftmaxDesc(float(shift), rounds, row_len, len(exp_coeffs) - 1, rdeg, C.cast(ec, C.POINTER(C.c_double)),
                         C.cast(rc, C.POINTER(C.c_double)), exp_m, rsqrt_m)
        need = int(load().ckks_softmax_workspace_bytes(self._h, C.byref(d), ct.level))
        if need == 0:
            raise CkksError(ERR_ARG)
        if ws is None:
            ws = self.workspace(need)
        out = self.empty_ct(ct.level)
        ci, co = _cct(ct), _cct(out)
        crlk = CEvk(_dev_u64(rlk.data).data_ptr(), 0)
        ka = (CEvk * max(1, len(keys)))(*[CEvk(_dev_u64(k.data).data_ptr(), k.galois) for k in keys])
        self._check(load().ckks_softmax(self._h, C.byref(d), C.byref(ci), C.byref(crlk), ka, len(keys), C.byref(co), ws.data_ptr(), ws.numel(),
                                        _stream_ptr(stream)))
        res = Ciphertext(out.data.view(-1)[: 2 * co.level * self.N].view(2, co.level, self.N), co.scale)
        return res

    # ------------------------------------------------------------ attention in the diagonal-block layout
    @staticmethod
    def _softmax_desc(shift, rounds, exp_coeffs, rsqrt_coeffs, row_len=0):
        ec = (C.c_double * len(exp_coeffs))(*[float(v) for v in exp_coeffs])
        flat = [float(v) for row in rsqrt_coeffs for v in row] if rounds else []
        rc = (C.c_double * max(1, len(flat)))(*flat)
        rdeg = (len(rsqrt_coeffs[0]) - 1) if rounds else 0
        d = CSoftmaxDesc(float(shift), rounds, row_len, len(exp_coeffs) - 1, rdeg, C.cast(ec, C.POINTER(C.c_double)),
                         C.cast(rc, C.POINTER(C.c_double)), 0, 0)
        d._keep = (ec, rc)          # the arrays must outlive the descriptor
        return d

    def _cut(self, out: Ciphertext, c: CCt) -> Ciphertext:
        """The first c.level limbs per component of a buffer written densely as [2][c.level][N]."""
        return Ciphertext(out.data.view(-1)[: 2 * c.level * self.N].view(2, c.level, self.N), c.scale)

    def attention_rotations(self, tokens: int, heads: int, diag_block: int, group_baby: int = 1):
        d = CAttnDesc(tokens, heads, diag_block, group_baby)
        n = load().ckks_attention_rotations(self._h, C.byref(d), None, 0)
        if n < 0:
            raise CkksError(n)
        buf = (C.c_int64 * max(n, 1))()
        load().ckks_attention_rotations(self._h, C.byref(d), buf, n)
        return list(buf)[:n]

    def attention_pack_rotations(self, kind: int, dim: int, tokens: int, heads: int, diag_block: int, token_inner: int):
        d = CAttnDesc(tokens, heads, diag_block, 1, token_inner)
        n = load().ckks_attention_pack_rotations(self._h, C.byref(d), kind, dim, None, 0)
        if n < 0:
            raise CkksError(n)
        buf = (C.c_int64 * max(n, 1))()
        load().ckks_attention_pack_rotations(self._h, C.byref(d), kind, dim, buf, n)
        return list(buf)[:n]

    def attention_pack(self, kind: int, cts, dim: int, keys, tokens: int, heads: int, diag_block: int, token_inner: int, stream=None):
        """Conversion between token-shard ciphertexts in channel-major feature order and the attention operands: kind
        ATTN_QUERY / ATTN_KEY_VALUE take the shards to dim operands, ATTN_TO_SHARDS takes dim outputs back to the shards."""
        d = CAttnDesc(tokens, heads, diag_block, 1, token_inner)
        level = cts[0].level
        need = int(load().ckks_attention_pack_workspace_bytes(self._h, C.byref(d), kind, level, dim))
        if need == 0:
            raise CkksError(ERR_UNSUPPORTED)
        ws = self.workspace(need)
        nout = tokens // max(1, token_inner) if kind == ATTN_TO_SHARDS else dim
        outs = [self.empty_ct(level - 1) for _ in range(nout)]
        ia = (CCt * len(cts))(*[_cct(x) for x in cts])
        oa = (CCt * nout)(*[_cct(x) for x in outs])
        ra = (CEvk * max(1, len(keys)))(*[CEvk(_dev_u64(x.data).data_ptr(), x.galois) for x in keys])
        self._check(load().ckks_attention_pack(self._h, C.byref(d), kind, ia, dim, ra, len(keys), oa, ws.data_ptr(), ws.numel(), _stream_ptr(stream)))
        return [self._cut(o, c) for o, c in zip(outs, oa)]

    def attention_scores(self, q, k, rlk: SwitchKey, keys, tokens, heads, diag_block, ws: torch.Tensor = None, stream=None,
                         group_baby: int = 1):
        """Score ciphertexts S_g (one per group of diag_block diagonals) from the channel operands q[d], k[d]; group_baby > 1
        splits the groups into baby and giant steps."""
        d = CAttnDesc(tokens, heads, diag_block, group_baby)
        level, G = q[0].level, tokens // diag_block
        outs = [self.empty_ct(level - 1) for _ in range(G)]
        if ws is None:
            ws = self.workspace(int(load().ckks_attention_scores_workspace_bytes(self._h, C.byref(d), level, len(q))))
        qa = (CCt * len(q))(*[_cct(x) for x in q])
        ka = (CCt * len(k))(*[_cct(x) for x in k])
        oa = (CCt * G)(*[_cct(x) for x in outs])
        ck = CEvk(_dev_u64(rlk.data).data_ptr(), 0)
        ra = (CEvk * max(1, len(keys)))(*[CEvk(_dev_u64(x.data).data_ptr(), x.galois) for x in keys])
        self._check(load().ckks_attention_scores(self._h, C.byref(d), qa, ka, len(q), C.byref(ck), ra, len(keys), oa, ws.data_ptr(), ws.numel(),
                                                 _stream_ptr(stream)))
        for o, c in zip(outs, oa):
            o.scale = c.scale
        return outs

    def softmax_rows(self, cts, shift, rounds, exp_coeffs, rsqrt_coeffs, rlk: SwitchKey, keys, tokens, heads, diag_block, stream=None):
        """Softmax by doubling on score rows spread over the groups' ciphertexts (slots (e, i, h) of every group)."""
        d = CAttnDesc(tokens, heads, diag_block, 1)
        sd = self._softmax_desc(shift, rounds, exp_coeffs, rsqrt_coeffs)
        level = cts[0].level
        need = int(load().ckks_softmax_rows_workspace_bytes(self._h, C.byref(d), C.byref(sd), level))
        if need == 0:
            raise CkksError(ERR_ARG)
        ws = self.workspace(need)
        outs = [self.empty_ct(level) for _ in cts]
        ia = (CCt * len(cts))(*[_cct(x) for x in cts])
        oa = (CCt * len(outs))(*[_cct(x) for x in outs])
        ck = CEvk(_dev_u64(rlk.data).data_ptr(), 0)
        ra = (CEvk * max(1, len(keys)))(*[CEvk(_dev_u64(x.data).data_ptr(), x.galois) for x in keys])
        self._check(load().ckks_softmax_rows(self._h, C.byref(d), C.byref(sd), ia, C.byref(ck), ra, len(keys), oa, ws.data_ptr(), ws.numel(),
                                             _stream_ptr(stream)))
        return [self._cut(o, c) for o, c in zip(outs, oa)]

    def attention_values(self, probs, v, rlk: SwitchKey, keys, tokens, heads, diag_block, stream=None):
        """Output channels sum over key tokens of probability x value, in the query operand's layout."""
        d = CAttnDesc(tokens, heads, diag_block, 1)
        lp = probs[0].level
        ws = self.workspace(int(load().ckks_attention_values_workspace_bytes(self._h, C.byref(d), lp)))
        outs = [self.empty_ct(lp - 1) for _ in v]
        pa = (CCt * len(probs))(*[_cct(x) for x in probs])
        va = (CCt * len(v))(*[_cct(x) for x in v])
        oa = (CCt * len(outs))(*[_cct(x) for x in outs])
        ck = CEvk(_dev_u64(rlk.data).data_ptr(), 0)
        ra = (CEvk * max(1, len(keys)))(*[CEvk(_dev_u64(x.data).data_ptr(), x.galois) for x in keys])
        self._check(load().ckks_attention_values(self._h, C.byref(d), pa, va, len(v), C.byref(ck), ra, len(keys), oa, ws.data_ptr(), ws.numel(),
                                                 _stream_ptr(stream)))
        for o, c in zip(outs, oa):
            o.scale = c.scale
        return outs

    def attention(self, q, k, v, shift, rounds, exp_coeffs, rsqrt_coeffs, rlk: SwitchKey, keys, tokens, heads, diag_block,
                  ws: torch.Tensor = None, stream=None, group_baby: int = 1):
        """Scores, Softmax over the score rows and probability x value in one call; returns the output channels."""
        d = CAttnDesc(tokens, heads, diag_block, group_baby)
        sd = self._softmax_desc(shift, rounds, exp_coeffs, rsqrt_coeffs)
        level = q[0].level
        need = int(load().ckks_attention_workspace_bytes(self._h, C.byref(d), C.byref(sd), level, len(q)))
        if need == 0:
            raise CkksError(ERR_ARG)
        if ws is None:
            ws = self.workspace(need)
        outs = [self.empty_ct(level - 1) for _ in v]
        qa = (CCt * len(q))(*[_cct(x) for x in q])
        ka = (CCt * len(k))(*[_cct(x) for x in k])
        va = (CCt * len(v))(*[_cct(x) for x in v])
        oa = (CCt * len(outs))(*[_cct(x) for x in outs])
        ck = CEvk(_dev_u64(rlk.data).data_ptr(), 0)
        ra = (CEvk * max(1, len(keys)))(*[CEvk(_dev_u64(x.data).data_ptr(), x.galois) for x in keys])
        self._check(load().ckks_attention(self._h, C.byref(d), C.byref(sd), qa, ka, len(q), va, len(v), C.byref(ck), ra, len(keys), oa,
                                          ws.data_ptr(), ws.numel(), _stream_ptr(stream)))
        return [self._cut(o, c) for o, c in zip(outs, oa)]

    def rotate_sum(self, cts, keys, out: Ciphertext = None, ws: torch.Tensor = None, stream=None):
        """sum_i rotate(cts[i], keys[i]) formed in the key-switching basis and divided by P once."""
        level = cts[0].level
        out = out or self.empty_ct(level)
        if ws is None:
            ws = self.workspace(self.workspace_bytes(OP_ROTATE_SUM, level, len(cts)))
        ia = (CCt * len(cts))(*[_cct(x) for x in cts])
        ka = (CEvk * len(keys))(*[CEvk(_dev_u64(k.data).data_ptr(), k.galois) for k in keys])
        co = _cct(out)
        self._check(load().ckks_rotate_sum(self._h, ia, ka, len(cts), C.byref(co), ws.data_ptr(), ws.numel(), _stream_ptr(stream)))
        out.scale = co.scale
        return out

    def rotate_batch(self, cts, key: SwitchKey, outs=None, ws: torch.Tensor = None, stream=None):
        """[rotate(ct, key) for ct in cts] with the key switches of up to 16 ciphertexts running side by side."""
        level = cts[0].level
        outs = outs or [self.empty_ct(level) for _ in cts]
        if ws is None:
            ws = self.workspace(self.workspace_bytes(OP_ROTATE_BATCH, level, len(cts)))
        ia = (CCt * len(cts))(*[_cct(x) for x in cts])
        oa = (CCt * len(outs))(*[_cct(x) for x in outs])
        ck = CEvk(_dev_u64(key.data).data_ptr(), key.galois)
        self._check(load().ckks_rotate_batch(self._h, ia, len(cts), C.byref(ck), oa, ws.data_ptr(), ws.numel(), _stream_ptr(stream)))
        for o, c in zip(outs, oa):
            o.scale = c.scale
        return outs

    def mul_relin_batch(self, a, b, rlk: SwitchKey, outs=None, ws: torch.Tensor = None, stream=None):
        """[mul_relin(a[i], b[i]) for i] with the key switches of up to 16 products running side by side."""
        if len(a) != len(b) or not a:
            raise ValueError("a and b must be non-empty lists of the same length")
        level = a[0].level
        outs = outs or [self.empty_ct(level) for _ in a]
        if ws is None:
            ws = self.workspace(self.workspace_bytes(OP_MUL_RELIN_BATCH, level, len(a)))
        aa = (CCt * len(a))(*[_cct(x) for x in a])
        ba = (CCt * len(b))(*[_cct(x) for x in b])
        oa = (CCt * len(outs))(*[_cct(x) for x in outs])
        ck = CEvk(_dev_u64(rlk.data).data_ptr(), rlk.galois)
        self._check(load().ckks_mul_relin_batch(self._h, aa, ba, len(a), C.byref(ck), oa, ws.data_ptr(), ws.numel(), _stream_ptr(stream)))
        for o, c in zip(outs, oa):
            o.scale = c.scale
        return outs

    def mul_relin_sum(self, a, b, rlk: SwitchKey, out: Ciphertext = None, stream=None):
        """relin(sum_i a[i] (x) b[i]) with a single key switch; a, b: equally long lists of ciphertexts."""
        if len(a) != len(b) or not a:
            raise ValueError("a and b must be non-empty lists of the same length")
        level = a[0].level
        out = out or self.empty_ct(level)
        ws = self.workspace(self.workspace_bytes(OP_MUL_RELIN, level))
        aa = (CCt * len(a))(*[_cct(x) for x in a])
        ba = (CCt * len(b))(*[_cct(x) for x in b])
        co, ck = _cct(out), CEvk(_dev_u64(rlk.data).data_ptr(), rlk.galois)
        self._check(load().ckks_mul_relin_sum(self._h, aa, ba, len(a), C.byref(ck), C.byref(co), ws.data_ptr(), ws.numel(),
                                              _stream_ptr(stream)))
        out.scale = co.scale
        return out

    def rotate(self, ct: Ciphertext, key: SwitchKey, out: Ciphertext = None, stream=None):
        out = out or self.empty_ct(ct.level)
        ws = self.workspace(self.workspace_bytes(OP_ROTATE, ct.level))
        co, ck = _cct(out), CEvk(_dev_u64(key.data).data_ptr(), key.galois)
        self._check(load().ckks_rotate(self._h, C.byref(_cct(ct)), C.byref(ck), C.byref(co), ws.data_ptr(), ws.numel(),
                                       _stream_ptr(stream)))
        out.scale = co.scale
        return out

    def rotate_hoisted(self, ct: Ciphertext, keys, outs=None, stream=None):
        n = len(keys)
        outs = outs or [self.empty_ct(ct.level) for _ in keys]
        ws = self.workspace(self.workspace_bytes(OP_ROTATE_HOISTED, ct.level, n))
        ka = (CEvk * n)(*[CEvk(_dev_u64(k.data).data_ptr(), k.galois) for k in keys])
        oa = (CCt * n)(*[_cct(o) for o in outs])
        self._check(load().ckks_rotate_hoisted(self._h, C.byref(_cct(ct)), ka, n, oa, ws.data_ptr(), ws.numel(),
                                               _stream_ptr(stream)))
        for o, c in zip(outs, oa):
            o.scale = c.scale
        return outs

    def linear_proj_multi(self, cts, Ws, keys, d_in, d_outs, tokens_per_shard, nshards, baby, pt_scale=0.0,
                          ws: torch.Tensor = None, stream=None, lazy_moddown=False):
        """[X W_0, X W_1, ...] for weight matrices sharing their input (Q/K/V, gate/up): the baby-step rotations of
        the inputs are computed once.  Returns one list of output ciphertexts per matrix, each bit-identical to a
        separate linear_proj call."""
        nmat = len(Ws)
        for W, d_out in zip(Ws, d_outs):
            if not (W.is_cuda and W.dtype == torch.float64 and W.is_contiguous() and tuple(W.shape) == (d_in, d_out)):
                raise TypeError("every W must be a contiguous CUDA float64 [d_in][d_out] tensor")
        da = (CProjDesc * nmat)(*[self._desc(d_in, d_out, tokens_per_shard, nshards, baby, pt_scale, lazy_moddown) for d_out in d_outs])
        level = cts[0].level
        F = self.n // tokens_per_shard
        outs = [[self.empty_ct(level - 1) for _ in range(nshards * -(-d_out // F))] for d_out in d_outs]
        flat = [o for m in outs for o in m]
        if ws is None:
            ws = self.workspace(int(load().ckks_linear_proj_multi_workspace_bytes(self._h, da, nmat, level)))
        ia = (CCt * len(cts))(*[_cct(c) for c in cts])
        oa = (CCt * len(flat))(*[_cct(o) for o in flat])
        wa = (C.c_void_p * nmat)(*[W.data_ptr() for W in Ws])
        ka = (CEvk * len(keys))(*[CEvk(_dev_u64(k.data).data_ptr(), k.galois) for k in keys])
        self._check(load().ckks_linear_proj_multi(self._h, da, nmat, ia, wa, ka, len(keys), oa, ws.data_ptr(), ws.numel(),
                                                  _stream_ptr(stream)))
        for o, c in zip(flat, oa):
            o.scale = c.scale
        return outs

    def rescale(self, ct: Ciphertext, out: Ciphertext = None, stream=None):
        out = out or self.empty_ct(ct.level - 1, ct.ncomp)
        ws = self.workspace(self.workspace_bytes(OP_RESCALE, ct.level))
        co = _cct(out)
        co.level = ct.level - 1
        self._check(load().ckks_rescale(self._h, C.byref(_cct(ct)), C.byref(co), ws.data_ptr(), ws.numel(), _stream_ptr(stream)))
        out.scale = co.scale
        return out

    # ----------------------------------------------------- linear projection
    def _desc(self, d_in, d_out, tokens_per_shard, nshards, baby, pt_scale=0.0, lazy_moddown=False):
        return CProjDesc(d_in, d_out, tokens_per_shard, nshards, baby, PROJ_LAZY_MODDOWN if lazy_moddown else 0, float(pt_scale))

    def linear_proj_rotations(self, d_in, d_out, tokens_per_shard, nshards, baby):
        d = self._desc(d_in, d_out, tokens_per_shard, nshards, baby)
        n = load().ckks_linear_proj_rotations(self._h, C.byref(d), None, 0)
        if n < 0:
            raise CkksError(n)
        buf = (C.c_int64 * max(n, 1))()
        load().ckks_linear_proj_rotations(self._h, C.byref(d), buf, n)
        return list(buf)[:n]

    def linear_proj_workspace_bytes(self, d_in, d_out, tokens_per_shard, nshards, baby, level, lazy_moddown=False):
        d = self._desc(d_in, d_out, tokens_per_shard, nshards, baby, 0.0, lazy_moddown)
        return int(load().ckks_linear_proj_workspace_bytes(self._h, C.byref(d), level))

    def linear_proj(self, cts, W: torch.Tensor, keys, d_in, d_out, tokens_per_shard, nshards, baby, pt_scale=0.0,
                    outs=None, ws: torch.Tensor = None, stream=None, lazy_moddown=False):
        """Y = X W.  cts: nshards * n_in_blocks ciphertexts; W: fp64 [d_in][d_out] on the device;
        keys: rotation SwitchKeys.  Returns nshards * n_out_blocks ciphertexts at level - 1."""
        if not (W.is_cuda and W.dtype == torch.float64 and W.is_contiguous() and tuple(W.shape) == (d_in, d_out)):
            raise TypeError("W must be a contiguous CUDA float64 [d_in][d_out] tensor")
        d = self._desc(d_in, d_out, tokens_per_shard, nshards, baby, pt_scale, lazy_moddown)
        level = cts[0].level
        F = self.n // tokens_per_shard
        nob = -(-d_out // F)
        if outs is None:
            outs = [self.empty_ct(level - 1) for _ in range(nshards * nob)]
        if ws is None:
            ws = self.workspace(self.linear_proj_workspace_bytes(d_in, d_out, tokens_per_shard, nshards, baby, level, lazy_moddown))
        ia = (CCt * len(cts))(*[_cct(c) for c in cts])
        oa = (CCt * len(outs))(*[_cct(o) for o in outs])
        for o in oa:
            o.level = level - 1
        ka = (CEvk * len(keys))(*[CEvk(_dev_u64(k.data).data_ptr(), k.galois) for k in keys])
        self._check(load().ckks_linear_proj(self._h, C.byref(d), ia, W.data_ptr(), ka, len(keys), oa, ws.data_ptr(),
                                            ws.numel(), _stream_ptr(stream)))
        for o, c in zip(outs, oa):
            o.scale = c.scale
        return outs

"""Python face of the CPU checker (test infrastructure, not the product).

Thin ctypes wrappers over ``ckks_oracle.c`` plus the two composites that are
easier to read in Python than in C: key derivation helpers and the linear
projection by diagonals (Eq. 5) in its baby-step/giant-step schedule.

Nothing here imports the CUDA package.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass

import numpy as np

from . import build as _build

_u64p = C.POINTER(C.c_uint64)
_i64p = C.POINTER(C.c_int64)
_f64p = C.POINTER(C.c_double)
_ldp = C.POINTER(C.c_longdouble)


def _p(a, typ):
    return a.ctypes.data_as(typ) if a is not None else None


def _u64(a):
    a = np.ascontiguousarray(a, dtype=np.uint64)
    return a


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        L.orc_create.restype = C.c_void_p
        L.orc_create.argtypes = [C.c_uint32] * 4 + [_u64p, _u64p]
        L.orc_destroy.argtypes = [C.c_void_p]
        L.orc_root.restype = C.c_uint64
        L.orc_root.argtypes = [C.c_void_p, C.c_uint32]
        L.orc_galois_element.restype = C.c_uint64
        L.orc_galois_element.argtypes = [C.c_void_p, C.c_int64]
        L.orc_encode_coeffs.restype = C.c_int
        L.orc_encode.restype = C.c_int
        _lib = L
    return _lib


@dataclass
class ProjDesc:
    """Shape of one linear projection Y = X W in the feature-major token-shard layout."""
    d_in: int
    d_out: int
    tokens_per_shard: int
    nshards: int
    baby: int
    pt_scale: float = 0.0      # 0 => q_{level-1}
    lazy_moddown: bool = False  # giant-step results summed in the extended basis, one ModDown per output


@dataclass
class AttnDesc:
    """Shape of one attention block in the diagonal-block layout.  Every operand and every score ciphertext uses the slot
    index ((e * tokens + i) * heads + h) * R + r: i a token position, h a head, e < diag_block one of the score diagonals
    a ciphertext holds side by side, r < R = n / (diag_block * tokens * heads) trailing copies."""
    tokens: int
    heads: int
    diag_block: int
    group_baby: int = 1      # attention_scores: baby-step count of the split of the score groups (1 = every group by itself)
    token_inner: int = 1     # tokens kept innermost in the slot index (divides diag_block): slot =
                             # (((e P + pos) heads + h) token_inner + t) R + r, token = pos token_inner + t, P = tokens / token_inner

    def groups(self) -> int:
        return self.tokens // self.diag_block


class Oracle:
    def __init__(self, log_n: int, q, p, dnum: int):
        self.log_n, self.N, self.n, self.M = log_n, 1 << log_n, 1 << (log_n - 1), 2 << log_n
        self.q = [int(x) for x in q]
        self.p = [int(x) for x in p]
        self.L, self.K, self.dnum = len(self.q), len(self.p), dnum
        self.alpha = -(-self.L // dnum)
        self.mod = self.q + self.p
        qa = np.array(self.q, dtype=np.uint64)
        pa = np.array(self.p if self.p else [0], dtype=np.uint64)
        self._h = C.c_void_p(lib().orc_create(log_n, self.L, self.K, dnum, _p(qa, _u64p), _p(pa, _u64p)))

    def __del__(self):
        try:
            lib().orc_destroy(self._h)
        except Exception:
            pass

    # ------------------------------------------------------------ parameters
    def root(self, t: int) -> int:
        return int(lib().orc_root(self._h, t))

    def galois_element(self, r: int) -> int:
        return int(lib().orc_galois_element(self._h, r))

    # ------------------------------------------------------------------- NTT
    def ntt_definition(self, a, t: int):
        a = _u64(a); out = np.empty_like(a)
        lib().orc_ntt_definition(self._h, C.c_uint32(t), _p(a, _u64p), _p(out, _u64p))
        return out

    def intt_definition(self, a, t: int):
        a = _u64(a); out = np.empty_like(a)
        lib().orc_intt_definition(self._h, C.c_uint32(t), _p(a, _u64p), _p(out, _u64p))
        return out

    def ntt(self, polys, first: int = 0):
        """polys [..., nlimbs, N] -> forward NTT of every limb (copy)."""
        a = _u64(polys).copy()
        nl = a.shape[-2] if a.ndim >= 2 else 1
        batch = a.size // (nl * self.N)
        lib().orc_ntt_batch(self._h, _p(a, _u64p), C.c_uint32(batch), C.c_uint32(first), C.c_uint32(nl))
        return a

    def intt(self, polys, first: int = 0):
        a = _u64(polys).copy()
        nl = a.shape[-2] if a.ndim >= 2 else 1
        batch = a.size // (nl * self.N)
        lib().orc_intt_batch(self._h, _p(a, _u64p), C.c_uint32(batch), C.c_uint32(first), C.c_uint32(nl))
        return a

    # ---------------------------------------------------------------- encode
    def encode_coeffs(self, z, scale: float):
        z = np.asarray(z)
        re = np.ascontiguousarray(z.real, dtype=np.float64)
        im = np.ascontiguousarray(z.imag, dtype=np.float64) if np.iscomplexobj(z) else None
        m = np.empty(self.N, dtype=np.int64)
        rc = lib().orc_encode_coeffs(self._h, _p(re, _f64p), _p(im, _f64p), C.c_double(scale), _p(m, _i64p))
        if rc:
            raise OverflowError("scaled value out of range")
        return m

    def encode(self, z, scale: float, level: int):
        z = np.asarray(z)
        re = np.ascontiguousarray(z.real, dtype=np.float64)
        im = np.ascontiguousarray(z.imag, dtype=np.float64) if np.iscomplexobj(z) else None
        out = np.empty((level, self.N), dtype=np.uint64)
        rc = lib().orc_encode(self._h, _p(re, _f64p), _p(im, _f64p), C.c_double(scale), C.c_uint32(level), _p(out, _u64p))
        if rc:
            raise OverflowError("scaled value out of range")
        return out

    def small_to_limbs(self, poly, first: int, nl: int):
        poly = np.ascontiguousarray(poly, dtype=np.int64)
        out = np.empty((nl, self.N), dtype=np.uint64)
        lib().orc_small_to_limbs(self._h, _p(poly, _i64p), C.c_uint32(first), C.c_uint32(nl), _p(out, _u64p))
        return out

    def decode(self, coeffs, scale: float, direct: bool = False):
        m = np.ascontiguousarray(coeffs, dtype=np.longdouble)
        re = np.empty(self.n); im = np.empty(self.n)
        f = lib().orc_decode_direct if direct else lib().orc_decode
        f(self._h, _p(m, _ldp), C.c_double(scale), _p(re, _f64p), _p(im, _f64p))
        return re + 1j * im

    # ------------------------------------------------- keys, encrypt, decrypt
    def encrypt(self, pt, a, e, s):
        pt = _u64(pt); level = pt.shape[0]
        a = _u64(a); e = np.ascontiguousarray(e, dtype=np.int64); s = np.ascontiguousarray(s, dtype=np.int64)
        ct = np.empty((2, level, self.N), dtype=np.uint64)
        lib().orc_encrypt(self._h, _p(pt, _u64p), _p(a, _u64p), _p(e, _i64p), _p(s, _i64p), C.c_uint32(level), _p(ct, _u64p))
        return ct

    def decrypt(self, ct, s, exact: bool = False):
        """Centred plaintext coefficients: long double array, or Python ints when exact."""
        ct = _u64(ct); ncomp, level = ct.shape[0], ct.shape[1]
        s = np.ascontiguousarray(s, dtype=np.int64)
        if exact:
            buf = np.empty((self.N, 2), dtype=np.uint64)
            lib().orc_decrypt(self._h, _p(ct, _u64p), C.c_uint32(ncomp), C.c_uint32(level), _p(s, _i64p),
                              C.c_void_p(buf.ctypes.data), None)
            out = []
            for lo, hi in buf.tolist():
                v = (hi << 64) | lo
                out.append(v - (1 << 128) if v >> 127 else v)
            return out
        m = np.empty(self.N, dtype=np.longdouble)
        lib().orc_decrypt(self._h, _p(ct, _u64p), C.c_uint32(ncomp), C.c_uint32(level), _p(s, _i64p), None, _p(m, _ldp))
        return m

    def decrypt_decode(self, ct, s, scale: float):
        return self.decode(self.decrypt(ct, s), scale)

    def switch_keygen(self, s, sprime_limbs, a, e):
        s = np.ascontiguousarray(s, dtype=np.int64)
        sp = _u64(sprime_limbs); a = _u64(a); e = np.ascontiguousarray(e, dtype=np.int64)
        T = self.L + self.K
        assert sp.shape == (T, self.N) and a.shape == (self.dnum, T, self.N) and e.shape == (self.dnum, self.N)
        evk = np.empty((self.dnum, 2, T, self.N), dtype=np.uint64)
        lib().orc_switch_keygen(self._h, _p(s, _i64p), _p(sp, _u64p), _p(a, _u64p), _p(e, _i64p), _p(evk, _u64p))
        return evk

    def automorphism_small(self, a, g: int):
        a = np.ascontiguousarray(a, dtype=np.int64); out = np.empty_like(a)
        lib().orc_automorphism_small(self._h, _p(a, _i64p), C.c_uint64(g), _p(out, _i64p))
        return out

    def rotation_key(self, s, g: int, a, e):
        """Key switching sigma_g(s) -> s."""
        sg = self.automorphism_small(s, g)
        return self.switch_keygen(s, self.small_to_limbs(sg, 0, self.L + self.K), a, e)

    def relin_key(self, s, a, e):
        """Key switching s^2 -> s."""
        T = self.L + self.K
        sl = self.small_to_limbs(s, 0, T)
        s2 = np.empty_like(sl)
        lib().orc_pointwise_mul(self._h, _p(sl, _u64p), _p(sl, _u64p), C.c_uint32(0), C.c_uint32(T), _p(s2, _u64p))
        return self.switch_keygen(s, s2, a, e)

    # ------------------------------------------------------------- pointwise
    def mul_plain_acc(self, ct, pt, acc=None):
        ct = _u64(ct); pt = _u64(pt); level = ct.shape[1]
        init = acc is None
        if init:
            acc = np.empty_like(ct)
        lib().orc_mul_plain_acc(self._h, _p(ct, _u64p), _p(pt, _u64p), _p(acc, _u64p), C.c_uint32(level), C.c_int(int(init)))
        return acc

    def add(self, a, b):
        a = _u64(a); b = _u64(b); out = np.empty_like(a)
        lib().orc_add(self._h, _p(a, _u64p), _p(b, _u64p), _p(out, _u64p), C.c_uint32(a.shape[0]), C.c_uint32(a.shape[1]))
        return out

    def mul_const(self, ct, v: int):
        """ct times the constant polynomial v (a signed integer)."""
        ct = _u64(ct); out = np.empty_like(ct)
        lib().orc_mul_const(self._h, _p(ct, _u64p), C.c_int64(v), C.c_uint32(ct.shape[0]), C.c_uint32(ct.shape[1]), _p(out, _u64p))
        return out

    def add_const(self, ct, v: int):
        """ct plus the constant polynomial v (a signed integer), i.e. v added to component 0."""
        ct = _u64(ct); out = np.empty_like(ct)
        lib().orc_add_const(self._h, _p(ct, _u64p), C.c_int64(v), C.c_uint32(ct.shape[0]), C.c_uint32(ct.shape[1]), _p(out, _u64p))
        return out

    def poly_eval(self, x, scale: float, coeffs, rlk):
        """Horner evaluation of sum_k coeffs[k] x^k (degree d = len(coeffs) - 1 >= 1) on a ciphertext, in this order:
        r = x * round(c_d * q_{l-1});  rescale;  r += round(c_{d-1} * scale(r));  then for k = d-2 .. 0:
        r = mul_relin(r, x truncated to r's level);  rescale;  r += round(c_k * scale(r)).
        Scales are tracked as doubles, multiplied and divided in exactly this order.  Returns (ct, scale) at level
        l - d."""
        x = _u64(x); level = x.shape[1]; d = len(coeffs) - 1
        if d < 1 or level < d + 1:
            raise ValueError("degree must be >= 1 and the ciphertext needs degree + 1 limbs")
        cs = float(self.q[level - 1])
        r = self.mul_const(x, int(np.rint(coeffs[d] * cs)))
        rs = scale * cs
        r = self.rescale(r); rs = rs / float(self.q[level - 1]); lvl = level - 1
        r = self.add_const(r, int(np.rint(coeffs[d - 1] * rs)))
        for k in range(d - 2, -1, -1):
            r = self.mul_relin(r, x[:, :lvl], rlk); rs = rs * scale
            r = self.rescale(r); rs = rs / float(self.q[lvl - 1]); lvl -= 1
            r = self.add_const(r, int(np.rint(coeffs[k] * rs)))
        return r, rs

    def poly_eval_tree(self, x, scale: float, coeffs, rlk):
        """sum_k coeffs[k] x^k (degree d >= 2) in depth ceil(log2 d) + 1 instead of d.  Order of steps:
        powers: pw[1] = x; for k = 2..d: a = k // 2, b = k - a, lv = min(level[a], level[b]),
          pw[k] = rescale(mul_relin(pw[a][:, :lv], pw[b][:, :lv])), scale[k] = scale[a] * scale[b] / q_{lv-1};
        combination at level Lt = level[d] and scale T = scale(x) * q_{Lt-1}:
          acc = sum over k = 1..d with coeffs[k] != 0, in increasing k, of pw[k][:, :Lt] * round(coeffs[k] * (T / scale[k]));
        result = rescale(acc) + round(coeffs[0] * (T / q_{Lt-1})).  Returns (ct, scale) at level Lt - 1."""
        x = _u64(x); level = x.shape[1]; d = len(coeffs) - 1
        depth = (d - 1).bit_length()
        if d < 2 or level < depth + 2:
            raise ValueError("degree must be >= 2 and the ciphertext needs ceil(log2 degree) + 2 limbs")
        pw, sc = {1: x}, {1: scale}
        for k in range(2, d + 1):
            a = k // 2; b = k - a
            lv = min(pw[a].shape[1], pw[b].shape[1])
            t = self.mul_relin(pw[a][:, :lv], pw[b][:, :lv], rlk)
            pw[k] = self.rescale(t)
            sc[k] = sc[a] * sc[b] / float(self.q[lv - 1])
        Lt = pw[d].shape[1]
        T = scale * float(self.q[Lt - 1])
        acc = None
        for k in range(1, d + 1):
            if coeffs[k] == 0.0:
                continue
            term = self.mul_const(pw[k][:, :Lt], int(np.rint(coeffs[k] * (T / sc[k]))))
            acc = term if acc is None else self.add(acc, term)
        if acc is None:
            raise ValueError("all non-constant coefficients are zero")
        out = self.rescale(acc)
        so = T / float(self.q[Lt - 1])
        return self.add_const(out, int(np.rint(coeffs[0] * so))), so

    def poly_eval_bsgs(self, x, scale: float, coeffs, rlk, m: int):
        """sum_k coeffs[k] x^k by baby steps and giant steps (m a power of two, 2 <= m <= degree): about m + 2 d / m
        products instead of the tree's d - 1, one key switch for the whole giant-step sum.  With blocks
        B_i(x) = sum_{j<m} coeffs[i m + j] x^j, G = d // m + 1 and y = x^m the polynomial is sum_{i<G} B_i(x) y^i.
        Order of steps:
          baby powers pw[k], k = 2..m, and giant powers gp[i] = y^i, i = 2..G-1, as poly_eval_tree forms its powers
            (operands k // 2 and k - k // 2, truncated to their common level; mul_relin; rescale);
          Lb = level of pw[m-1] (of x for m = 2), Lc = min(level of gp[G-1], Lb - 1), Tp = scale(x) * q_{Lc-1};
          block i >= 1 with a non-constant part: at level Lb and scale Ti = (Tp / scale(gp[i])) * q_{Lb-1} the sum over
            j = 1..m-1 (coefficient != 0, increasing j) of pw[j][:Lb] * round(c (Ti / scale(pw[j]))), rescaled, plus
            round(coeffs[i m] * (Ti / q_{Lb-1})); a block that is only a constant enters as gp[i][:Lc] * round(c (Tp / scale(gp[i])));
          S = mul_relin_sum of the non-constant blocks (truncated to Lc) with their gp[i][:Lc], in increasing i;
          then block 0's terms pw[j][:Lc] * round(c_j (Tp / scale(pw[j]))), j = 1..m-1, and the constant-only blocks are added
          to S in that order; result = rescale(S) + round(coeffs[0] * (Tp / q_{Lc-1})).
        Returns (ct, scale = Tp / q_{Lc-1}) at level Lc - 1."""
        x = _u64(x); level = x.shape[1]; d = len(coeffs) - 1
        if m < 2 or m & (m - 1) or m > d:
            raise ValueError("m must be a power of two between 2 and the degree")
        G = d // m + 1
        c = lambda k: float(coeffs[k]) if k <= d else 0.0
        q = lambda l: float(self.q[l - 1])

        def powers(base, sbase, top):
            pw, sc = {1: base}, {1: sbase}
            for k in range(2, top + 1):
                a = k // 2; b = k - a
                lv = min(pw[a].shape[1], pw[b].shape[1])
                pw[k] = self.rescale(self.mul_relin(pw[a][:, :lv], pw[b][:, :lv], rlk))
                sc[k] = sc[a] * sc[b] / q(lv)
            return pw, sc
        pw, sc = powers(x, scale, m)
        gp, sg = powers(pw[m], sc[m], G - 1)
        Lb = pw[m - 1].shape[1]
        Lc = min(gp[G - 1].shape[1], Lb - 1)
        if Lc < 2:
            raise ValueError("not enough limbs")
        Tp = scale * q(Lc)
        A, B, consts = [], [], []
        for i in range(1, G):
            Ti = (Tp / sg[i]) * q(Lb)
            acc = None
            for j in range(1, m):
                if c(i * m + j) == 0.0:
                    continue
                term = self.mul_const(pw[j][:, :Lb], int(np.rint(c(i * m + j) * (Ti / sc[j]))))
                acc = term if acc is None else self.add(acc, term)
            if acc is None:
                if c(i * m) != 0.0:
                    consts.append(self.mul_const(gp[i][:, :Lc], int(np.rint(c(i * m) * (Tp / sg[i])))))
                continue
            blk = self.add_const(self.rescale(acc), int(np.rint(c(i * m) * (Ti / q(Lb)))))
            A.append(blk[:, :Lc]); B.append(gp[i][:, :Lc])
        S = self.mul_relin_sum(np.stack(A), np.stack(B), rlk) if A else None
        for j in range(1, m):
            if c(j) == 0.0:
                continue
            term = self.mul_const(pw[j][:, :Lc], int(np.rint(c(j) * (Tp / sc[j]))))
            S = term if S is None else self.add(S, term)
        for t in consts:
            S = t if S is None else self.add(S, t)
        if S is None:
            raise ValueError("all non-constant coefficients are zero")
        so = Tp / q(Lc)
        return self.add_const(self.rescale(S), int(np.rint(c(0) * so))), so

    def softmax_doubling(self, x, scale: float, shift: float, rounds: int, row_len: int, exp_coeffs, rsqrt_coeffs, rlk, keys: dict,
                         exp_m: int = 0, rsqrt_m: int = 0):
        """Softmax by doubling with a public shift (Algorithm 1) on one ciphertext of score rows.  Row r holds its
        row_len scores in slots i * (n / row_len) + r, so that rotations by (n / row_len) 2^i, i < log2 row_len,
        add up a whole row in every one of its slots.  exp_coeffs: the polynomial p_exp(z / 2^k) as a polynomial in z;
        rsqrt_coeffs[j]: round j's inverse-square-root polynomial.  Order of steps:
          z = x + round(-shift * scale);  u = poly_eval_tree(z, exp_coeffs);
          per round: sq = rescale(mul_relin(u, u));  s = sq, then s = s + rotate(s, (n / row_len) 2^i) for i = 0, 1, ..;
                     lam = poly_eval_tree(s, rsqrt_coeffs[j]);  v = rescale(mul_relin(lam, u truncated to lam's level));
                     u = rescale(mul_relin(v, v)).
        Scales are doubles, multiplied and divided in this order.  keys maps a Galois element to its key.
        exp_m / rsqrt_m != 0 evaluate that polynomial by poly_eval_bsgs with blocks of m instead of the power tree.
        Returns (ct, scale)."""
        x = _u64(x)
        stride = self.n // row_len
        if row_len < 2 or row_len & (row_len - 1) or self.n % row_len:
            raise ValueError("row_len must be a power of two dividing the slot count")
        z = self.add_const(x, int(np.rint(-shift * scale)))
        poly = lambda c_, s_, co, m_: self.poly_eval_bsgs(c_, s_, co, rlk, m_) if m_ else self.poly_eval_tree(c_, s_, co, rlk)
        u, su = poly(z, scale, exp_coeffs, exp_m)
        for j in range(rounds):
            lv = u.shape[1]
            sq = self.rescale(self.mul_relin(u, u, rlk)); ss = su * su / float(self.q[lv - 1])
            s = sq
            i = 1
            while i < row_len:
                ge = self.galois_element(stride * i)
                s = self.add(s, self.rotate(s, keys[ge], ge))
                i *= 2
            lam, sl = poly(s, ss, rsqrt_coeffs[j], rsqrt_m)
            ll = lam.shape[1]
            v = self.rescale(self.mul_relin(lam, u[:, :ll], rlk)); sv = sl * su / float(self.q[ll - 1])
            u = self.rescale(self.mul_relin(v, v, rlk)); su = sv * sv / float(self.q[ll - 2])
        return u, su

    # -------------------------------------------------------------- attention
    def attention_rotations(self, desc: AttnDesc):
        """(token rotations, ladder rotations) in slots: key rotations by g * diag_block tokens, g = 1 .. groups - 1, and
        the rotate-and-add ladder over the diag_block blocks of a ciphertext (by tokens * heads * R * 2^k slots)."""
        E, Tk, H = desc.diag_block, desc.tokens, desc.heads
        if Tk % E or self.n % (E * Tk * H) or E & (E - 1) or Tk & (Tk - 1):
            raise ValueError("diag_block must divide tokens, and diag_block * tokens * heads the slot count (powers of two)")
        if desc.token_inner < 1 or E % desc.token_inner:
            raise ValueError("token_inner must divide diag_block")
        R = self.n // (E * Tk * H)
        tok = [g * E * H * R for g in range(1, desc.groups())]
        lad, k = [], 1
        while k < E:
            lad.append(Tk * H * R * k); k *= 2
        return tok, lad

    def attention_query_rotations(self, desc: AttnDesc):
        """Rotations (in slots, negative: to the right) of the query operands when the score groups are split into
        group_baby baby steps and groups / group_baby giant steps: -g1 * group_baby * diag_block tokens, g1 >= 1."""
        tok, _ = self.attention_rotations(desc)
        Gb, G = desc.group_baby, desc.groups()
        if Gb < 1 or G % Gb:
            raise ValueError("group_baby must divide the number of score groups")
        return [-tok[g1 * Gb - 1] for g1 in range(1, G // Gb)] if Gb > 1 else []

    def attention_scores(self, desc: AttnDesc, q, k, rlk, keys: dict):
        """Score ciphertexts S_g, g < groups = tokens / diag_block, from the channel operands q[d], k[d] (d < dim,
        [dim][2][level][N], layout of AttnDesc with the query repeated in every block e and the key operand holding token
        i + e in block e):  S_g = rescale(mul_relin_sum_d(q[d], rotate(k[d], g * diag_block tokens))).
        Slot (e, i, h) of S_g is the score of query i and head h against one key token; over all g and e every key token
        occurs exactly once, so the score row of (i, h) is spread over the groups x diag_block slots (e, i, h) of the S_g.
        One relinearisation per S_g; the products of a group are summed before it.  With desc.group_baby = Gb > 1 the
        groups are split g = g1 Gb + g0:  S_g = rotate(rescale(mul_relin_sum_d(rotate(q[d], -g1 Gb diag_block tokens),
        rotate(k[d], g0 diag_block tokens))), g1 Gb diag_block tokens), the same slot values from other integers (the last
        rotation is left out for g1 = 0).  Returns [groups][2][level-1][N]."""
        q = _u64(q); k = _u64(k); level = q.shape[2]
        tok, _ = self.attention_rotations(desc)
        out = np.empty((desc.groups(), 2, level - 1, self.N), dtype=np.uint64)
        if desc.group_baby > 1:
            # Baby-step / giant-step split of the groups, g = g1 * Gb + g0: a rotation is a ring automorphism, so
            #   q[d] * rot_g(k[d]) = rot_{g1 Gb}( rot_{-g1 Gb}(q[d]) * rot_{g0}(k[d]) )
            # and the query operand is the same in every block, so its right rotation is again a query operand (of the
            # tokens shifted cyclically).  Per channel Gb - 1 key and G / Gb - 1 query rotations instead of G - 1 key
            # rotations; every group with g1 > 0 is rotated back once, after its rescale.
            Gb, G = desc.group_baby, desc.groups()
            neg = self.attention_query_rotations(desc)
            dim = q.shape[0]
            kr, qr = [k], [q]
            for g0 in range(1, Gb):
                ge = self.galois_element(tok[g0 - 1])
                kr.append(np.stack([self.rotate(k[d], keys[ge], ge) for d in range(dim)]))
            for r in neg:
                ge = self.galois_element(r)
                qr.append(np.stack([self.rotate(q[d], keys[ge], ge) for d in range(dim)]))
            for g in range(G):
                g1, g0 = divmod(g, Gb)
                t = self.rescale(self.mul_relin_sum(qr[g1], kr[g0], rlk))
                if g1:
                    ge = self.galois_element(tok[g1 * Gb - 1])
                    t = self.rotate(t, keys[ge], ge)
                out[g] = t
            return out
        for g in range(desc.groups()):
            if g == 0:
                kr = k
            else:
                ge = self.galois_element(tok[g - 1])
                kr = np.stack([self.rotate(k[d], keys[ge], ge) for d in range(k.shape[0])])
            out[g] = self.rescale(self.mul_relin_sum(q, kr, rlk))
        return out

    def _block_ladder(self, desc: AttnDesc, s, keys: dict):
        _, lad = self.attention_rotations(desc)
        for r in lad:
            ge = self.galois_element(r)
            s = self.add(s, self.rotate(s, keys[ge], ge))
        return s

    def softmax_rows(self, desc: AttnDesc, S, scale: float, shift: float, rounds: int, exp_coeffs, rsqrt_coeffs, rlk, keys: dict):
        """Softmax by doubling with a public shift (Algorithm 1) on score rows spread over several ciphertexts: the row of
        (i, h) consists of the slots (e, i, h), e < diag_block, of every S_g.  Order of steps:
          u_g = poly_eval_tree(S_g + round(-shift * scale), exp_coeffs) for every g;
          per round: t = rescale(mul_relin_sum_g(u_g, u_g)); t = t + rotate(t, r) for the ladder rotations r in ascending
                     order (the row sum, in every slot of the row); lam = poly_eval_tree(t, rsqrt_coeffs[j]);
                     for every g: v = rescale(mul_relin(lam, u_g truncated to lam's level)); u_g = rescale(mul_relin(v, v)).
        The row sums and the inverse square root are formed once for all groups.  Returns ([groups][2][l][N], scale)."""
        S = _u64(S)
        G = S.shape[0]
        u, su = [], None
        for g in range(G):
            z = self.add_const(S[g], int(np.rint(-shift * scale)))
            ug, su = self.poly_eval_tree(z, scale, exp_coeffs, rlk)
            u.append(ug)
        for j in range(rounds):
            lv = u[0].shape[1]
            U = np.stack(u)
            t = self.rescale(self.mul_relin_sum(U, U, rlk)); st = su * su / float(self.q[lv - 1])
            t = self._block_ladder(desc, t, keys)
            lam, sl = self.poly_eval_tree(t, st, rsqrt_coeffs[j], rlk)
            ll = lam.shape[1]
            sv = sl * su / float(self.q[ll - 1])
            for g in range(G):
                v = self.rescale(self.mul_relin(lam, u[g][:, :ll], rlk))
                u[g] = self.rescale(self.mul_relin(v, v, rlk))
            su = sv * sv / float(self.q[ll - 2])
        return np.stack(u), su

    def attention_values(self, desc: AttnDesc, P, v, rlk, keys: dict):
        """Output channels from the probability ciphertexts P_g ([groups][2][lp][N], layout of the scores) and the value
        operands v[d] ([dim_v][2][level][N], level >= lp, layout of the key operand):
          vt = v[d] truncated to lp limbs;  o = rescale(mul_relin_sum_g(P_g, rotate(vt, g * diag_block tokens)));
          o = o + rotate(o, r) for the ladder rotations in ascending order.
        Slot (e, i, h) of output d then holds sum over all key tokens of probability x value for query i, head h, in every
        block e (the layout of the query operand).  Returns [dim_v][2][lp-1][N]."""
        P = _u64(P); v = _u64(v)
        G, lp = P.shape[0], P.shape[2]
        tok, _ = self.attention_rotations(desc)
        out = np.empty((v.shape[0], 2, lp - 1, self.N), dtype=np.uint64)
        for d in range(v.shape[0]):
            vt = np.ascontiguousarray(v[d][:, :lp])
            vr = [vt]
            for g in range(1, G):
                ge = self.galois_element(tok[g - 1])
                vr.append(self.rotate(vt, keys[ge], ge))
            o = self.rescale(self.mul_relin_sum(P, np.stack(vr), rlk))
            out[d] = self._block_ladder(desc, o, keys)
        return out

    def attention(self, desc: AttnDesc, q, k, v, scale: float, v_scale: float, shift: float, rounds: int, exp_coeffs, rsqrt_coeffs,
                  rlk, keys: dict):
        """Scores, Softmax over the score rows, output channels: attention_scores, softmax_rows, attention_values in a row,
        with the scales a sequence of doubles: scores scale^2 / q_{l-1}, the Softmax's own, then times v_scale / q_{lp-1}.
        Returns ([dim_v][2][lp-1][N], scale)."""
        level = _u64(q).shape[2]
        S = self.attention_scores(desc, q, k, rlk, keys)
        ss = scale * scale / float(self.q[level - 1])
        P, sp = self.softmax_rows(desc, S, ss, shift, rounds, exp_coeffs, rsqrt_coeffs, rlk, keys)
        lp = P.shape[2]
        return self.attention_values(desc, P, v, rlk, keys), sp * v_scale / float(self.q[lp - 1])

    # ---- conversion between the projections' token-shard layout and the attention operands ------------------------
    def _pack_shape(self, desc: AttnDesc):
        E, Tk, H, Ti = desc.diag_block, desc.tokens, desc.heads, desc.token_inner
        self.attention_rotations(desc)
        if E * Tk * H != self.n:
            raise ValueError("the conversions need diag_block * tokens * heads = slot count (no trailing copies)")
        return E, Tk // Ti, H * Ti, Ti                 # blocks, positions per block, slots per position, tokens per position

    def _slot_mask(self, B: int, lo: int, hi: int, Ti: int, t0: int, t1: int):
        """1.0 on the slots x with lo <= x // B < hi and t0 <= x % Ti < t1, else 0.0."""
        x = np.arange(self.n)
        return (((x // B >= lo) & (x // B < hi) & (x % Ti >= t0) & (x % Ti < t1))).astype(np.float64)

    def attention_pack_rotations(self, desc: AttnDesc, kind: int, dim: int):
        """Rotations (in slots) attention_pack uses.  Block moves: -c B for shard c < P and d B for channel d < dim (B = heads
        * token_inner slots per position); kind 0 (query): the ladder over the blocks; kind 1 (key / value): -P B (a second
        copy of block 0) and, per block e with e = a token_inner + b, the token shifts a B + b - e P B (slots with
        t < token_inner - b) and (a + 1) B + b - token_inner - e P B (the others, which take their token from the next
        position)."""
        E, P, B, Ti = self._pack_shape(desc)
        move = [-c * B for c in range(1, P)] + [d * B for d in range(1, dim)]
        if kind == 0:
            return move, self.attention_rotations(desc)[1]
        shift = []
        for e in range(E):
            a, b = divmod(e, Ti)
            shift.append((a * B + b - e * P * B, (a + 1) * B + b - Ti - e * P * B if b else None))
        return move, ([-P * B] if E > 1 else []), shift

    def _move_blocks(self, desc: AttnDesc, X, nout: int, keys: dict):
        """out[y] = rotate( rescale( sum_x rotate(X[x], -x B) * mask(block x + y) ), y B ),  y < nout: block y of input x ends up
        as block x of output y (a transpose between the ciphertext index and the block index).  Every input and every
        output is rotated once; the sums in between are plaintext multiplications by 0/1 masks (encoded at the scale of the
        level's last prime) and additions.  Blocks are counted cyclically over the n / B blocks of a ciphertext."""
        E, P, B, Ti = self._pack_shape(desc)
        X = _u64(X); nin, level = X.shape[0], X.shape[2]
        pt_scale = float(self.q[level - 1])
        nblk = self.n // B
        Xp = []
        for x in range(nin):
            if x:
                ge = self.galois_element(-x * B)
                Xp.append(self.rotate(X[x], keys[ge], ge))
            else:
                Xp.append(X[0])
        acc = [None] * nout
        for j in range(min(nin + nout - 1, nblk)):
            mask = None
            for x in range(nin):
                for y in range(nout):
                    if (x + y) % nblk != j:
                        continue
                    if mask is None:
                        mask = self.encode(self._slot_mask(B, j, j + 1, Ti, 0, Ti), pt_scale, level)
                    acc[y] = self.mul_plain_acc(Xp[x], mask, acc[y])
        out = []
        for y in range(nout):
            w = self.rescale(acc[y])
            if y:
                ge = self.galois_element(y * B)
                w = self.rotate(w, keys[ge], ge)
            out.append(w)
        return np.stack(out)

    def _gather_channels(self, desc: AttnDesc, X, dim: int, keys: dict):
        """gathered[d], d < dim: block 0 holds channel d of every shard at the shard's position (position c = shard c).
        X: [P][2][level][N] with slot (d heads + h) token_inner + t = value of token c token_inner + t, head h, channel d.
        Returns [dim][2][level-1][N]."""
        return self._move_blocks(desc, X, dim, keys)

    def attention_pack(self, desc: AttnDesc, kind: int, X, dim: int, keys: dict):
        """Attention operands from token-shard ciphertexts in channel-major feature order (the projections' layout with
        token_inner tokens per shard): X [P][2][level][N], slot (d heads + h) token_inner + t.
        gathered[d] = rotate( rescale( sum_c rotate(X[c], -c B) * mask(block c + d) ), d B ) (_move_blocks): position c of block
        0 holds channel d of shard c.
          kind 0 (query):  q[d] = ladder(gathered[d]): channel d of every token in every block e.  Level - 1.
          kind 1 (key, value): k0 = gathered[d]; k0 = k0 + rotate(k0, -P B) (blocks 0 and 1 hold the tokens); then
            k[d] = rescale( sum_e [ rotate(k0, sA_e) * mask(block e, t < token_inner - b) + rotate(k0, sB_e) * mask(block e,
            t >= token_inner - b) ] ) with the shifts of attention_pack_rotations: block e holds token i + e.  Level - 2
            (level - 1 if diag_block = 1: nothing to shift).
        Masks are encoded at the scale of the last prime of their level, so that every rescale returns the input's scale.
        Returns [dim][2][l'][N]."""
        E, P, B, Ti = self._pack_shape(desc)
        g = self._gather_channels(desc, X, dim, keys)
        if kind == 0:
            return np.stack([self._block_ladder(desc, g[d], keys) for d in range(dim)])
        if E == 1:
            return g
        _, dbl, shift = self.attention_pack_rotations(desc, 1, dim)
        level = g.shape[2]
        pt_scale = float(self.q[level - 1])
        out = []
        for d in range(dim):
            ge = self.galois_element(dbl[0])
            k0 = self.add(g[d], self.rotate(g[d], keys[ge], ge))
            acc = None
            for e in range(E):
                b = e % Ti
                for part, r in enumerate(shift[e]):
                    if r is None:
                        continue
                    mask = self._slot_mask(B, e * P, (e + 1) * P, Ti, 0, Ti - b) if part == 0 else self._slot_mask(B, e * P, (e + 1) * P, Ti, Ti - b, Ti)
                    if r % self.n:
                        ge = self.galois_element(r)
                        kr = self.rotate(k0, keys[ge], ge)
                    else:
                        kr = k0
                    acc = self.mul_plain_acc(kr, self.encode(mask, pt_scale, level), acc)
            out.append(self.rescale(acc))
        return np.stack(out)

    def attention_unpack_rotations(self, desc: AttnDesc, dim: int):
        """Block moves of attention_unpack: -d B for channel d < dim, c B for shard c < P."""
        E, P, B, Ti = self._pack_shape(desc)
        return [-d * B for d in range(1, dim)] + [c * B for c in range(1, P)]

    def attention_unpack(self, desc: AttnDesc, O, keys: dict):
        """Token-shard ciphertexts in channel-major feature order from attention outputs in the query operand's layout
        (O [dim][2][level][N], every block e alike): the same transpose between ciphertext index and block index the other
        way, X[c] = rotate( rescale( sum_d rotate(O[d], -d B) * mask(block c + d) ), c B ): slot (d heads + h) token_inner + t
        of X[c] holds channel d of token c token_inner + t, head h.  Returns [P][2][level-1][N]."""
        E, P, B, Ti = self._pack_shape(desc)
        return self._move_blocks(desc, O, P, keys)

    def automorphism_coeff(self, a, g: int, t: int):
        a = _u64(a); out = np.empty_like(a)
        lib().orc_automorphism_coeff(self._h, C.c_uint32(t), _p(a, _u64p), C.c_uint64(g), _p(out, _u64p))
        return out

    def automorphism_eval(self, a, g: int):
        a = _u64(a); out = np.empty_like(a)
        lib().orc_automorphism_eval(self._h, _p(a, _u64p), C.c_uint64(g), _p(out, _u64p))
        return out

    # ------------------------------------------------------------ key switch
    def num_digits(self, level: int) -> int:
        return -(-level // self.alpha)

    def modup_digit(self, d_coeff, j: int):
        d = _u64(d_coeff); level = d.shape[0]
        ext = np.empty((level + self.K, self.N), dtype=np.uint64)
        lib().orc_modup_digit(self._h, _p(d, _u64p), C.c_uint32(level), C.c_uint32(j), _p(ext, _u64p))
        return ext

    def moddown(self, u, level: int):
        u = _u64(u); out = np.empty((level, self.N), dtype=np.uint64)
        lib().orc_moddown(self._h, _p(u, _u64p), C.c_uint32(level), _p(out, _u64p))
        return out

    def keyswitch(self, d, evk):
        d = _u64(d); evk = _u64(evk); level = d.shape[0]
        k = np.empty((2, level, self.N), dtype=np.uint64)
        lib().orc_keyswitch(self._h, _p(d, _u64p), _p(evk, _u64p), C.c_uint32(level), _p(k, _u64p))
        return k

    def rotate(self, ct, evk, g: int):
        ct = _u64(ct); evk = _u64(evk); level = ct.shape[1]
        out = np.empty_like(ct)
        lib().orc_rotate(self._h, _p(ct, _u64p), _p(evk, _u64p), C.c_uint64(g), C.c_uint32(level), _p(out, _u64p))
        return out

    def rotate_hoisted(self, ct, evks, gs):
        ct = _u64(ct); level = ct.shape[1]; nrot = len(gs)
        evks = [_u64(k) for k in evks]
        ptrs = (C.c_void_p * nrot)(*[k.ctypes.data for k in evks])
        ga = np.array(gs, dtype=np.uint64)
        outs = np.empty((nrot, 2, level, self.N), dtype=np.uint64)
        lib().orc_rotate_hoisted(self._h, _p(ct, _u64p), ptrs, _p(ga, _u64p), C.c_uint32(nrot), C.c_uint32(level), _p(outs, _u64p))
        return outs

    def modup_all(self, d):
        """d [level][N] evaluation domain -> all digits extended and transformed, [beta][level+K][N]."""
        d = _u64(d); level = d.shape[0]
        ext = np.empty((self.num_digits(level), level + self.K, self.N), dtype=np.uint64)
        lib().orc_modup_all(self._h, _p(d, _u64p), C.c_uint32(level), _p(ext, _u64p))
        return ext

    def inner_product(self, ext, evk):
        """<ext, evk> in the extended basis: [2][level+K][N], before any ModDown."""
        ext = _u64(ext); evk = _u64(evk); level = ext.shape[1] - self.K
        u = np.empty((2, level + self.K, self.N), dtype=np.uint64)
        lib().orc_inner_product(self._h, _p(ext, _u64p), _p(evk, _u64p), C.c_uint32(level), _p(u, _u64p))
        return u

    def rotate_sum(self, cts, evks, gs):
        """sum_i rotate(cts[i], evks[i], gs[i]) with the sum taken in the extended basis and one ModDown."""
        cts = _u64(cts); n, level = cts.shape[0], cts.shape[2]
        evks = [_u64(k) for k in evks]
        ptrs = (C.c_void_p * n)(*[k.ctypes.data for k in evks])
        ga = np.array(gs, dtype=np.uint64)
        out = np.empty((2, level, self.N), dtype=np.uint64)
        lib().orc_rotate_sum(self._h, _p(cts, _u64p), ptrs, _p(ga, _u64p), C.c_uint32(n), C.c_uint32(level), _p(out, _u64p))
        return out

    def rescale(self, ct):
        ct = _u64(ct); ncomp, level = ct.shape[0], ct.shape[1]
        out = np.empty((ncomp, level - 1, self.N), dtype=np.uint64)
        lib().orc_rescale(self._h, _p(ct, _u64p), C.c_uint32(ncomp), C.c_uint32(level), _p(out, _u64p))
        return out

    def tensor(self, a, b):
        a = _u64(a); b = _u64(b); level = a.shape[1]
        e = np.empty((3, level, self.N), dtype=np.uint64)
        lib().orc_tensor(self._h, _p(a, _u64p), _p(b, _u64p), C.c_uint32(level), _p(e, _u64p))
        return e

    def mul_relin(self, a, b, rlk):
        a = _u64(a); b = _u64(b); rlk = _u64(rlk); level = a.shape[1]
        out = np.empty_like(a)
        lib().orc_mul_relin(self._h, _p(a, _u64p), _p(b, _u64p), _p(rlk, _u64p), C.c_uint32(level), _p(out, _u64p))
        return out

    def mul_relin_sum(self, a, b, rlk):
        """relin(sum_i a_i (x) b_i): a, b [n][2][level][N]; one key switch for the whole sum."""
        a = _u64(a); b = _u64(b); rlk = _u64(rlk); n, level = a.shape[0], a.shape[2]
        out = np.empty_like(a[0])
        lib().orc_mul_relin_sum(self._h, _p(a, _u64p), _p(b, _u64p), C.c_uint32(n), _p(rlk, _u64p), C.c_uint32(level), _p(out, _u64p))
        return out

    # ----------------------------------------------------- linear projection
    def proj_blocks(self, desc: ProjDesc):
        """Feature blocks of the input and output: lists of (start, size).  F = n / T_s
        features fit one ciphertext; a trailing block smaller than F must divide F."""
        F = self.n // desc.tokens_per_shard

        def split(d):
            blocks, s = [], 0
            while s < d:
                m = min(F, d - s)
                if F % m:
                    raise ValueError("remainder block must divide F")
                blocks.append((s, m)); s += m
            return blocks
        return F, split(desc.d_in), split(desc.d_out)

    def proj_rotations(self, desc: ProjDesc):
        """Slot rotations (hence Galois keys) the schedule uses: baby, giant, fold."""
        F, ins, outs = self.proj_blocks(desc)
        T, B = desc.tokens_per_shard, desc.baby
        rots = set(b * T for b in range(1, B))
        for (_, mo) in outs:
            for (_, mi) in ins:
                nd = min(mi, mo)
                rots |= set(g * B * T for g in range(1, nd // B))
                f = mo
                while f < mi:
                    rots.add(f * T); f *= 2
        return sorted(rots)

    @staticmethod
    def diagonal(Wt_blk, k: int, F: int):
        """k-th generalised cyclic diagonal of the block A = W^T[out block, in block]
        (Eq. 5): d_k[r] = A[r mod m_out, (r + k) mod m_in], r < F."""
        mo, mi = Wt_blk.shape
        r = np.arange(F)
        return Wt_blk[r % mo, (r + k) % mi]

    def linear_proj(self, desc: ProjDesc, cts, W, keys: dict, ct_scale: float):
        """Y = X W on token-shard ciphertexts by the diagonal method (Eq. 5), schedule:
        baby rotations hoisted per input ciphertext; for every giant step g the
        pre-rotated diagonals are encoded and multiply-accumulated; acc_g is rotated by
        g*B*T_s (plain rotation) and summed; optional fold; one rescale.  With
        desc.lazy_moddown the rotated accumulators of g >= 1 are summed by rotate_sum
        (one ModDown for all of them) and added to acc_0.

        cts [nshards * n_in_blocks][2][level][N]; W [d_in][d_out] fp64; keys maps a
        Galois element to its switching key.  Returns (outs [nshards*n_out_blocks][2]
        [level-1][N], out_scale).
        """
        cts = _u64(cts); level = cts.shape[2]
        F, ins, outs_b = self.proj_blocks(desc)
        T, B = desc.tokens_per_shard, desc.baby
        pt_scale = desc.pt_scale if desc.pt_scale else float(self.q[level - 1])
        nib, nob = len(ins), len(outs_b)
        A = np.asarray(W, dtype=np.float64).T                     # [d_out][d_in]
        outs = np.empty((desc.nshards * nob, 2, level - 1, self.N), dtype=np.uint64)
        gal = lambda r: self.galois_element(r)
        # Encoded pre-rotated diagonals are independent of the shard: cache per (ob, ib, g, b).
        pt_cache = {}

        def plaintext(ob, ib, g, b):
            key = (ob, ib, g, b)
            if key not in pt_cache:
                (os_, mo), (is_, mi) = outs_b[ob], ins[ib]
                d = self.diagonal(A[os_:os_ + mo, is_:is_ + mi], g * B + b, F)
                dpre = np.roll(d, g * B)                          # d'[r] = d[(r - gB) mod F]
                pt_cache[key] = self.encode(np.repeat(dpre, T), pt_scale, level)
            return pt_cache[key]

        for c in range(desc.nshards):
            baby = []
            for ib in range(nib):
                x = cts[c * nib + ib]
                gs = [gal(b * T) for b in range(1, B)]
                rot = self.rotate_hoisted(x, [keys[g] for g in gs], gs) if gs else []
                baby.append([x] + [rot[i] for i in range(len(gs))])
            for ob, (os_, mo) in enumerate(outs_b):
                nds = [min(mi, mo) for (_, mi) in ins]
                folds = {mi // mo if mi > mo else 1 for (_, mi) in ins}
                if len(folds) != 1:
                    raise ValueError("input blocks of one output block need the same fold count")
                total, later = None, []
                for g in range(max(nds) // B):
                    acc = None
                    for ib in range(nib):
                        if g >= nds[ib] // B:
                            continue
                        for b in range(B):
                            acc = self.mul_plain_acc(baby[ib][b], plaintext(ob, ib, g, b), acc)
                    if g and desc.lazy_moddown:
                        later.append(acc)
                        continue
                    if g:
                        ge = gal(g * B * T)
                        acc = self.rotate(acc, keys[ge], ge)
                    total = acc if total is None else self.add(total, acc)
                if later:
                    ges = [gal(g * B * T) for g in range(1, len(later) + 1)]
                    total = self.add(total, self.rotate_sum(np.stack(later), [keys[ge] for ge in ges], ges))
                f, fold = mo, folds.pop()
                while fold > 1:
                    ge = gal(f * T)
                    total = self.add(total, self.rotate(total, keys[ge], ge))
                    f *= 2; fold //= 2
                outs[c * nob + ob] = self.rescale(total)
        return outs, ct_scale * pt_scale / float(self.q[level - 1])

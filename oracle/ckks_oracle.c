/*
 * CPU checker ("oracle") for the CKKS RNS primitive layer.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow,
 * definition-level implementation in exact 128-bit integer arithmetic and
 * fp64, written only so that the CUDA library can be compared against
 * something that can be checked by eye.  It shares no code, header, table or
 * constant generator with the CUDA path.  Only the tests, the smoke check and
 * the benchmark's CPU-baseline leg may call it.
 *
 * The paper names the primitives it relies on -- Encode, Add, PCMult, Mult,
 * Rot_k, KeySwitch, Rescale (Section 2.1, "The CKKS Computation Model") -- and
 * the diagonal matrix-vector identity (Eq. 5), but defines none of the
 * arithmetic; that follows the full-RNS form of the scheme it cites.  Every
 * function below states which primitive it realises and which reading of the
 * silent parts it takes.
 *
 * Conventions
 *   N ring degree, n = N/2 slots, M = 2N.  Prime index space: 0..L-1 are the
 *   ciphertext primes q_i, L..L+K-1 the special primes p_k.  A "limb" is N
 *   residues in [0, prime).  Stored polynomials are in the evaluation domain,
 *   bit-reversed order: stored[p] = a(psi^(2*brev(p)+1)).  A ciphertext is
 *   [ncomp][level][N]; a switching key is [dnum][2][L+K][N].
 *
 * Pins (tests/test_oracle_*.py): schoolbook negacyclic convolution, closed
 * forms NTT(1), NTT(X), Horner evaluation, the q=17 N=8 worked example,
 * decode(encode(z)) = z, constant and cosine closed forms, direct O(n*N)
 * embedding sums, exact big-integer CRT checks of ModUp / ModDown / rescale,
 * decrypt(rotate(enc z)) = rotated z, slot products after relinearisation,
 * and Eq. 5 in the clear.  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef unsigned __int128 u128;
typedef __int128 i128;

typedef struct orc_ctx {
    uint32_t log_n, L, K, dnum, alpha;
    uint64_t N, n, M;
    uint64_t *mod;      /* [L+K] primes, q then p                         */
    uint64_t *psi;      /* [L+K] smallest primitive 2N-th root per prime  */
    uint64_t **pw;      /* pw[t][j] = psi_t^j mod prime_t, j < 2N         */
    uint64_t *n_inv;    /* [L+K] N^-1 mod prime                           */
    uint32_t *brev;     /* [N] bit reversal on log_n bits                 */
    uint64_t *pow5;     /* [n] 5^j mod M                                  */
    double *om_re, *om_im; /* [n] omega^t = exp(2 pi i t / n)             */
    double *ze_re, *ze_im; /* [n] zeta^k  = exp(2 pi i k / M)             */
} orc_ctx;

/* ---------------------------------------------------------------- scalars */

static uint64_t mulmod(uint64_t a, uint64_t b, uint64_t q) { return (uint64_t)((u128)a * b % q); }
static uint64_t addmod(uint64_t a, uint64_t b, uint64_t q) { uint64_t s = a + b; return s >= q ? s - q : s; }
static uint64_t submod(uint64_t a, uint64_t b, uint64_t q) { return a >= b ? a - b : a + q - b; }
static uint64_t powmod(uint64_t a, uint64_t e, uint64_t q) {
    uint64_t r = 1 % q;
    a %= q;
    while (e) { if (e & 1) r = mulmod(r, a, q); a = mulmod(a, a, q); e >>= 1; }
    return r;
}
static uint64_t invmod(uint64_t a, uint64_t q) { return powmod(a, q - 2, q); } /* q prime */
/* canonical residue of a signed value */
static uint64_t reduce_signed(i128 v, uint64_t q) { i128 r = v % (i128)q; if (r < 0) r += q; return (uint64_t)r; }
/* centred representative of y in [0,q): the one in (-q/2, q/2); q odd so no tie */
static int64_t centre(uint64_t y, uint64_t q) { return y > (q - 1) / 2 ? (int64_t)y - (int64_t)q : (int64_t)y; }

static uint32_t bitrev(uint32_t x, uint32_t bits) {
    uint32_t r = 0;
    for (uint32_t i = 0; i < bits; i++) { r = (r << 1) | (x & 1); x >>= 1; }
    return r;
}

/*
 * Smallest x in [2,q) with x^N = -1 (mod q): the minimum over the N primitive
 * 2N-th roots of unity.  Reading: the scheme leaves the root free; "smallest"
 * makes it a function of (q, N) alone.
 */
static uint64_t smallest_primitive_root_2n(uint64_t q, uint64_t N) {
    uint64_t r = 0;
    for (uint64_t x = 2; x < q; x++) {
        r = powmod(x, (q - 1) / (2 * N), q);
        if (powmod(r, N, q) == q - 1) break;   /* order exactly 2N (N a power of two) */
    }
    uint64_t r2 = mulmod(r, r, q), cur = r, best = r;
    for (uint64_t k = 1; k < 2 * N; k += 2) {   /* odd powers = all primitive 2N-th roots */
        if (cur < best) best = cur;
        cur = mulmod(cur, r2, q);
    }
    return best;
}

/* ---------------------------------------------------------------- context */

orc_ctx *orc_create(uint32_t log_n, uint32_t L, uint32_t K, uint32_t dnum, const uint64_t *q, const uint64_t *p) {
    orc_ctx *c = (orc_ctx *)calloc(1, sizeof(orc_ctx));
    c->log_n = log_n; c->L = L; c->K = K; c->dnum = dnum;
    c->alpha = (L + dnum - 1) / dnum;
    c->N = 1ull << log_n; c->n = c->N / 2; c->M = 2 * c->N;
    uint32_t T = L + K;
    c->mod = (uint64_t *)malloc(T * 8);
    c->psi = (uint64_t *)malloc(T * 8);
    c->n_inv = (uint64_t *)malloc(T * 8);
    c->pw = (uint64_t **)malloc(T * sizeof(uint64_t *));
    for (uint32_t t = 0; t < T; t++) c->mod[t] = t < L ? q[t] : p[t - L];
    #pragma omp parallel for
    for (uint32_t t = 0; t < T; t++) {
        uint64_t m = c->mod[t];
        c->psi[t] = smallest_primitive_root_2n(m, c->N);
        c->n_inv[t] = invmod(c->N % m, m);
        c->pw[t] = (uint64_t *)malloc(2 * c->N * 8);
        c->pw[t][0] = 1;
        for (uint64_t j = 1; j < 2 * c->N; j++) c->pw[t][j] = mulmod(c->pw[t][j - 1], c->psi[t], m);
    }
    c->brev = (uint32_t *)malloc(c->N * 4);
    for (uint64_t i = 0; i < c->N; i++) c->brev[i] = bitrev((uint32_t)i, log_n);
    uint64_t n = c->n ? c->n : 1;
    c->pow5 = (uint64_t *)malloc(n * 8);
    c->pow5[0] = 1 % c->M;
    for (uint64_t j = 1; j < n; j++) c->pow5[j] = c->pow5[j - 1] * 5 % c->M;
    c->om_re = (double *)malloc(n * 8); c->om_im = (double *)malloc(n * 8);
    c->ze_re = (double *)malloc(n * 8); c->ze_im = (double *)malloc(n * 8);
    /* Reading: twiddles are the host libm's cos/sin of 2.0*M_PI*t/n evaluated in double. */
    for (uint64_t t = 0; t < n; t++) {
        c->om_re[t] = cos(2.0 * M_PI * (double)t / (double)c->n);
        c->om_im[t] = sin(2.0 * M_PI * (double)t / (double)c->n);
        c->ze_re[t] = cos(2.0 * M_PI * (double)t / (double)c->M);
        c->ze_im[t] = sin(2.0 * M_PI * (double)t / (double)c->M);
    }
    return c;
}

void orc_destroy(orc_ctx *c) {
    if (!c) return;
    for (uint32_t t = 0; t < c->L + c->K; t++) free(c->pw[t]);
    free(c->pw); free(c->mod); free(c->psi); free(c->n_inv); free(c->brev); free(c->pow5);
    free(c->om_re); free(c->om_im); free(c->ze_re); free(c->ze_im);
    free(c);
}

uint64_t orc_root(const orc_ctx *c, uint32_t t) { return c->psi[t]; }
uint64_t orc_modulus(const orc_ctx *c, uint32_t t) { return c->mod[t]; }

/* ------------------------------------------------------------------- NTT */

/*
 * Negacyclic NTT, plain definition, O(N^2):
 *   nat[k] = sum_j a_j psi^((2k+1) j) mod q,   out[p] = nat[brev(p)].
 */
void orc_ntt_definition(const orc_ctx *c, uint32_t t, const uint64_t *a, uint64_t *out) {
    uint64_t q = c->mod[t], N = c->N, M = c->M;
    for (uint64_t p = 0; p < N; p++) {
        uint64_t k = c->brev[p], e = 2 * k + 1, acc = 0;
        for (uint64_t j = 0; j < N; j++) acc = addmod(acc, mulmod(a[j], c->pw[t][e * j % M], q), q);
        out[p] = acc;
    }
}

/* Inverse by definition: a_j = N^-1 sum_k nat[k] psi^(-(2k+1) j). */
void orc_intt_definition(const orc_ctx *c, uint32_t t, const uint64_t *in, uint64_t *a) {
    uint64_t q = c->mod[t], N = c->N, M = c->M;
    for (uint64_t j = 0; j < N; j++) {
        uint64_t acc = 0;
        for (uint64_t p = 0; p < N; p++) {
            uint64_t k = c->brev[p], e = (2 * k + 1) * j % M;
            acc = addmod(acc, mulmod(in[p], c->pw[t][(M - e) % M], q), q);
        }
        a[j] = mulmod(acc, c->n_inv[t], q);
    }
}

/*
 * Textbook radix-2 cyclic transform of size N with root w = psi^(2*dir):
 * bit-reverse the input, then log N butterfly stages; natural-order output
 * x[k] = sum_j in[j] w^(kj).  dir = +1 forward, -1 inverse (unnormalised).
 */
static void cyclic_transform(const orc_ctx *c, uint32_t t, uint64_t *x, int dir) {
    uint64_t q = c->mod[t], N = c->N, M = c->M;
    for (uint64_t i = 0; i < N; i++) {
        uint64_t r = c->brev[i];
        if (i < r) { uint64_t tmp = x[i]; x[i] = x[r]; x[r] = tmp; }
    }
    for (uint64_t len = 2; len <= N; len <<= 1) {
        uint64_t step = M / len;                 /* w_len = psi^(2N/len) */
        for (uint64_t i = 0; i < N; i += len)
            for (uint64_t j = 0; j < len / 2; j++) {
                uint64_t e = step * j;
                uint64_t w = c->pw[t][dir > 0 ? e : (M - e) % M];
                uint64_t u = x[i + j], v = mulmod(x[i + j + len / 2], w, q);
                x[i + j] = addmod(u, v, q);
                x[i + j + len / 2] = submod(u, v, q);
            }
    }
}

/* Fast forward NTT, in place: twist by psi^j, cyclic transform, store bit-reversed. */
void orc_ntt(const orc_ctx *c, uint32_t t, uint64_t *a) {
    uint64_t q = c->mod[t], N = c->N;
    uint64_t *x = (uint64_t *)malloc(N * 8);
    for (uint64_t j = 0; j < N; j++) x[j] = mulmod(a[j], c->pw[t][j], q);
    cyclic_transform(c, t, x, +1);
    for (uint64_t p = 0; p < N; p++) a[p] = x[c->brev[p]];
    free(x);
}

/* Fast inverse NTT, in place. */
void orc_intt(const orc_ctx *c, uint32_t t, uint64_t *a) {
    uint64_t q = c->mod[t], N = c->N, M = c->M;
    uint64_t *x = (uint64_t *)malloc(N * 8);
    for (uint64_t k = 0; k < N; k++) x[k] = a[c->brev[k]];
    cyclic_transform(c, t, x, -1);
    for (uint64_t j = 0; j < N; j++)
        a[j] = mulmod(mulmod(x[j], c->n_inv[t], q), c->pw[t][(M - j) % M], q);
    free(x);
}

/* Batched helpers: `polys` is [batch][nlimbs][N], limb i under prime first+i. */
void orc_ntt_batch(const orc_ctx *c, uint64_t *polys, uint32_t batch, uint32_t first, uint32_t nlimbs) {
    #pragma omp parallel for
    for (uint32_t x = 0; x < batch * nlimbs; x++) orc_ntt(c, first + x % nlimbs, polys + (uint64_t)x * c->N);
}
void orc_intt_batch(const orc_ctx *c, uint64_t *polys, uint32_t batch, uint32_t first, uint32_t nlimbs) {
    #pragma omp parallel for
    for (uint32_t x = 0; x < batch * nlimbs; x++) orc_intt(c, first + x % nlimbs, polys + (uint64_t)x * c->N);
}

/* ---------------------------------------------------------------- Encode */

/*
 * Encode, fp64 part (Section 2.1 "Encode(m) returns a plaintext polynomial
 * whose slots represent the vector m").  Slot j sits at the root zeta^(5^j).
 *   m_k = round( (Delta/n) Re sum_j z_j zeta^(-5^j k) ),  k < N.
 * Steps, in this order (each product and each sum rounded on its own, no FMA):
 *   E1  Z[e_j] = z_j, e_j = ((5^j mod M) - 1) / 4
 *   E2  b_k = sum_e Z[e] omega^(-e k): bit-reverse, then stages m = 2,4,..,n of
 *       radix-2 butterflies (u, v) -> (u + w v, u - w v), w = conj(omega^(j n/m))
 *   E3  a_k = b_k conj(zeta^k)
 *   E4  m_k = rint(Re a_k * (Delta/n)), m_(k+n) = rint(Im a_k * (Delta/n)),
 *       round-half-even
 * Returns 0, or -1 if a scaled value is not below 2^62 in magnitude.
 */
int orc_encode_coeffs(const orc_ctx *c, const double *re, const double *im, double scale, int64_t *m) {
    uint64_t n = c->n, M = c->M;
    double *vr = (double *)calloc(n, 8), *vi = (double *)calloc(n, 8);
    uint32_t bits = c->log_n - 1;
    for (uint64_t j = 0; j < n; j++) {                    /* E1 then the bit-reverse of E2 */
        uint64_t e = (c->pow5[j] % M - 1) / 4;
        uint64_t pos = bitrev((uint32_t)e, bits);
        vr[pos] = re[j];
        vi[pos] = im ? im[j] : 0.0;
    }
    for (uint64_t m2 = 2; m2 <= n; m2 <<= 1) {            /* E2 */
        uint64_t half = m2 / 2, stride = n / m2;
        for (uint64_t k0 = 0; k0 < n; k0 += m2)
            for (uint64_t j = 0; j < half; j++) {
                double wr = c->om_re[j * stride], wi = -c->om_im[j * stride];
                double xr = vr[k0 + j + half], xi = vi[k0 + j + half];
                double p0 = wr * xr, p1 = wi * xi, p2 = wr * xi, p3 = wi * xr;
                double tr = p0 - p1, ti = p2 + p3;
                double ur = vr[k0 + j], ui = vi[k0 + j];
                vr[k0 + j] = ur + tr;        vi[k0 + j] = ui + ti;
                vr[k0 + j + half] = ur - tr; vi[k0 + j + half] = ui - ti;
            }
    }
    double s = scale / (double)n;
    int rc = 0;
    for (uint64_t k = 0; k < n; k++) {                    /* E3, E4 */
        double wr = c->ze_re[k], wi = -c->ze_im[k];
        double p0 = wr * vr[k], p1 = wi * vi[k], p2 = wr * vi[k], p3 = wi * vr[k];
        double ar = p0 - p1, ai = p2 + p3;
        double xr = ar * s, xi = ai * s;
        if (!(fabs(xr) < 4611686018427387904.0) || !(fabs(xi) < 4611686018427387904.0)) { rc = -1; xr = xi = 0.0; }
        m[k] = (int64_t)llrint(xr);
        m[k + n] = (int64_t)llrint(xi);
    }
    free(vr); free(vi);
    return rc;
}

/* Encode to RNS limbs: E5 canonical residues of m_k, E6 NTT per limb.  out is [level][N]. */
int orc_encode(const orc_ctx *c, const double *re, const double *im, double scale, uint32_t level, uint64_t *out) {
    uint64_t N = c->N;
    int64_t *m = (int64_t *)malloc(N * 8);
    int rc = orc_encode_coeffs(c, re, im, scale, m);
    #pragma omp parallel for
    for (uint32_t i = 0; i < level; i++) {
        uint64_t q = c->mod[i];
        for (uint64_t k = 0; k < N; k++) out[i * N + k] = reduce_signed(m[k], q);
        orc_ntt(c, i, out + i * N);
    }
    free(m);
    return rc;
}

/* Small signed coefficients (secret, error, sigma_g(s), ...) to limbs under primes first..first+nl-1. */
void orc_small_to_limbs(const orc_ctx *c, const int64_t *poly, uint32_t first, uint32_t nl, uint64_t *out) {
    uint64_t N = c->N;
    #pragma omp parallel for
    for (uint32_t i = 0; i < nl; i++) {
        uint64_t q = c->mod[first + i];
        for (uint64_t k = 0; k < N; k++) out[i * N + k] = reduce_signed(poly[k], q);
        orc_ntt(c, first + i, out + i * N);
    }
}

/*
 * Decode: z_j = (1/Delta) sum_{k<n} (m_k + i m_(k+n)) zeta^(5^j k), in long double,
 * by the plain O(n^2) sum (used for pins on small rings) ...
 */
void orc_decode_direct(const orc_ctx *c, const long double *m, double scale, double *re, double *im) {
    uint64_t n = c->n, M = c->M;
    const long double tau = 6.283185307179586476925286766559005768L;
    for (uint64_t j = 0; j < n; j++) {
        long double sr = 0, si = 0;
        for (uint64_t k = 0; k < n; k++) {
            uint64_t e = c->pow5[j] * k % M;
            long double cr = cosl(tau * (long double)e / (long double)M), ci = sinl(tau * (long double)e / (long double)M);
            sr += m[k] * cr - m[k + n] * ci;
            si += m[k] * ci + m[k + n] * cr;
        }
        re[j] = (double)(sr / scale);
        im[j] = (double)(si / scale);
    }
}

/* ... and by the same sum organised as a size-n transform (twist by zeta^k, then B_e = sum_k a_k omega^(e k)). */
void orc_decode(const orc_ctx *c, const long double *m, double scale, double *re, double *im) {
    uint64_t n = c->n, M = c->M;
    const long double tau = 6.283185307179586476925286766559005768L;
    long double *vr = (long double *)malloc(n * sizeof(long double)), *vi = (long double *)malloc(n * sizeof(long double));
    uint32_t bits = c->log_n - 1;
    for (uint64_t k = 0; k < n; k++) {
        long double cr = cosl(tau * (long double)k / (long double)M), ci = sinl(tau * (long double)k / (long double)M);
        uint64_t pos = bitrev((uint32_t)k, bits);
        vr[pos] = m[k] * cr - m[k + n] * ci;
        vi[pos] = m[k] * ci + m[k + n] * cr;
    }
    for (uint64_t m2 = 2; m2 <= n; m2 <<= 1) {
        uint64_t half = m2 / 2;
        for (uint64_t k0 = 0; k0 < n; k0 += m2)
            for (uint64_t j = 0; j < half; j++) {
                long double ang = tau * (long double)j / (long double)m2;
                long double wr = cosl(ang), wi = sinl(ang);
                long double xr = vr[k0 + j + half], xi = vi[k0 + j + half];
                long double tr = wr * xr - wi * xi, ti = wr * xi + wi * xr;
                long double ur = vr[k0 + j], ui = vi[k0 + j];
                vr[k0 + j] = ur + tr;        vi[k0 + j] = ui + ti;
                vr[k0 + j + half] = ur - tr; vi[k0 + j + half] = ui - ti;
            }
    }
    for (uint64_t j = 0; j < n; j++) {
        uint64_t e = (c->pow5[j] % M - 1) / 4;
        re[j] = (double)(vr[e] / scale);
        im[j] = (double)(vi[e] / scale);
    }
    free(vr); free(vi);
}

/* ------------------------------------------------- keys, encrypt, decrypt */

/*
 * Symmetric encryption of an encoded plaintext: c1 = a, c0 = -a s + e + m.
 * `a` [level][N] uniform residues (taken as evaluation-domain values), `e`
 * int64[N] rounded Gaussian, `s` int64[N] ternary -- all drawn by the caller.
 * ct is [2][level][N].
 */
void orc_encrypt(const orc_ctx *c, const uint64_t *pt, const uint64_t *a, const int64_t *e, const int64_t *s,
                 uint32_t level, uint64_t *ct) {
    uint64_t N = c->N;
    uint64_t *sl = (uint64_t *)malloc((uint64_t)level * N * 8), *el = (uint64_t *)malloc((uint64_t)level * N * 8);
    orc_small_to_limbs(c, s, 0, level, sl);
    orc_small_to_limbs(c, e, 0, level, el);
    for (uint32_t i = 0; i < level; i++) {
        uint64_t q = c->mod[i];
        for (uint64_t k = 0; k < N; k++) {
            uint64_t x = i * N + k;
            uint64_t as = mulmod(a[x], sl[x], q);
            ct[x] = addmod(submod(el[x], as, q), pt[x], q);
            ct[(uint64_t)level * N + x] = a[x];
        }
    }
    free(sl); free(el);
}

/*
 * Decrypt: c0 + c1 s (+ c2 s^2) on limbs 0 and 1 only, CRT over q_0 q_1,
 * centred lift (valid while the plaintext stays below q_0 q_1 / 2), returned
 * both exactly (__int128) and as long double.  Either output may be NULL.
 */
void orc_decrypt(const orc_ctx *c, const uint64_t *ct, uint32_t ncomp, uint32_t level, const int64_t *s,
                 i128 *exact, long double *approx) {
    uint64_t N = c->N;
    uint32_t nl = level >= 2 ? 2 : 1;
    uint64_t *sl = (uint64_t *)malloc(2 * N * 8), *acc = (uint64_t *)malloc(2 * N * 8);
    orc_small_to_limbs(c, s, 0, nl, sl);
    for (uint32_t i = 0; i < nl; i++) {
        uint64_t q = c->mod[i];
        for (uint64_t k = 0; k < N; k++) {
            uint64_t v = 0;                                  /* Horner in s over the components */
            for (int comp = (int)ncomp - 1; comp >= 0; comp--)
                v = addmod(mulmod(v, sl[i * N + k], q), ct[((uint64_t)comp * level + i) * N + k], q);
            acc[i * N + k] = v;
        }
        orc_intt(c, i, acc + i * N);
    }
    uint64_t q0 = c->mod[0], q1 = nl == 2 ? c->mod[1] : 1;
    u128 Q = (u128)q0 * q1;
    uint64_t q0_inv_q1 = nl == 2 ? invmod(q0 % q1, q1) : 0;
    for (uint64_t k = 0; k < N; k++) {
        u128 v = acc[k];
        if (nl == 2) {                                       /* v = r0 + q0 * ((r1 - r0) q0^-1 mod q1) */
            uint64_t d = submod(acc[N + k], acc[k] % q1, q1);
            v += (u128)q0 * mulmod(d, q0_inv_q1, q1);
        }
        i128 sv = v > Q / 2 ? (i128)v - (i128)Q : (i128)v;
        if (exact) exact[k] = sv;
        if (approx) approx[k] = (long double)sv;
    }
    free(sl); free(acc);
}

/*
 * Switching key from s' to s (hybrid key switching, dnum digits):
 *   digit j, limb t:  a_j[t] uniform,  b_j[t] = -a_j[t] s + e_j + [t in D_j] (P mod t) s'
 * (the gadget factor P * Qhat_j * Qhat_j^-1 is P on the digit's own limbs and
 * 0 on the others, so the key does not depend on the level).
 * `sprime` [L+K][N] evaluation-domain limbs of s'; `a` [dnum][L+K][N]; `e`
 * [dnum][N] int64.  evk is [dnum][2][L+K][N] with component 0 = b, 1 = a.
 */
void orc_switch_keygen(const orc_ctx *c, const int64_t *s, const uint64_t *sprime, const uint64_t *a,
                       const int64_t *e, uint64_t *evk) {
    uint64_t N = c->N;
    uint32_t T = c->L + c->K;
    uint64_t *sl = (uint64_t *)malloc((uint64_t)T * N * 8), *el = (uint64_t *)malloc((uint64_t)T * N * 8);
    orc_small_to_limbs(c, s, 0, T, sl);
    for (uint32_t j = 0; j < c->dnum; j++) {
        orc_small_to_limbs(c, e + (uint64_t)j * N, 0, T, el);
        #pragma omp parallel for
        for (uint32_t t = 0; t < T; t++) {
            uint64_t m = c->mod[t];
            int own = t < c->L && t / c->alpha == j;
            uint64_t Pm = 1;
            for (uint32_t k = 0; k < c->K; k++) Pm = mulmod(Pm, c->mod[c->L + k] % m, m);
            const uint64_t *at = a + ((uint64_t)j * T + t) * N;
            uint64_t *bo = evk + (((uint64_t)j * 2 + 0) * T + t) * N;
            uint64_t *ao = evk + (((uint64_t)j * 2 + 1) * T + t) * N;
            for (uint64_t k = 0; k < N; k++) {
                uint64_t v = submod(el[t * N + k], mulmod(at[k], sl[t * N + k], m), m);
                if (own) v = addmod(v, mulmod(Pm, sprime[t * N + k], m), m);
                bo[k] = v;
                ao[k] = at[k];
            }
        }
    }
    free(sl); free(el);
}

/* ------------------------------------------------------- pointwise family */

/* PCMult + Add: acc[c][i][.] (+)= ct[c][i][.] * pt[i][.], c in {0,1}. */
void orc_mul_plain_acc(const orc_ctx *c, const uint64_t *ct, const uint64_t *pt, uint64_t *acc, uint32_t level, int init) {
    uint64_t N = c->N;
    #pragma omp parallel for collapse(2)
    for (uint32_t comp = 0; comp < 2; comp++)
        for (uint32_t i = 0; i < level; i++) {
            uint64_t q = c->mod[i];
            for (uint64_t k = 0; k < N; k++) {
                uint64_t x = ((uint64_t)comp * level + i) * N + k;
                uint64_t v = mulmod(ct[x], pt[i * N + k], q);
                acc[x] = init ? v : addmod(acc[x], v, q);
            }
        }
}

/* Add: out = a + b, `nl` limbs under primes 0..level-1 repeated per component. */
void orc_add(const orc_ctx *c, const uint64_t *a, const uint64_t *b, uint64_t *out, uint32_t ncomp, uint32_t level) {
    uint64_t N = c->N;
    for (uint32_t x = 0; x < ncomp * level; x++) {
        uint64_t q = c->mod[x % level];
        for (uint64_t k = 0; k < N; k++) out[x * N + k] = addmod(a[x * N + k], b[x * N + k], q);
    }
}

/*
 * Multiplication and addition of a real constant (Section 2.1: Mult and Add with a plaintext that encodes the
 * same value in every slot).  Such a plaintext is the constant polynomial v = round(c * scale), whose
 * evaluation-domain image is v in every position.  v is passed as a signed integer (the caller rounds).
 *   mul: out = ct * v on every component and limb;   add: out = ct with v added to component 0.
 */
void orc_mul_const(const orc_ctx *c, const uint64_t *in, int64_t v, uint32_t ncomp, uint32_t level, uint64_t *out) {
    uint64_t N = c->N;
    for (uint32_t x = 0; x < ncomp * level; x++) {
        uint64_t q = c->mod[x % level], r = reduce_signed((i128)v, q);
        for (uint64_t k = 0; k < N; k++) out[x * N + k] = mulmod(in[x * N + k], r, q);
    }
}
void orc_add_const(const orc_ctx *c, const uint64_t *in, int64_t v, uint32_t ncomp, uint32_t level, uint64_t *out) {
    uint64_t N = c->N;
    for (uint32_t x = 0; x < ncomp * level; x++) {
        uint64_t q = c->mod[x % level], r = x < level ? reduce_signed((i128)v, q) : 0;
        for (uint64_t k = 0; k < N; k++) out[x * N + k] = addmod(in[x * N + k], r, q);
    }
}

/* Galois automorphism by definition, coefficient domain: a(X) -> a(X^g), X^N = -1. */
void orc_automorphism_coeff(const orc_ctx *c, uint32_t t, const uint64_t *a, uint64_t g, uint64_t *out) {
    uint64_t q = c->mod[t], N = c->N, M = c->M;
    for (uint64_t j = 0; j < N; j++) {
        uint64_t e = (u128)j * g % M;
        if (e < N) out[e] = a[j];
        else out[e - N] = a[j] ? q - a[j] : 0;
    }
}
/* Same on small signed coefficients (for sigma_g of the secret). */
void orc_automorphism_small(const orc_ctx *c, const int64_t *a, uint64_t g, int64_t *out) {
    uint64_t N = c->N, M = c->M;
    for (uint64_t j = 0; j < N; j++) {
        uint64_t e = (u128)j * g % M;
        if (e < N) out[e] = a[j]; else out[e - N] = -a[j];
    }
}

/*
 * Galois automorphism in the stored (evaluation, bit-reversed) domain: since
 * stored[p] = a(psi^(2 brev(p)+1)) and sigma_g(a)(x) = a(x^g),
 *   out[p] = in[p'],  2 brev(p') + 1 = g (2 brev(p) + 1) mod 2N.
 * The modulus plays no part.  Pinned against the coefficient-domain definition.
 */
void orc_automorphism_eval(const orc_ctx *c, const uint64_t *in, uint64_t g, uint64_t *out) {
    uint64_t N = c->N, M = c->M;
    for (uint64_t p = 0; p < N; p++) {
        uint64_t e = (u128)g * (2 * (uint64_t)c->brev[p] + 1) % M;
        out[p] = in[c->brev[(e - 1) / 2]];
    }
}

/* 5^r mod 2N with r reduced mod n: the Galois element of a left rotation by r slots (Eq. 5's rho^r). */
uint64_t orc_galois_element(const orc_ctx *c, int64_t r) {
    int64_t n = (int64_t)c->n;
    r %= n; if (r < 0) r += n;
    return c->pow5[r];
}

/* ------------------------------------------------------------ key switch */

static uint32_t num_digits(const orc_ctx *c, uint32_t level) { return (level + c->alpha - 1) / c->alpha; }

/*
 * ModUp of one digit (fast basis conversion, centred, no floating-point
 * correction).  d is [level][N] coefficient domain.  Digit j has the active
 * limbs D = {j alpha .. min((j+1) alpha, level) - 1}, Q_j their product,
 * qhat_i = Q_j / q_i.   y_i = centre([d_i qhat_i^-1]_{q_i});
 * target t not in D:  sum_i y_i (qhat_i mod t) mod t;   t in D: d_t.
 * ext is [level+K][N] ordered q_0..q_{level-1}, p_0..p_{K-1}.
 */
void orc_modup_digit(const orc_ctx *c, const uint64_t *d, uint32_t level, uint32_t j, uint64_t *ext) {
    uint64_t N = c->N;
    uint32_t lo = j * c->alpha, hi = lo + c->alpha < level ? lo + c->alpha : level, nd = hi - lo;
    uint32_t nt = level + c->K;
    uint64_t *hat_inv = (uint64_t *)malloc(nd * 8);
    uint64_t *hat_mod = (uint64_t *)malloc((uint64_t)nd * nt * 8);
    for (uint32_t a = 0; a < nd; a++) {
        uint64_t qi = c->mod[lo + a], h = 1;
        for (uint32_t b = 0; b < nd; b++) if (b != a) h = mulmod(h, c->mod[lo + b] % qi, qi);
        hat_inv[a] = invmod(h, qi);
        for (uint32_t x = 0; x < nt; x++) {
            uint64_t t = c->mod[x < level ? x : c->L + (x - level)], v = 1 % t;
            for (uint32_t b = 0; b < nd; b++) if (b != a) v = mulmod(v, c->mod[lo + b] % t, t);
            hat_mod[a * nt + x] = v;
        }
    }
    #pragma omp parallel for
    for (uint32_t x = 0; x < nt; x++) {
        uint64_t *o = ext + (uint64_t)x * N;
        if (x >= lo && x < hi) { memcpy(o, d + (uint64_t)x * N, N * 8); continue; }
        uint64_t t = c->mod[x < level ? x : c->L + (x - level)];
        for (uint64_t k = 0; k < N; k++) {
            i128 acc = 0;
            for (uint32_t a = 0; a < nd; a++) {
                uint64_t qi = c->mod[lo + a];
                int64_t y = centre(mulmod(d[(uint64_t)(lo + a) * N + k], hat_inv[a], qi), qi);
                acc += (i128)y * hat_mod[a * nt + x];
            }
            o[k] = reduce_signed(acc, t);
        }
    }
    free(hat_inv); free(hat_mod);
}

/*
 * ModDown of one component.  u is [level+K][N] evaluation domain.  iNTT the K
 * special limbs; y_k = centre([u_{p_k} Phat_k^-1]_{p_k}); conv_i = sum_k y_k
 * (Phat_k mod q_i) mod q_i; NTT conv_i; out_i = (u_i - conv_i) P^-1 mod q_i.
 * out is [level][N] evaluation domain.
 */
void orc_moddown(const orc_ctx *c, const uint64_t *u, uint32_t level, uint64_t *out) {
    uint64_t N = c->N;
    uint32_t K = c->K, L = c->L;
    uint64_t *sp = (uint64_t *)malloc((uint64_t)K * N * 8);
    memcpy(sp, u + (uint64_t)level * N, (uint64_t)K * N * 8);
    orc_intt_batch(c, sp, 1, L, K);
    uint64_t *hat_inv = (uint64_t *)malloc(K * 8);
    for (uint32_t a = 0; a < K; a++) {
        uint64_t pa = c->mod[L + a], h = 1;
        for (uint32_t b = 0; b < K; b++) if (b != a) h = mulmod(h, c->mod[L + b] % pa, pa);
        hat_inv[a] = invmod(h, pa);
    }
    #pragma omp parallel for
    for (uint32_t i = 0; i < level; i++) {
        uint64_t q = c->mod[i], Pm = 1;
        uint64_t *hat_mod = (uint64_t *)malloc(K * 8);
        for (uint32_t a = 0; a < K; a++) {
            uint64_t v = 1;
            for (uint32_t b = 0; b < K; b++) if (b != a) v = mulmod(v, c->mod[L + b] % q, q);
            hat_mod[a] = v;
            Pm = mulmod(Pm, c->mod[L + a] % q, q);
        }
        uint64_t Pinv = invmod(Pm, q);
        uint64_t *conv = (uint64_t *)malloc(N * 8);
        for (uint64_t k = 0; k < N; k++) {
            i128 acc = 0;
            for (uint32_t a = 0; a < K; a++) {
                uint64_t pa = c->mod[L + a];
                int64_t y = centre(mulmod(sp[(uint64_t)a * N + k], hat_inv[a], pa), pa);
                acc += (i128)y * hat_mod[a];
            }
            conv[k] = reduce_signed(acc, q);
        }
        orc_ntt(c, i, conv);
        for (uint64_t k = 0; k < N; k++)
            out[(uint64_t)i * N + k] = mulmod(submod(u[(uint64_t)i * N + k], conv[k], q), Pinv, q);
        free(conv); free(hat_mod);
    }
    free(sp); free(hat_inv);
}

/*
 * ModUp of all active digits followed by the NTT of every extended limb:
 * d [level][N] evaluation domain -> ext [beta][level+K][N] evaluation domain.
 */
void orc_modup_all(const orc_ctx *c, const uint64_t *d, uint32_t level, uint64_t *ext) {
    uint64_t N = c->N;
    uint32_t beta = num_digits(c, level), nt = level + c->K;
    uint64_t *dc = (uint64_t *)malloc((uint64_t)level * N * 8);
    memcpy(dc, d, (uint64_t)level * N * 8);
    orc_intt_batch(c, dc, 1, 0, level);
    for (uint32_t j = 0; j < beta; j++) {
        uint64_t *e = ext + (uint64_t)j * nt * N;
        orc_modup_digit(c, dc, level, j, e);
        orc_ntt_batch(c, e, 1, 0, level);
        orc_ntt_batch(c, e + (uint64_t)level * N, 1, c->L, c->K);
    }
    free(dc);
}

/*
 * Evaluation-key inner product in the extended basis: ext [beta][level+K][N]
 * evaluation domain, evk [dnum][2][L+K][N].  u_c[t] = sum_j ext_j[t] * evk_{j,c}[t]
 * over the active limbs (key limbs of dropped q's are skipped).  u is
 * [2][level+K][N].
 */
void orc_inner_product(const orc_ctx *c, const uint64_t *ext, const uint64_t *evk, uint32_t level, uint64_t *u) {
    uint64_t N = c->N;
    uint32_t beta = num_digits(c, level), nt = level + c->K, T = c->L + c->K;
    #pragma omp parallel for
    for (uint32_t x = 0; x < 2 * nt; x++) {
        uint32_t comp = x / nt, lx = x % nt;
        uint32_t kt = lx < level ? lx : c->L + (lx - level);       /* index into the key / prime space */
        uint64_t m = c->mod[kt];
        for (uint64_t p = 0; p < N; p++) {
            uint64_t acc = 0;
            for (uint32_t j = 0; j < beta; j++)
                acc = addmod(acc, mulmod(ext[((uint64_t)j * nt + lx) * N + p],
                                         evk[(((uint64_t)j * 2 + comp) * T + kt) * N + p], m), m);
            u[(uint64_t)x * N + p] = acc;
        }
    }
}

/* The inner product followed by the ModDown of each component.  k is [2][level][N]. */
void orc_inner_moddown(const orc_ctx *c, const uint64_t *ext, const uint64_t *evk, uint32_t level, uint64_t *k) {
    uint64_t N = c->N;
    uint32_t nt = level + c->K;
    uint64_t *u = (uint64_t *)malloc(2ull * nt * N * 8);
    orc_inner_product(c, ext, evk, level, u);
    orc_moddown(c, u, level, k);
    orc_moddown(c, u + (uint64_t)nt * N, level, k + (uint64_t)level * N);
    free(u);
}

/* KeySwitch core: d [level][N] evaluation domain -> (k0,k1) [2][level][N] with k0 + k1 s ~ d s'. */
void orc_keyswitch(const orc_ctx *c, const uint64_t *d, const uint64_t *evk, uint32_t level, uint64_t *k) {
    uint32_t beta = num_digits(c, level), nt = level + c->K;
    uint64_t *ext = (uint64_t *)malloc((uint64_t)beta * nt * c->N * 8);
    orc_modup_all(c, d, level, ext);
    orc_inner_moddown(c, ext, evk, level, k);
    free(ext);
}

/*
 * Rot_k (Section 2.1), plain: apply sigma_g to both components, key-switch the
 * permuted c1, add.  out = (sigma c0 + k0, k1).  Scale and level unchanged.
 */
void orc_rotate(const orc_ctx *c, const uint64_t *ct, const uint64_t *evk, uint64_t g, uint32_t level, uint64_t *out) {
    uint64_t N = c->N;
    uint64_t *perm = (uint64_t *)malloc(2ull * level * N * 8), *k = (uint64_t *)malloc(2ull * level * N * 8);
    for (uint32_t x = 0; x < 2 * level; x++) orc_automorphism_eval(c, ct + (uint64_t)x * N, g, perm + (uint64_t)x * N);
    orc_keyswitch(c, perm + (uint64_t)level * N, evk, level, k);
    for (uint32_t i = 0; i < level; i++) {
        uint64_t q = c->mod[i];
        for (uint64_t p = 0; p < N; p++) {
            out[(uint64_t)i * N + p] = addmod(perm[(uint64_t)i * N + p], k[(uint64_t)i * N + p], q);
            out[((uint64_t)level + i) * N + p] = k[((uint64_t)level + i) * N + p];
        }
    }
    free(perm); free(k);
}

/*
 * A sum of rotated ciphertexts with one ModDown ("lazy" ModDown: the sum is
 * formed in the extended basis, where the key-switched terms live before
 * they are divided by P):
 *   U = sum_i <ModUp(sigma_{g_i} c1_i), evk_i>   over the limbs of Q_level P,
 *   out = (sum_i sigma_{g_i} c0_i + ModDown(U_0), ModDown(U_1)).
 * It decrypts to the same sum as adding up orc_rotate's results, with one
 * division rounding instead of n.  cts is [n][2][level][N], evks[i] points at
 * the key of Galois element gs[i].
 */
void orc_rotate_sum(const orc_ctx *c, const uint64_t *cts, const uint64_t *const *evks, const uint64_t *gs, uint32_t n,
                    uint32_t level, uint64_t *out) {
    uint64_t N = c->N;
    uint32_t beta = num_digits(c, level), nt = level + c->K;
    uint64_t *perm = (uint64_t *)malloc(2ull * level * N * 8), *ext = (uint64_t *)malloc((uint64_t)beta * nt * N * 8);
    uint64_t *u = (uint64_t *)malloc(2ull * nt * N * 8), *U = (uint64_t *)calloc(2ull * nt * N, 8);
    uint64_t *z = (uint64_t *)calloc((uint64_t)level * N, 8);
    for (uint32_t r = 0; r < n; r++) {
        const uint64_t *ct = cts + (uint64_t)r * 2 * level * N;
        for (uint32_t x = 0; x < 2 * level; x++) orc_automorphism_eval(c, ct + (uint64_t)x * N, gs[r], perm + (uint64_t)x * N);
        orc_modup_all(c, perm + (uint64_t)level * N, level, ext);
        orc_inner_product(c, ext, evks[r], level, u);
        for (uint32_t x = 0; x < 2 * nt; x++) {
            uint32_t lx = x % nt;
            uint64_t m = c->mod[lx < level ? lx : c->L + (lx - level)];
            for (uint64_t p = 0; p < N; p++) U[(uint64_t)x * N + p] = addmod(U[(uint64_t)x * N + p], u[(uint64_t)x * N + p], m);
        }
        for (uint32_t i = 0; i < level; i++)
            for (uint64_t p = 0; p < N; p++) z[(uint64_t)i * N + p] = addmod(z[(uint64_t)i * N + p], perm[(uint64_t)i * N + p], c->mod[i]);
    }
    orc_moddown(c, U, level, out);
    orc_moddown(c, U + (uint64_t)nt * N, level, out + (uint64_t)level * N);
    for (uint32_t i = 0; i < level; i++)
        for (uint64_t p = 0; p < N; p++) out[(uint64_t)i * N + p] = addmod(out[(uint64_t)i * N + p], z[(uint64_t)i * N + p], c->mod[i]);
    free(perm); free(ext); free(u); free(U); free(z);
}

/*
 * Hoisted rotations: one iNTT + ModUp + NTT of c1 shared by all rotations;
 * for each g: permute every extended limb of every digit by sigma_g, inner
 * product with evk_g, ModDown, add sigma_g(c0).  The steps are taken in
 * this order; the result is bit-identical to the plain form because the
 * centred conversion is odd (centre(q - v) = -centre(v) for odd q), hence
 * commutes with the permutation and sign flips of sigma_g (pinned by a test).
 * evks[r] points at key r; outs is
 * [nrot][2][level][N].
 */
void orc_rotate_hoisted(const orc_ctx *c, const uint64_t *ct, const uint64_t *const *evks, const uint64_t *gs,
                        uint32_t nrot, uint32_t level, uint64_t *outs) {
    uint64_t N = c->N;
    uint32_t beta = num_digits(c, level), nt = level + c->K;
    uint64_t ext_sz = (uint64_t)beta * nt * N;
    uint64_t *ext = (uint64_t *)malloc(ext_sz * 8), *pe = (uint64_t *)malloc(ext_sz * 8);
    uint64_t *k = (uint64_t *)malloc(2ull * level * N * 8), *c0 = (uint64_t *)malloc(N * 8);
    orc_modup_all(c, ct + (uint64_t)level * N, level, ext);
    for (uint32_t r = 0; r < nrot; r++) {
        uint64_t *out = outs + (uint64_t)r * 2 * level * N;
        #pragma omp parallel for
        for (uint32_t x = 0; x < beta * nt; x++) orc_automorphism_eval(c, ext + (uint64_t)x * N, gs[r], pe + (uint64_t)x * N);
        orc_inner_moddown(c, pe, evks[r], level, k);
        for (uint32_t i = 0; i < level; i++) {
            uint64_t q = c->mod[i];
            orc_automorphism_eval(c, ct + (uint64_t)i * N, gs[r], c0);
            for (uint64_t p = 0; p < N; p++) {
                out[(uint64_t)i * N + p] = addmod(c0[p], k[(uint64_t)i * N + p], q);
                out[((uint64_t)level + i) * N + p] = k[((uint64_t)level + i) * N + p];
            }
        }
    }
    free(ext); free(pe); free(k); free(c0);
}

/*
 * Rescale (Section 2.1): drop the last limb with exact rounding.
 *   r = centre(c_{l-1});  out_i = (c_i - (r mod q_i)) q_{l-1}^-1 mod q_i,  i < l-1.
 * Works per coefficient, so the last limb goes to the coefficient domain and
 * its lift comes back under each remaining prime.  in [ncomp][level][N] ->
 * out [ncomp][level-1][N].
 */
void orc_rescale(const orc_ctx *c, const uint64_t *in, uint32_t ncomp, uint32_t level, uint64_t *out) {
    uint64_t N = c->N;
    uint32_t last = level - 1;
    uint64_t ql = c->mod[last];
    for (uint32_t comp = 0; comp < ncomp; comp++) {
        uint64_t *lc = (uint64_t *)malloc(N * 8);
        memcpy(lc, in + ((uint64_t)comp * level + last) * N, N * 8);
        orc_intt(c, last, lc);
        #pragma omp parallel for
        for (uint32_t i = 0; i < last; i++) {
            uint64_t q = c->mod[i], qinv = invmod(ql % q, q);
            uint64_t *r = (uint64_t *)malloc(N * 8);
            for (uint64_t k = 0; k < N; k++) r[k] = reduce_signed(centre(lc[k], ql), q);
            orc_ntt(c, i, r);
            for (uint64_t k = 0; k < N; k++)
                out[((uint64_t)comp * last + i) * N + k] =
                    mulmod(submod(in[((uint64_t)comp * level + i) * N + k], r[k], q), qinv, q);
            free(r);
        }
        free(lc);
    }
}

/* Tensor product of two 2-component ciphertexts: (c0 d0, c0 d1 + c1 d0, c1 d1), [3][level][N]. */
void orc_tensor(const orc_ctx *c, const uint64_t *a, const uint64_t *b, uint32_t level, uint64_t *e) {
    uint64_t N = c->N, S = (uint64_t)level * N;
    for (uint32_t i = 0; i < level; i++) {
        uint64_t q = c->mod[i];
        for (uint64_t k = 0; k < N; k++) {
            uint64_t x = (uint64_t)i * N + k;
            e[x] = mulmod(a[x], b[x], q);
            e[S + x] = addmod(mulmod(a[x], b[S + x], q), mulmod(a[S + x], b[x], q), q);
            e[2 * S + x] = mulmod(a[S + x], b[S + x], q);
        }
    }
}

/* Mult (Section 2.1) with relinearisation: out = (e0 + k0, e1 + k1), (k0,k1) = KeySwitch(e2, rlk).  No rescale inside. */
void orc_mul_relin(const orc_ctx *c, const uint64_t *a, const uint64_t *b, const uint64_t *rlk, uint32_t level, uint64_t *out) {
    uint64_t N = c->N, S = (uint64_t)level * N;
    uint64_t *e = (uint64_t *)malloc(3 * S * 8), *k = (uint64_t *)malloc(2 * S * 8);
    orc_tensor(c, a, b, level, e);
    orc_keyswitch(c, e + 2 * S, rlk, level, k);
    for (uint32_t x = 0; x < 2 * level; x++) {
        uint64_t q = c->mod[x % level];
        for (uint64_t p = 0; p < N; p++) out[x * N + p] = addmod(e[x * N + p], k[x * N + p], q);
    }
    free(e); free(k);
}

/*
 * Sum of n products with one relinearisation (the lazy form of a sum of Mults, Section 4: the attention
 * products add up many ciphertext x ciphertext terms): e = sum_i tensor(a_i, b_i) component-wise modulo each
 * prime, (k0,k1) = KeySwitch(e2, rlk), out = (e0 + k0, e1 + k1).  a, b: [n][2][level][N].  For n = 1 this is
 * orc_mul_relin.  Not the same integers as the sum of n separately relinearised products (the key switch's
 * rounding acts on the sum once instead of on every term); both decrypt to the sum of the slot products.
 */
void orc_mul_relin_sum(const orc_ctx *c, const uint64_t *a, const uint64_t *b, uint32_t n, const uint64_t *rlk, uint32_t level,
                       uint64_t *out) {
    uint64_t N = c->N, S = (uint64_t)level * N;
    uint64_t *e = (uint64_t *)calloc(3 * S, 8), *t = (uint64_t *)malloc(3 * S * 8), *k = (uint64_t *)malloc(2 * S * 8);
    for (uint32_t i = 0; i < n; i++) {
        orc_tensor(c, a + (uint64_t)i * 2 * S, b + (uint64_t)i * 2 * S, level, t);
        for (uint32_t x = 0; x < 3 * level; x++) {
            uint64_t q = c->mod[x % level];
            for (uint64_t p = 0; p < N; p++) e[x * N + p] = addmod(e[x * N + p], t[x * N + p], q);
        }
    }
    orc_keyswitch(c, e + 2 * S, rlk, level, k);
    for (uint32_t x = 0; x < 2 * level; x++) {
        uint64_t q = c->mod[x % level];
        for (uint64_t p = 0; p < N; p++) out[x * N + p] = addmod(e[x * N + p], k[x * N + p], q);
    }
    free(e); free(t); free(k);
}

/* Pointwise product of limb arrays under primes first..first+nl-1 (used to form s^2 for the relinearisation key). */
void orc_pointwise_mul(const orc_ctx *c, const uint64_t *a, const uint64_t *b, uint32_t first, uint32_t nl, uint64_t *out) {
    uint64_t N = c->N;
    for (uint32_t i = 0; i < nl; i++) {
        uint64_t q = c->mod[first + i];
        for (uint64_t k = 0; k < N; k++) out[i * N + k] = mulmod(a[i * N + k], b[i * N + k], q);
    }
}

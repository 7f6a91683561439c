// Shared declarations of the ckks_b200 library: context, device tables,
// modular arithmetic for 50-bit primes, kernel launch entry points.
#pragma once
#include <algorithm>

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "../../include/ckks_b200.h"

typedef unsigned long long u64;
typedef unsigned __int128 u128;

// ---------------------------------------------------------------------------
// Device-side view of the context tables (plain pointers, passed by value).
// Prime index space t: 0..L-1 = q_i, L..L+K-1 = p_k.
// ---------------------------------------------------------------------------
struct DevTables {
    uint32_t log_n, N, L, K, alpha, T, dnum;
    const u64 *mod;          // [T]
    const u64 *mu;           // [T] floor(2^112 / prime)
    const u64 *mu64;         // [T] floor(2^64 / prime)
    const double2 *modd;     // [T] {prime, 1/prime} as doubles
    const ulonglong2 *tw_fwd;  // [T][N] {psi^bitrev(i), Shoup companion}, index m+i
    const ulonglong2 *tw_inv;  // [T][N] inverses of the same
    const ulonglong2 *n_inv;   // [T] {N^-1, Shoup}
    // fp64 copies for the double-precision NTT path (N = 2^16 only): the centred representative of w as a double, same
    // indexing (the transform estimates a product's quotient from the rounded product and 1/q, so the table holds w alone)
    const double *twd_fwd, *twd_inv;    // [T][N]
    const double2 *n_inv_d;             // [T][2] {N^-1, N^-1/q}, {w N^-1, that/q} for the inverse's last twiddle w, all centred
    // inverse-transform scalings that deliver the basis conversions' first factor y = [d qhat^-1] (N = 2^16 only), pairs
    // {N^-1 qhat^-1, last inverse twiddle times that}, each {v, v / prime} centred
    const double2 *inv_scale_up;   // [(L+1)][L][2]   ModUp: level, limb
    const double2 *inv_scale_dn;   // [K][2]          ModDown: special limb
    // ModUp, per level l (1..L), digit j, source a < alpha:
    const ulonglong2 *up_hat_inv;  // [(L+1)][dnum][alpha]        {qhat^-1 mod q_src, Shoup}
    const u64 *up_hat_mod;         // [(L+1)][dnum][alpha][T]     qhat mod target
    const double2 *up_hat_mod_d;   // same shape, {c, c / target prime} as doubles
    // ModDown:
    const ulonglong2 *dn_hat_inv;  // [K]      {Phat_k^-1 mod p_k, Shoup}
    const u64 *dn_hat_mod;         // [L][K]   Phat_k mod q_i
    const double2 *dn_hat_mod_d;   // [L][K]   {c, c / q_i} as doubles
    const ulonglong2 *dn_p_inv;    // [L]      {P^-1 mod q_i, Shoup}
    const double2 *dn_p_inv_d;     // [L]      {P^-1 mod q_i, that / q_i} as doubles
    const double *dn_p_mod_d;      // [L]      P mod q_i as a double
    // Tensor-core basis conversion (conv_mma.cu; conv_groups = 0 when alpha or K exceeds 8 sources): byte matrices of
    // the conversion constants in the B-fragment order of mma.m16n8k32, [group of 8 targets][13 diagonals][2 k-steps]
    // [lane][2] words; targets are the non-own limbs of the digit in ascending order (ModUp) or q_0.. (ModDown)
    const uint32_t *up_bmat;       // [(L+1)][dnum][conv_groups][13][2][64]
    const uint32_t *dn_bmat;       // [conv_groups][13][2][64]
    const double2 *two52_d;        // [T] {2^52 mod prime, that / prime}
    uint32_t conv_groups;
    // Rescale: [L(last)][L(i)] {q_last^-1 mod q_i, Shoup}
    const ulonglong2 *rs_inv;
    // Encode:
    const uint32_t *enc_src;       // [n] slot index feeding FFT input position pos (bit-reversed e_j)
    const double2 *enc_omega;      // [n] exp(2 pi i t / n)
    const double2 *enc_omega_st;   // [min(n, 1024)] the same values stage by stage: entry half + j = omega^(j n / (2 half)), half = 1, 2, .. (entry 0 unused)
    const double2 *enc_omega_st2;  // [n] second-pass twiddles by stage and row: entry (hr + jr) * ch + col = omega^((jr ch + col) n / (2 hr ch)), ch = min(n, 1024)
    const double2 *enc_zeta;       // [n] exp(2 pi i k / 2N)
    int *range_flag;               // [0] sticky encode overflow flag, [1] sticky device-side wait timeout flag
};

struct ckks_ctx {
    uint32_t log_n, N, n, L, K, dnum, alpha, T;
    int device;
    std::vector<u64> mod;        // host copy of the primes
    std::vector<u64> pow5;       // 5^j mod 2N, j < n (host)
    DevTables dev;               // pointers into `allocs`
    std::vector<void *> allocs;  // device allocations owned by the context
    std::string cuda_error;
    // options (ckks_context_set_option); host-side state read when a call is made
    uint32_t ntt_fp_share = 8;               // of every 8 limbs, how many take the double-precision NTT path
    int ntt_bulk_store = 1;                  // forward row pass (N = 2^16): results leave as 128-byte bulk copies from shared memory
    int conv_kernel = 0;                     // basis conversions: 0 = FP64 pipe, 1 = tensor cores (conv_mma.cu)
    int mac_kernel = 82;                     // projection multiply-accumulate kernel (see launch_mac_mma)
    long long wait_cycles = 2000000000ll;    // clock bound of every device-side wait (about a second)
    // Streams of the context.  Composite calls whose work is many independent single-ciphertext chains (the attention
    // entry points) spread those chains over `lanes` streams, lane 0 being the caller's: a single ciphertext's kernels fill
    // the GPU for at most one wave, so independent chains overlap.  Forked from and joined to the caller's stream by events.
    int lanes = 4;
    cudaStream_t lane_stream[3] = {nullptr, nullptr, nullptr};
    cudaEvent_t lane_event[4] = {nullptr, nullptr, nullptr, nullptr};
};

// The context's streams as lanes for independent chains: lane 0 is the caller's stream.  fork() makes the other lanes wait
// for what the caller's stream has been given so far, join() makes the caller's stream wait for all of them.
struct Lanes {
    ckks_ctx *c;
    cudaStream_t caller;
    uint32_t n;
    Lanes(ckks_ctx *ctx, void *stream) : c(ctx), caller((cudaStream_t)stream), n((uint32_t)std::max(1, std::min(ctx->lanes, 4))) {}
    void *at(uint32_t i) const { return i % n == 0 ? (void *)caller : (void *)c->lane_stream[i % n - 1]; }
    void fork() const {
        if (n == 1) return;
        int prev = 0;
        cudaGetDevice(&prev);
        cudaSetDevice(c->device);
        cudaEventRecord(c->lane_event[0], caller);
        for (uint32_t i = 1; i < n; i++) cudaStreamWaitEvent(c->lane_stream[i - 1], c->lane_event[0], 0);
        cudaSetDevice(prev);
    }
    void join() const {
        if (n == 1) return;
        int prev = 0;
        cudaGetDevice(&prev);
        cudaSetDevice(c->device);
        for (uint32_t i = 1; i < n; i++) {
            cudaEventRecord(c->lane_event[i], c->lane_stream[i - 1]);
            cudaStreamWaitEvent(caller, c->lane_event[i], 0);
        }
        cudaSetDevice(prev);
    }
};
inline uint32_t lane_count(const ckks_ctx *c) { return (uint32_t)std::max(1, std::min(c->lanes, 4)); }

// ---------------------------------------------------------------------------
// "Tiled" operand layout of the projection's multiply-accumulate.  R rows (one row = one plaintext, or one
// component of one ciphertext) of [level][N] words are stored so that, for a limb i and a block of 64
// coefficients, all R rows are adjacent:   index(r, i, p) = (((i * N/64) + p/64) * R + r) * 64 + p % 64.
// The multiply-accumulate walks all rows of a few coefficients; in the plain [row][level][N] layout those
// words are 12-24 MiB apart (one TLB entry and one DRAM page per 64 bytes), here they are one 512-byte step apart.
// ---------------------------------------------------------------------------
__host__ __device__ inline size_t tiled_index(uint32_t R, uint32_t N, uint32_t r, uint32_t i, uint32_t p) {
    return ((((size_t)i * (N >> 6)) + (p >> 6)) * R + r) * 64 + (p & 63);
}
// where a key-switch result goes when it is written straight into a tiled buffer: component c of batch entry b
// becomes row row0 + b * row_stride + c of a buffer with R rows (R = 0: plain layout)
struct TiledOut { uint32_t R = 0, row0 = 0, row_stride = 0; };

// ---------------------------------------------------------------------------
// Limb addressing for batched limb-wise kernels (NTT): limb y of a buffer
// [..][period][N] -> prime index, or -1 to skip the limb.
//   kind 0: prime = first + y % period
//   kind 1: "extended" layout [batch][digit][level + K]: x = y % period is q_x for
//           x < level, else p_{x-level}; with skip_own the digit's own limbs
//           (which never leave the evaluation domain) are skipped.
// ---------------------------------------------------------------------------
struct LimbMap {
    uint32_t kind, first, period, pitch, level, L, alpha, nbeta, skip_own;
};
// limbs [..][period][N] contiguous, limb x of every period under prime first + x
inline LimbMap plain_map(uint32_t first, uint32_t period) { return LimbMap{0, first, period, period, 0, 0, 0, 1, 0}; }
// same, but consecutive periods start `pitch` limbs apart (a sub-range of limbs of a larger array)
inline LimbMap pitched_map(uint32_t first, uint32_t period, uint32_t pitch) { return LimbMap{0, first, period, pitch, 0, 0, 0, 1, 0}; }
// extended digits [batch][beta][level + K]
inline LimbMap ext_map(uint32_t level, uint32_t K, uint32_t L, uint32_t alpha, uint32_t beta) {
    return LimbMap{1, 0, level + K, level + K, level, L, alpha, beta, 1};
}

__host__ __device__ inline int limb_prime(const LimbMap &m, uint32_t y) {
    uint32_t x = y % m.period;
    if (m.kind == 0) return (int)(m.first + x);
    if (m.skip_own) {
        uint32_t j = (y / m.period) % m.nbeta, lo = j * m.alpha, hi = lo + m.alpha < m.level ? lo + m.alpha : m.level;
        if (x >= lo && x < hi) return -1;
    }
    return x < m.level ? (int)x : (int)(m.L + (x - m.level));
}
// index (in limbs) of limb y from the base pointer
__host__ __device__ inline size_t limb_index(const LimbMap &m, uint32_t y) { return (size_t)(y / m.period) * m.pitch + y % m.period; }

// ---------------------------------------------------------------------------
// Modular arithmetic, primes in (2^49, 2^50).
// ---------------------------------------------------------------------------

// x * w mod q for a constant w with companion wp = floor(w 2^64 / q); result in [0, 2q) for ANY 64-bit x.
__device__ __forceinline__ u64 mul_shoup_lazy(u64 x, u64 w, u64 wp, u64 q) {
    return x * w - __umul64hi(x, wp) * q;
}
__device__ __forceinline__ u64 mul_shoup(u64 x, u64 w, u64 wp, u64 q) {
    u64 r = mul_shoup_lazy(x, w, wp, q);
    return r >= q ? r - q : r;
}
__device__ __forceinline__ u64 add_mod(u64 a, u64 b, u64 q) { u64 s = a + b; return s >= q ? s - q : s; }
__device__ __forceinline__ u64 sub_mod(u64 a, u64 b, u64 q) { return a >= b ? a - b : a + q - b; }

// (hi:lo) mod q for a value below 2^112; mu = floor(2^112 / q).
// qhat = floor((x >> 48) mu / 2^64) is in (x/q - 2, x/q], so one conditional subtraction finishes.
__device__ __forceinline__ u64 barrett112(u64 hi, u64 lo, u64 q, u64 mu) {
    u64 xh = (hi << 16) | (lo >> 48);
    u64 qhat = __umul64hi(xh, mu);
    u64 r = lo - qhat * q;
    return r >= q ? r - q : r;
}
__device__ __forceinline__ u64 mul_mod(u64 a, u64 b, u64 q, u64 mu) {
    return barrett112(__umul64hi(a, b), a * b, q, mu);
}
// 128-bit lazy accumulator: acc += a * b
__device__ __forceinline__ void mac128(u64 &hi, u64 &lo, u64 a, u64 b) {
    u64 pl = a * b, ph = __umul64hi(a, b);
    lo += pl;
    hi += ph + (lo < pl);
}
// Representative of the centred lift of y (mod src) taken modulo dst, for primes of equal bit length:
// y <= (src-1)/2 stays, else y - src + dst (positive because dst > src/2).
__device__ __forceinline__ u64 centred_to(u64 y, u64 src, u64 dst) {
    return y > (src >> 1) ? y + dst - src : y;
}

// ---------------------------------------------------------------------------
// Double-precision modular arithmetic for 50-bit primes (FP64 pipe).  Values are
// signed integers held in doubles, exact while below 2^53 in magnitude.
//   mulmod_d: y * w - k q with k = round(y * (w/q)); exact; |result| <= (1/2 + |y| 2^-53) q
//             (COARSE: k rounded to even, valid for |y w / q| < 2^52, |result| <= (1 + ..) q).
// ---------------------------------------------------------------------------
constexpr double MAGIC0 = 6755399441055744.0;    // 1.5 * 2^52: rounds |v| < 2^51 to the nearest integer
constexpr double MAGIC1 = 13510798882111488.0;   // 1.5 * 2^53: rounds |v| < 2^52 to the nearest even integer
constexpr double TWO52 = 4503599627370496.0;

template <int COARSE>
__device__ __forceinline__ double mulmod_d(double y, double2 w, double q) {
    const double p = __dmul_rn(y, w.x);
    const double e = __fma_rn(y, w.x, -p);
    const double M = COARSE ? MAGIC1 : MAGIC0;
    const double k = __dsub_rn(__fma_rn(y, w.y, M), M);
    return __dadd_rn(__fma_rn(-k, q, p), e);
}
// The same with the quotient estimated from the rounded product, k = round(p * (1/q)): p and 1/q are each within 2^-53
// relative, so the estimate is as close as with a precomputed w * (1/q), and no per-twiddle multiply is needed.
template <int COARSE>
__device__ __forceinline__ double mulmod_pq(double y, double w, double q, double qinv) {
    const double p = __dmul_rn(y, w);
    const double e = __fma_rn(y, w, -p);
    const double M = COARSE ? MAGIC1 : MAGIC0;
    const double k = __dsub_rn(__fma_rn(p, qinv, M), M);
    return __dadd_rn(__fma_rn(-k, q, p), e);
}
// x * y - k q for two variable residues 0 <= x, y < q (as doubles): exact, |result| <= 0.75 q
__device__ __forceinline__ double mulmod_dd(double x, double y, double q, double qinv) {
    const double p = __dmul_rn(x, y);
    const double e = __fma_rn(x, y, -p);
    const double k = __dsub_rn(__fma_rn(p, qinv, MAGIC0), MAGIC0);
    return __dadd_rn(__fma_rn(-k, q, p), e);
}
__device__ __forceinline__ double reduce_d(double v, double q, double qinv) {   // to |v| <= q/2
    const double k = __dsub_rn(__fma_rn(v, qinv, MAGIC0), MAGIC0);
    return __fma_rn(-k, q, v);
}
__device__ __forceinline__ double u64_to_d(u64 x) { return __dsub_rn(__longlong_as_double((long long)(x | 0x4330000000000000ull)), TWO52); }
__device__ __forceinline__ u64 d_to_u64(double v) { return (u64)__double_as_longlong(__dadd_rn(v, TWO52)) & 0x000FFFFFFFFFFFFFull; }
__device__ __forceinline__ u64 canonical_d(double v, double q) { return d_to_u64(v < 0.0 ? __dadd_rn(v, q) : v); }

__device__ __forceinline__ uint32_t bitrev_n(uint32_t x, uint32_t bits) { return __brev(x) >> (32 - bits); }
// index p' with stored[p] of sigma_g(a) = stored[p'] of a (evaluation domain, bit-reversed); g = 1: identity
__device__ __forceinline__ uint32_t galois_src(uint32_t p, u64 g, uint32_t log_n, uint32_t N) {
    if (g == 1) return p;
    const u64 e = (g * (2ull * bitrev_n(p, log_n) + 1)) & (2ull * N - 1);
    return bitrev_n((uint32_t)((e - 1) >> 1), log_n);
}

// Kernel launches issued by this library since it was loaded (all contexts, all streams).
extern unsigned long long g_kernel_launches;
inline void count_launches(unsigned n = 1) { g_kernel_launches += n; }

// ---------------------------------------------------------------------------
// Internal launchers (each validates nothing; the C ABI layer does).
// ---------------------------------------------------------------------------
// Optional epilogue of the forward transform (N = 2^16 path): instead of storing NTT(conv) the last pass finishes the
// ModDown: out[b][comp][i][p] (+)= (u[b][comp][i][p] - NTT(conv)[p]) P^-1 + sigma_g(add_comp)[b][i][p], for a buffer of
// limbs laid out [b][comp][level]; `out` in the plain layout (out_stride words per b) or tiled (tl.R != 0).
// mode 2: the transform's own result is stored, but into a tiled buffer: limb y = b * level + i becomes row
// tl.row0 + b * tl.row_stride, limb i.
// Up to KS_MULTI key switches that share one set of extended digits but differ in key, Galois element and output
// buffer (hoisted rotations): batch entry b uses evk[b], galois[b], out[b].
constexpr uint32_t KS_MULTI = 16;
struct KsMulti {
    const u64 *evk[KS_MULTI];
    u64 galois[KS_MULTI];
    u64 *out[KS_MULTI];
    // group > 0 (N = 2^16 only): `group` ciphertexts with their own digits take every one of the keys; batch entry
    // b = r * group + m is key r applied to member m's digits, added to member m's addend, and written to the tiled
    // row  row0 + r * rot_rows + m * row_stride + component  (out[] is not used)
    uint32_t group, rot_rows;
};

struct NttEpilogue {
    int mode;      // 1 = ModDown tail, 2 = tiled store
    const u64 *u, *add0, *add1;
    u64 *out;
    size_t add_stride, out_stride;
    u64 galois;
    uint32_t level, nt;
    int accumulate;
    TiledOut tl;
    int multi;             // mode 1: batch entry b adds through mgalois[b] and writes to mout[b]
    u64 mgalois[KS_MULTI];
    u64 *mout[KS_MULTI];
    uint32_t group, rot_rows;   // KsMulti's grouped form
};
// coef_src (forward, N = 2^16 path only): the first pass reads signed 64-bit coefficients [batch][N] (batch = limb
// index / map.period) and reduces them modulo the limb's prime on the fly instead of reading `base`.
// inv_src (inverse, N = 2^16 path only): the first pass reads its limbs from another buffer whose periods start
// inv_src_pitch limbs apart, so the transform runs out of place and the input stays intact.
// inv_scale (inverse, N = 2^16 path only): pairs [map.period][2] that replace {N^-1, last twiddle N^-1} for limb x of every
// period (device pointer), so that the output is scaled by a per-limb constant.
void launch_ntt(const ckks_ctx *c, u64 *base, uint32_t nlimbs_total, const LimbMap &map, bool inverse, cudaStream_t s,
                const NttEpilogue *ep = nullptr, const long long *coef_src = nullptr, const u64 *inv_src = nullptr,
                uint32_t inv_src_pitch = 0, const double2 *inv_scale = nullptr);

void launch_mul_plain_acc(const ckks_ctx *c, const u64 *const *cts, u64 *const *accs, uint32_t ncts, const u64 *pt,
                          uint32_t level, bool init, cudaStream_t s);
void launch_add(const ckks_ctx *c, const u64 *a, const u64 *b, u64 *out, uint32_t ncomp, uint32_t level, cudaStream_t s);
void launch_automorphism(const ckks_ctx *c, const u64 *in, u64 *out, uint32_t nlimbs, u64 galois, cudaStream_t s);
void launch_tensor(const ckks_ctx *c, const u64 *a, const u64 *b, u64 *e01, u64 *e2, uint32_t level, cudaStream_t s);
// slot values 1.0 on the slots x with lo <= x / B < hi and t0 <= x % Ti < t1, else 0.0 (n doubles on the device)
void launch_slot_mask(const ckks_ctx *c, double *out, uint32_t B, uint32_t lo, uint32_t hi, uint32_t Ti, uint32_t t0, uint32_t t1, cudaStream_t s);
// out = in * v or in + v (component 0 only) for the constant polynomial v
void launch_const(const ckks_ctx *c, const u64 *in, long long v, bool mul, u64 *out, uint32_t ncomp, uint32_t level, cudaStream_t s);
// e01, e2 = sum_i tensor(a_i, b_i) (host arrays of n device pointers, [2][level][N] each)
constexpr uint32_t TS_MAX = 16;
struct TensorSumArgs { const u64 *a[TS_MAX]; const u64 *b[TS_MAX]; };
void launch_tensor_sum(const ckks_ctx *c, const u64 *const *a, const u64 *const *b, uint32_t n, u64 *e01, u64 *e2, uint32_t level,
                       cudaStream_t s);

// Key switch pieces.  Sizes in limbs: d [level], ext [beta][level+K], u [2][level+K], conv [2][level].
struct KsWorkspace { u64 *dcoef, *ext, *u, *conv; };
size_t ks_workspace_limbs(const ckks_ctx *c, uint32_t level);
KsWorkspace ks_carve(const ckks_ctx *c, uint32_t level, void *ws, uint32_t nb = 1);
// nb key switches side by side (batch entry b reads d + b * d_stride words, d_stride a multiple of N):
// d (evaluation domain, [level][N]) -> ext (evaluation domain, all digits).  A rotation applies its sigma_g to the
// extended digits when the inner product reads them (ext_galois below): the centred conversion commutes with the
// permutation and the sign flips of sigma_g, so this equals extending sigma_g(d), and d is never copied.
void ks_modup(const ckks_ctx *c, const u64 *d, uint32_t level, const KsWorkspace &w, cudaStream_t s, uint32_t nb = 1, size_t d_stride = 0);
// inner product with evk (digits read through sigma_{ext_galois}; 1 = identity), ModDown, and the final
// combination out_c (+)= sigma_{add_galois}(add_c) + k_c.  add0/add1 may be null.
void ks_inner_moddown(const ckks_ctx *c, const u64 *evk, uint32_t level, u64 ext_galois, const KsWorkspace &w,
                      const u64 *add0, const u64 *add1, u64 add_galois, u64 *out, cudaStream_t s, uint32_t nb = 1,
                      size_t add_stride = 0, size_t out_stride = 0, bool accumulate = false, TiledOut tiled = TiledOut(),
                      const KsMulti *multi = nullptr);
// The two halves of ks_inner_moddown.  ks_inner leaves u = <digits, evk> in the extended basis (w.u, nb entries); with
// acc_u it adds to what w.u holds, so that a sum of key-switched terms can share one ks_moddown.
void ks_inner(const ckks_ctx *c, const u64 *evk, uint32_t level, u64 ext_galois, const KsWorkspace &w, cudaStream_t s, uint32_t nb = 1,
              bool acc_u = false, const KsMulti *multi = nullptr);
void ks_moddown(const ckks_ctx *c, uint32_t level, const KsWorkspace &w, const u64 *add0, const u64 *add1, u64 add_galois, u64 *out,
                cudaStream_t s, uint32_t nb = 1, size_t add_stride = 0, size_t out_stride = 0, bool accumulate = false,
                TiledOut tiled = TiledOut(), const KsMulti *multi = nullptr);
// A sum of up to IP_TERMS key-switched terms in one pass over the extended basis:
//   u[b] (+)= sum_t ( <ext[t][b] read through sigma_{g_t}, evk_t>  +  P sigma_{g_t}(c0_t[b]) on component 0's q-limbs )
// ext holds term t's digits of batch entry b at ext + t * term_stride + b * beta * (level + K) * N words; c0[t]
// (may be null) points at term t's first-component limbs, entries c0_stride words apart.  Adding P c0 before the
// ModDown equals adding c0 after it, exactly.
constexpr uint32_t IP_TERMS = 4;
struct IpTerms {
    const u64 *evk[IP_TERMS];
    u64 galois[IP_TERMS];
    const u64 *c0[IP_TERMS];
};
void ks_inner_terms(const ckks_ctx *c, uint32_t level, const KsWorkspace &w, size_t term_stride, const IpTerms &terms, uint32_t nterm,
                    size_t c0_stride, cudaStream_t s, uint32_t nb, bool acc_u);
// The basis conversions on the tensor cores (N = 2^16 layout rules: any N that is a multiple of 1024).  Return false if
// the context has no byte matrices (more than 8 sources) and nothing was launched.
bool launch_modup_mma(const ckks_ctx *c, const u64 *dcoef, const u64 *deval, size_t deval_stride, u64 *ext, uint32_t level, uint32_t nb,
                      cudaStream_t s);
bool launch_moddown_conv_mma(const ckks_ctx *c, const u64 *u, u64 *conv, uint32_t level, uint32_t nb, cudaStream_t s);
// rows of [level][N] words, src_stride words apart, into rows row0, row0 + row_step, .. of a tiled buffer with R rows
void launch_to_tiled(const ckks_ctx *c, const u64 *src, size_t src_stride, uint32_t nrows, u64 *dst, uint32_t R, uint32_t row0,
                     uint32_t row_step, uint32_t level, cudaStream_t s);

// Tensor-core multiply-accumulate of a giant-step group (mac_mma.cu)
bool mac_mma_supported(const ckks_ctx *c, uint32_t J);
// baby, pts: tiled buffers with 2 * S * J rows ((shard * J + j) * 2 + component) and G * J rows (g * J + j)
// the baby buffer may hold Jx >= J rows per shard and component, of which rows j0 .. j0 + J - 1 are used (Jx = 0: J);
// accumulate: add to acc instead of overwriting it
bool launch_mac_mma(const ckks_ctx *c, const u64 *baby, const u64 *pts, u64 *acc, uint32_t J, uint32_t S, uint32_t G, uint32_t level,
                    cudaStream_t s, uint32_t Jx = 0, uint32_t j0 = 0, bool accumulate = false);

// the same contraction on the integer pipe, any J (mac_tile.cu): baby rows (s J + j) 2 + c, pts rows g J + j, both tiled
void launch_mac_tile(const ckks_ctx *c, const u64 *baby, const u64 *pts, u64 *acc, uint32_t J, uint32_t S, uint32_t G, uint32_t level,
                     cudaStream_t s);

// register-resident forward butterflies (measurement aid, ntt.cu); sink: device scratch of SMs * 4 * 256 words
uint64_t launch_butterfly_probe(const ckks_ctx *c, uint32_t iters, u64 *sink, cudaStream_t s);

// the same on tcgen05 / TMEM (mac_umma.cu); J <= 64
bool mac_umma_supported(const ckks_ctx *c, uint32_t J);
bool launch_mac_umma(const ckks_ctx *c, const u64 *baby, const u64 *pts, u64 *acc, uint32_t J, uint32_t S, uint32_t G, uint32_t level,
                     cudaStream_t s, uint32_t Jx = 0, uint32_t j0 = 0, bool accumulate = false);

void launch_rescale(const ckks_ctx *c, const u64 *in, u64 *out, uint32_t ncomp, uint32_t level, u64 *ws, cudaStream_t s);

size_t encode_workspace_bytes(const ckks_ctx *c, uint32_t batch);
// tiled.R != 0 (N = 2^16 only): plaintext b is written as row tiled.row0 + b * tiled.row_stride of the tiled buffer
// `tiled_out`; `out` is then only the scratch between the two NTT passes.
void launch_encode(const ckks_ctx *c, const double *re, const double *im, uint32_t batch, double scale, uint32_t level,
                   u64 *out, void *ws, cudaStream_t s, TiledOut tiled = TiledOut(), u64 *tiled_out = nullptr);
// Slot vectors of pre-rotated generalised diagonals, [count][n] fp64, for k = k0 .. k0+count-1 of one block pair.
void launch_extract_diagonals(const ckks_ctx *c, const double *W, uint32_t d_out_total, uint32_t in0, uint32_t m_in,
                              uint32_t out0, uint32_t m_out, uint32_t F, uint32_t T, uint32_t k0, uint32_t count,
                              uint32_t pre_rot, double *slots, cudaStream_t s);

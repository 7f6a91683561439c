// Batched negacyclic NTT / inverse NTT.
//
// Forward: merged Cooley-Tukey, natural-order input, bit-reversed output, stages
// m = 1, 2, .., N/2 with butterfly distance t = N/(2m) and twiddle psi^bitrev(m+i)
// for block i.  Inverse: Gentleman-Sande, the same stages backwards, then N^-1.
//
// Generic path (N < 2^16).  A limb is viewed as R rows of 256 coefficients (R = N/256).  The stages with
// distance >= 256 couple rows only ("column pass": a CTA owns all R rows of a
// 16-column strip in shared memory); the stages with distance < 256 stay inside
// a row ("row pass": a CTA owns 8 rows).  Each limb therefore makes two trips
// through HBM per transform.
#include "common.cuh"

namespace {

constexpr uint32_t ROW = 256;       // coefficients per row
constexpr uint32_t COLS = 16;       // columns per CTA in the column pass
constexpr uint32_t ROWS_PER_CTA = 8;
constexpr uint32_t THREADS = 256;

// ---- column pass: stages m = 1 .. R/2 (forward) / R/2 .. 1 (inverse) ------
template <bool INV>
__global__ void __launch_bounds__(THREADS) ntt_cols(DevTables c, u64 *base, LimbMap map) {
    extern __shared__ u64 sm[];
    const int prime = limb_prime(map, blockIdx.y);
    if (prime < 0) return;
    const uint32_t N = c.N, R = N / ROW;
    const u64 q = c.mod[prime];
    const ulonglong2 *tw = (INV ? c.tw_inv : c.tw_fwd) + (size_t)prime * N;
    u64 *g = base + limb_index(map, blockIdx.y) * N + blockIdx.x * COLS;
    for (uint32_t x = threadIdx.x; x < R * COLS; x += THREADS) sm[x] = g[(size_t)(x / COLS) * ROW + x % COLS];
    __syncthreads();
    if (!INV) {
        for (uint32_t m = 1, tr = R / 2; m < R; m <<= 1, tr >>= 1) {
            for (uint32_t x = threadIdx.x; x < (R / 2) * COLS; x += THREADS) {
                uint32_t cc = x % COLS, b = x / COLS, i = b / tr, r1 = 2 * i * tr + b % tr;
                ulonglong2 w = tw[m + i];
                u64 U = sm[r1 * COLS + cc], V = mul_shoup(sm[(r1 + tr) * COLS + cc], w.x, w.y, q);
                sm[r1 * COLS + cc] = add_mod(U, V, q);
                sm[(r1 + tr) * COLS + cc] = sub_mod(U, V, q);
            }
            __syncthreads();
        }
    } else {
        for (uint32_t m = R / 2, tr = 1; m >= 1; m >>= 1, tr <<= 1) {
            for (uint32_t x = threadIdx.x; x < (R / 2) * COLS; x += THREADS) {
                uint32_t cc = x % COLS, b = x / COLS, i = b / tr, r1 = 2 * i * tr + b % tr;
                ulonglong2 w = tw[m + i];
                u64 U = sm[r1 * COLS + cc], V = sm[(r1 + tr) * COLS + cc];
                sm[r1 * COLS + cc] = add_mod(U, V, q);
                sm[(r1 + tr) * COLS + cc] = mul_shoup(sub_mod(U, V, q), w.x, w.y, q);
            }
            __syncthreads();
        }
        ulonglong2 ni = c.n_inv[prime];
        for (uint32_t x = threadIdx.x; x < R * COLS; x += THREADS) sm[x] = mul_shoup(sm[x], ni.x, ni.y, q);
        __syncthreads();
    }
    for (uint32_t x = threadIdx.x; x < R * COLS; x += THREADS) g[(size_t)(x / COLS) * ROW + x % COLS] = sm[x];
}

// ---- row pass: stages m = R .. N/2 (forward) / N/2 .. R (inverse) ---------
template <bool INV>
__global__ void __launch_bounds__(THREADS) ntt_rows(DevTables c, u64 *base, LimbMap map, uint32_t rows) {
    __shared__ u64 sm[ROWS_PER_CTA * ROW];
    const int prime = limb_prime(map, blockIdx.y);
    if (prime < 0) return;
    const uint32_t N = c.N, R = N / ROW;
    const u64 q = c.mod[prime];
    const ulonglong2 *tw = (INV ? c.tw_inv : c.tw_fwd) + (size_t)prime * N;
    const uint32_t row0 = blockIdx.x * rows;
    u64 *g = base + limb_index(map, blockIdx.y) * N + (size_t)row0 * ROW;
    for (uint32_t x = threadIdx.x; x < rows * ROW; x += THREADS) sm[x] = g[x];
    __syncthreads();
    // local stage mp = 1 .. 128: global stage m = R*mp, distance t = 128/mp, twiddle index mp*(R + row) + i_local
    if (!INV) {
        for (uint32_t mp = 1, t = ROW / 2; mp < ROW; mp <<= 1, t >>= 1) {
            for (uint32_t x = threadIdx.x; x < rows * ROW / 2; x += THREADS) {
                uint32_t rl = x / (ROW / 2), b = x % (ROW / 2), i = b / t, c1 = rl * ROW + 2 * i * t + b % t;
                ulonglong2 w = tw[mp * (R + row0 + rl) + i];
                u64 U = sm[c1], V = mul_shoup(sm[c1 + t], w.x, w.y, q);
                sm[c1] = add_mod(U, V, q);
                sm[c1 + t] = sub_mod(U, V, q);
            }
            __syncthreads();
        }
    } else {
        for (uint32_t mp = ROW / 2, t = 1; mp >= 1; mp >>= 1, t <<= 1) {
            for (uint32_t x = threadIdx.x; x < rows * ROW / 2; x += THREADS) {
                uint32_t rl = x / (ROW / 2), b = x % (ROW / 2), i = b / t, c1 = rl * ROW + 2 * i * t + b % t;
                ulonglong2 w = tw[mp * (R + row0 + rl) + i];
                u64 U = sm[c1], V = sm[c1 + t];
                sm[c1] = add_mod(U, V, q);
                sm[c1 + t] = mul_shoup(sub_mod(U, V, q), w.x, w.y, q);
            }
            __syncthreads();
        }
    }
    for (uint32_t x = threadIdx.x; x < rows * ROW; x += THREADS) g[x] = sm[x];
}


// ===========================================================================
// Fast path for N = 2^16 (256 x 256): every pass is two radix-16 steps held in
// registers (4 butterfly stages each, 16 coefficients per thread) with a single
// shared-memory exchange in between, so a limb crosses shared memory once per
// pass instead of once per stage.
//
// Lazy arithmetic.  Residues travel as 64-bit words that are only congruent to
// the value: with 50-bit primes there are 14 spare bits.  The twiddle product
// uses an under-estimate of floor(x w'/2^64) built from three 32x32 products
// (the low x low product is dropped, the cross products keep their high halves),
// at most 3 below the exact quotient, so the product lands in [0, 5q) for ANY
// 64-bit x.  Forward (Cooley-Tukey): X' = X + T, Y' = X - T + 5q; magnitudes grow
// by at most 5q per stage, 81q < 2^57 after 16 stages, one exact reduction at the
// end.  Inverse (Gentleman-Sande): X' = U + V doubles the bound per stage,
// Y' = (U - V + bound q) w' is back in [0, 5q); 8 stages keep everything below
// 1280 q < 2^61, so one lazy reduction between the passes suffices.
// ===========================================================================

constexpr uint32_t F_THREADS = 256;
// CTAs per SM the compiler is asked to fit.  The forward kernels take their quotients from the rounded products (no
// {w, w/q} pairs in registers) and run four CTAs of 64 registers per SM: 0.422 us per limb against 0.440 with pairs at three
// CTAs.  The row pass with the ModDown tail would spill at 64 registers and the inverse kernels lose at four CTAs
// (0.447 against 0.440 us per limb), so those stay at three.
constexpr uint32_t FWD_CTAS = 4, INV_CTAS = 3;

__device__ __forceinline__ u64 mulhi_under(u64 x, u64 a) {
    const uint32_t x0 = (uint32_t)x, x1 = (uint32_t)(x >> 32), a0 = (uint32_t)a, a1 = (uint32_t)(a >> 32);
    return (u64)x1 * a1 + __umulhi(x1, a0) + __umulhi(x0, a1);
}
// x * w mod q up to a multiple of q, in [0, 5q), for any 64-bit x
__device__ __forceinline__ u64 mul_tw(u64 x, ulonglong2 w, u64 q) { return x * w.x - mulhi_under(x, w.y) * q; }

// 4 Cooley-Tukey stages on 16 registers; stage twiddles tw[ml*base + i], ml = 1,2,4,8
__device__ __forceinline__ void fwd16(u64 (&x)[16], const ulonglong2 *__restrict__ tw, uint32_t base, u64 q, u64 q5) {
#pragma unroll
    for (uint32_t ml = 1; ml < 16; ml <<= 1) {
        const uint32_t tl = 8 / ml;
#pragma unroll
        for (uint32_t i = 0; i < ml; i++) {
            const ulonglong2 w = __ldg(&tw[ml * base + i]);
#pragma unroll
            for (uint32_t j = 0; j < tl; j++) {
                const uint32_t k1 = 2 * i * tl + j, k2 = k1 + tl;
                const u64 t = mul_tw(x[k2], w, q);
                x[k2] = x[k1] + q5 - t;
                x[k1] = x[k1] + t;
            }
        }
    }
}

// 4 Gentleman-Sande stages (ml = 8,4,2,1); `bound` = multiple of q bounding the inputs on entry
template <uint32_t BOUND>
__device__ __forceinline__ void inv16(u64 (&x)[16], const ulonglong2 *__restrict__ tw, uint32_t base, u64 q) {
    uint32_t b = BOUND;
#pragma unroll
    for (uint32_t ml = 8; ml >= 1; ml >>= 1) {
        const uint32_t tl = 8 / ml;
        const u64 off = (u64)b * q;
#pragma unroll
        for (uint32_t i = 0; i < ml; i++) {
            const ulonglong2 w = __ldg(&tw[ml * base + i]);
#pragma unroll
            for (uint32_t j = 0; j < tl; j++) {
                const uint32_t k1 = 2 * i * tl + j, k2 = k1 + tl;
                const u64 u = x[k1], v = x[k2];
                x[k1] = u + v;
                x[k2] = mul_tw(u + off - v, w, q);
            }
        }
        b = 2 * b > 5 ? 2 * b : 5;
    }
}
// bound after the 4 stages of inv16<b>: b -> max(2b, 5) four times, i.e. 1 -> 40, 5 -> 80, 40 -> 640, 80 -> 1280

// exact reduction of a lazy word (< 2^64) to [0, q): qinv64 = floor(2^64 / q)
__device__ __forceinline__ u64 reduce_exact(u64 x, u64 q, u64 qinv64) {
    u64 r = x - __umul64hi(x, qinv64) * q;     // in [0, 2q)
    return r >= q ? r - q : r;
}

// ---------------------------------------------------------------------------
// Double-precision variant of the same butterflies.  The FP64 pipe multiplies
// 53-bit operands in one instruction where the integer pipe needs several
// 32x32 products, so for 50-bit primes a twiddle product is cheaper there:
//   p = y w (rounded), e = fma(y, w, -p) (exact low part),
//   k = round(p * (1/q))  by adding and subtracting 1.5 * 2^52 (or 1.5 * 2^53),
//   r = fma(-k, q, p) + e  =  y w - k q   exactly, |r| <= (1/2 + eps) q  (or (1 + eps) q).
// Values are signed integers held in doubles; everything is exact while they stay
// below 2^53 in magnitude, so each group of four stages starts by reducing its 16
// values to |v| <= q/2 (forward), and the inverse reduces again after two stages.
// A limb is handled by the integer or by the double path in BOTH passes (the
// intermediate written between the passes is a lazy word in one case and a double
// in the other); the result is the same canonical residue either way.
// ---------------------------------------------------------------------------
// ML consecutive twiddles w (ML = 1, 2, 4, 8; the index is a multiple of ML) with the widest loads that fit.  The quotient
// of a twiddle product is estimated from the rounded product and fl(1/q) (mulmod_pq): within 2^-52 relative of y w / q,
// which the stage bounds allow for, and one multiply per twiddle and half the twiddle registers less than with {w, w/q}.
template <uint32_t ML>
__device__ __forceinline__ void load_tw(const double *p, double (&v)[ML]) {
    if (ML == 1) v[0] = __ldg(p);
    if (ML == 2) asm volatile("ld.global.nc.v2.f64 {%0,%1}, [%2];" : "=d"(v[0]), "=d"(v[1]) : "l"(p));
    if (ML >= 4) {
#pragma unroll
        for (uint32_t i = 0; i < ML; i += 4)
            asm volatile("ld.global.nc.v4.f64 {%0,%1,%2,%3}, [%4];" : "=d"(v[i]), "=d"(v[(i + 1) % ML]), "=d"(v[(i + 2) % ML]), "=d"(v[(i + 3) % ML]) : "l"(p + i));
    }
}
__device__ __forceinline__ void stg_4(u64 *p, u64 a, u64 b, u64 c, u64 d) {
    asm volatile("st.global.v4.b64 [%0], {%1,%2,%3,%4};" ::"l"(p), "l"(a), "l"(b), "l"(c), "l"(d) : "memory");
}
__device__ __forceinline__ void ldg_4(const u64 *p, u64 &a, u64 &b, u64 &c, u64 &d) {
    asm volatile("ld.global.v4.b64 {%0,%1,%2,%3}, [%4];" : "=l"(a), "=l"(b), "=l"(c), "=l"(d) : "l"(p) : "memory");
}

// Range bookkeeping of the double-precision path (B = bound in units of q).  The twiddle tables hold centred
// representatives, |w| <= q/2, and the quotient estimate is within 2^-52 relative, so for |y| <= B q the product y w - k q comes out below
//   T(B) = (1/2 + B/8) q   when k is rounded to the nearest integer (needs B <= 4:  |y w/q| < 2^51), and below
//   Tc(B) = (1 + B/8) q    when k is rounded to the nearest even integer (needs |y w/q| < 2^52, sums below 2^53 ~ 8 q).
// A Cooley-Tukey stage takes B to B + T(B): from a canonical input (B = 1) four stages reach 1.63, 2.33, 3.12, 4.01;
// from a reduced one (B = 1/2) 1.06, 1.70, 2.41, 3.21.  The sixteen stages of a transform therefore need the
// three-instruction reduction only twice on the way (after stage 6 and before stage 13) and once at the end:
//   column pass  canonical 1 | 1.63 2.33 3.12 4.01 | exchange | 5.51c 7.20c | reduce | 1.06 1.70 | stored as doubles
//   row pass     1.70 | 2.41 3.21 4.11 5.63c | exchange | reduce | 1.06 1.70 2.41 3.21 | exact reduction, canonical word
// (c = even rounding).  A Gentleman-Sande stage doubles the bound (x1 = u + v) and multiplies u - v, |u - v| <= 2 B:
// from a reduced input four stages reach 1, 2, 4, 8 (the last product with even rounding, 8 q < 2^53), so the inverse
// reduces once per group of four stages.
template <uint32_t ML, int COARSE>
__device__ __forceinline__ void fwd_stage_d(double (&x)[16], const double *__restrict__ tw, uint32_t base, double q, double qinv) {
    constexpr uint32_t tl = 8 / ML;
    double w[ML];
    load_tw<ML>(tw + ML * base, w);
#pragma unroll
    for (uint32_t i = 0; i < ML; i++)
#pragma unroll
        for (uint32_t j = 0; j < tl; j++) {
            const uint32_t k1 = 2 * i * tl + j, k2 = k1 + tl;
                        const double t = mulmod_pq<COARSE>(x[k2], w[i], q, qinv);
            x[k2] = __dsub_rn(x[k1], t);
            x[k1] = __dadd_rn(x[k1], t);
        }
}
__device__ __forceinline__ void reduce16(double (&x)[16], double q, double qinv) {
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) x[k] = reduce_d(x[k], q, qinv);
}
// stages 1-4 (canonical or reduced input, bound 4.01 q out) and 9-12 (1.70 q in, 5.63 q out): no reduction
template <int LAST_COARSE>
__device__ __forceinline__ void fwd16_open(double (&x)[16], const double *__restrict__ tw, uint32_t base, double q, double qinv) {
    fwd_stage_d<1, 0>(x, tw, base, q, qinv);
    fwd_stage_d<2, 0>(x, tw, base, q, qinv);
    fwd_stage_d<4, 0>(x, tw, base, q, qinv);
    fwd_stage_d<8, LAST_COARSE>(x, tw, base, q, qinv);
}
// stages 5-8: two stages with even rounding (4.01 q in, 7.20 q), the reduction, two more (1.70 q out)
__device__ __forceinline__ void fwd16_mid(double (&x)[16], const double *__restrict__ tw, uint32_t base, double q, double qinv) {
    fwd_stage_d<1, 1>(x, tw, base, q, qinv);
    fwd_stage_d<2, 1>(x, tw, base, q, qinv);
    reduce16(x, q, qinv);
    fwd_stage_d<4, 0>(x, tw, base, q, qinv);
    fwd_stage_d<8, 0>(x, tw, base, q, qinv);
}
// stages 13-16, and the groups of the register-resident probe: reduction first, outputs below 3.21 q
__device__ __forceinline__ void fwd16_d(double (&x)[16], const double *__restrict__ tw, uint32_t base, double q, double qinv) {
    reduce16(x, q, qinv);
    fwd_stage_d<1, 0>(x, tw, base, q, qinv);
    fwd_stage_d<2, 0>(x, tw, base, q, qinv);
    fwd_stage_d<4, 0>(x, tw, base, q, qinv);
    fwd_stage_d<8, 0>(x, tw, base, q, qinv);
}

// 4 Gentleman-Sande stages after one reduction; outputs below 8 q (the last stage's products with even rounding).
template <uint32_t ML, int COARSE>
__device__ __forceinline__ void inv_stage_d(double (&x)[16], const double *__restrict__ tw, uint32_t base, double q, double qinv) {
    constexpr uint32_t tl = 8 / ML;
    double w[ML];
    load_tw<ML>(tw + ML * base, w);
#pragma unroll
    for (uint32_t i = 0; i < ML; i++)
#pragma unroll
        for (uint32_t j = 0; j < tl; j++) {
            const uint32_t k1 = 2 * i * tl + j, k2 = k1 + tl;
            const double u = x[k1], v = x[k2];
            x[k1] = __dadd_rn(u, v);
            x[k2] = mulmod_pq<COARSE>(__dsub_rn(u, v), w[i], q, qinv);
        }
}
__device__ __forceinline__ void inv16_d(double (&x)[16], const double *__restrict__ tw, uint32_t base, double q, double qinv) {
    reduce16(x, q, qinv);
    inv_stage_d<8, 0>(x, tw, base, q, qinv);     // |u - v| <= 1 q
    inv_stage_d<4, 0>(x, tw, base, q, qinv);     // 2 q
    inv_stage_d<2, 0>(x, tw, base, q, qinv);     // 4 q
    inv_stage_d<1, 1>(x, tw, base, q, qinv);     // 8 q: even rounding; sums reach 8 q < 2^53
}
// The last group of the inverse transform (stages m = 8, 4, 2, 1 of the column pass, twiddle base 1): three stages, a
// second reduction, and the last stage with N^-1 folded in: x1 = (u + v) N^-1, x2 = (u - v) (w N^-1), both products of
// values below 1 q, so the results are within 0.63 q and one conditional addition makes them canonical.
// nw = {N^-1, N^-1/q}, wn = {w_1 N^-1, that / q}, centred.
__device__ __forceinline__ void inv16_last(double (&x)[16], const double *__restrict__ tw, double q, double qinv, double2 nw, double2 wn) {
    reduce16(x, q, qinv);
    inv_stage_d<8, 0>(x, tw, 1, q, qinv);
    inv_stage_d<4, 0>(x, tw, 1, q, qinv);
    inv_stage_d<2, 0>(x, tw, 1, q, qinv);
    reduce16(x, q, qinv);
#pragma unroll
    for (uint32_t j = 0; j < 8; j++) {
        const double u = x[j], v = x[j + 8];
        x[j] = mulmod_d<0>(__dadd_rn(u, v), nw, q);
        x[j + 8] = mulmod_d<0>(__dsub_rn(u, v), wn, q);
    }
}

// ---- measurement aid: the forward butterflies of the N = 2^16 kernels on registers only ------------------
// Every thread runs `iters` radix-16 groups (4 stages, 32 butterflies, with the same range reductions and twiddle
// fetches, the latter from a 64 KiB window that stays in L1/L2) on 16 registers; nothing else touches memory.
__global__ void __launch_bounds__(F_THREADS, 3) butterfly_probe_kernel(DevTables c, uint32_t iters, u64 *sink) {
    const double q = c.modd[0].x, qinv = c.modd[0].y;
    const double *tw = c.twd_fwd;
    double x[16];
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) x[k] = (double)(threadIdx.x * 16 + k + 1);
    uint32_t base = 16 + (threadIdx.x & 255);
    for (uint32_t it = 0; it < iters; it++) {
        fwd16_d(x, tw, base, q, qinv);
        base = 16 + ((base * 5 + 1) & 255);
    }
    double acc = 0.0;
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) acc = __dadd_rn(acc, x[k]);
    if (acc == 0.5) sink[blockIdx.x * F_THREADS + threadIdx.x] = 1;      // never true for integer-valued sums
}

// ---- forward, column pass (stages m = 1..128): CTA = strip of 16 columns -----------------
template <bool ALLFP>
__global__ void __launch_bounds__(F_THREADS, FWD_CTAS) ntt16_fwd_cols(DevTables c, u64 *base, LimbMap map, uint32_t fp_share, const long long *coef_src) {
    __shared__ u64 sm[256 * 16];
    const int prime = limb_prime(map, blockIdx.y);
    if (prime < 0) return;
    if (ALLFP || (blockIdx.y & 7) < fp_share) {
        const double q = c.modd[prime].x, qinv = c.modd[prime].y;
        const double *tw = c.twd_fwd + ((size_t)prime << 16);
        const uint32_t cc = threadIdx.x & 15, r = threadIdx.x >> 4;
        u64 *g = base + (limb_index(map, blockIdx.y) << 16) + blockIdx.x * 16 + cc;
        double *smd = reinterpret_cast<double *>(sm);
        double x[16];
        if (coef_src) {     // signed coefficients shared by all limbs of a batch entry, reduced here
            const long long *cs = coef_src + ((size_t)(blockIdx.y / map.period) << 16) + blockIdx.x * 16 + cc;
            const u64 qi = c.mod[prime], mu = c.mu[prime];
#pragma unroll
            for (uint32_t k = 0; k < 16; k++) {
                const long long v = cs[(size_t)(r + 16 * k) * 256];
                const u64 m = barrett112(0, v < 0 ? (u64)(-v) : (u64)v, qi, mu);
                x[k] = u64_to_d((v < 0 && m) ? qi - m : m);
            }
        } else {
#pragma unroll
            for (uint32_t k = 0; k < 16; k++) x[k] = u64_to_d(g[(size_t)(r + 16 * k) * 256]);
        }
        fwd16_open<0>(x, tw, 1, q, qinv);                 // canonical input: no reduction before stage 1
#pragma unroll
        for (uint32_t k = 0; k < 16; k++) smd[(r + 16 * k) * 16 + cc] = x[k];
        __syncthreads();
#pragma unroll
        for (uint32_t k = 0; k < 16; k++) x[k] = smd[(16 * r + k) * 16 + cc];
        fwd16_mid(x, tw, 16 + r, q, qinv);
#pragma unroll
        for (uint32_t k = 0; k < 16; k++) reinterpret_cast<double *>(g)[(size_t)(16 * r + k) * 256] = x[k];
        return;
    }
    if (ALLFP) return;
    const u64 q = c.mod[prime], q5 = 5 * q;
    const ulonglong2 *tw = c.tw_fwd + ((size_t)prime << 16);
    const uint32_t cc = threadIdx.x & 15, r = threadIdx.x >> 4;
    u64 *g = base + (limb_index(map, blockIdx.y) << 16) + blockIdx.x * 16 + cc;
    u64 x[16];
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) x[k] = g[(size_t)(r + 16 * k) * 256];
    fwd16(x, tw, 1, q, q5);
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) sm[(r + 16 * k) * 16 + cc] = x[k];
    __syncthreads();
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) x[k] = sm[(16 * r + k) * 16 + cc];
    fwd16(x, tw, 16 + r, q, q5);
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) g[(size_t)(16 * r + k) * 256] = x[k];
}

// padded index inside a 256-coefficient row: two spare words per 16, so that a thread's 16 consecutive coefficients
// form a 16-byte aligned block of 128 bytes at a pitch of 144 (strided 8-byte accesses by consecutive lanes and
// 16-byte accesses to the own block are both conflict free, and the block can be the source of a bulk copy)
__device__ __forceinline__ uint32_t padded(uint32_t i) { return i + 2 * (i >> 4); }
constexpr uint32_t ROW_PAD = 256 + 32;
// Results leave the row pass as one 128-byte bulk copy per thread (shared -> global, no multicast, this GPU's memory):
// a thread writes its 16 canonical words into its own block of the exchange row with 16-byte stores and hands the
// block to the copy engine, which takes the stores off the load/store pipe (four 32-byte global stores per thread cost
// it one pass per lane and sector: the row pass's busiest unit).
__device__ __forceinline__ void bulk_store_128(u64 *gdst, const void *ssrc) {
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], 128;\n" ::"l"(gdst), "r"((uint32_t)__cvta_generic_to_shared(ssrc)) : "memory");
    asm volatile("cp.async.bulk.commit_group;\n" ::: "memory");
}
__device__ __forceinline__ void bulk_store_wait() { asm volatile("cp.async.bulk.wait_group.read 0;\n" ::: "memory"); }

// The mirror for loads: a warp's 32 threads each fetch their 128-byte block (global -> shared, this GPU's memory, no
// multicast) and wait on the warp's mbarrier for the 4096 bytes.  The wait is bounded by the SM clock.
__device__ __forceinline__ void warp_bulk_load_128(uint32_t bar, void *sdst, const u64 *gsrc, uint32_t lane) {
    if (lane == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(bar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    __syncwarp();
    if (lane == 0) asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], 4096;\n" ::"r"(bar) : "memory");
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], 128, [%2];\n"
                 ::"r"((uint32_t)__cvta_generic_to_shared(sdst)), "l"(gsrc), "r"(bar) : "memory");
}
// true once the warp's copies have landed; the answer is the warp's (one vote)
__device__ __forceinline__ bool warp_bulk_wait(uint32_t bar, long long limit) {
    const long long t0 = clock64();
    uint32_t ok = 0;
    do {
        asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\nselp.u32 %0, 1, 0, p;\n}\n" : "=r"(ok) : "r"(bar) : "memory");
    } while (!ok && clock64() - t0 < limit);
    return __all_sync(0xffffffffu, ok != 0);
}

// ---- forward, row pass (stages m = 256..32768): CTA = 16 rows, 16 threads per row ---------
template <bool ALLFP, int EP, bool BULK = false>
__global__ void __launch_bounds__(F_THREADS, EP == 1 ? 3 : FWD_CTAS) ntt16_fwd_rows(DevTables c, u64 *base, LimbMap map, uint32_t fp_share, NttEpilogue ep) {
    constexpr int has_ep = EP;
    __shared__ __align__(16) u64 sm[16 * ROW_PAD];
    const int prime = limb_prime(map, blockIdx.y);
    if (prime < 0) return;
    if (ALLFP || (blockIdx.y & 7) < fp_share) {
        const double q = c.modd[prime].x, qinv = c.modd[prime].y;
        const double *tw = c.twd_fwd + ((size_t)prime << 16);
        const uint32_t t = threadIdx.x & 15, rl = threadIdx.x >> 4, row = blockIdx.x * 16 + rl;
        u64 *g = base + (limb_index(map, blockIdx.y) << 16) + (size_t)row * 256;
        double *s = reinterpret_cast<double *>(sm) + rl * ROW_PAD;
        double x[16];
#pragma unroll
        for (uint32_t k = 0; k < 16; k++) x[k] = reinterpret_cast<const double *>(g)[t + 16 * k];
        fwd16_open<1>(x, tw, 256 + row, q, qinv);     // 1.70 q in, 5.63 q out
#pragma unroll
        for (uint32_t k = 0; k < 16; k++) s[padded(t + 16 * k)] = x[k];
        __syncwarp();
        double *blk = s + 18 * t;                 // this thread's 16 consecutive coefficients: 16-byte aligned, 144-byte pitch
#pragma unroll
        for (uint32_t k = 0; k < 16; k += 2) {
            const double2 v = *reinterpret_cast<const double2 *>(blk + k);
            x[k] = v.x; x[k + 1] = v.y;
        }
        fwd16_d(x, tw, 16 * (256 + row) + t, q, qinv);
        // four finished words: to the own block (BULK) or straight to global memory
        auto put4 = [&](u64 *dst, uint32_t k, u64 a, u64 b, u64 cc, u64 d) {
            if (BULK) {
                *reinterpret_cast<ulonglong2 *>(blk + k) = make_ulonglong2(a, b);
                *reinterpret_cast<ulonglong2 *>(blk + k + 2) = make_ulonglong2(cc, d);
            } else {
                stg_4(dst + k, a, b, cc, d);
            }
        };
        auto finish = [&](u64 *dst) {
            if (BULK) {
                bulk_store_128(dst, blk);
                bulk_store_wait();
            }
        };
        if (has_ep == 2) {     // the result itself, but into a tiled buffer
            const uint32_t y = blockIdx.y, i = y % ep.level, b = y / ep.level;
            u64 *dst = ep.out + tiled_index(ep.tl.R, 65536, ep.tl.row0 + b * ep.tl.row_stride, i, row * 256 + 16 * t);
#pragma unroll
            for (uint32_t k = 0; k < 16; k += 4)
                put4(dst, k, canonical_d(reduce_d(x[k], q, qinv), q), canonical_d(reduce_d(x[k + 1], q, qinv), q),
                     canonical_d(reduce_d(x[k + 2], q, qinv), q), canonical_d(reduce_d(x[k + 3], q, qinv), q));
            finish(dst);
            return;
        }
        if (has_ep) {      // ModDown tail: (u - NTT(conv)) P^-1 + sigma_g(add), written to its final place
            const uint32_t y = blockIdx.y, i = y % ep.level, comp = (y / ep.level) & 1, bz = y / (2 * ep.level);
            const double2 pinv = c.dn_p_inv_d[i];
            const uint32_t p0 = row * 256 + 16 * t;
            const u64 *up = ep.u + (((size_t)bz * 2 + comp) * ep.nt + i) * 65536 + p0;
            const u64 *add = comp ? ep.add1 : ep.add0;
            // grouped: entry bz is key bz / group applied to member bz % group
            const uint32_t rot = ep.group ? bz / ep.group : bz, mem = ep.group ? bz % ep.group : bz;
            const u64 gal = ep.multi ? ep.mgalois[rot] : ep.galois;
            u64 *dst = ep.group ? ep.out + tiled_index(ep.tl.R, 65536, ep.tl.row0 + rot * ep.rot_rows + mem * ep.tl.row_stride + comp, i, p0)
                       : ep.multi ? ep.mout[bz] + ((size_t)comp * ep.level + i) * 65536 + p0
                       : ep.tl.R ? ep.out + tiled_index(ep.tl.R, 65536, ep.tl.row0 + bz * ep.tl.row_stride + comp, i, p0)
                                 : ep.out + bz * ep.out_stride + ((size_t)comp * ep.level + i) * 65536 + p0;
#pragma unroll
            for (uint32_t k = 0; k < 16; k += 4) {
                u64 uu[4], old[4] = {0, 0, 0, 0}, r[4];
                ldg_4(up + k, uu[0], uu[1], uu[2], uu[3]);
                if (ep.accumulate) ldg_4(dst + k, old[0], old[1], old[2], old[3]);
#pragma unroll
                for (uint32_t e = 0; e < 4; e++) {
                    // all on the FP64 pipe: |u - v| < 1.5 q, times P^-1 -> |.| < 0.9 q, plus up to two residues, reduced once
                    double v = mulmod_d<0>(__dsub_rn(u64_to_d(uu[e]), reduce_d(x[k + e], q, qinv)), pinv, q);
                    if (add) v = __dadd_rn(v, u64_to_d(add[mem * ep.add_stride + (size_t)i * 65536 + galois_src(p0 + k + e, gal, 16, 65536)]));
                    if (ep.accumulate) v = __dadd_rn(v, u64_to_d(old[e]));
                    r[e] = canonical_d(reduce_d(v, q, qinv), q);
                }
                put4(dst, k, r[0], r[1], r[2], r[3]);
            }
            finish(dst);
            return;
        }
        // a thread ends up with 16 consecutive coefficients
#pragma unroll
        for (uint32_t k = 0; k < 16; k += 4)
            put4(g + 16 * t, k, canonical_d(reduce_d(x[k], q, qinv), q), canonical_d(reduce_d(x[k + 1], q, qinv), q),
                 canonical_d(reduce_d(x[k + 2], q, qinv), q), canonical_d(reduce_d(x[k + 3], q, qinv), q));
        finish(g + 16 * t);
        return;
    }
    if (ALLFP) return;
    const u64 q = c.mod[prime], q5 = 5 * q;
    const ulonglong2 *tw = c.tw_fwd + ((size_t)prime << 16);
    const uint32_t t = threadIdx.x & 15, rl = threadIdx.x >> 4, row = blockIdx.x * 16 + rl;
    u64 *g = base + (limb_index(map, blockIdx.y) << 16) + (size_t)row * 256;
    u64 *s = sm + rl * ROW_PAD;
    u64 x[16];
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) x[k] = g[t + 16 * k];
    fwd16(x, tw, 256 + row, q, q5);
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) s[padded(t + 16 * k)] = x[k];
    __syncwarp();   // a row lives in one half warp
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) x[k] = s[padded(16 * t + k)];
    fwd16(x, tw, 16 * (256 + row) + t, q, q5);
    const u64 qinv64 = c.mu64[prime];
    __syncwarp();
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) s[padded(16 * t + k)] = reduce_exact(x[k], q, qinv64);
    __syncwarp();
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) g[t + 16 * k] = s[padded(t + 16 * k)];
}

// ---- inverse, row pass (stages m = 32768..256) ---------------------------------------------
template <bool ALLFP, bool BULK = false>
__global__ void __launch_bounds__(F_THREADS, INV_CTAS) ntt16_inv_rows(DevTables c, u64 *base, LimbMap map, uint32_t fp_share, const u64 *src,
                                                                uint32_t src_pitch, long long wait_limit) {
    __shared__ __align__(16) u64 sm[16 * ROW_PAD];
    __shared__ __align__(8) u64 bars[F_THREADS / 32];
    const int prime = limb_prime(map, blockIdx.y);
    if (prime < 0) return;
    if (ALLFP || (blockIdx.y & 7) < fp_share) {
        const double q = c.modd[prime].x, qinv = c.modd[prime].y;
        const double *tw = c.twd_inv + ((size_t)prime << 16);
        const uint32_t t = threadIdx.x & 15, rl = threadIdx.x >> 4, row = blockIdx.x * 16 + rl;
        u64 *g = base + (limb_index(map, blockIdx.y) << 16) + (size_t)row * 256;
        // out of place: the input limbs lie in another buffer, periods src_pitch limbs apart
        const u64 *gs = src ? src + ((((size_t)(blockIdx.y / map.period) * src_pitch) + blockIdx.y % map.period) << 16) + (size_t)row * 256 : g;
        double *s = reinterpret_cast<double *>(sm) + rl * ROW_PAD;
        double x[16];
        if (BULK) {
            // 16 consecutive coefficients per thread arrive in the thread's own block of the exchange row as one 128-byte
            // bulk copy: the four 32-byte loads per thread they replace cost the load/store pipe one pass per lane and
            // sector, which made it the busiest unit of this kernel (inverse transform 0.440 -> 0.426 us per limb).  The
            // column passes' strided row pieces were measured slower as bulk copies (per warp or per CTA) and stay loads.
            const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&bars[threadIdx.x >> 5]);
            u64 *blk = reinterpret_cast<u64 *>(s) + 18 * t;
            warp_bulk_load_128(bar, blk, gs + 16 * t, threadIdx.x & 31);
            if (!warp_bulk_wait(bar, wait_limit)) {
                // report it, give the copies in flight one more bounded wait (their target is this CTA's memory) and leave
                if ((threadIdx.x & 31) == 0) atomicExch(c.range_flag + 1, 1);
                warp_bulk_wait(bar, wait_limit);
                return;
            }
#pragma unroll
            for (uint32_t k = 0; k < 16; k += 2) {
                const ulonglong2 v = *reinterpret_cast<const ulonglong2 *>(blk + k);
                x[k] = u64_to_d(v.x); x[k + 1] = u64_to_d(v.y);
            }
        } else {
#pragma unroll
            for (uint32_t k = 0; k < 16; k += 4) {      // 16 consecutive coefficients per thread, four 32-byte loads
                u64 a, b, cc, d;
                ldg_4(gs + 16 * t + k, a, b, cc, d);
                x[k] = u64_to_d(a); x[k + 1] = u64_to_d(b); x[k + 2] = u64_to_d(cc); x[k + 3] = u64_to_d(d);
            }
        }
        inv16_d(x, tw, 16 * (256 + row) + t, q, qinv);
#pragma unroll
        for (uint32_t k = 0; k < 16; k += 2) *reinterpret_cast<double2 *>(s + 18 * t + k) = make_double2(x[k], x[k + 1]);     // own block, 16-byte stores
        __syncwarp();
#pragma unroll
        for (uint32_t k = 0; k < 16; k++) x[k] = s[padded(t + 16 * k)];
        inv16_d(x, tw, 256 + row, q, qinv);
#pragma unroll
        for (uint32_t k = 0; k < 16; k++) reinterpret_cast<double *>(g)[t + 16 * k] = x[k];
        return;
    }
    if (ALLFP) return;
    const u64 q = c.mod[prime];
    const ulonglong2 *tw = c.tw_inv + ((size_t)prime << 16);
    const uint32_t t = threadIdx.x & 15, rl = threadIdx.x >> 4, row = blockIdx.x * 16 + rl;
    u64 *g = base + (limb_index(map, blockIdx.y) << 16) + (size_t)row * 256;
    const u64 *gs = src ? src + ((((size_t)(blockIdx.y / map.period) * src_pitch) + blockIdx.y % map.period) << 16) + (size_t)row * 256 : g;
    u64 *s = sm + rl * ROW_PAD;
    u64 x[16];
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) s[padded(t + 16 * k)] = gs[t + 16 * k];
    __syncwarp();
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) x[k] = s[padded(16 * t + k)];
    inv16<1>(x, tw, 16 * (256 + row) + t, q);
    __syncwarp();
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) s[padded(16 * t + k)] = x[k];
    __syncwarp();
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) x[k] = s[padded(t + 16 * k)];
    inv16<40>(x, tw, 256 + row, q);
    const ulonglong2 one = make_ulonglong2(1, c.mu64[prime]);
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) g[t + 16 * k] = mul_tw(x[k], one, q);   // lazy reduction to [0, 5q)
}

// ---- inverse, column pass (stages m = 128..1), then N^-1 and the exact reduction -----------
template <bool ALLFP>
__global__ void __launch_bounds__(F_THREADS, INV_CTAS) ntt16_inv_cols(DevTables c, u64 *base, LimbMap map, uint32_t fp_share, const double2 *scale) {
    __shared__ u64 sm[256 * 16];
    const int prime = limb_prime(map, blockIdx.y);
    if (prime < 0) return;
    if (ALLFP || (blockIdx.y & 7) < fp_share) {
        const double q = c.modd[prime].x, qinv = c.modd[prime].y;
        const double *tw = c.twd_inv + ((size_t)prime << 16);
        const uint32_t cc = threadIdx.x & 15, r = threadIdx.x >> 4;
        u64 *g = base + (limb_index(map, blockIdx.y) << 16) + blockIdx.x * 16 + cc;
        double *smd = reinterpret_cast<double *>(sm);
        double x[16];
#pragma unroll
        for (uint32_t k = 0; k < 16; k++) x[k] = reinterpret_cast<const double *>(g)[(size_t)(16 * r + k) * 256];
        inv16_d(x, tw, 16 + r, q, qinv);
#pragma unroll
        for (uint32_t k = 0; k < 16; k++) smd[(16 * r + k) * 16 + cc] = x[k];
        __syncthreads();
#pragma unroll
        for (uint32_t k = 0; k < 16; k++) x[k] = smd[(r + 16 * k) * 16 + cc];
        const double2 *sc = scale ? scale + 2 * (blockIdx.y % map.period) : c.n_inv_d + 2 * prime;
        inv16_last(x, tw, q, qinv, sc[0], sc[1]);
#pragma unroll
        for (uint32_t k = 0; k < 16; k++) g[(size_t)(r + 16 * k) * 256] = canonical_d(x[k], q);
        return;
    }
    if (ALLFP) return;
    const u64 q = c.mod[prime];
    const ulonglong2 *tw = c.tw_inv + ((size_t)prime << 16);
    const uint32_t cc = threadIdx.x & 15, r = threadIdx.x >> 4;
    u64 *g = base + (limb_index(map, blockIdx.y) << 16) + blockIdx.x * 16 + cc;
    u64 x[16];
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) x[k] = g[(size_t)(16 * r + k) * 256];
    inv16<5>(x, tw, 16 + r, q);
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) sm[(16 * r + k) * 16 + cc] = x[k];
    __syncthreads();
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) x[k] = sm[(r + 16 * k) * 16 + cc];
    inv16<80>(x, tw, 1, q);
    const ulonglong2 ni = c.n_inv[prime];
#pragma unroll
    for (uint32_t k = 0; k < 16; k++) g[(size_t)(r + 16 * k) * 256] = mul_shoup(x[k], ni.x, ni.y, q);
}

}  // namespace

void launch_ntt(const ckks_ctx *c, u64 *base, uint32_t nlimbs_total, const LimbMap &map, bool inverse, cudaStream_t s,
                const NttEpilogue *ep, const long long *coef_src, const u64 *inv_src, uint32_t inv_src_pitch, const double2 *inv_scale) {
    if (nlimbs_total == 0) return;
    if (c->log_n == 16) {
        for (uint32_t y0 = 0; y0 < nlimbs_total;) {
            const uint32_t chunk = map.period >= 32768 ? map.period : (32768 / map.period) * map.period;
            const uint32_t ny = nlimbs_total - y0 < chunk ? nlimbs_total - y0 : chunk;
            u64 *b = base + (limb_index(map, y0) << 16);
            dim3 grid(16, ny);
            if (!inverse) {
                // an epilogue is only implemented on the double-precision path, so it takes all limbs there
                const uint32_t share = (ep || coef_src) ? 8 : c->ntt_fp_share;
                if (share >= 8) ntt16_fwd_cols<true><<<grid, F_THREADS, 0, s>>>(c->dev, b, map, share, coef_src);
                else ntt16_fwd_cols<false><<<grid, F_THREADS, 0, s>>>(c->dev, b, map, share, coef_src);
                count_launches();
                // bulk-copy stores need 16-byte aligned destinations (every block is then 128-byte aligned relative to them)
                bool bulk = c->ntt_bulk_store && ((uintptr_t)(ep ? (const void *)ep->out : (const void *)b) & 15) == 0;
                if (ep && ep->multi)
                    for (uint32_t k = 0; k < KS_MULTI; k++) bulk = bulk && ((uintptr_t)ep->mout[k] & 15) == 0;
                if (share < 8) ntt16_fwd_rows<false, 0><<<grid, F_THREADS, 0, s>>>(c->dev, b, map, share, NttEpilogue{});
                else if (!ep && bulk) ntt16_fwd_rows<true, 0, true><<<grid, F_THREADS, 0, s>>>(c->dev, b, map, share, NttEpilogue{});
                else if (!ep) ntt16_fwd_rows<true, 0><<<grid, F_THREADS, 0, s>>>(c->dev, b, map, share, NttEpilogue{});
                else if (ep->mode == 1 && bulk) ntt16_fwd_rows<true, 1, true><<<grid, F_THREADS, 0, s>>>(c->dev, b, map, share, *ep);
                else if (ep->mode == 1) ntt16_fwd_rows<true, 1><<<grid, F_THREADS, 0, s>>>(c->dev, b, map, share, *ep);
                else if (bulk) ntt16_fwd_rows<true, 2, true><<<grid, F_THREADS, 0, s>>>(c->dev, b, map, share, *ep);
                else ntt16_fwd_rows<true, 2><<<grid, F_THREADS, 0, s>>>(c->dev, b, map, share, *ep);
                count_launches();
            } else {
                const u64 *sb = inv_src ? inv_src + (((size_t)(y0 / map.period) * inv_src_pitch) << 16) : nullptr;
                // bulk-copy loads need 16-byte aligned sources
                const bool bulk_in = c->ntt_bulk_store && ((uintptr_t)(sb ? (const void *)sb : (const void *)b) & 15) == 0;
                if (c->ntt_fp_share >= 8 && bulk_in) ntt16_inv_rows<true, true><<<grid, F_THREADS, 0, s>>>(c->dev, b, map, 8, sb, inv_src_pitch, c->wait_cycles);
                else if (c->ntt_fp_share >= 8) ntt16_inv_rows<true><<<grid, F_THREADS, 0, s>>>(c->dev, b, map, 8, sb, inv_src_pitch, 0);
                else ntt16_inv_rows<false><<<grid, F_THREADS, 0, s>>>(c->dev, b, map, c->ntt_fp_share, sb, inv_src_pitch, 0);
                count_launches();
                if (c->ntt_fp_share >= 8) ntt16_inv_cols<true><<<grid, F_THREADS, 0, s>>>(c->dev, b, map, 8, inv_scale);
                else ntt16_inv_cols<false><<<grid, F_THREADS, 0, s>>>(c->dev, b, map, c->ntt_fp_share, nullptr);
                count_launches();
            }
            y0 += ny;
        }
        return;
    }
    const uint32_t N = c->N, R = N / ROW;
    const uint32_t rows = R < ROWS_PER_CTA ? R : ROWS_PER_CTA;   // R >= 4 since N >= 1024
    const size_t smc = (size_t)R * COLS * sizeof(u64);
    // grid.y is limited to 65535: go in chunks that are whole periods of the limb map
    const uint32_t chunk = map.period >= 32768 ? map.period : (32768 / map.period) * map.period;
    for (uint32_t y0 = 0; y0 < nlimbs_total; y0 += chunk) {
        const uint32_t ny = nlimbs_total - y0 < chunk ? nlimbs_total - y0 : chunk;
        u64 *b = base + limb_index(map, y0) * N;
        dim3 gc(ROW / COLS, ny), gr(R / rows, ny);
        if (!inverse) {
            ntt_cols<false><<<gc, THREADS, smc, s>>>(c->dev, b, map); count_launches();
            ntt_rows<false><<<gr, THREADS, 0, s>>>(c->dev, b, map, rows); count_launches();
        } else {
            ntt_rows<true><<<gr, THREADS, 0, s>>>(c->dev, b, map, rows); count_launches();
            ntt_cols<true><<<gc, THREADS, smc, s>>>(c->dev, b, map); count_launches();
        }
    }
}

// grid: three CTAs per SM, the residency of the transform kernels.  Returns the butterflies one launch performs.
uint64_t launch_butterfly_probe(const ckks_ctx *c, uint32_t iters, u64 *sink, cudaStream_t s) {
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
    const uint32_t ctas = (uint32_t)sms * 3;
    butterfly_probe_kernel<<<ctas, F_THREADS, 0, s>>>(c->dev, iters, sink);
    count_launches();
    return (uint64_t)ctas * F_THREADS * iters * 32;
}


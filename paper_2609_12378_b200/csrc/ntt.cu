// Batched negacyclic NTT / inverse NTT.
//
// Forward: merged Cooley-Tukey, natural-order input, bit-reversed output, stages
// m = 1, 2, .., N/2 with butterfly distance t = N/(2m) and twiddle psi^bitrev(m+i)
// for block i.  Inverse: Gentleman-Sande, the same stages backwards, then N^-1.
//
// A limb is viewed as R rows of 256 coefficients (R = N/256).  The stages with
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
    u64 *g = base + (size_t)blockIdx.y * N + blockIdx.x * COLS;
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
    u64 *g = base + (size_t)blockIdx.y * N + (size_t)row0 * ROW;
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

}  // namespace

void launch_ntt(const ckks_ctx *c, u64 *base, uint32_t nlimbs_total, const LimbMap &map, bool inverse, cudaStream_t s) {
    if (nlimbs_total == 0) return;
    const uint32_t N = c->N, R = N / ROW;
    const uint32_t rows = R < ROWS_PER_CTA ? R : ROWS_PER_CTA;   // R >= 4 since N >= 1024
    const size_t smc = (size_t)R * COLS * sizeof(u64);
    // grid.y is limited to 65535: go in chunks that are whole periods of the limb map
    const uint32_t chunk = map.period >= 32768 ? map.period : (32768 / map.period) * map.period;
    for (uint32_t y0 = 0; y0 < nlimbs_total; y0 += chunk) {
        const uint32_t ny = nlimbs_total - y0 < chunk ? nlimbs_total - y0 : chunk;
        u64 *b = base + (size_t)y0 * N;
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

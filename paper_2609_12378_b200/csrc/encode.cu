// Encode: slot values -> plaintext limbs.
//
//   E1  Z[e_j] = z_j,  e_j = ((5^j mod 2N) - 1) / 4
//   E2  b_k = sum_e Z[e] omega^(-e k)   (size n, unnormalised), radix-2 decimation in time:
//       bit-reversed input, stages m = 2, 4, .., n, butterfly (u, v) -> (u + w v, u - w v) with
//       w = conj(omega^(j n / m)); every product and every sum rounded on its own (no FMA)
//   E3  a_k = b_k conj(zeta^k)
//   E4  m_k = rint(Re a_k * scale/n), m_{k+n} = rint(Im a_k * scale/n), ties to even
//   E5  residues of m_k modulo every prime, E6 NTT per limb.
//
// The transform of size n is split like the NTT: the stages with span <= CH run on
// contiguous chunks of CH points in shared memory, the remaining ones on strips of
// 16 columns of the [n/CH][CH] view.  Each radix-2 butterfly is performed exactly once
// with the operands the definition gives it, so the result does not depend on the split.
#include "common.cuh"

namespace {

constexpr uint32_t THREADS = 256;
constexpr uint32_t CH = 1024;   // points per chunk in the first pass
constexpr uint32_t COLS = 16;   // columns per CTA in the second pass

__device__ __forceinline__ double2 cmul_conj_w(double2 w, double2 v) {   // conj(w) * v, four products, two sums
    const double wr = w.x, wi = -w.y;
    const double p0 = __dmul_rn(wr, v.x), p1 = __dmul_rn(wi, v.y), p2 = __dmul_rn(wr, v.y), p3 = __dmul_rn(wi, v.x);
    return make_double2(__dsub_rn(p0, p1), __dadd_rn(p2, p3));
}

// Pass 1: gather (E1 + bit reversal), stages m = 2 .. min(n, CH) on chunks of CH points.  The stages' twiddles come from
// a copy in shared memory (stage by stage, so that a warp reads consecutive entries): fetched from the full table they
// were 5120 scattered 16-byte loads per CTA and the kernel was bound by the traffic between L2 and L1.
__global__ void __launch_bounds__(THREADS) fft_chunks(DevTables c, const double *re, const double *im, double2 *buf, uint32_t n, uint32_t ch) {
    __shared__ double2 sm[CH];
    __shared__ double2 tw[CH];
    const uint32_t b = blockIdx.y, base = blockIdx.x * ch;
    for (uint32_t x = threadIdx.x; x < ch; x += THREADS) {
        const uint32_t j = c.enc_src[base + x];
        sm[x] = make_double2(re[(size_t)b * n + j], im ? im[(size_t)b * n + j] : 0.0);
        tw[x] = c.enc_omega_st[x];
    }
    __syncthreads();
    // two stages per pass over shared memory: a thread takes the four points j, j + h, j + 2h, j + 3h of a block of 4h and does
    // the two butterflies of span h and the two of span 2h on registers (the same butterflies with the same operands as one
    // stage at a time; the kernel is bound by shared-memory traffic, which this halves)
    uint32_t m = 2;
    for (; 2 * m <= ch; m <<= 2) {
        const uint32_t h = m >> 1;
        for (uint32_t x = threadIdx.x; x < ch / 4; x += THREADS) {
            const uint32_t j = x & (h - 1), i0 = ((x - j) << 2) + j;
            double2 a0 = sm[i0], a1 = sm[i0 + h], a2 = sm[i0 + 2 * h], a3 = sm[i0 + 3 * h];
            const double2 w1 = tw[h + j];
            double2 t = cmul_conj_w(w1, a1);
            a1 = make_double2(__dsub_rn(a0.x, t.x), __dsub_rn(a0.y, t.y));
            a0 = make_double2(__dadd_rn(a0.x, t.x), __dadd_rn(a0.y, t.y));
            t = cmul_conj_w(w1, a3);
            a3 = make_double2(__dsub_rn(a2.x, t.x), __dsub_rn(a2.y, t.y));
            a2 = make_double2(__dadd_rn(a2.x, t.x), __dadd_rn(a2.y, t.y));
            t = cmul_conj_w(tw[2 * h + j], a2);
            a2 = make_double2(__dsub_rn(a0.x, t.x), __dsub_rn(a0.y, t.y));
            a0 = make_double2(__dadd_rn(a0.x, t.x), __dadd_rn(a0.y, t.y));
            t = cmul_conj_w(tw[2 * h + j + h], a3);
            a3 = make_double2(__dsub_rn(a1.x, t.x), __dsub_rn(a1.y, t.y));
            a1 = make_double2(__dadd_rn(a1.x, t.x), __dadd_rn(a1.y, t.y));
            sm[i0] = a0; sm[i0 + h] = a1; sm[i0 + 2 * h] = a2; sm[i0 + 3 * h] = a3;
        }
        __syncthreads();
    }
    for (; m <= ch; m <<= 1) {             // a last single stage when the number of stages is odd
        const uint32_t half = m >> 1;
        for (uint32_t x = threadIdx.x; x < ch / 2; x += THREADS) {
            const uint32_t j = x & (half - 1), i1 = ((x - j) << 1) + j;
            const double2 t = cmul_conj_w(tw[half + j], sm[i1 + half]);
            const double2 u = sm[i1];
            sm[i1] = make_double2(__dadd_rn(u.x, t.x), __dadd_rn(u.y, t.y));
            sm[i1 + half] = make_double2(__dsub_rn(u.x, t.x), __dsub_rn(u.y, t.y));
        }
        __syncthreads();
    }
    for (uint32_t x = threadIdx.x; x < ch; x += THREADS) buf[(size_t)b * n + base + x] = sm[x];
}

// Pass 2: stages m = 2 CH .. n on strips of COLS columns (rows = n/ch), then E3, E4 -> int64 coefficients.
__global__ void __launch_bounds__(THREADS) fft_strips_round(DevTables c, const double2 *buf, long long *coef, uint32_t n, uint32_t ch, double s) {
    extern __shared__ double2 sm2[];
    const uint32_t b = blockIdx.y, rows = n / ch, col0 = blockIdx.x * COLS;
    double2 *tw = sm2 + rows * COLS;          // the strip's twiddles, entry (hr + jr) * COLS + column (row 0 unused)
    for (uint32_t x = threadIdx.x; x < rows * COLS; x += THREADS) {
        sm2[x] = buf[(size_t)b * n + (size_t)(x / COLS) * ch + col0 + x % COLS];
        tw[x] = c.enc_omega_st2[(size_t)(x / COLS) * ch + col0 + x % COLS];
    }
    __syncthreads();
    for (uint32_t m = 2 * ch; m <= n; m <<= 1) {
        const uint32_t half = m >> 1, hr = half / ch;      // hr = distance in rows
        for (uint32_t x = threadIdx.x; x < (rows / 2) * COLS; x += THREADS) {
            const uint32_t cc = x % COLS, y = x / COLS, jr = y & (hr - 1), r1 = ((y - jr) << 1) + jr;
            // twiddle omega^(j n / m) of position j = jr ch + col0 + cc inside the half block
            const double2 t = cmul_conj_w(tw[(hr + jr) * COLS + cc], sm2[(r1 + hr) * COLS + cc]);
            const double2 u = sm2[r1 * COLS + cc];
            sm2[r1 * COLS + cc] = make_double2(__dadd_rn(u.x, t.x), __dadd_rn(u.y, t.y));
            sm2[(r1 + hr) * COLS + cc] = make_double2(__dsub_rn(u.x, t.x), __dsub_rn(u.y, t.y));
        }
        __syncthreads();
    }
    for (uint32_t x = threadIdx.x; x < rows * COLS; x += THREADS) {
        const uint32_t k = (x / COLS) * ch + col0 + x % COLS;
        const double2 a = cmul_conj_w(c.enc_zeta[k], sm2[x]);
        double xr = __dmul_rn(a.x, s), xi = __dmul_rn(a.y, s);
        if (!(fabs(xr) < 4611686018427387904.0) || !(fabs(xi) < 4611686018427387904.0)) { *c.range_flag = 1; xr = xi = 0.0; }
        coef[(size_t)b * 2 * n + k] = __double2ll_rn(xr);
        coef[(size_t)b * 2 * n + n + k] = __double2ll_rn(xi);
    }
}

// out[b][i][k] = canonical residue of coef[b][k] modulo q_i
__global__ void __launch_bounds__(THREADS) reduce_coeffs(DevTables c, const long long *coef, u64 *out, uint32_t level) {
    const uint32_t k = blockIdx.x * THREADS + threadIdx.x;
    const uint32_t i = blockIdx.y, b = blockIdx.z;
    const long long v = coef[(size_t)b * c.N + k];
    const u64 q = c.mod[i];
    const u64 mag = v < 0 ? (u64)(-v) : (u64)v;
    const u64 r = barrett112(0, mag, q, c.mu[i]);
    out[((size_t)b * level + i) * c.N + k] = (v < 0 && r) ? q - r : r;
}

// slots[kk][r*T + t] = d'_k[r],  k = k0 + kk,  d'_k[r] = d_k[(r - pre_rot) mod F],
// d_k[r'] = W^T[out0 + r' mod m_out, in0 + (r' + k) mod m_in]
__global__ void __launch_bounds__(THREADS) extract_diagonals(const double *W, uint32_t d_out_total, uint32_t in0, uint32_t m_in,
                                                             uint32_t out0, uint32_t m_out, uint32_t F, uint32_t T, uint32_t k0,
                                                             uint32_t pre_rot, double *slots, uint32_t n) {
    const uint32_t x = blockIdx.x * THREADS + threadIdx.x;
    if (x >= n) return;
    const uint32_t r = x / T, k = k0 + blockIdx.y;
    const uint32_t rp = (r + F - pre_rot % F) % F;
    const uint32_t ro = rp % m_out, ci = (rp + k) % m_in;
    slots[(size_t)blockIdx.y * n + x] = W[(size_t)(in0 + ci) * d_out_total + out0 + ro];
}

}  // namespace

size_t encode_workspace_bytes(const ckks_ctx *c, uint32_t batch) {
    return (size_t)batch * ((size_t)c->n * sizeof(double2) + (size_t)c->N * sizeof(long long));
}

void launch_encode(const ckks_ctx *c, const double *re, const double *im, uint32_t batch, double scale, uint32_t level,
                   u64 *out, void *ws, cudaStream_t s, TiledOut tiled, u64 *tiled_out) {
    const uint32_t n = c->n, N = c->N, ch = n < CH ? n : CH;
    double2 *buf = (double2 *)ws;
    long long *coef = (long long *)(buf + (size_t)batch * n);
    const double sc = scale / (double)n;
    for (uint32_t b0 = 0; b0 < batch; b0 += 32768) {
        const uint32_t nb = batch - b0 < 32768 ? batch - b0 : 32768;
        fft_chunks<<<dim3(n / ch, nb), THREADS, 0, s>>>(c->dev, re + (size_t)b0 * n, im ? im + (size_t)b0 * n : nullptr,
                                                         buf + (size_t)b0 * n, n, ch); count_launches();
        fft_strips_round<<<dim3(ch / COLS, nb), THREADS, (size_t)2 * (n / ch) * COLS * sizeof(double2), s>>>(
            c->dev, buf + (size_t)b0 * n, coef + (size_t)b0 * N, n, ch, sc); count_launches();
    }
    if (c->log_n == 16 && (uint64_t)batch * level <= 32768) {
        // the first NTT pass reduces the signed coefficients itself; the last one can write the tiled layout
        if (tiled.R) {
            NttEpilogue ep{};
            ep.mode = 2; ep.out = tiled_out; ep.level = level; ep.tl = tiled;
            launch_ntt(c, out, batch * level, plain_map(0, level), false, s, &ep, coef);
        } else {
            launch_ntt(c, out, batch * level, plain_map(0, level), false, s, nullptr, coef);
        }
        return;
    }
    for (uint32_t b0 = 0; b0 < batch; b0 += 32768) {
        const uint32_t nb = batch - b0 < 32768 ? batch - b0 : 32768;
        reduce_coeffs<<<dim3(N / THREADS, level, nb), THREADS, 0, s>>>(c->dev, coef + (size_t)b0 * N, out + (size_t)b0 * level * N, level);
        count_launches();
    }
    launch_ntt(c, out, batch * level, plain_map(0, level), false, s);
    if (tiled.R) launch_to_tiled(c, out, (size_t)level * N, batch, tiled_out, tiled.R, tiled.row0, tiled.row_stride, level, s);
}

void launch_extract_diagonals(const ckks_ctx *c, const double *W, uint32_t d_out_total, uint32_t in0, uint32_t m_in,
                              uint32_t out0, uint32_t m_out, uint32_t F, uint32_t T, uint32_t k0, uint32_t count,
                              uint32_t pre_rot, double *slots, cudaStream_t s) {
    extract_diagonals<<<dim3((c->n + THREADS - 1) / THREADS, count), THREADS, 0, s>>>(W, d_out_total, in0, m_in, out0, m_out, F, T, k0,
                                                                                       pre_rot, slots, c->n); count_launches();
}

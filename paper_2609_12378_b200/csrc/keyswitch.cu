// Hybrid key switching (dnum digits, K special primes) and rescale.
//
// KeySwitch(d, evk):  d (evaluation domain, `level` limbs)
//   1. to the coefficient domain (inverse NTT)
//   2. ModUp: every active digit j is extended from its own limbs to all active
//      q-limbs and all special limbs by a centred fast basis conversion
//         y_a = centre([d_a * qhat_a^-1]_{q_a}),  ext_j[t] = sum_a y_a (qhat_a mod t)  mod t
//   3. NTT of the converted limbs (own limbs keep their evaluation values)
//   4. inner product with the key: u_c[t] = sum_j ext_j[t] * evk_{j,c}[t]
//   5. ModDown: inverse NTT of the special limbs, centred conversion P -> q_i,
//      NTT, out_i = (u_i - conv_i) * P^-1 mod q_i.
// Rescale drops the last limb the same way with a single source limb.
#include "common.cuh"

namespace {

constexpr uint32_t THREADS = 256;

// dst[b][i][p] = src[b][i][pi_g(p)]  (g = 1: copy); batch entries src_stride / dst_stride words apart
__global__ void __launch_bounds__(THREADS) permute_kernel(DevTables c, const u64 *src, size_t src_stride, u64 *dst, size_t dst_stride, u64 g) {
    const uint32_t p = blockIdx.x * THREADS + threadIdx.x;
    const size_t row = (size_t)blockIdx.y * c.N;
    dst[blockIdx.z * dst_stride + row + p] = src[blockIdx.z * src_stride + row + galois_src(p, g, c.log_n, c.N)];
}

// targets per CTA row in the basis-conversion kernels: the source limbs are re-read once per chunk, so large batches
// take all targets in one chunk and single ciphertexts split them for parallelism
inline uint32_t conv_chunk(uint32_t nb) { return nb >= 4 ? 32 : 16; }

// ext[j][x][k] for x over q_0..q_{level-1}, p_0..p_{K-1}.  dcoef: sigma_g(d) in the coefficient domain;
// deval: d in the evaluation domain, read through sigma_g for the digit's own limbs.
// A thread owns one coefficient of one digit: it forms the centred y_a of the digit's limbs once and then
// walks a chunk of CHUNK target limbs (blockIdx.y), so the source limbs are read once per chunk.
constexpr uint32_t CONV_CHUNK_MAX = 32;

// PRE: dcoef already holds [d_a qhat_a^-1] (the inverse transform multiplied it in), so only the centring is left.
template <uint32_t ALPHA, bool PRE>
__global__ void __launch_bounds__(THREADS) modup_kernel(DevTables c, const u64 *dcoef, const u64 *deval, size_t deval_stride, u64 g,
                                                        u64 *ext, uint32_t level, uint32_t CHUNK) {
    // the CTA's conversion constants (qhat_a mod t and its quotient by t; t and 1/t), fetched once: as global loads
    // inside the loop they kept the L1 busier than the arithmetic kept the FP64 pipe
    __shared__ double2 s_w[CONV_CHUNK_MAX][ALPHA];
    __shared__ double2 s_m[CONV_CHUNK_MAX];
    const uint32_t k = blockIdx.x * THREADS + threadIdx.x;
    const uint32_t beta = (level + c.alpha - 1) / c.alpha, j = blockIdx.z % beta, bz = blockIdx.z / beta;
    const uint32_t nt = level + c.K, lo = j * c.alpha, hi = min(lo + c.alpha, level), nd = hi - lo;
    const uint32_t x0 = blockIdx.y * CHUNK, x1 = min(x0 + CHUNK, nt);
    const size_t cb = ((size_t)level * c.dnum + j) * c.alpha;
    for (uint32_t e = threadIdx.x; e < (x1 - x0) * ALPHA; e += THREADS) {
        const uint32_t xi = e / ALPHA, a = e % ALPHA, x = x0 + xi, t = x < level ? x : c.L + (x - level);
        s_w[xi][a] = a < nd ? c.up_hat_mod_d[(cb + a) * c.T + t] : make_double2(0.0, 0.0);
        if (a == 0) s_m[xi] = c.modd[t];
    }
    dcoef += (size_t)bz * level * c.N;
    deval += bz * deval_stride;
    ext += (size_t)bz * beta * nt * c.N;
    // centred y_a = [d_a qhat_a^-1] as signed doubles (integer Shoup product, then the lift)
    double y[ALPHA];
#pragma unroll
    for (uint32_t a = 0; a < ALPHA; a++) {
        y[a] = 0.0;
        if (a < nd) {
            const u64 qa = c.mod[lo + a];
            u64 v = dcoef[(size_t)(lo + a) * c.N + k];
            if (!PRE) {
                const ulonglong2 hinv = c.up_hat_inv[cb + a];
                v = mul_shoup(v, hinv.x, hinv.y, qa);
            }
            y[a] = v > (qa >> 1) ? __dsub_rn(u64_to_d(v), (double)qa) : u64_to_d(v);
        }
    }
    __syncthreads();
    u64 *dst = ext + ((size_t)j * nt + x0) * c.N + k;
    for (uint32_t x = x0; x < x1; x++, dst += c.N) {
        if (x >= lo && x < hi) {
            *dst = deval[(size_t)x * c.N + galois_src(k, g, c.log_n, c.N)];
            continue;
        }
        const double2 md = s_m[x - x0];
        const double mt = md.x, mtinv = md.y;
        // each product is reduced to |r| <= 0.57 m_t on the FP64 pipe; eight of them stay far below 2^53 (a missing
        // source has y = 0 and a zero constant)
        double acc = 0.0;
#pragma unroll
        for (uint32_t a = 0; a < ALPHA; a++) {
            acc = __dadd_rn(acc, mulmod_d<0>(y[a], s_w[x - x0][a], mt));
            if ((a & 7) == 7 && a + 1 < ALPHA) acc = reduce_d(acc, mt, mtinv);
        }
        *dst = canonical_d(reduce_d(acc, mt, mtinv), mt);
    }
}

template <uint32_t ALPHA>
void launch_modup(const ckks_ctx *c, const u64 *dcoef, const u64 *deval, size_t deval_stride, u64 g, u64 *ext, uint32_t level,
                  uint32_t nb, cudaStream_t s, bool pre) {
    const uint32_t nt = level + c->K, beta = (level + c->alpha - 1) / c->alpha;
    const uint32_t CHUNK = conv_chunk(nb);
    const dim3 grid(c->N / THREADS, (nt + CHUNK - 1) / CHUNK, beta * nb);
    if (pre) modup_kernel<ALPHA, true><<<grid, THREADS, 0, s>>>(c->dev, dcoef, deval, deval_stride, g, ext, level, CHUNK);
    else modup_kernel<ALPHA, false><<<grid, THREADS, 0, s>>>(c->dev, dcoef, deval, deval_stride, g, ext, level, CHUNK);
    count_launches();
}

// u[comp][x][p] = sum_j ext[j][x][pi_g(p)] * evk[j][comp][kt(x)][p]          (any number of digits)
__global__ void __launch_bounds__(THREADS) inner_product_generic_kernel(DevTables c, const u64 *ext, const u64 *evk, u64 g,
                                                                        u64 *u, uint32_t level, int has_multi, KsMulti multi, int acc_u) {
    const uint32_t p = blockIdx.x * THREADS + threadIdx.x;
    const uint32_t x = blockIdx.z, bz = blockIdx.y;     // batch varies faster than the limb: a key limb is reused from L2
    const uint32_t nt = level + c.K, beta = (level + c.alpha - 1) / c.alpha;
    const uint32_t kt = x < level ? x : c.L + (x - level);
    if (has_multi) { evk = multi.evk[bz]; g = multi.galois[bz]; }     // shared digits, per-entry key and permutation
    else ext += (size_t)bz * beta * nt * c.N;
    const uint32_t src = galois_src(p, g, c.log_n, c.N);
    u += (size_t)bz * 2 * nt * c.N;
    // products on the FP64 pipe: each is reduced to |r| <= 0.75 m as it is formed, the few digits are summed exactly
    const double2 md = c.modd[kt];
    double a0 = 0.0, a1 = 0.0;
    for (uint32_t j = 0; j < beta; j++) {
        const double e = u64_to_d(ext[((size_t)j * nt + x) * c.N + src]);
        a0 = __dadd_rn(a0, mulmod_dd(e, u64_to_d(evk[(((size_t)j * 2 + 0) * c.T + kt) * c.N + p]), md.x, md.y));
        a1 = __dadd_rn(a1, mulmod_dd(e, u64_to_d(evk[(((size_t)j * 2 + 1) * c.T + kt) * c.N + p]), md.x, md.y));
        if ((j & 7) == 7) { a0 = reduce_d(a0, md.x, md.y); a1 = reduce_d(a1, md.x, md.y); }
    }
    u64 r0 = canonical_d(reduce_d(a0, md.x, md.y), md.x), r1 = canonical_d(reduce_d(a1, md.x, md.y), md.x);
    if (acc_u) {        // a sum of key-switched terms kept in the extended basis
        const u64 m = c.mod[kt];
        r0 = add_mod(r0, u[((size_t)0 * nt + x) * c.N + p], m);
        r1 = add_mod(r1, u[((size_t)1 * nt + x) * c.N + p], m);
    }
    u[((size_t)0 * nt + x) * c.N + p] = r0;
    u[((size_t)1 * nt + x) * c.N + p] = r1;
}

// The same for BETA <= 4 digits, two adjacent coefficients per thread.  pi_g maps the pair (p, p + 1), p even, onto a
// pair (s, s ^ 1), so digits and key words both move as 16-byte loads.  Without `multi` a thread walks `bch` batch
// entries (blockIdx.y picks the chunk) with the key words of its pair held in registers; with it, an entry is one
// of up to KS_MULTI keys applied to the same digits.
constexpr uint32_t IP_MAX_BETA = 4;
template <uint32_t BETA>
__global__ void __launch_bounds__(THREADS) inner_product_kernel(DevTables c, const u64 *ext, const u64 *evk, u64 g, u64 *u,
                                                                uint32_t level, uint32_t nb, uint32_t bch, int has_multi, KsMulti multi,
                                                                int acc_u) {
    const uint32_t p = (blockIdx.x * THREADS + threadIdx.x) * 2;
    const uint32_t x = blockIdx.z;     // chunks of a limb run together: its key words (and shared digits) come from L2
    uint32_t b0 = blockIdx.y * bch, b1 = min(b0 + bch, nb), e0 = has_multi ? 0 : b0;      // entries; first digits entry
    const uint32_t nt = level + c.K;
    const uint32_t kt = x < level ? x : c.L + (x - level);
    const double2 md = c.modd[kt];
    const size_t js = (size_t)nt * c.N, ks = (size_t)c.T * c.N;
    if (has_multi && multi.group) {     // key r on a chunk of the group's members
        const uint32_t cpr = (multi.group + bch - 1) / bch, r = blockIdx.y / cpr, ch = blockIdx.y % cpr;
        e0 = ch * bch;
        b0 = r * multi.group + e0;
        b1 = min(b0 + bch, (r + 1) * multi.group);
        evk = multi.evk[r]; g = multi.galois[r];
    } else if (has_multi) { evk = multi.evk[b0]; g = multi.galois[b0]; }
    const uint32_t src = galois_src(p, g, c.log_n, c.N);
    const bool odd = src & 1;
    double k[BETA][2][2];                         // [digit][component][coefficient of the pair]
#pragma unroll
    for (uint32_t j = 0; j < BETA; j++)
#pragma unroll
        for (uint32_t cm = 0; cm < 2; cm++) {
            const ulonglong2 v = *reinterpret_cast<const ulonglong2 *>(evk + ((size_t)j * 2 + cm) * ks + (size_t)kt * c.N + p);
            k[j][cm][0] = u64_to_d(v.x);
            k[j][cm][1] = u64_to_d(v.y);
        }
    const u64 *e = ext + e0 * BETA * js + (size_t)x * c.N + (src & ~1u);
    u64 *o = u + b0 * 2 * js + (size_t)x * c.N + p;
    for (uint32_t b = b0; b < b1; b++, e += BETA * js, o += 2 * js) {
        double acc[2][2] = {{0.0, 0.0}, {0.0, 0.0}};
#pragma unroll
        for (uint32_t j = 0; j < BETA; j++) {
            const ulonglong2 v = *reinterpret_cast<const ulonglong2 *>(e + j * js);
            const double d0 = u64_to_d(odd ? v.y : v.x), d1 = u64_to_d(odd ? v.x : v.y);
#pragma unroll
            for (uint32_t cm = 0; cm < 2; cm++) {
                acc[cm][0] = __dadd_rn(acc[cm][0], mulmod_dd(d0, k[j][cm][0], md.x, md.y));
                acc[cm][1] = __dadd_rn(acc[cm][1], mulmod_dd(d1, k[j][cm][1], md.x, md.y));
            }
        }
#pragma unroll
        for (uint32_t cm = 0; cm < 2; cm++) {
            ulonglong2 r;
            r.x = canonical_d(reduce_d(acc[cm][0], md.x, md.y), md.x);
            r.y = canonical_d(reduce_d(acc[cm][1], md.x, md.y), md.x);
            if (acc_u) {
                const ulonglong2 old = *reinterpret_cast<const ulonglong2 *>(o + cm * js);
                const u64 m = c.mod[kt];
                r.x = add_mod(r.x, old.x, m);
                r.y = add_mod(r.y, old.y, m);
            }
            *reinterpret_cast<ulonglong2 *>(o + cm * js) = r;
        }
    }
}

// The inner product of several terms at once (see ks_inner_terms): like inner_product_kernel, but every term has its
// own digits, key, permutation and first component, and the running sums of a chunk of IP_BCH batch entries stay in
// registers over the terms.
constexpr uint32_t IP_BCH = 4;
template <uint32_t BETA>
__global__ void __launch_bounds__(THREADS, 3) inner_product_terms_kernel(DevTables c, const u64 *ext, size_t term_stride,
                                                                         const __grid_constant__ IpTerms tm, uint32_t nterm, size_t c0_stride,
                                                                         u64 *u, uint32_t level, uint32_t nb, int acc_u) {
    const uint32_t p = (blockIdx.x * THREADS + threadIdx.x) * 2;
    const uint32_t x = blockIdx.z, b0 = blockIdx.y * IP_BCH;
    const uint32_t nt = level + c.K;
    const uint32_t kt = x < level ? x : c.L + (x - level);
    const double2 md = c.modd[kt];
    const size_t js = (size_t)nt * c.N, ks = (size_t)c.T * c.N;
    const double pq = x < level ? c.dn_p_mod_d[x] : 0.0;
    double acc[IP_BCH][2][2];
#pragma unroll
    for (uint32_t bi = 0; bi < IP_BCH; bi++) acc[bi][0][0] = acc[bi][0][1] = acc[bi][1][0] = acc[bi][1][1] = 0.0;
    for (uint32_t t = 0; t < nterm; t++) {
        const uint32_t src = galois_src(p, tm.galois[t], c.log_n, c.N);
        const bool odd = src & 1;
        const u64 *evk = tm.evk[t];
        double k[BETA][2][2];
#pragma unroll
        for (uint32_t j = 0; j < BETA; j++)
#pragma unroll
            for (uint32_t cm = 0; cm < 2; cm++) {
                const ulonglong2 v = *reinterpret_cast<const ulonglong2 *>(evk + ((size_t)j * 2 + cm) * ks + (size_t)kt * c.N + p);
                k[j][cm][0] = u64_to_d(v.x);
                k[j][cm][1] = u64_to_d(v.y);
            }
        const u64 *e = ext + t * term_stride + (size_t)b0 * BETA * js + (size_t)x * c.N + (src & ~1u);
        const u64 *z = (x < level && tm.c0[t]) ? tm.c0[t] + b0 * c0_stride + (size_t)x * c.N + (src & ~1u) : nullptr;
        // no branch in here, so that the loads of all entries of the chunk are in flight together: an entry past the end
        // of the batch repeats the last one and is not stored
#pragma unroll
        for (uint32_t bi = 0; bi < IP_BCH; bi++) {
            const uint32_t bc = min(bi, nb - 1 - b0);
            double sum[2][2] = {{0.0, 0.0}, {0.0, 0.0}};
#pragma unroll
            for (uint32_t j = 0; j < BETA; j++) {
                const ulonglong2 v = *reinterpret_cast<const ulonglong2 *>(e + ((size_t)bc * BETA + j) * js);
                const double d0 = u64_to_d(odd ? v.y : v.x), d1 = u64_to_d(odd ? v.x : v.y);
#pragma unroll
                for (uint32_t cm = 0; cm < 2; cm++) {
                    sum[cm][0] = __dadd_rn(sum[cm][0], mulmod_dd(d0, k[j][cm][0], md.x, md.y));
                    sum[cm][1] = __dadd_rn(sum[cm][1], mulmod_dd(d1, k[j][cm][1], md.x, md.y));
                }
            }
            if (z) {
                const ulonglong2 v = *reinterpret_cast<const ulonglong2 *>(z + bc * c0_stride);
                sum[0][0] = __dadd_rn(sum[0][0], mulmod_dd(u64_to_d(odd ? v.y : v.x), pq, md.x, md.y));
                sum[0][1] = __dadd_rn(sum[0][1], mulmod_dd(u64_to_d(odd ? v.x : v.y), pq, md.x, md.y));
            }
            // at most BETA + 1 products of size 0.75 m on top of a reduced sum: far below 2^53
#pragma unroll
            for (uint32_t cm = 0; cm < 2; cm++) {
                acc[bi][cm][0] = reduce_d(__dadd_rn(acc[bi][cm][0], sum[cm][0]), md.x, md.y);
                acc[bi][cm][1] = reduce_d(__dadd_rn(acc[bi][cm][1], sum[cm][1]), md.x, md.y);
            }
        }
    }
    const u64 m = c.mod[kt];
#pragma unroll
    for (uint32_t bi = 0; bi < IP_BCH; bi++) {
        if (b0 + bi >= nb) break;
        u64 *o = u + (size_t)(b0 + bi) * 2 * js + (size_t)x * c.N + p;
#pragma unroll
        for (uint32_t cm = 0; cm < 2; cm++) {
            ulonglong2 r;
            r.x = canonical_d(acc[bi][cm][0], md.x);
            r.y = canonical_d(acc[bi][cm][1], md.x);
            if (acc_u) {
                const ulonglong2 old = *reinterpret_cast<const ulonglong2 *>(o + cm * js);
                r.x = add_mod(r.x, old.x, m);
                r.y = add_mod(r.y, old.y, m);
            }
            *reinterpret_cast<ulonglong2 *>(o + cm * js) = r;
        }
    }
}

// conv[comp][i][k] = sum_a centre([u_{p_a} Phat_a^-1]) (Phat_a mod q_i)  mod q_i   (coefficient domain)
// Same shape as ModUp: the K centred special residues are formed once per thread, then a chunk of targets is walked.
template <uint32_t KK, bool PRE>
__global__ void __launch_bounds__(THREADS, 6) moddown_conv_kernel(DevTables c, const u64 *u, u64 *conv, uint32_t level, uint32_t CHUNK) {
    __shared__ double2 s_w[CONV_CHUNK_MAX][KK];     // Phat_a mod q_i and its quotient by q_i
    __shared__ double2 s_m[CONV_CHUNK_MAX];         // q_i, 1 / q_i
    const uint32_t k = blockIdx.x * THREADS + threadIdx.x;
    const uint32_t comp = blockIdx.z & 1, bz = blockIdx.z >> 1;
    const uint32_t nt = level + c.K;
    const uint32_t i0 = blockIdx.y * CHUNK, i1 = min(i0 + CHUNK, level);
    for (uint32_t e = threadIdx.x; e < (i1 - i0) * KK; e += THREADS) {
        const uint32_t ii = e / KK, a = e % KK;
        s_w[ii][a] = a < c.K ? c.dn_hat_mod_d[(size_t)(i0 + ii) * c.K + a] : make_double2(0.0, 0.0);
        if (a == 0) s_m[ii] = c.modd[i0 + ii];
    }
    u += (size_t)bz * 2 * nt * c.N;
    conv += (size_t)bz * 2 * level * c.N;
    double y[KK];
#pragma unroll
    for (uint32_t a = 0; a < KK; a++) {
        y[a] = 0.0;
        if (a < c.K) {
            const u64 pa = c.mod[c.L + a];
            u64 v = u[((size_t)comp * nt + level + a) * c.N + k];
            if (!PRE) {
                const ulonglong2 hinv = c.dn_hat_inv[a];
                v = mul_shoup(v, hinv.x, hinv.y, pa);
            }
            y[a] = v > (pa >> 1) ? __dsub_rn(u64_to_d(v), (double)pa) : u64_to_d(v);
        }
    }
    __syncthreads();
    u64 *dst = conv + ((size_t)comp * level + i0) * c.N + k;
    for (uint32_t i = i0; i < i1; i++, dst += c.N) {
        const double2 md = s_m[i - i0];
        const double q = md.x, qinv = md.y;
        double acc = 0.0;
#pragma unroll
        for (uint32_t a = 0; a < KK; a++) {
            acc = __dadd_rn(acc, mulmod_d<0>(y[a], s_w[i - i0][a], q));
            if ((a & 7) == 7 && a + 1 < KK) acc = reduce_d(acc, q, qinv);
        }
        *dst = canonical_d(reduce_d(acc, q, qinv), q);
    }
}

template <uint32_t KK>
void launch_moddown_conv(const ckks_ctx *c, const u64 *u, u64 *conv, uint32_t level, uint32_t nb, cudaStream_t s, bool pre) {
    const uint32_t CHUNK = conv_chunk(nb);
    const dim3 grid(c->N / THREADS, (level + CHUNK - 1) / CHUNK, 2 * nb);
    if (pre) moddown_conv_kernel<KK, true><<<grid, THREADS, 0, s>>>(c->dev, u, conv, level, CHUNK);
    else moddown_conv_kernel<KK, false><<<grid, THREADS, 0, s>>>(c->dev, u, conv, level, CHUNK);
    count_launches();
}

// register-array size for a digit / special-prime count: next of 1, 2, 4, 8, 16, 32, 64
#define DISPATCH_POW2(n, CALL)                      \
    do {                                            \
        if ((n) <= 1) { CALL(1); }                  \
        else if ((n) <= 2) { CALL(2); }             \
        else if ((n) <= 4) { CALL(4); }             \
        else if ((n) <= 8) { CALL(8); }             \
        else if ((n) <= 16) { CALL(16); }           \
        else if ((n) <= 32) { CALL(32); }           \
        else { CALL(64); }                          \
    } while (0)

// out[b][comp][i][p] (+)= (u[b][comp][i][p] - conv[b][comp][i][p]) P^-1 + add_comp[b][i][pi_g(p)]
__global__ void __launch_bounds__(THREADS) moddown_final_kernel(DevTables c, const u64 *u, const u64 *conv, const u64 *add0,
                                                                const u64 *add1, size_t add_stride, u64 g, u64 *out,
                                                                size_t out_stride, int accumulate, uint32_t level, TiledOut tl) {
    const uint32_t p = blockIdx.x * THREADS + threadIdx.x;
    const uint32_t i = blockIdx.y, comp = blockIdx.z & 1, bz = blockIdx.z >> 1;
    const uint32_t nt = level + c.K;
    const u64 q = c.mod[i];
    const ulonglong2 pinv = c.dn_p_inv[i];
    u64 r = sub_mod(u[(((size_t)bz * 2 + comp) * nt + i) * c.N + p], conv[(((size_t)bz * 2 + comp) * level + i) * c.N + p], q);
    r = mul_shoup(r, pinv.x, pinv.y, q);
    const u64 *add = comp ? add1 : add0;
    if (add) r = add_mod(r, add[bz * add_stride + (size_t)i * c.N + galois_src(p, g, c.log_n, c.N)], q);
    u64 *dst = tl.R ? out + tiled_index(tl.R, c.N, tl.row0 + bz * tl.row_stride + comp, i, p)
                    : out + bz * out_stride + ((size_t)comp * level + i) * c.N + p;
    if (accumulate) r = add_mod(r, *dst, q);
    *dst = r;
}

// dst row (row0 + r * row_step) of a tiled buffer <- src + r * src_stride ([level][N] words)
__global__ void __launch_bounds__(THREADS) to_tiled_kernel(DevTables c, const u64 *src, size_t src_stride, u64 *dst, uint32_t R,
                                                           uint32_t row0, uint32_t row_step) {
    const uint32_t p = (blockIdx.x * THREADS + threadIdx.x) * 2, i = blockIdx.y, r = blockIdx.z;
    const ulonglong2 v = *reinterpret_cast<const ulonglong2 *>(src + r * src_stride + (size_t)i * c.N + p);
    *reinterpret_cast<ulonglong2 *>(dst + tiled_index(R, c.N, row0 + r * row_step, i, p)) = v;
}

// tmp[comp][i][k] = centred lift of last[comp][k] (mod q_last) taken mod q_i
__global__ void __launch_bounds__(THREADS) rescale_lift_kernel(DevTables c, const u64 *last, u64 *tmp, uint32_t level) {
    const uint32_t k = blockIdx.x * THREADS + threadIdx.x;
    const uint32_t i = blockIdx.y, comp = blockIdx.z;
    tmp[((size_t)comp * (level - 1) + i) * c.N + k] = centred_to(last[(size_t)comp * c.N + k], c.mod[level - 1], c.mod[i]);
}

// out[comp][i][p] = (in[comp][i][p] - tmp[comp][i][p]) q_last^-1
__global__ void __launch_bounds__(THREADS) rescale_final_kernel(DevTables c, const u64 *in, const u64 *tmp, u64 *out, uint32_t level) {
    const uint32_t p = blockIdx.x * THREADS + threadIdx.x;
    const uint32_t i = blockIdx.y, comp = blockIdx.z;
    const u64 q = c.mod[i];
    const ulonglong2 inv = c.rs_inv[(size_t)(level - 1) * c.L + i];
    const u64 r = sub_mod(in[((size_t)comp * level + i) * c.N + p], tmp[((size_t)comp * (level - 1) + i) * c.N + p], q);
    out[((size_t)comp * (level - 1) + i) * c.N + p] = mul_shoup(r, inv.x, inv.y, q);
}

// u[b][0][i][p] += P sigma_g(c0[b][i])[p]   (first component's q-limbs of the extended-basis sum)
__global__ void __launch_bounds__(THREADS) p_c0_acc_kernel(DevTables c, const u64 *c0, size_t c0_stride, u64 g, u64 *u, size_t u_stride) {
    const uint32_t p = blockIdx.x * THREADS + threadIdx.x, i = blockIdx.y, b = blockIdx.z;
    const double2 md = c.modd[i];
    u64 *d = u + b * u_stride + (size_t)i * c.N + p;
    const double v = mulmod_dd(u64_to_d(c0[b * c0_stride + (size_t)i * c.N + galois_src(p, g, c.log_n, c.N)]), c.dn_p_mod_d[i], md.x, md.y);
    *d = add_mod(*d, canonical_d(reduce_d(v, md.x, md.y), md.x), c.mod[i]);
}

}  // namespace

size_t ks_workspace_limbs(const ckks_ctx *c, uint32_t level) {
    const size_t beta = (level + c->alpha - 1) / c->alpha, nt = level + c->K;
    return level + beta * nt + 2 * nt + 2 * (size_t)level;
}

// Workspace for nb key switches running side by side: dcoef [nb][level], ext [nb][beta][level+K],
// u [nb][2][level+K], conv [nb][2][level].
KsWorkspace ks_carve(const ckks_ctx *c, uint32_t level, void *ws, uint32_t nb) {
    const size_t beta = (level + c->alpha - 1) / c->alpha, nt = level + c->K, N = c->N;
    KsWorkspace w;
    w.dcoef = (u64 *)ws;
    w.ext = w.dcoef + (size_t)nb * level * N;
    w.u = w.ext + (size_t)nb * beta * nt * N;
    w.conv = w.u + (size_t)nb * 2 * nt * N;
    return w;
}

void ks_modup(const ckks_ctx *c, const u64 *d, uint32_t level, const KsWorkspace &w, cudaStream_t s, uint32_t nb, size_t d_stride) {
    const uint32_t N = c->N, beta = (level + c->alpha - 1) / c->alpha, nt = level + c->K;
    // N = 2^16 with the FP64 transform and conversion: the inverse transform's last stage multiplies qhat^-1 in
    const bool pre = c->log_n == 16 && c->ntt_fp_share >= 8 && c->conv_kernel != CKKS_CONV_TENSOR;
    if (c->log_n == 16) {      // the inverse transform reads d and writes the coefficient copy
        launch_ntt(c, w.dcoef, nb * level, plain_map(0, level), true, s, nullptr, nullptr, d, (uint32_t)(d_stride / N),
                   pre ? c->dev.inv_scale_up + (size_t)level * c->L * 2 : nullptr);
    } else {
        permute_kernel<<<dim3(N / THREADS, level, nb), THREADS, 0, s>>>(c->dev, d, d_stride, w.dcoef, (size_t)level * N, 1); count_launches();
        launch_ntt(c, w.dcoef, nb * level, plain_map(0, level), true, s);
    }
    // the context option CKKS_CONV_TENSOR takes the tensor-core conversion of conv_mma.cu: bit-identical, 2 % slower on B200
    if (c->conv_kernel != CKKS_CONV_TENSOR || !launch_modup_mma(c, w.dcoef, d, d_stride, w.ext, level, nb, s)) {
#define CALL_UP(A) launch_modup<A>(c, w.dcoef, d, d_stride, 1, w.ext, level, nb, s, pre)
        DISPATCH_POW2(c->alpha, CALL_UP);
#undef CALL_UP
    }
    launch_ntt(c, w.ext, nb * beta * nt, ext_map(level, c->K, c->L, c->alpha, beta), false, s);
}

void ks_inner(const ckks_ctx *c, const u64 *evk, uint32_t level, u64 ext_galois, const KsWorkspace &w, cudaStream_t s, uint32_t nb,
              bool acc_u, const KsMulti *multi) {
    const uint32_t N = c->N, nt = level + c->K;
    const uint32_t beta = (level + c->alpha - 1) / c->alpha;
    const int au = acc_u ? 1 : 0;
    bool aligned = ((uintptr_t)w.ext & 15) == 0 && ((uintptr_t)w.u & 15) == 0 && (multi || ((uintptr_t)evk & 15) == 0);
    const uint32_t nkeys = multi ? (multi->group ? nb / multi->group : nb) : 0;
    for (uint32_t b = 0; b < nkeys; b++) aligned = aligned && ((uintptr_t)multi->evk[b] & 15) == 0;
    const bool fast = beta <= IP_MAX_BETA && N >= 2 * THREADS && aligned;
    if (multi && multi->group && !fast) {       // grouped entries without the fast kernel: one key at a time
        for (uint32_t r = 0; r < nkeys; r++) {
            KsWorkspace wr = w;
            wr.u = w.u + (size_t)r * multi->group * 2 * nt * N;
            ks_inner(c, multi->evk[r], level, multi->galois[r], wr, s, multi->group, acc_u, nullptr);
        }
        return;
    }
    if (fast) {
        // batch entries per thread: enough chunks left to fill the machine, key words reused across a chunk
        const uint32_t grp = multi ? multi->group : 0, per = grp ? grp : nb;
        const uint32_t bch = (multi && !grp) ? 1 : (per >= 8 ? 4 : (per >= 4 ? 2 : 1));
        const dim3 grid(N / (2 * THREADS), grp ? (nb / grp) * ((grp + bch - 1) / bch) : (nb + bch - 1) / bch, nt);
        const KsMulti m = multi ? *multi : KsMulti{};
        switch (beta) {
        case 1: inner_product_kernel<1><<<grid, THREADS, 0, s>>>(c->dev, w.ext, evk, ext_galois, w.u, level, nb, bch, multi ? 1 : 0, m, au); break;
        case 2: inner_product_kernel<2><<<grid, THREADS, 0, s>>>(c->dev, w.ext, evk, ext_galois, w.u, level, nb, bch, multi ? 1 : 0, m, au); break;
        case 3: inner_product_kernel<3><<<grid, THREADS, 0, s>>>(c->dev, w.ext, evk, ext_galois, w.u, level, nb, bch, multi ? 1 : 0, m, au); break;
        default: inner_product_kernel<4><<<grid, THREADS, 0, s>>>(c->dev, w.ext, evk, ext_galois, w.u, level, nb, bch, multi ? 1 : 0, m, au); break;
        }
    } else {
        inner_product_generic_kernel<<<dim3(N / THREADS, nb, nt), THREADS, 0, s>>>(c->dev, w.ext, evk, ext_galois, w.u, level, multi ? 1 : 0,
                                                                                     multi ? *multi : KsMulti{}, au);
    }
    count_launches();
}

void ks_moddown(const ckks_ctx *c, uint32_t level, const KsWorkspace &w, const u64 *add0, const u64 *add1, u64 add_galois, u64 *out,
                cudaStream_t s, uint32_t nb, size_t add_stride, size_t out_stride, bool accumulate, TiledOut tiled, const KsMulti *multi) {
    const uint32_t N = c->N, nt = level + c->K, K = c->K;
    // the K special limbs of every (batch, component): groups of K limbs, nt limbs apart; at N = 2^16 the inverse
    // transform's last stage multiplies Phat^-1 in
    const bool pre = c->log_n == 16 && c->ntt_fp_share >= 8 && c->conv_kernel != CKKS_CONV_TENSOR;
    launch_ntt(c, w.u + (size_t)level * N, nb * 2 * K, pitched_map(c->L, K, nt), true, s, nullptr, nullptr, nullptr, 0,
               pre ? c->dev.inv_scale_dn : nullptr);
    if (c->conv_kernel != CKKS_CONV_TENSOR || !launch_moddown_conv_mma(c, w.u, w.conv, level, nb, s)) {
#define CALL_DN(A) launch_moddown_conv<A>(c, w.u, w.conv, level, nb, s, pre)
        DISPATCH_POW2(K, CALL_DN);
#undef CALL_DN
    }
    if (c->log_n == 16) {      // the last NTT pass finishes the ModDown itself
        NttEpilogue ep{1, w.u, add0, add1, out, add_stride, out_stride, add_galois, level, nt, accumulate ? 1 : 0, tiled};
        ep.multi = multi ? 1 : 0;
        ep.group = multi ? multi->group : 0;
        ep.rot_rows = multi ? multi->rot_rows : 0;
        if (multi)
            for (uint32_t b = 0; b < KS_MULTI; b++) { ep.mgalois[b] = multi->galois[b]; ep.mout[b] = multi->out[b]; }
        launch_ntt(c, w.conv, nb * 2 * level, plain_map(0, level), false, s, &ep);
        return;
    }
    launch_ntt(c, w.conv, nb * 2 * level, plain_map(0, level), false, s);
    if (multi) {
        for (uint32_t b = 0; b < nb; b++) {
            moddown_final_kernel<<<dim3(N / THREADS, level, 2), THREADS, 0, s>>>(c->dev, w.u + (size_t)b * 2 * nt * N, w.conv + (size_t)b * 2 * level * N,
                                                                                  add0, add1, 0, multi->galois[b], multi->out[b], 0, 0, level, TiledOut());
            count_launches();
        }
        return;
    }
    moddown_final_kernel<<<dim3(N / THREADS, level, 2 * nb), THREADS, 0, s>>>(c->dev, w.u, w.conv, add0, add1, add_stride, add_galois, out,
                                                                               out_stride, accumulate ? 1 : 0, level, tiled);
    count_launches();
}

void ks_inner_moddown(const ckks_ctx *c, const u64 *evk, uint32_t level, u64 ext_galois, const KsWorkspace &w,
                      const u64 *add0, const u64 *add1, u64 add_galois, u64 *out, cudaStream_t s, uint32_t nb,
                      size_t add_stride, size_t out_stride, bool accumulate, TiledOut tiled, const KsMulti *multi) {
    ks_inner(c, evk, level, ext_galois, w, s, nb, false, multi);
    ks_moddown(c, level, w, add0, add1, add_galois, out, s, nb, add_stride, out_stride, accumulate, tiled, multi);
}

void ks_inner_terms(const ckks_ctx *c, uint32_t level, const KsWorkspace &w, size_t term_stride, const IpTerms &terms, uint32_t nterm,
                    size_t c0_stride, cudaStream_t s, uint32_t nb, bool acc_u) {
    const uint32_t N = c->N, nt = level + c->K, beta = (level + c->alpha - 1) / c->alpha;
    bool aligned = ((uintptr_t)w.ext & 15) == 0 && ((uintptr_t)w.u & 15) == 0 && (term_stride & 1) == 0 && (c0_stride & 1) == 0;
    for (uint32_t t = 0; t < nterm; t++) aligned = aligned && ((uintptr_t)terms.evk[t] & 15) == 0 && ((uintptr_t)terms.c0[t] & 15) == 0;
    if (beta <= IP_MAX_BETA && N >= 2 * THREADS && aligned) {
        const dim3 grid(N / (2 * THREADS), (nb + IP_BCH - 1) / IP_BCH, nt);
        const int au = acc_u ? 1 : 0;
        switch (beta) {
        case 1: inner_product_terms_kernel<1><<<grid, THREADS, 0, s>>>(c->dev, w.ext, term_stride, terms, nterm, c0_stride, w.u, level, nb, au); break;
        case 2: inner_product_terms_kernel<2><<<grid, THREADS, 0, s>>>(c->dev, w.ext, term_stride, terms, nterm, c0_stride, w.u, level, nb, au); break;
        case 3: inner_product_terms_kernel<3><<<grid, THREADS, 0, s>>>(c->dev, w.ext, term_stride, terms, nterm, c0_stride, w.u, level, nb, au); break;
        default: inner_product_terms_kernel<4><<<grid, THREADS, 0, s>>>(c->dev, w.ext, term_stride, terms, nterm, c0_stride, w.u, level, nb, au); break;
        }
        count_launches();
        return;
    }
    // any number of digits, any alignment: one term at a time through the generic kernel, then its P c0
    for (uint32_t t = 0; t < nterm; t++) {
        inner_product_generic_kernel<<<dim3(N / THREADS, nb, nt), THREADS, 0, s>>>(c->dev, w.ext + t * term_stride, terms.evk[t], terms.galois[t],
                                                                                     w.u, level, 0, KsMulti{}, (acc_u || t > 0) ? 1 : 0);
        count_launches();
        if (terms.c0[t]) {
            p_c0_acc_kernel<<<dim3(N / THREADS, level, nb), THREADS, 0, s>>>(c->dev, terms.c0[t], c0_stride, terms.galois[t], w.u, (size_t)2 * nt * N);
            count_launches();
        }
    }
}

void launch_to_tiled(const ckks_ctx *c, const u64 *src, size_t src_stride, uint32_t nrows, u64 *dst, uint32_t R, uint32_t row0,
                     uint32_t row_step, uint32_t level, cudaStream_t s) {
    for (uint32_t r0 = 0; r0 < nrows; r0 += 32768) {
        const uint32_t nr = nrows - r0 < 32768 ? nrows - r0 : 32768;
        to_tiled_kernel<<<dim3(c->N / (2 * THREADS), level, nr), THREADS, 0, s>>>(c->dev, src + r0 * src_stride, src_stride, dst, R,
                                                                                   row0 + r0 * row_step, row_step);
        count_launches();
    }
}

// ws: [ncomp][N] last limbs + [ncomp][level-1][N]
void launch_rescale(const ckks_ctx *c, const u64 *in, u64 *out, uint32_t ncomp, uint32_t level, u64 *ws, cudaStream_t s) {
    const uint32_t N = c->N;
    u64 *last = ws, *tmp = ws + (size_t)ncomp * N;
    for (uint32_t comp = 0; comp < ncomp; comp++)
        cudaMemcpyAsync(last + (size_t)comp * N, in + ((size_t)comp * level + level - 1) * N, (size_t)N * 8,
                        cudaMemcpyDeviceToDevice, s);
    launch_ntt(c, last, ncomp, plain_map(level - 1, 1), true, s);
    rescale_lift_kernel<<<dim3(N / THREADS, level - 1, ncomp), THREADS, 0, s>>>(c->dev, last, tmp, level); count_launches();
    launch_ntt(c, tmp, ncomp * (level - 1), plain_map(0, level - 1), false, s);
    rescale_final_kernel<<<dim3(N / THREADS, level - 1, ncomp), THREADS, 0, s>>>(c->dev, in, tmp, out, level); count_launches();
}

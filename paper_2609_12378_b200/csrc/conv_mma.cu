// Basis conversion (the matrix product inside ModUp and ModDown) on the tensor cores.
//
// For every coefficient the conversion is  out[x] = sum_a centre(v_a) C[a][x]  mod t_x  with v_a = [d_a qhat_a^-1]_{q_a}
// (at most 8 sources a, 24 targets x) and a constant matrix C that is the same for all 2^16 coefficients: a dense
// contraction.  The 50-bit words are taken as 7 bytes: row k = 8 a + b of the k-dimension is byte b of v_a, byte 7
// carrying the flag "v_a > q_a / 2", and column (x, d) of the constant byte matrix collects what has weight 2^(8 d)
// (byte d - b of C[a][x]; for the flag byte d of (-q_a C[a][x]) mod t_x, which turns v_a into its centred
// representative).  mma.m16n8k32 (u8 x u8 -> s32) over k = 64 then leaves, for 16 coefficients x 8 targets, the 13
// diagonal sums D_d < 2^22 in the registers of one thread each, and
//     sum_d D_d 2^(8 d) = sum_a v_a C[a][x] + flags   (< 2^103)
// is put together with shifts, split at bit 52 and reduced on the FP64 pipe.  Every output is the canonical residue,
// so the results are bit-identical to the FP64 kernels of keyswitch.cu.  The constant matrices are built at context
// creation in the B-fragment order (context.cu).
//
// Status: opt-in (CKKS_CONV=mma).  On B200 it is no faster than the FP64 kernels (ModDown conversion of 16 entries:
// 297 us against 258-290 us; 4096 x 4096 projection 299 ms against 293 ms): putting the 13 sums together and reducing
// them costs about 50 instructions per output, the kernel issues on 45 % of its cycles with 16 warps per SM (122
// registers), and the tensor, FP64 and integer pipes each stay below 30 %.
#include "common.cuh"

namespace {

constexpr uint32_t CM_THREADS = 256, CM_TILES = 8;      // a CTA converts CM_TILES x 128 coefficients of one item
constexpr uint32_t CM_DIAG = 13, CM_GWORDS = CM_DIAG * 2 * 64;

__device__ __forceinline__ void mma_u8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// sum_q E_q 2^(16 q), q < 7, E_q < 2^31, as four 32-bit words (the value stays below 2^103)
__device__ __forceinline__ void assemble7(const uint32_t (&E)[7], uint32_t &w0, uint32_t &w1, uint32_t &w2, uint32_t &w3) {
    asm("{\n"
        ".reg .u32 a1, b1, t1, a3, b3, t2, a5, b5, t3;\n"
        "shl.b32 a1, %5, 16;\n"
        "shr.u32 b1, %5, 16;\n"
        "add.u32 t1, b1, %6;\n"
        "shl.b32 a3, %7, 16;\n"
        "shr.u32 b3, %7, 16;\n"
        "add.u32 t2, b3, %8;\n"
        "shl.b32 a5, %9, 16;\n"
        "shr.u32 b5, %9, 16;\n"
        "add.u32 t3, b5, %10;\n"
        "add.cc.u32 %0, %4, a1;\n"
        "addc.cc.u32 %1, t1, a3;\n"
        "addc.cc.u32 %2, t2, a5;\n"
        "addc.u32 %3, t3, 0;\n"
        "}\n"
        : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3)
        : "r"(E[0]), "r"(E[1]), "r"(E[2]), "r"(E[3]), "r"(E[4]), "r"(E[5]), "r"(E[6]));
}

// MODE 0: ModUp.   item = (batch b, digit j); sources dcoef[b][lo + a]; targets the limbs of ext[b][j] outside the digit.
// MODE 1: ModDown. item = (batch b, component); sources the special limbs of u; targets conv[b][comp][0 .. level).
template <int MODE>
__global__ void __launch_bounds__(CM_THREADS, 2) conv_mma_kernel(DevTables c, const u64 *src, const u64 *deval, size_t deval_stride, u64 *dst,
                                                                 uint32_t level) {
    extern __shared__ __align__(16) uint32_t bs[];
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const uint32_t nt = level + c.K, N = c.N;
    uint32_t nsrc, ntgt, lo = 0, nd = 0, qbase;
    const u64 *sbase;
    u64 *dbase;
    const uint32_t *bm;
    const ulonglong2 *hinv;
    if (MODE == 0) {
        const uint32_t beta = (level + c.alpha - 1) / c.alpha, b = blockIdx.z / beta, j = blockIdx.z % beta;
        lo = j * c.alpha;
        nd = min(lo + c.alpha, level) - lo;
        nsrc = nd; ntgt = nt - nd; qbase = lo;
        sbase = src + ((size_t)b * level + lo) * N;
        dbase = dst + (size_t)(b * beta + j) * nt * N;
        bm = c.up_bmat + ((size_t)level * c.dnum + j) * c.conv_groups * CM_GWORDS;
        hinv = c.up_hat_inv + ((size_t)level * c.dnum + j) * c.alpha;
        deval += b * deval_stride;
    } else {
        nsrc = c.K; ntgt = level; qbase = c.L;
        sbase = src + ((size_t)blockIdx.z * nt + level) * N;
        dbase = dst + (size_t)blockIdx.z * level * N;
        bm = c.dn_bmat;
        hinv = c.dn_hat_inv;
    }
    const uint32_t ngroups = (ntgt + 7) / 8;
    // the byte matrix and the targets' constants
    double2 *tm = reinterpret_cast<double2 *>(bs + ngroups * CM_GWORDS);       // {t, 1 / t}
    double2 *tc = tm + ngroups * 8;                                            // {2^52 mod t, that / t}
    uint32_t *tlimb = reinterpret_cast<uint32_t *>(tc + ngroups * 8);          // destination limb, ~0 for padding
    for (uint32_t w = tid; w < ngroups * CM_GWORDS / 4; w += CM_THREADS)
        reinterpret_cast<uint4 *>(bs)[w] = reinterpret_cast<const uint4 *>(bm)[w];
    for (uint32_t x = tid; x < ngroups * 8; x += CM_THREADS) {
        if (x < ntgt) {
            const uint32_t xp = MODE == 0 ? (x < lo ? x : x + nd) : x;
            const uint32_t prime = MODE == 0 ? (xp < level ? xp : c.L + (xp - level)) : xp;
            tm[x] = c.modd[prime];
            tc[x] = c.two52_d[prime];
            tlimb[x] = xp;
        } else {
            tm[x] = make_double2(1.0, 1.0);
            tc[x] = make_double2(0.0, 0.0);
            tlimb[x] = 0xffffffffu;
        }
    }
    const uint32_t kcta = blockIdx.x * (CM_TILES * 128);
    if (MODE == 0)      // the digit's own limbs are copied as they are (evaluation domain)
        for (uint32_t e = tid; e < nd * (CM_TILES * 128); e += CM_THREADS) {
            const uint32_t a = e / (CM_TILES * 128), k = kcta + e % (CM_TILES * 128);
            dbase[(size_t)(lo + a) * N + k] = deval[(size_t)(lo + a) * N + k];
        }
    __syncthreads();

    // this thread prepares the words of sources t and 4 + t for rows g and g + 8 of its warp's 16 coefficients
    u64 qa[2];
    ulonglong2 hv[2];
#pragma unroll
    for (uint32_t i = 0; i < 2; i++) {
        const uint32_t a = 4 * i + t;
        qa[i] = a < nsrc ? c.mod[qbase + a] : 0;
        hv[i] = a < nsrc ? hinv[a] : make_ulonglong2(0, 0);
    }
    const uint32_t src1 = (lane & ~3u) | (t >> 1), src2 = src1 + 2;
    const bool hi_half = t & 1;
    const uint2 *bs2 = reinterpret_cast<const uint2 *>(bs);

    // the source words of a tile are fetched while the tile before it is converted
    u64 nxt[2][2];
#pragma unroll
    for (uint32_t i = 0; i < 2; i++)
#pragma unroll
        for (uint32_t r = 0; r < 2; r++) nxt[i][r] = qa[i] ? sbase[(size_t)(4 * i + t) * N + kcta + warp * 16 + g + 8 * r] : 0;
    for (uint32_t tile = 0; tile < CM_TILES; tile++) {
        const uint32_t k0 = kcta + tile * 128 + warp * 16;
        uint32_t wlo[2][2], whi[2][2];
#pragma unroll
        for (uint32_t i = 0; i < 2; i++)
#pragma unroll
            for (uint32_t r = 0; r < 2; r++) {
                u64 wd = 0;
                if (qa[i]) {
                    const u64 v = mul_shoup(nxt[i][r], hv[i].x, hv[i].y, qa[i]);
                    wd = v | ((u64)(v > (qa[i] >> 1)) << 56);
                    if (tile + 1 < CM_TILES) nxt[i][r] = sbase[(size_t)(4 * i + t) * N + k0 + 128 + g + 8 * r];
                }
                wlo[i][r] = (uint32_t)wd;
                whi[i][r] = (uint32_t)(wd >> 32);
            }
        // A fragments: a0/a1 = rows g, g + 8 at k-bytes 4t .. 4t + 3 (word t / 2 of the k-step, half t % 2), a2/a3 the
        // same 16 bytes further (word 2 + t / 2); the words live in the lanes of this quad
        uint32_t afr[2][4];
#pragma unroll
        for (uint32_t ks = 0; ks < 2; ks++)
#pragma unroll
            for (uint32_t r = 0; r < 2; r++) {
                const uint32_t l1 = __shfl_sync(0xffffffffu, wlo[ks][r], src1), h1 = __shfl_sync(0xffffffffu, whi[ks][r], src1);
                const uint32_t l2 = __shfl_sync(0xffffffffu, wlo[ks][r], src2), h2 = __shfl_sync(0xffffffffu, whi[ks][r], src2);
                afr[ks][r] = hi_half ? h1 : l1;
                afr[ks][2 + r] = hi_half ? h2 : l2;
            }
        for (uint32_t gr = 0; gr < ngroups; gr++) {
            int acc[CM_DIAG][4];
#pragma unroll
            for (uint32_t d = 0; d < CM_DIAG; d++) acc[d][0] = acc[d][1] = acc[d][2] = acc[d][3] = 0;
#pragma unroll
            for (uint32_t d = 0; d < CM_DIAG; d++)
#pragma unroll
                for (uint32_t ks = 0; ks < 2; ks++) {
                    const uint2 bw = bs2[((gr * CM_DIAG + d) * 2 + ks) * 32 + lane];
                    mma_u8(acc[d], afr[ks], bw.x, bw.y);
                }
            // acc[d][o]: o & 1 = target 2t + (o & 1) of the group, o >> 1 = row g + 8 (o >> 1)
#pragma unroll
            for (uint32_t o = 0; o < 4; o++) {
                const uint32_t xi = gr * 8 + 2 * t + (o & 1);
                const uint32_t limb = tlimb[xi];
                const double2 md = tm[xi], c52 = tc[xi];
                uint32_t E[7];
#pragma unroll
                for (uint32_t q = 0; q < 6; q++) E[q] = (uint32_t)acc[2 * q][o] + ((uint32_t)acc[2 * q + 1][o] << 8);
                E[6] = (uint32_t)acc[12][o];
                uint32_t w0, w1, w2, w3;
                assemble7(E, w0, w1, w2, w3);
                // split at bit 52; both parts go into the mantissa of 2^52 (an integer below 2^52 each)
                const double dlo = __dsub_rn(__hiloint2double((int)((w1 & 0x000FFFFFu) | 0x43300000u), (int)w0), TWO52);
                const double dhi = __dsub_rn(__hiloint2double((int)(__funnelshift_r(w2, w3, 20) | 0x43300000u), (int)__funnelshift_r(w1, w2, 20)), TWO52);
                const double r = __dadd_rn(mulmod_d<0>(dhi, c52, md.x), reduce_d(dlo, md.x, md.y));
                const u64 res = canonical_d(reduce_d(r, md.x, md.y), md.x);
                if (limb != 0xffffffffu) dbase[(size_t)limb * N + k0 + g + 8 * (o >> 1)] = res;
            }
        }
    }
}

size_t conv_smem(uint32_t ngroups) { return (size_t)ngroups * (CM_GWORDS * 4 + 8 * (16 + 16 + 4)); }

}  // namespace

bool launch_modup_mma(const ckks_ctx *c, const u64 *dcoef, const u64 *deval, size_t deval_stride, u64 *ext, uint32_t level, uint32_t nb,
                      cudaStream_t s) {
    if (!c->dev.conv_groups || c->N % (CM_TILES * 128)) return false;
    const uint32_t beta = (level + c->alpha - 1) / c->alpha, nt = level + c->K;
    const size_t smem = conv_smem((nt + 7) / 8);
    if (cudaFuncSetAttribute(conv_mma_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
    conv_mma_kernel<0><<<dim3(c->N / (CM_TILES * 128), 1, beta * nb), CM_THREADS, smem, s>>>(c->dev, dcoef, deval, deval_stride, ext, level);
    count_launches();
    return true;
}

bool launch_moddown_conv_mma(const ckks_ctx *c, const u64 *u, u64 *conv, uint32_t level, uint32_t nb, cudaStream_t s) {
    if (!c->dev.conv_groups || c->N % (CM_TILES * 128)) return false;
    const size_t smem = conv_smem((level + 7) / 8);
    if (cudaFuncSetAttribute(conv_mma_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
    conv_mma_kernel<1><<<dim3(c->N / (CM_TILES * 128), 1, 2 * nb), CM_THREADS, smem, s>>>(c->dev, u, nullptr, 0, conv, level);
    count_launches();
    return true;
}

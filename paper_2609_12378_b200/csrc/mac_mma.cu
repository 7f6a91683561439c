// Tensor-core form of the projection's ciphertext x plaintext multiply-accumulate.
//
// For one coefficient (limb i, index p) a giant-step group's work is a small dense contraction
//   out[g][s'] = sum_j w[g][j] x[j][s']        g < 16 giant steps, s' = 2 shard + component, j < J,
// exact in integer tensor-core arithmetic after splitting every 50-bit word into 7 bytes: the byte
// products of equal weight a + b = d are summed over j by mma.m16n8k32 (u8 x u8 -> s32; J * 7 * 255^2 stays
// far below 2^31), which yields 13 diagonal sums D_d per output, and out = sum_d D_d 2^(8d) < 2^110 is
// reduced modulo the prime once.
//
// Mapping.  A warp owns one coefficient: M = 16 giants, N = 16 columns s' (two n-tiles), K = 32 values of j
// per step.  A CTA (8 warps) owns 8 adjacent coefficients, so a row of operands (one (g, j) or (s', j) pair) is
// 64 contiguous bytes; both operand arrays are in the tiled layout (all rows of a 64-coefficient block adjacent, see
// tiled_index), so the 1024 rows of a step are 512 bytes apart.  A row is fetched as four 16-byte cp.async.cg
// chunks into a 3-deep ring.  Rows are stored
// [g or s'][j][8 coefficients] with a pitch of 2112 bytes per g and the 16-byte chunks of a row XOR-swizzled
// by (j / 4) mod 4, which brings the fragment reads (same coefficient, rows gid and 4 tig + e) down to a
// two-way bank conflict.  CTAs are persistent and walk tiles (column tile fastest, then coefficient block,
// then limb), keeping the ring running across tile boundaries.  Rows beyond the group's giants or beyond the
// last column re-read row 0; their results are never stored.
#include "common.cuh"

namespace {

constexpr uint32_t COEF = 8, MG = 16, MS = 16, MK = 32, STAGES = 3;
constexpr uint32_t GPITCH = MK * 64 + 64;                 // bytes per g (or s') block of 32 rows
constexpr uint32_t BOX_BYTES = MG * GPITCH;               // one operand of one stage
constexpr uint32_t STAGE_BYTES = 2 * BOX_BYTES;
constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 128 /* alignment slack */;

__device__ __forceinline__ void cp_async16(void *smem, const void *gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int NLEFT>
__device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(NLEFT) : "memory"); }

// byte offset of (block a, row j, 16-byte chunk ch) inside an operand tile
__device__ __forceinline__ uint32_t tile_off(uint32_t a, uint32_t j, uint32_t ch) { return a * GPITCH + j * 64 + ((ch ^ ((j >> 2) & 3)) << 4); }

__device__ __forceinline__ void mma_u8(int (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
// byte PLANE of four words, packed lowest word first
template <uint32_t PLANE>
__device__ __forceinline__ uint32_t pack_plane(const u64 (&w)[4]) {
    constexpr uint32_t bsel = PLANE & 3;
    const uint32_t x0 = PLANE < 4 ? (uint32_t)w[0] : (uint32_t)(w[0] >> 32), x1 = PLANE < 4 ? (uint32_t)w[1] : (uint32_t)(w[1] >> 32);
    const uint32_t x2 = PLANE < 4 ? (uint32_t)w[2] : (uint32_t)(w[2] >> 32), x3 = PLANE < 4 ? (uint32_t)w[3] : (uint32_t)(w[3] >> 32);
    const uint32_t t0 = __byte_perm(x0, x1, bsel | ((4 + bsel) << 4)), t1 = __byte_perm(x2, x3, bsel | ((4 + bsel) << 4));
    return __byte_perm(t0, t1, 0x5410);
}
template <uint32_t NREG>
__device__ __forceinline__ void planes7(const u64 (&w)[NREG][4], uint32_t (&f)[7][NREG]) {
#pragma unroll
    for (uint32_t r = 0; r < NREG; r++) {
        f[0][r] = pack_plane<0>(w[r]); f[1][r] = pack_plane<1>(w[r]); f[2][r] = pack_plane<2>(w[r]); f[3][r] = pack_plane<3>(w[r]);
        f[4][r] = pack_plane<4>(w[r]); f[5][r] = pack_plane<5>(w[r]); f[6][r] = pack_plane<6>(w[r]);
    }
}
__device__ __forceinline__ u64 tile_word(const uint8_t *tile, uint32_t a, uint32_t j, uint32_t coef) {
    return *reinterpret_cast<const u64 *>(tile + tile_off(a, j, coef >> 1) + (coef & 1) * 8);
}

__global__ void __launch_bounds__(256, 1) mac_mma_kernel(DevTables c, const u64 *__restrict__ baby, const u64 *__restrict__ pts,
                                                         u64 *__restrict__ acc, uint32_t J, uint32_t S, uint32_t G, uint32_t level,
                                                         uint32_t ntiles) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *ring = reinterpret_cast<uint8_t *>(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, gid = lane >> 2, tig = lane & 3;
    const uint32_t ncol = 2 * S, coltiles = (ncol + MS - 1) / MS, gtiles = (G + MG - 1) / MG, ztiles = coltiles * gtiles;
    const uint32_t xblocks = c.N / COEF;
    const size_t lN = (size_t)level * c.N, ctl = 2 * lN;
    const uint32_t nk = J / MK;
    const uint32_t my_tiles = blockIdx.x < ntiles ? (ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const uint32_t nsteps = my_tiles * nk;

    struct Tile { uint32_t col0, g0, off, i, xb; };
    auto decode = [&](uint32_t t) {
        const uint32_t tile = blockIdx.x + t * gridDim.x;
        const uint32_t z = tile % ztiles, rest = tile / ztiles, xb = rest % xblocks, i = rest / xblocks;
        Tile r;
        r.col0 = (z % coltiles) * MS;
        r.g0 = (z / coltiles) * MG;
        r.off = i * c.N + xb * COEF;          // position inside the [level][N] plane, < 2^32
        r.i = i;
        r.xb = xb;
        return r;
    };
    // loader: a thread always fetches the 16-byte chunk ch = tid & 3 of row j = 32 ks + (tid >> 3) and walks
    // blocks a = (tid >> 2 & 1) + 2 it of W and of X, so every address is a base plus a constant stride
    const uint32_t ch = tid & 3, ah = (tid >> 2) & 1, jj = tid >> 3;
    const uint32_t Rw = G * J, Rx = 2 * S * J;
    auto issue = [&](uint32_t step) {
        if (step < nsteps) {
            const Tile tl = decode(step / nk);
            const uint32_t j = (step % nk) * MK + jj;
            uint8_t *st = ring + (size_t)(step % STAGES) * STAGE_BYTES;
            // tiled_index(R, N, r, i, p) = blk * R * 64 + r * 64 + p % 64, blk = i * N/64 + p/64
            const size_t blk = (size_t)tl.i * (c.N >> 6) + (tl.xb >> 3);
            const u64 *wb = pts + blk * Rw * 64 + (tl.xb & 7) * 8 + 2 * ch;
            const u64 *xb = baby + blk * Rx * 64 + (tl.xb & 7) * 8 + 2 * ch;
            const uint32_t gleft = G - tl.g0, cleft = ncol - tl.col0;      // valid giants / columns in this tile
#pragma unroll
            for (uint32_t it = 0; it < MG / 2; it++) {
                const uint32_t a = 2 * it + ah;
                cp_async16(st + tile_off(a, jj, ch), wb + (size_t)((a < gleft ? tl.g0 + a : 0) * J + j) * 64);
            }
#pragma unroll
            for (uint32_t it = 0; it < MS / 2; it++) {
                const uint32_t a = 2 * it + ah, col = a < cleft ? tl.col0 + a : 0;
                cp_async16(st + BOX_BYTES + tile_off(a, jj, ch), xb + (size_t)(((col >> 1) * J + j) * 2 + (col & 1)) * 64);
            }
        }
        cp_commit();
    };
#pragma unroll
    for (uint32_t s = 0; s < STAGES - 1; s++) issue(s);

    int dsum[2][13][4];
    for (uint32_t step = 0; step < nsteps; step++) {
        const uint32_t ks = step % nk, slot = step % STAGES;
        if (ks == 0) {
#pragma unroll
            for (uint32_t n = 0; n < 2; n++)
#pragma unroll
                for (uint32_t d = 0; d < 13; d++)
#pragma unroll
                    for (uint32_t r = 0; r < 4; r++) dsum[n][d][r] = 0;
        }
        cp_wait<STAGES - 2>();
        __syncthreads();                       // everyone's chunks of this step have landed; the previous step's slot is free
        issue(step + STAGES - 1);
        const uint8_t *Wt = ring + (size_t)slot * STAGE_BYTES, *Xt = Wt + BOX_BYTES;
        uint32_t A[7][4];
        {
            u64 w[4][4];                       // fragment register r + 2h: row g = gid + 8r, j = 16h + 4 tig + e
#pragma unroll
            for (uint32_t r = 0; r < 2; r++)
#pragma unroll
                for (uint32_t h = 0; h < 2; h++)
#pragma unroll
                    for (uint32_t e = 0; e < 4; e++) w[r + 2 * h][e] = tile_word(Wt, gid + 8 * r, 16 * h + 4 * tig + e, warp);
            planes7<4>(w, A);
        }
#pragma unroll
        for (uint32_t n = 0; n < 2; n++) {
            uint32_t Bf[7][2];
            {
                u64 x[2][4];                   // fragment register h: column 8n + gid, j = 16h + 4 tig + e
#pragma unroll
                for (uint32_t h = 0; h < 2; h++)
#pragma unroll
                    for (uint32_t e = 0; e < 4; e++) x[h][e] = tile_word(Xt, 8 * n + gid, 16 * h + 4 * tig + e, warp);
                planes7<2>(x, Bf);
            }
#pragma unroll
            for (uint32_t a = 0; a < 7; a++)
#pragma unroll
                for (uint32_t b = 0; b < 7; b++) mma_u8(dsum[n][a + b], A[a], Bf[b]);
        }
        if (ks == nk - 1) {
            const Tile tl = decode(step / nk);
            const uint32_t i = tl.off / c.N;
            const u64 q = c.mod[i], mu = c.mu[i];
#pragma unroll
            for (uint32_t n = 0; n < 2; n++)
#pragma unroll
                for (uint32_t r = 0; r < 4; r++) {
                    const uint32_t g = tl.g0 + gid + 8 * (r >> 1), col = tl.col0 + 8 * n + 2 * tig + (r & 1);
                    u128 t = 0;
#pragma unroll
                    for (uint32_t d = 0; d < 13; d++) t += (u128)(uint32_t)dsum[n][d][r] << (8 * d);
                    if (g < G && col < ncol)
                        acc[((size_t)g * S + (col >> 1)) * ctl + (col & 1) * lN + tl.off + warp] = barrett112((u64)(t >> 64), (u64)t, q, mu);
                }
        }
    }
    cp_wait<0>();
}

}  // namespace

bool mac_mma_supported(const ckks_ctx *c, uint32_t J) { return J % MK == 0 && J > 0 && c->N % COEF == 0; }

// acc[g][s][c][i][p] = sum_{j < J} baby[s][j][c][i][p] * pts[g][j][i][p] with baby and pts in the tiled layout
// (rows (s J + j) 2 + c and g J + j); acc in the plain layout.  Returns false if nothing was launched.
bool launch_mac_mma(const ckks_ctx *c, const u64 *baby, const u64 *pts, u64 *acc, uint32_t J, uint32_t S, uint32_t G, uint32_t level,
                    cudaStream_t s) {
    if (!mac_mma_supported(c, J)) return false;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(mac_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES) != cudaSuccess) return false;
        attr_set = true;
    }
    const uint32_t coltiles = (2 * S + MS - 1) / MS, gt = (G + MG - 1) / MG;
    const uint32_t ntiles = (c->N / COEF) * level * coltiles * gt;
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
    mac_mma_kernel<<<ntiles < (uint32_t)sms ? ntiles : (uint32_t)sms, 256, SMEM_BYTES, s>>>(c->dev, baby, pts, acc, J, S, G, level, ntiles);
    count_launches();
    return true;
}

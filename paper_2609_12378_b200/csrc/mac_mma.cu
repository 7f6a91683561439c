// Tensor-core form of the projection's ciphertext x plaintext multiply-accumulate.
//
// For one coefficient (limb i, index p) a giant-step group's work is a small dense contraction
//   out[g][s'] = sum_j w[g][j] x[j][s']        g < 16 giant steps, s' = 2 shard + component, j < J,
// exact in integer tensor-core arithmetic after splitting every 50-bit word into 7 bytes: the byte
// products of equal weight a + b = d are summed over j by mma.m16n8k32 (u8 x u8 -> s32; J * 7 * 255^2 stays
// far below 2^31), which yields 13 diagonal sums D_d per output, and out = sum_d D_d 2^(8d) < 2^110 is
// reduced modulo the prime once.
//
// Mapping.  A tile is M = 16 giants x N = 16 columns s' x COEF adjacent coefficients, walked in steps of K = 32
// values of j.  A warp owns one coefficient of the tile (NW = 2: both 8-column halves, NW = 1: one half).  Both
// operand arrays are in the tiled layout (all rows of a 64-coefficient block adjacent, see tiled_index), so the 1024
// rows of a step are 512 bytes apart and a CTA takes COEF * 8 contiguous bytes of each.  A row is fetched as 16-byte
// cp.async.cg chunks into a 3-deep ring, issued a few at a time between the products of the step before.  Rows are
// stored [g or s'][j][COEF coefficients] with a padded pitch per g and the 16-byte chunks XOR-swizzled by
// (j / 4) mod 4, which keeps the fragment reads (same coefficient, rows gid and 4 tig + e) at the two wavefronts an
// 8-byte access needs.  A CTA walks a contiguous run of tiles (column tile fastest, then giant tile, then
// coefficient block, then limb), keeping the ring running across tile boundaries.  Finished tiles are staged in
// shared memory and written after the next barrier as whole COEF * 8-byte rows: stores of single words to 256
// rows that are megabytes apart were the most expensive part of the first version of this kernel.
#include "common.cuh"

namespace {

constexpr uint32_t MG = 16, MS = 16, MK = 32, STAGES = 3;

template <uint32_t COEF>
struct Geo {
    static constexpr uint32_t CH = COEF / 2;                        // 16-byte chunks per row
    static constexpr uint32_t ROW = COEF * 8;                       // bytes per row
    static constexpr uint32_t GPITCH = MK * ROW + (CH == 4 ? 64 : 16);   // bytes per g (or s') block of 32 rows
    static constexpr uint32_t BOX_BYTES = MG * GPITCH;              // one operand of one stage
    static constexpr uint32_t STAGE_BYTES = 2 * BOX_BYTES;
    static constexpr uint32_t OBUF_BYTES = MG * MS * COEF * 8;      // one tile of results, staged for whole-row stores
    static constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + OBUF_BYTES + 64 /* mbarriers */ + 128 /* alignment slack */;
    // byte offset of (block a, row j, 16-byte chunk ch) inside an operand tile
    static __device__ __forceinline__ uint32_t tile_off(uint32_t a, uint32_t j, uint32_t ch) {
        return a * GPITCH + (((j * CH + ch) ^ (((j >> 2) & 3) * (4 / CH))) << 4);
    }
    static __device__ __forceinline__ u64 tile_word(const uint8_t *tile, uint32_t a, uint32_t j, uint32_t coef) {
        return *reinterpret_cast<const u64 *>(tile + tile_off(a, j, coef >> 1) + (coef & 1) * 8);
    }
};

__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int NLEFT>
__device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(NLEFT) : "memory"); }

__device__ __forceinline__ void mma_u8(int (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
__device__ __forceinline__ u64 mad_wide(uint32_t a, uint32_t b, u64 c) {
    u64 d;
    asm("mad.wide.u32 %0, %1, %2, %3;\n" : "=l"(d) : "r"(a), "r"(b), "l"(c));
    return d;
}
// The seven byte planes of four words, each packed lowest word first: a 4 x 4 byte transpose of the low halves
// (8 permutes), 7 more for bytes 4, 5, 6 of the high halves.
__device__ __forceinline__ void planes7(const u64 (&w)[4], uint32_t (&f)[7]) {
    const uint32_t l0 = (uint32_t)w[0], l1 = (uint32_t)w[1], l2 = (uint32_t)w[2], l3 = (uint32_t)w[3];
    const uint32_t h0 = (uint32_t)(w[0] >> 32), h1 = (uint32_t)(w[1] >> 32), h2 = (uint32_t)(w[2] >> 32), h3 = (uint32_t)(w[3] >> 32);
    const uint32_t t0 = __byte_perm(l0, l1, 0x5140), t1 = __byte_perm(l2, l3, 0x5140);     // bytes 0, 1 of each word
    const uint32_t t2 = __byte_perm(l0, l1, 0x7362), t3 = __byte_perm(l2, l3, 0x7362);     // bytes 2, 3
    const uint32_t t4 = __byte_perm(h0, h1, 0x5140), t5 = __byte_perm(h2, h3, 0x5140);     // bytes 4, 5
    const uint32_t t6 = __byte_perm(h0, h1, 0x6262), t7 = __byte_perm(h2, h3, 0x6262);     // byte 6
    f[0] = __byte_perm(t0, t1, 0x5410); f[1] = __byte_perm(t0, t1, 0x7632);
    f[2] = __byte_perm(t2, t3, 0x5410); f[3] = __byte_perm(t2, t3, 0x7632);
    f[4] = __byte_perm(t4, t5, 0x5410); f[5] = __byte_perm(t4, t5, 0x7632);
    f[6] = __byte_perm(t6, t7, 0x5410);
}

// position of a CTA in its run of tiles: column tile fastest, then giant tile, then coefficient block, then limb
struct TileIt {
    uint32_t zc, zg, xb, i;
    __device__ __forceinline__ void init(uint32_t tile, uint32_t coltiles, uint32_t gtiles, uint32_t xblocks) {
        zc = tile % coltiles; tile /= coltiles;
        zg = tile % gtiles; tile /= gtiles;
        xb = tile % xblocks; i = tile / xblocks;
    }
    __device__ __forceinline__ void next(uint32_t coltiles, uint32_t gtiles, uint32_t xblocks) {
        if (++zc == coltiles) {
            zc = 0;
            if (++zg == gtiles) {
                zg = 0;
                if (++xb == xblocks) { xb = 0; i++; }
            }
        }
    }
};

template <uint32_t COEF, uint32_t NW>
__global__ void __launch_bounds__(COEF * 64 / NW, 8 / COEF) mac_mma_kernel(DevTables c, const u64 *__restrict__ baby,
                                                                           const u64 *__restrict__ pts, u64 *__restrict__ acc, uint32_t J,
                                                                           uint32_t S, uint32_t G, uint32_t level, uint32_t ntiles,
                                                                           uint32_t Jx, uint32_t j0, uint32_t accumulate) {
    using T = Geo<COEF>;
    constexpr uint32_t THREADS = COEF * 64 / NW, CH = T::CH;
    constexpr uint32_t AH = THREADS / (CH * MK);      // blocks a loaded side by side; a thread walks a = arow + AH it
    constexpr uint32_t NIT = MG / AH;                 // cp.async per operand per thread and step
    constexpr uint32_t XB64 = 64 / COEF;              // tiles per 64-coefficient block
    extern __shared__ uint8_t smem_raw[];
    uint8_t *ring = reinterpret_cast<uint8_t *>(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    u64 *obuf = reinterpret_cast<u64 *>(ring + STAGES * T::STAGE_BYTES);
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, gid = lane >> 2, tig = lane & 3;
    const uint32_t coef = NW == 2 ? warp : warp >> 1, n0 = NW == 2 ? 0 : (warp & 1);
    const uint32_t ncol = 2 * S, coltiles = (ncol + MS - 1) / MS, gtiles = (G + MG - 1) / MG;
    const uint32_t xblocks = c.N / COEF;
    const uint32_t nk = J / MK;
    // a CTA takes a contiguous run of tiles
    const uint32_t t_begin = (uint32_t)(((u64)ntiles * blockIdx.x) / gridDim.x), t_end = (uint32_t)(((u64)ntiles * (blockIdx.x + 1)) / gridDim.x);
    const uint32_t nsteps = (t_end - t_begin) * nk;

    // loader: a thread always fetches the 16-byte chunk ch of row jj of the step and walks blocks a = arow + AH it of
    // W and of X, so its shared-memory addresses are one base plus constants
    const uint32_t ch = tid % CH, jj = (tid / CH) % MK, arow = tid / (CH * MK);
    const uint32_t Rw = G * J, Rx = 2 * S * Jx;          // the baby buffer has Jx rows per shard and component; this launch uses rows j0 .. j0 + J - 1
    const uint32_t sm_thread = (uint32_t)__cvta_generic_to_shared(ring) + T::tile_off(arow, jj, ch);
    TileIt lt;                                    // tile of the step the loader issues next
    lt.init(t_begin, coltiles, gtiles, xblocks);
    uint32_t lks = 0, lstep = 0;
    const u64 *wrow = nullptr, *xrow = nullptr;   // row j of the step, giant 0 / shard 0, this thread's chunk
    uint32_t lg0 = 0, lsh0 = 0, lsm = 0;
    auto load_begin = [&]() {
        if (lstep < nsteps) {
            // tiled_index(R, N, r, i, p) = blk * R * 64 + r * 64 + p % 64, blk = i * N/64 + p/64
            const size_t blk = (size_t)lt.i * (c.N >> 6) + lt.xb / XB64;
            const uint32_t in_blk = (lt.xb % XB64) * COEF + 2 * ch, j = lks * MK + jj;
            wrow = pts + blk * Rw * 64 + in_blk + (size_t)j * 64;
            xrow = baby + blk * Rx * 64 + in_blk + (size_t)(2 * (j0 + j) + (arow & 1)) * 64;
            lg0 = lt.zg * MG + arow;
            lsh0 = lt.zc * (MS / 2) + (arow >> 1);
            lsm = sm_thread + (lstep % STAGES) * T::STAGE_BYTES;
        }
    };
    // rows beyond the last giant or shard re-read the last valid one; their results are never stored
    auto load_w = [&](uint32_t k) {
        if (lstep < nsteps) {
            const uint32_t g = min(lg0 + AH * k, G - 1);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(lsm + k * AH * T::GPITCH), "l"(wrow + (size_t)g * J * 64) : "memory");
        }
    };
    auto load_x = [&](uint32_t k) {
        if (lstep < nsteps) {
            const uint32_t sh = min(lsh0 + (AH / 2) * k, S - 1);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(lsm + T::BOX_BYTES + k * AH * T::GPITCH), "l"(xrow + (size_t)sh * Jx * 128)
                         : "memory");
        }
    };
    auto load_end = [&]() {
        cp_commit();
        lstep++;
        if (++lks == nk) { lks = 0; lt.next(coltiles, gtiles, xblocks); }
    };
#pragma unroll 1
    for (uint32_t s = 0; s < STAGES - 1; s++) {
        load_begin();
#pragma unroll
        for (uint32_t k = 0; k < NIT; k++) { load_w(k); load_x(k); }
        load_end();
    }

    TileIt ct;                                    // tile being computed
    ct.init(t_begin, coltiles, gtiles, xblocks);
    uint32_t ks = 0, slot = 0, qi = ct.i;
    u64 q = c.mod[qi], mu = c.mu[qi];
    int dsum[NW][13][4];
    // results of a finished tile wait in obuf[row = 16 g + col][coefficient ^ (g mod COEF)] and are written after the
    // next barrier, COEF lanes per row
    u64 *pend = nullptr;
    uint32_t pend_g0 = 0, pend_col0 = 0;
    u64 pend_q = 0;
    const size_t lN = (size_t)level * c.N;
    auto flush = [&]() {
#pragma unroll
        for (uint32_t k = 0; k < MG * MS * COEF / THREADS; k++) {
            const uint32_t row = k * (THREADS / COEF) + tid / COEF, sl = tid % COEF, gl = row >> 4, cl = row & 15;
            const uint32_t g = pend_g0 + gl, col = pend_col0 + cl;
            if (g < G && col < ncol) {
                u64 *dst = pend + ((size_t)g * ncol + col) * lN + (sl ^ (gl % COEF));
                const u64 v = obuf[row * COEF + sl];
                *dst = accumulate ? add_mod(v, *dst, pend_q) : v;
            }
        }
        pend = nullptr;
    };
#pragma unroll 1
    for (uint32_t step = 0; step < nsteps; step++) {
        if (ks == 0) {
#pragma unroll
            for (uint32_t n = 0; n < NW; n++)
#pragma unroll
                for (uint32_t d = 0; d < 13; d++)
#pragma unroll
                    for (uint32_t r = 0; r < 4; r++) dsum[n][d][r] = 0;
        }
        cp_wait<STAGES - 2>();
        __syncthreads();                       // everyone's chunks of this step have landed; the previous step's slot is free
        if (pend) flush();
        load_begin();
        const uint8_t *Wt = ring + (size_t)slot * T::STAGE_BYTES, *Xt = Wt + T::BOX_BYTES;
        uint32_t A[7][4];
#pragma unroll
        for (uint32_t r = 0; r < 2; r++)
#pragma unroll
            for (uint32_t h = 0; h < 2; h++) {
                u64 w[4];                      // fragment register r + 2h: row g = gid + 8r, j = 16h + 4 tig + e
                uint32_t f[7];
#pragma unroll
                for (uint32_t e = 0; e < 4; e++) w[e] = T::tile_word(Wt, gid + 8 * r, 16 * h + 4 * tig + e, coef);
                planes7(w, f);
#pragma unroll
                for (uint32_t pl = 0; pl < 7; pl++) A[pl][r + 2 * h] = f[pl];
            }
#pragma unroll
        for (uint32_t n = 0; n < NW; n++) {
            uint32_t Bf[7][2];
#pragma unroll
            for (uint32_t h = 0; h < 2; h++) {
                u64 x[4];                      // fragment register h: column 8n + gid, j = 16h + 4 tig + e
                uint32_t f[7];
#pragma unroll
                for (uint32_t e = 0; e < 4; e++) x[e] = T::tile_word(Xt, 8 * (n0 + n) + gid, 16 * h + 4 * tig + e, coef);
                planes7(x, f);
#pragma unroll
                for (uint32_t pl = 0; pl < 7; pl++) Bf[pl][h] = f[pl];
            }
#pragma unroll
            for (uint32_t a = 0; a < 7; a++) {
#pragma unroll
                for (uint32_t b = 0; b < 7; b++) mma_u8(dsum[n][a + b], A[a], Bf[b]);
                // the next-but-one step's loads go out a few at a time between the products
                constexpr uint32_t SLOTS = 7 * NW, NCP = 2 * NIT;
                const uint32_t sl = n * 7 + a;
#pragma unroll
                for (uint32_t k = 0; k < NCP; k++)
                    if (k * SLOTS / NCP == sl) {
                        if (k < NIT) load_w(k); else load_x(k - NIT);
                    }
            }
        }
        load_end();
        if (ks == nk - 1) {
            if (ct.i != qi) { qi = ct.i; q = c.mod[qi]; mu = c.mu[qi]; }
            if (nk == 1) __syncthreads();       // single-step tiles: the previous tile's rows were read after this step's barrier
#pragma unroll
            for (uint32_t n = 0; n < NW; n++)
#pragma unroll
                for (uint32_t r = 0; r < 4; r++) {
                    const uint32_t gl = gid + 8 * (r >> 1), cl = 8 * (n0 + n) + 2 * tig + (r & 1);
                    // sum_d D_d 2^(8d) as four 56-bit pieces of weights 1, 2^32, 2^64, 2^96
                    u64 e[3];
#pragma unroll
                    for (uint32_t k = 0; k < 3; k++) {
                        e[k] = mad_wide((uint32_t)dsum[n][4 * k + 1][r], 1u << 8, (u64)(uint32_t)dsum[n][4 * k][r]);
                        e[k] = mad_wide((uint32_t)dsum[n][4 * k + 2][r], 1u << 16, e[k]);
                        e[k] = mad_wide((uint32_t)dsum[n][4 * k + 3][r], 1u << 24, e[k]);
                    }
                    const u64 lo = e[0] + (e[1] << 32);
                    const u64 hi = (e[1] >> 32) + e[2] + ((u64)(uint32_t)dsum[n][12][r] << 32) + (lo < e[0]);
                    obuf[(gl * 16 + cl) * COEF + (coef ^ (gl % COEF))] = barrett112(hi, lo, q, mu);
                }
            pend_g0 = ct.zg * MG;
            pend_col0 = ct.zc * MS;
            pend_q = q;
            pend = acc + (size_t)ct.i * c.N + ct.xb * COEF;
        }
        if (++ks == nk) { ks = 0; ct.next(coltiles, gtiles, xblocks); }
        if (++slot == STAGES) slot = 0;
    }
    cp_wait<0>();
    __syncthreads();
    if (pend) flush();
}

// ---------------------------------------------------------------------------
// The same computation without CTA-wide barriers.  Each ring stage has a "full" mbarrier (every thread's cp.async
// arrive on it as they complete) and an "empty" one (a warp arrives when it has read its fragments), and the result
// staging buffer has the same pair, so warps drift up to a step apart: while one splits bytes or reduces results,
// another keeps the tensor pipe busy.  Every wait is bounded by the clock; on a timeout the kernel raises the
// context's sticky timeout flag and returns.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cp_async(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];\n" ::"r"(bar) : "memory");
}
// Bounded wait, called by all 32 lanes of a warp together; the answer is the warp's (every lane gets the same one, so
// a timeout never splits a warp in front of a warp-wide instruction).  limit: SM clock cycles.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, long long limit) {
    const long long t0 = clock64();
    uint32_t ok = 0;
    // a non-blocking test first (try_wait may itself sleep for a while, which would make a limit of zero meaningless)
    asm volatile("{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    while (!ok && clock64() - t0 < limit) {
        asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    }
    return __all_sync(0xffffffffu, ok != 0);
}

template <uint32_t COEF, uint32_t NW>
__global__ void __launch_bounds__(COEF * 64 / NW, 8 / COEF) mac_mma_async_kernel(DevTables c, const u64 *__restrict__ baby,
                                                                                 const u64 *__restrict__ pts, u64 *__restrict__ acc,
                                                                                 uint32_t J, uint32_t S, uint32_t G, uint32_t level,
                                                                                 uint32_t ntiles, uint32_t Jx, uint32_t j0, uint32_t accumulate,
                                                                                 long long wait_limit) {
    using T = Geo<COEF>;
    constexpr uint32_t THREADS = COEF * 64 / NW, CH = T::CH, NWARPS = THREADS / 32;
    constexpr uint32_t AH = THREADS / (CH * MK), NIT = MG / AH, XB64 = 64 / COEF;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *ring = reinterpret_cast<uint8_t *>(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    u64 *obuf = reinterpret_cast<u64 *>(ring + STAGES * T::STAGE_BYTES);
    // mbarriers behind the staging buffer: full[STAGES], empty[STAGES], results full, results empty
    const uint32_t bars = (uint32_t)__cvta_generic_to_shared(ring) + STAGES * T::STAGE_BYTES + T::OBUF_BYTES;
    const uint32_t bar_ofull = bars + 2 * STAGES * 8, bar_oempty = bar_ofull + 8;
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, gid = lane >> 2, tig = lane & 3;
    if (tid == 0) {
        for (uint32_t k = 0; k < STAGES; k++) { mbar_init(bars + 8 * k, THREADS); mbar_init(bars + 8 * (STAGES + k), NWARPS); }
        mbar_init(bar_ofull, NWARPS);
        mbar_init(bar_oempty, NWARPS);
    }
    __syncthreads();
    const uint32_t coef = NW == 2 ? warp : warp >> 1, n0 = NW == 2 ? 0 : (warp & 1);
    const uint32_t ncol = 2 * S, coltiles = (ncol + MS - 1) / MS, gtiles = (G + MG - 1) / MG;
    const uint32_t xblocks = c.N / COEF;
    const uint32_t nk = J / MK;
    const uint32_t t_begin = (uint32_t)(((u64)ntiles * blockIdx.x) / gridDim.x), t_end = (uint32_t)(((u64)ntiles * (blockIdx.x + 1)) / gridDim.x);
    const uint32_t nsteps = (t_end - t_begin) * nk;

    const uint32_t ch = tid % CH, jj = (tid / CH) % MK, arow = tid / (CH * MK);
    const uint32_t Rw = G * J, Rx = 2 * S * Jx;          // the baby buffer has Jx rows per shard and component; this launch uses rows j0 .. j0 + J - 1
    const uint32_t sm_thread = (uint32_t)__cvta_generic_to_shared(ring) + T::tile_off(arow, jj, ch);
    TileIt lt;
    lt.init(t_begin, coltiles, gtiles, xblocks);
    uint32_t lks = 0, lstep = 0, lslot = 0, luse = 0;      // luse: how many times the loader has wrapped the ring
    const u64 *wrow = nullptr, *xrow = nullptr;
    uint32_t lg0 = 0, lsh0 = 0, lsm = 0;
    bool alive = true;
    // addresses of the next step to load; waits until every warp has read the stage's previous contents
    auto load_begin = [&]() {
        if (lstep < nsteps) {
            const size_t blk = (size_t)lt.i * (c.N >> 6) + lt.xb / XB64;
            const uint32_t in_blk = (lt.xb % XB64) * COEF + 2 * ch, j = lks * MK + jj;
            wrow = pts + blk * Rw * 64 + in_blk + (size_t)j * 64;
            xrow = baby + blk * Rx * 64 + in_blk + (size_t)(2 * (j0 + j) + (arow & 1)) * 64;
            lg0 = lt.zg * MG + arow;
            lsh0 = lt.zc * (MS / 2) + (arow >> 1);
            lsm = sm_thread + lslot * T::STAGE_BYTES;
            if (luse > 0 && !mbar_wait(bars + 8 * (STAGES + lslot), (luse - 1) & 1, wait_limit)) alive = false;
        }
    };
    auto load_w = [&](uint32_t k) {
        if (lstep < nsteps) {
            const uint32_t g = min(lg0 + AH * k, G - 1);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(lsm + k * AH * T::GPITCH), "l"(wrow + (size_t)g * J * 64) : "memory");
        }
    };
    auto load_x = [&](uint32_t k) {
        if (lstep < nsteps) {
            const uint32_t sh = min(lsh0 + (AH / 2) * k, S - 1);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(lsm + T::BOX_BYTES + k * AH * T::GPITCH), "l"(xrow + (size_t)sh * Jx * 128)
                         : "memory");
        }
    };
    auto load_end = [&]() {
        if (lstep < nsteps) mbar_arrive_cp_async(bars + 8 * lslot);
        lstep++;
        if (++lslot == STAGES) { lslot = 0; luse++; }
        if (++lks == nk) { lks = 0; lt.next(coltiles, gtiles, xblocks); }
    };
#pragma unroll 1
    for (uint32_t s = 0; s < STAGES - 1; s++) {
        load_begin();
#pragma unroll
        for (uint32_t k = 0; k < NIT; k++) { load_w(k); load_x(k); }
        load_end();
    }

    TileIt ct;
    ct.init(t_begin, coltiles, gtiles, xblocks);
    uint32_t ks = 0, slot = 0, use = 0, qi = ct.i, tiles_done = 0;
    u64 q = c.mod[qi], mu = c.mu[qi];
    int dsum[NW][13][4];
    u64 *pend = nullptr;
    uint32_t pend_g0 = 0, pend_col0 = 0, pend_tile = 0;
    u64 pend_q = 0;
    const size_t lN = (size_t)level * c.N;
    auto flush = [&]() {
        if (!mbar_wait(bar_ofull, pend_tile & 1, wait_limit)) alive = false;
#pragma unroll
        for (uint32_t k = 0; k < MG * MS * COEF / THREADS; k++) {
            const uint32_t row = k * (THREADS / COEF) + tid / COEF, sl = tid % COEF, gl = row >> 4, cl = row & 15;
            const uint32_t g = pend_g0 + gl, col = pend_col0 + cl;
            if (alive && g < G && col < ncol) {
                u64 *dst = pend + ((size_t)g * ncol + col) * lN + (sl ^ (gl % COEF));
                const u64 v = obuf[row * COEF + sl];
                *dst = accumulate ? add_mod(v, *dst, pend_q) : v;
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_oempty);
        pend = nullptr;
    };
#pragma unroll 1
    for (uint32_t step = 0; step < nsteps && alive; step++) {
        if (ks == 0) {
#pragma unroll
            for (uint32_t n = 0; n < NW; n++)
#pragma unroll
                for (uint32_t d = 0; d < 13; d++)
#pragma unroll
                    for (uint32_t r = 0; r < 4; r++) dsum[n][d][r] = 0;
        }
        if (!mbar_wait(bars + 8 * slot, use & 1, wait_limit)) { alive = false; break; }
        const uint8_t *Wt = ring + (size_t)slot * T::STAGE_BYTES, *Xt = Wt + T::BOX_BYTES;
        uint32_t A[7][4];
#pragma unroll
        for (uint32_t r = 0; r < 2; r++)
#pragma unroll
            for (uint32_t h = 0; h < 2; h++) {
                u64 w[4];
                uint32_t f[7];
#pragma unroll
                for (uint32_t e = 0; e < 4; e++) w[e] = T::tile_word(Wt, gid + 8 * r, 16 * h + 4 * tig + e, coef);
                planes7(w, f);
#pragma unroll
                for (uint32_t pl = 0; pl < 7; pl++) A[pl][r + 2 * h] = f[pl];
            }
#pragma unroll
        for (uint32_t n = 0; n < NW; n++) {
            uint32_t Bf[7][2];
#pragma unroll
            for (uint32_t h = 0; h < 2; h++) {
                u64 x[4];
                uint32_t f[7];
#pragma unroll
                for (uint32_t e = 0; e < 4; e++) x[e] = T::tile_word(Xt, 8 * (n0 + n) + gid, 16 * h + 4 * tig + e, coef);
                planes7(x, f);
#pragma unroll
                for (uint32_t pl = 0; pl < 7; pl++) Bf[pl][h] = f[pl];
            }
            if (n == NW - 1) {
                // this warp is done with the stage; the loads of the next-but-one step start now, a few between
                // the products of each plane a
                __syncwarp();
                if (lane == 0) mbar_arrive(bars + 8 * (STAGES + slot));
                load_begin();
            }
#pragma unroll
            for (uint32_t a = 0; a < 7; a++) {
#pragma unroll
                for (uint32_t b = 0; b < 7; b++) mma_u8(dsum[n][a + b], A[a], Bf[b]);
                if (n == NW - 1) {
                    constexpr uint32_t NCP = 2 * NIT;
#pragma unroll
                    for (uint32_t k = 0; k < NCP; k++)
                        if (k * 7 / NCP == a) {
                            if (k < NIT) load_w(k); else load_x(k - NIT);
                        }
                }
            }
        }
        load_end();
        if (pend) flush();
        if (ks == nk - 1 && alive) {
            if (ct.i != qi) { qi = ct.i; q = c.mod[qi]; mu = c.mu[qi]; }
            if (tiles_done > 0 && !mbar_wait(bar_oempty, (tiles_done - 1) & 1, wait_limit)) alive = false;
#pragma unroll
            for (uint32_t n = 0; n < NW; n++)
#pragma unroll
                for (uint32_t r = 0; r < 4; r++) {
                    const uint32_t gl = gid + 8 * (r >> 1), cl = 8 * (n0 + n) + 2 * tig + (r & 1);
                    u64 e[3];
#pragma unroll
                    for (uint32_t k = 0; k < 3; k++) {
                        e[k] = mad_wide((uint32_t)dsum[n][4 * k + 1][r], 1u << 8, (u64)(uint32_t)dsum[n][4 * k][r]);
                        e[k] = mad_wide((uint32_t)dsum[n][4 * k + 2][r], 1u << 16, e[k]);
                        e[k] = mad_wide((uint32_t)dsum[n][4 * k + 3][r], 1u << 24, e[k]);
                    }
                    const u64 lo = e[0] + (e[1] << 32);
                    const u64 hi = (e[1] >> 32) + e[2] + ((u64)(uint32_t)dsum[n][12][r] << 32) + (lo < e[0]);
                    obuf[(gl * 16 + cl) * COEF + (coef ^ (gl % COEF))] = barrett112(hi, lo, q, mu);
                }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_ofull);
            pend_g0 = ct.zg * MG;
            pend_col0 = ct.zc * MS;
            pend_tile = tiles_done++;
            pend_q = q;
            pend = acc + (size_t)ct.i * c.N + ct.xb * COEF;
        }
        if (++ks == nk) { ks = 0; ct.next(coltiles, gtiles, xblocks); }
        if (++slot == STAGES) { slot = 0; use++; }
    }
    if (pend && alive) flush();
    asm volatile("cp.async.wait_all;\n" ::: "memory");
    if (!alive) atomicExch(c.range_flag + 1, 1);
}

template <uint32_t COEF, uint32_t NW, bool ASYNC = false>
bool launch_as(const ckks_ctx *c, const u64 *baby, const u64 *pts, u64 *acc, uint32_t J, uint32_t S, uint32_t G, uint32_t level, cudaStream_t s,
               uint32_t Jx, uint32_t j0, bool accumulate) {
    // per device, so set on every launch (a host-side table update)
    const void *kernel = ASYNC ? (const void *)mac_mma_async_kernel<COEF, NW> : (const void *)mac_mma_kernel<COEF, NW>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Geo<COEF>::SMEM_BYTES) != cudaSuccess) return false;
    const uint32_t coltiles = (2 * S + MS - 1) / MS, gt = (G + MG - 1) / MG;
    const uint32_t ntiles = (c->N / COEF) * level * coltiles * gt;
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
    const uint32_t ctas = (uint32_t)sms * (8 / COEF), grid = ntiles < ctas ? ntiles : ctas;
    if (ASYNC)
        mac_mma_async_kernel<COEF, NW><<<grid, COEF * 64 / NW, Geo<COEF>::SMEM_BYTES, s>>>(c->dev, baby, pts, acc, J, S, G, level, ntiles, Jx, j0,
                                                                                            accumulate ? 1u : 0u, c->wait_cycles);
    else
        mac_mma_kernel<COEF, NW><<<grid, COEF * 64 / NW, Geo<COEF>::SMEM_BYTES, s>>>(c->dev, baby, pts, acc, J, S, G, level, ntiles, Jx, j0,
                                                                                      accumulate ? 1u : 0u);
    count_launches();
    return true;
}

}  // namespace

bool mac_mma_supported(const ckks_ctx *c, uint32_t J) { return J % MK == 0 && J > 0 && c->N % 64 == 0; }

// acc[g][s][c][i][p] (+)= sum_{j < J} baby[s][j0 + j][c][i][p] * pts[g][j][i][p] with baby and pts in the tiled layout
// (baby rows (s Jx + j) 2 + c, pts rows g J + j); acc in the plain layout.  Jx = 0 means Jx = J.  Returns false if
// nothing was launched.
bool launch_mac_mma(const ckks_ctx *c, const u64 *baby, const u64 *pts, u64 *acc, uint32_t J, uint32_t S, uint32_t G, uint32_t level,
                    cudaStream_t s, uint32_t Jx, uint32_t j0, bool accumulate) {
    if (!mac_mma_supported(c, J)) return false;
    if (!Jx) Jx = J;
    // context option CKKS_OPT_MAC_KERNEL: CKKS_MAC_TCGEN05 (the tcgen05 / TMEM kernel of mac_umma.cu, J <= 64), CKKS_MAC_MMA
    // (mma.sync, 8 coefficients per CTA, a warp per coefficient: the default), CKKS_MAC_MMA_ASYNC (the same without
    // CTA-wide barriers: 7 % faster, bounded mbarrier waits), CKKS_MAC_MMA_SPLIT (two warps per coefficient, 10 % slower)
    // or CKKS_MAC_MMA_HALF (4 coefficients per CTA, two CTAs per SM: the products overlap better, but operand rows
    // fetched 32 bytes at a time make the loads twice as slow as the whole kernel otherwise is)
    const int shape = c->mac_kernel;
    if (shape == 100 && launch_mac_umma(c, baby, pts, acc, J, S, G, level, s, Jx, j0, accumulate)) return true;
    if (shape == 83) return launch_as<8, 2, true>(c, baby, pts, acc, J, S, G, level, s, Jx, j0, accumulate);
    if (shape == 42) return launch_as<4, 2>(c, baby, pts, acc, J, S, G, level, s, Jx, j0, accumulate);
    if (shape == 81) return launch_as<8, 1>(c, baby, pts, acc, J, S, G, level, s, Jx, j0, accumulate);
    return launch_as<8, 2>(c, baby, pts, acc, J, S, G, level, s, Jx, j0, accumulate);
}

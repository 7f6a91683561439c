// The projection's ciphertext x plaintext multiply-accumulate on the fifth-generation tensor cores (tcgen05, TMEM).
//
// Same contraction as mac_mma.cu: for one coefficient, out[g][s'] = sum_j w[g][j] x[j][s'] over 50-bit words, exact
// through the 7 x 7 byte products.  Here the byte split costs nothing: operands stay 64-bit words in shared memory and
// the MMA reads them MN-major, so that row m = 8 g + a of A *is* byte a of word (g, j) and column n = 8 s' + b of B is
// byte b of word (j, s') (byte 7 is zero).  One tcgen05.mma (kind::i8, unsigned, M = 128, N = 64, K = 32) therefore forms
// all 64 byte-pair sums of 16 giants x 8 columns of one coefficient; two of them cover J = 64.  The accumulator
// (128 lanes x 64 columns of s32) lives in TMEM.  Four warps read it back (lane = (g, a), columns = (s', b)):
// every thread first folds b (weights 2^(8b)) for its 8 columns, then the 8 lanes of a giant fold a by a
// transpose-reduce over three shuffle rounds, which leaves each lane with the finished 128-bit sum of one column; one
// Barrett step reduces it.
//
// Shared-memory operand layout (no swizzle): the 16-byte unit along M (or N) is a pair of giants (columns), k runs
// at 16-byte stride inside a core matrix of 8, core matrices of a pair are contiguous (LBO = 128 bytes) and pairs are
// J * 16 bytes apart (SBO).  The loader builds it with 8-byte cp.async: the 8 coefficients of a 64-byte row piece go
// to the 8 coefficient tiles.
//
// Roles in a CTA (one per SM, persistent over blocks of 8 coefficients x 16 giants): 16 epilogue warps, one MMA
// warp (a single thread issues), four loader warps, one store warp.  W tiles (16 giants x J, 8 coefficients) are
// double-buffered per block; X tiles (8 columns x J) stream through a 2-slot ring; 8 TMEM accumulators rotate
// between the MMA thread and the epilogue warps; finished results are staged per column group and stored as
// 64-byte rows.  All hand-offs are mbarriers; every wait is bounded by the clock and raises the context's sticky
// timeout flag instead of hanging.
//
// Status: bit-identical to mac_mma.cu and selectable with the context option CKKS_MAC_TCGEN05, but not the default.  On B200 a
// giant-step group of the 4096 x 4096 projection (16 shards) takes 18.9 ms here against 13.8 ms with mma.sync: the
// tensor pipe is idle most of the time and the 16 epilogue warps are busy 85 % of it.  With accumulators in registers
// the products of equal weight a + b add up inside the MMA (13 sums per output); here all 49 arrive separately and
// are folded by integer instructions (about 300 per output).  Folding them in the MMA needs the byte-shifted copies
// of one operand along K (a Toeplitz expansion) and M = 64 giants per tile.  More read-back warps (20 or 24 instead of
// 16) change nothing (18.9 - 19.4 ms): the read-back is bound by instruction issue, not by latency.
#include "common.cuh"

namespace {

constexpr uint32_t UC = 8;                 // coefficients per block (one 64-byte row piece)
constexpr uint32_t UG = 16;                // giants per block: M = 8 * UG = 128
constexpr uint32_t UCG = 8;                // columns per accumulator: N = 8 * UCG = 64
constexpr uint32_t UK = 32;                // K of one MMA
constexpr uint32_t MAX_J = 64;
constexpr uint32_t E_WARPS = 16, L_WARPS = 4;      // loader warps: a multiple of 4 (128 threads cover 8 coefficients x 8 j x 2 parities)
constexpr uint32_t W_MMA = E_WARPS, W_LOAD = E_WARPS + 1, W_STORE = W_LOAD + L_WARPS, U_WARPS = W_STORE + 1;
constexpr uint32_t U_THREADS = U_WARPS * 32;
constexpr uint32_t NACC = 8;               // TMEM accumulators of 64 columns
constexpr uint32_t OBUF_BYTES = UG * UCG * UC * 8;
// mbarrier slots
constexpr uint32_t B_WFULL = 0, B_WEMPTY = 2, B_XFULL = 4, B_XEMPTY = 6, B_TFULL = 8, B_TEMPTY = 16, B_OFULL = 24, B_OEMPTY = 26, B_COUNT = 28;

struct Smem {
    uint32_t tsw, tsx;         // bytes per coefficient tile of W / X (padded by 16)
    uint32_t x0, o0, bars, tslot, total;
    __host__ __device__ uint32_t w(uint32_t k) const { return k * UC * tsw; }             // two W buffers
    __host__ __device__ uint32_t x(uint32_t k) const { return x0 + k * UC * tsx; }        // two X slots
    __host__ __device__ uint32_t o(uint32_t k) const { return o0 + k * OBUF_BYTES; }      // two result buffers
};
__host__ __device__ inline Smem smem_plan(uint32_t J) {
    Smem s;
    s.tsw = J * 16 * (UG / 2) + 16;
    s.tsx = J * 16 * (UCG / 2) + 16;
    s.x0 = 2 * UC * s.tsw;
    s.o0 = (s.x0 + 2 * UC * s.tsx + 127) & ~127u;
    s.bars = s.o0 + 2 * OBUF_BYTES;
    s.tslot = s.bars + B_COUNT * 8;
    s.total = s.tslot + 16 + 128;       // alignment slack
    return s;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory"); }
__device__ __forceinline__ void mbar_arrive_cp_async(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];\n" ::"r"(bar) : "memory");
}
// Bounded wait (limit in SM clock cycles).  WARP = true: all 32 lanes call it together and get the warp's common answer,
// so a timeout never splits a warp in front of a warp-wide instruction; WARP = false: a single thread waits (the MMA issuer).
template <bool WARP>
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
    return WARP ? __all_sync(0xffffffffu, ok != 0) : ok != 0;
}
// item n of a ring of depth D: the consumer waits for the fill of its slot, the producer for the drain of the item before
template <bool WARP = true>
__device__ __forceinline__ bool wait_full(uint32_t bars, uint32_t base, uint32_t n, uint32_t D, long long limit) {
    return mbar_wait<WARP>(bars + 8 * (base + n % D), (n / D) & 1, limit);
}
template <bool WARP = true>
__device__ __forceinline__ bool wait_empty(uint32_t bars, uint32_t base, uint32_t n, uint32_t D, long long limit) {
    return n < D ? true : mbar_wait<WARP>(bars + 8 * (base + n % D), ((n / D) - 1) & 1, limit);
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
// shared-memory matrix descriptor, no swizzle: start address, leading (k-group) and stride (MN-group) byte offsets, version 1
__device__ __forceinline__ uint64_t umma_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr >> 4) & 0x3FFF) | ((uint64_t)((lbo >> 4) & 0x3FFF) << 16) | ((uint64_t)((sbo >> 4) & 0x3FFF) << 32) | (1ull << 46);
}
// instruction descriptor: s32 accumulator, unsigned 8-bit A and B, both MN-major, N = 64, M = 128
constexpr uint32_t UMMA_IDESC = (2u << 4) | (1u << 15) | (1u << 16) | ((uint32_t)(8 * UCG >> 3) << 17) | ((uint32_t)(8 * UG >> 4) << 24);
__device__ __forceinline__ void umma_i8(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t accumulate) {
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
                 "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n}\n"
                 :: "r"(tmem_d), "l"(da), "l"(db), "r"(UMMA_IDESC), "r"(accumulate), "r"(0u) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, "
                 "%20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]),
                   "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
                   "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]),
                   "=r"(r[31])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}
// multi-word little-endian helpers (32-bit words)
template <int NW_IN, int NW_OUT>
__device__ __forceinline__ void shl_words(const uint32_t (&x)[NW_IN], uint32_t sh, uint32_t (&r)[NW_OUT]) {     // r = x << sh, sh < 32
#pragma unroll
    for (int i = 0; i < NW_OUT; i++) r[i] = __funnelshift_l(i ? x[i - 1] : 0u, i < NW_IN ? x[i] : 0u, sh);
}
template <int NWD>
__device__ __forceinline__ void add_words(uint32_t (&a)[NWD], const uint32_t (&b)[NWD]) {
    u64 t = 0;
#pragma unroll
    for (int i = 0; i < NWD; i++) {
        t = (u64)a[i] + b[i] + (t >> 32);
        a[i] = (uint32_t)t;
    }
}

struct BlockIt {           // blocks of a CTA: giant tile fastest, then coefficient block, then limb
    uint32_t zg, xb, i;
    __device__ __forceinline__ void init(uint32_t b, uint32_t gtiles, uint32_t xblocks) {
        zg = b % gtiles; b /= gtiles;
        xb = b % xblocks; i = b / xblocks;
    }
    __device__ __forceinline__ void next(uint32_t gtiles, uint32_t xblocks) {
        if (++zg == gtiles) {
            zg = 0;
            if (++xb == xblocks) { xb = 0; i++; }
        }
    }
};

__global__ void __launch_bounds__(U_THREADS, 1) mac_umma_kernel(DevTables c, const u64 *__restrict__ baby, const u64 *__restrict__ pts,
                                                                u64 *__restrict__ acc, uint32_t J, uint32_t S, uint32_t G, uint32_t level,
                                                                uint32_t nblocks, uint32_t Jx, uint32_t j0, uint32_t accumulate, long long wl) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = reinterpret_cast<uint8_t *>(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    const uint32_t sm0 = (uint32_t)__cvta_generic_to_shared(sm);
    const Smem L = smem_plan(J);
    const uint32_t bars = sm0 + L.bars;
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t ncol = 2 * S, ncg = (ncol + UCG - 1) / UCG, gtiles = (G + UG - 1) / UG, xblocks = c.N / UC;
    const uint32_t nk = J / UK, sbo = J * 16;
    const uint32_t b_begin = (uint32_t)(((u64)nblocks * blockIdx.x) / gridDim.x), b_end = (uint32_t)(((u64)nblocks * (blockIdx.x + 1)) / gridDim.x);
    const uint32_t myblocks = b_end - b_begin;

    if (tid == 0) {
        for (uint32_t k = 0; k < 2; k++) {
            mbar_init(bars + 8 * (B_WFULL + k), L_WARPS * 32); mbar_init(bars + 8 * (B_WEMPTY + k), 1);
            mbar_init(bars + 8 * (B_XFULL + k), L_WARPS * 32); mbar_init(bars + 8 * (B_XEMPTY + k), 1);
            mbar_init(bars + 8 * (B_OFULL + k), UC * 4);       mbar_init(bars + 8 * (B_OEMPTY + k), 1);
        }
        for (uint32_t k = 0; k < NACC; k++) { mbar_init(bars + 8 * (B_TFULL + k), 1); mbar_init(bars + 8 * (B_TEMPTY + k), 4); }
    }
    if (warp == W_MMA) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;\n" ::"r"(sm0 + L.tslot) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<const uint32_t *>(sm + L.tslot);
    bool alive = true;

    if (warp >= W_LOAD && warp < W_STORE) {
        // ---------------- loaders: 8-byte cp.async, lane -> coefficient p of a row piece ----------------
        // a thread keeps its coefficient p, its j mod 8 and the parity of its giant (column); it walks pairs and j / 8
        const uint32_t lt = tid - W_LOAD * 32, p = lt & 7, jr = (lt >> 3) & 7, par = (lt >> 6) & 1, sub = lt >> 7;
        constexpr uint32_t NSUB = L_WARPS / 4;                                  // thread groups sharing the pairs
        const uint32_t Rw = G * J, Rx = 2 * S * Jx, njb = J / 8;      // baby rows j0 .. j0 + J - 1 of Jx per shard and component
        BlockIt it;
        it.init(b_begin, gtiles, xblocks);
        uint32_t cgn = 0;                                                       // column groups issued so far
        for (uint32_t b = 0; b < myblocks && alive; b++, it.next(gtiles, xblocks)) {
            const size_t blk = (size_t)it.i * (c.N >> 6) + (it.xb >> 3);
            const uint32_t in_blk = (it.xb & 7) * UC + p;
            if (!wait_empty(bars, B_WEMPTY, b, 2, wl)) { alive = false; break; }
            const u64 *wsrc = pts + blk * Rw * 64 + in_blk + (size_t)jr * 64;
            const uint32_t wdst = sm0 + L.w(b & 1) + p * L.tsw + jr * 16 + par * 8;
            for (uint32_t gp = sub; gp < UG / 2; gp += NSUB) {
                const uint32_t g = min(it.zg * UG + 2 * gp + par, G - 1);
                const u64 *src = wsrc + (size_t)g * J * 64;
                uint32_t dst = wdst + gp * sbo;
                for (uint32_t jb = 0; jb < njb; jb++, src += 8 * 64, dst += 128)
                    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(dst), "l"(src) : "memory");
            }
            mbar_arrive_cp_async(bars + 8 * (B_WFULL + (b & 1)));
            const u64 *xsrc = baby + blk * Rx * 64 + in_blk + (size_t)(j0 + jr) * 128;
            for (uint32_t cg = 0; cg < ncg && alive; cg++, cgn++) {
                if (!wait_empty(bars, B_XEMPTY, cgn, 2, wl)) { alive = false; break; }
                const uint32_t xdst = sm0 + L.x(cgn & 1) + p * L.tsx + jr * 16 + par * 8;
                for (uint32_t cp = sub; cp < UCG / 2; cp += NSUB) {
                    const uint32_t col = min(cg * UCG + 2 * cp + par, ncol - 1);
                    const u64 *src = xsrc + ((size_t)(col >> 1) * Jx * 2 + (col & 1)) * 64;
                    uint32_t dst = xdst + cp * sbo;
                    for (uint32_t jb = 0; jb < njb; jb++, src += 16 * 64, dst += 128)
                        asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(dst), "l"(src) : "memory");
                }
                mbar_arrive_cp_async(bars + 8 * (B_XFULL + (cgn & 1)));
            }
        }
        asm volatile("cp.async.wait_all;\n" ::: "memory");
    } else if (warp == W_MMA) {
        // ---------------- MMA issue: one thread ----------------
        if (lane == 0) {
            uint32_t cgn = 0, an = 0;
            for (uint32_t b = 0; b < myblocks && alive; b++) {
                if (!wait_full<false>(bars, B_WFULL, b, 2, wl)) { alive = false; break; }
                for (uint32_t cg = 0; cg < ncg && alive; cg++, cgn++) {
                    if (!wait_full<false>(bars, B_XFULL, cgn, 2, wl)) { alive = false; break; }
                    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                    for (uint32_t p = 0; p < UC; p++, an++) {
                        if (!wait_empty<false>(bars, B_TEMPTY, an, NACC, wl)) { alive = false; break; }
                        tc_fence_after();
                        const uint32_t wa = sm0 + L.w(b & 1) + p * L.tsw, xa = sm0 + L.x(cgn & 1) + p * L.tsx;
                        for (uint32_t ks = 0; ks < nk; ks++)
                            umma_i8(tmem + (an % NACC) * 8 * UCG, umma_desc(wa + ks * UK * 16, 128, sbo), umma_desc(xa + ks * UK * 16, 128, sbo), ks);
                        tc_commit(bars + 8 * (B_TFULL + an % NACC));
                    }
                    tc_commit(bars + 8 * (B_XEMPTY + (cgn & 1)));
                }
                tc_commit(bars + 8 * (B_WEMPTY + (b & 1)));
            }
        }
    } else if (warp == W_STORE) {
        // ---------------- store: a finished column group as 64-byte rows ----------------
        const size_t lN = (size_t)level * c.N;
        BlockIt it;
        it.init(b_begin, gtiles, xblocks);
        uint32_t cgn = 0;
        for (uint32_t b = 0; b < myblocks && alive; b++, it.next(gtiles, xblocks)) {
            u64 *obase = acc + (size_t)it.i * c.N + it.xb * UC;
            for (uint32_t cg = 0; cg < ncg && alive; cg++, cgn++) {
                if (!wait_full(bars, B_OFULL, cgn, 2, wl)) { alive = false; break; }
                const u64 *ob = reinterpret_cast<const u64 *>(sm + L.o(cgn & 1));
#pragma unroll 4
                for (uint32_t k = 0; k < UG * UCG * UC / 32; k++) {
                    const uint32_t row = k * 4 + (lane >> 3), w = lane & 7, gl = row >> 3, cl = row & 7;
                    const uint32_t g = it.zg * UG + gl, col = cg * UCG + cl;
                    if (g < G && col < ncol) {
                        u64 *dst = obase + ((size_t)g * ncol + col) * lN + (w ^ (gl & 7));
                        const u64 v = ob[row * UC + w];
                        *dst = accumulate ? add_mod(v, *dst, c.mod[it.i]) : v;
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bars + 8 * (B_OEMPTY + (cgn & 1)));
            }
        }
    } else {
        // ---------------- epilogue: warp = (group eg, lane quarter q); group eg takes coefficients eg and eg + 4 ----------------
        const uint32_t eg = warp >> 2, q = warp & 3;
        const uint32_t a = lane & 7, gl = 4 * q + (lane >> 3);          // TMEM lane 32 q + lane = 8 gl + a
        const uint32_t sh1 = (a & 1) ? 8u : 0u, sh2 = (a & 2) ? 16u : 0u;
        const bool a0 = a & 1, a1 = a & 2, a2 = a & 4;
        BlockIt it;
        it.init(b_begin, gtiles, xblocks);
        uint32_t cgn = 0, qi = 0xffffffffu;
        u64 qmod = 0, mu = 0;
        for (uint32_t b = 0; b < myblocks && alive; b++, it.next(gtiles, xblocks)) {
            if (it.i != qi) { qi = it.i; qmod = c.mod[qi]; mu = c.mu[qi]; }
            for (uint32_t cg = 0; cg < ncg && alive; cg++, cgn++) {
                for (uint32_t half = 0; half < 2; half++) {
                    const uint32_t p = eg + 4 * half, an = cgn * UC + p;
                    if (!wait_full(bars, B_TFULL, an, NACC, wl)) { alive = false; break; }
                    tc_fence_after();
                    // fold b: S[cl] = sum_b D[cl][b] 2^(8b) as three 32-bit words (below 2^72)
                    uint32_t T[8][3];
#pragma unroll
                    for (uint32_t h = 0; h < 2; h++) {
                        uint32_t v[32];
                        tmem_ld32(tmem + ((32 * q) << 16) + (an % NACC) * 8 * UCG + 32 * h, v);
#pragma unroll
                        for (uint32_t cc = 0; cc < 4; cc++) {
                            const uint32_t *d = v + 8 * cc;
                            // every D is below 2^22 (J <= 64), so byte pairs combine in 32 bits
                            const uint32_t t01 = d[0] + (d[1] << 8), t23 = d[2] + (d[3] << 8), t45 = d[4] + (d[5] << 8);
                            const u64 lo = (u64)t01 + ((u64)t23 << 16);
                            const u64 hi = (u64)t45 + ((u64)d[6] << 16) + (lo >> 32);
                            // times 2^(8 (a & 1)) before the first exchange
                            const uint32_t s[3] = {(uint32_t)lo, (uint32_t)hi, (uint32_t)(hi >> 32)};
                            shl_words<3, 3>(s, sh1, T[4 * h + cc]);
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bars + 8 * (B_TEMPTY + an % NACC));
                    // fold a over the 8 lanes of a giant.  First exchange (lane ^ 1): a even keeps columns 0..3, odd keeps 4..7
                    uint32_t V[4][3];
#pragma unroll
                    for (uint32_t k = 0; k < 4; k++) {
                        uint32_t r[3];
#pragma unroll
                        for (uint32_t w = 0; w < 3; w++) {
                            const uint32_t keep = a0 ? T[4 + k][w] : T[k][w], send = a0 ? T[k][w] : T[4 + k][w];
                            V[k][w] = keep;
                            r[w] = __shfl_xor_sync(0xffffffffu, send, 1);
                        }
                        add_words<3>(V[k], r);
                    }
                    // second exchange (lane ^ 2): weights 2^(16 (a >> 1 & 1)); a1 = 0 keeps the first two of its four columns
                    uint32_t U[2][4];
                    {
                        uint32_t X4[4][4];
#pragma unroll
                        for (uint32_t k = 0; k < 4; k++) shl_words<3, 4>(V[k], sh2, X4[k]);
#pragma unroll
                        for (uint32_t k = 0; k < 2; k++) {
                            uint32_t r[4];
#pragma unroll
                            for (uint32_t w = 0; w < 4; w++) {
                                const uint32_t keep = a1 ? X4[2 + k][w] : X4[k][w], send = a1 ? X4[k][w] : X4[2 + k][w];
                                U[k][w] = keep;
                                r[w] = __shfl_xor_sync(0xffffffffu, send, 2);
                            }
                            add_words<4>(U[k], r);
                        }
                    }
                    // third exchange (lane ^ 4): weights 2^(32 (a >> 2)), a word shift; a2 = 0 keeps the first of its two columns
                    uint32_t Z[4];
                    {
                        uint32_t r[4];
#pragma unroll
                        for (uint32_t w = 0; w < 4; w++) {
                            const uint32_t k0 = a2 ? (w ? U[0][w - 1] : 0u) : U[0][w], k1 = a2 ? (w ? U[1][w - 1] : 0u) : U[1][w];
                            Z[w] = a2 ? k1 : k0;
                            r[w] = __shfl_xor_sync(0xffffffffu, a2 ? k0 : k1, 4);
                        }
                        add_words<4>(Z, r);
                    }
                    const uint32_t cl = (a0 ? 4u : 0u) + (a1 ? 2u : 0u) + (a2 ? 1u : 0u);     // the column this lane finished
                    const u64 res = barrett112(((u64)Z[3] << 32) | Z[2], ((u64)Z[1] << 32) | Z[0], qmod, mu);
                    if (!wait_empty(bars, B_OEMPTY, cgn, 2, wl)) { alive = false; break; }
                    reinterpret_cast<u64 *>(sm + L.o(cgn & 1))[(gl * UCG + cl) * UC + (p ^ (gl & 7))] = res;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bars + 8 * (B_OFULL + (cgn & 1)));
                }
            }
        }
    }
    if (!alive) atomicExch(c.range_flag + 1, 1);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == W_MMA) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;\n" ::"r"(tmem) : "memory");
}

}  // namespace

bool mac_umma_supported(const ckks_ctx *c, uint32_t J) { return J % UK == 0 && J > 0 && J <= MAX_J && c->N % 64 == 0; }

// Same contract as launch_mac_mma.
bool launch_mac_umma(const ckks_ctx *c, const u64 *baby, const u64 *pts, u64 *acc, uint32_t J, uint32_t S, uint32_t G, uint32_t level,
                     cudaStream_t s, uint32_t Jx, uint32_t j0, bool accumulate) {
    if (!mac_umma_supported(c, J)) return false;
    if (!Jx) Jx = J;
    const Smem L = smem_plan(J);
    // per device, so set on every launch (a host-side table update)
    if (cudaFuncSetAttribute(mac_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_plan(MAX_J).total) != cudaSuccess) return false;
    const uint32_t gtiles = (G + UG - 1) / UG, nblocks = (c->N / UC) * level * gtiles;
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
    mac_umma_kernel<<<nblocks < (uint32_t)sms ? nblocks : (uint32_t)sms, U_THREADS, L.total, s>>>(c->dev, baby, pts, acc, J, S, G, level, nblocks, Jx, j0,
                                                                                                  accumulate ? 1u : 0u, c->wait_cycles);
    count_launches();
    return true;
}

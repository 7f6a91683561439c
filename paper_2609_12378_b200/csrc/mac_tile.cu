// Integer-pipe form of the projection's ciphertext x plaintext multiply-accumulate: the fallback for baby-step counts
// the tensor-core kernels do not take (B not a multiple of 32).
#include "common.cuh"

namespace {

constexpr uint32_t MAC_GT = 4, MAC_ST = 2;   // register tile: giants x shards

// Multiply-accumulate of one giant-step group:
//   acc[g][s][c][i][p] = sum_{j < J} baby[s][j][c][i][p] * pts[g][j][i][p]      (j = input block * B + baby step)
// A thread owns one coefficient p of one limb i and a register tile of MAC_GT giant steps x MAC_ST shards x 2
// components; per j it loads MAC_ST*2 ciphertext words and MAC_GT plaintext words for MAC_GT*MAC_ST*2 products.
//
// Exact lazy accumulation without carries: every 50-bit word is split at bit 25, x = xh 2^25 + xl, and the
// three sums  LL = sum xl wl,  HH = sum xh wh,  MM = sum (xl + xh)(wl + wh)  are kept in plain 64-bit
// registers (each product is below 2^52, so 2^11 terms fit).  The sum of products is then
// LL + (MM - LL - HH) 2^25 + HH 2^50 < 2^112, reduced once.  Three 32x32->64 multiply-adds per product.
// Tiles of one coefficient range are adjacent in the grid (blockIdx.x), so re-reads of the same words by other
// tiles hit L2 rather than HBM.
struct Split { uint32_t l, h, s; };
__device__ __forceinline__ Split split25(u64 x) {
    Split r;
    r.l = (uint32_t)x & 0x1FFFFFFu;
    r.h = (uint32_t)(x >> 25);
    r.s = r.l + r.h;
    return r;
}

constexpr uint32_t MAC_THREADS = 128, MAC_DEPTH = 6, MAC_WORDS = MAC_GT + MAC_ST * 2;

__device__ __forceinline__ void cp_async8(void *smem, const void *gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int NLEFT>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(NLEFT) : "memory"); }

// Operands are staged through a MAC_DEPTH-deep ring in shared memory filled by cp.async, so that several j steps
// of loads are in flight per thread while the products of the current step are formed; a thread only ever reads
// back the words it requested itself, so no block-wide barrier is needed.
__global__ void __launch_bounds__(MAC_THREADS) mac_tile_kernel(DevTables c, const u64 *__restrict__ baby, const u64 *__restrict__ pts,
                                                               u64 *__restrict__ acc, uint32_t J, uint32_t S, uint32_t G, uint32_t level) {
    __shared__ u64 ring[MAC_DEPTH][MAC_WORDS][MAC_THREADS];
    const uint32_t stiles = (S + MAC_ST - 1) / MAC_ST;
    const uint32_t s0 = (blockIdx.x % stiles) * MAC_ST, g0 = (blockIdx.x / stiles) * MAC_GT;
    const uint32_t tid = threadIdx.x, p = blockIdx.y * MAC_THREADS + tid, i = blockIdx.z;
    const size_t lN = (size_t)level * c.N, ctl = 2 * lN;
    const u64 q = c.mod[i], mu = c.mu[i];
    const size_t off = (size_t)i * c.N + p;
    constexpr uint32_t NX = MAC_ST * 2;
    u64 LL[MAC_GT][NX], HH[MAC_GT][NX], MM[MAC_GT][NX];
#pragma unroll
    for (uint32_t g = 0; g < MAC_GT; g++)
#pragma unroll
        for (uint32_t x = 0; x < NX; x++) LL[g][x] = HH[g][x] = MM[g][x] = 0;
    // operands are tiled (tiled_index): row g J + j of pts, row (s J + j) 2 + c of baby; consecutive j are 64 (128) words apart
    const u64 *wp[MAC_GT], *xp[NX];
    bool wok[MAC_GT], xok[NX];
    const uint32_t Rw = G * J, Rx = 2 * S * J;
#pragma unroll
    for (uint32_t g = 0; g < MAC_GT; g++) {
        wok[g] = g0 + g < G;                      // out-of-range tiles read tile 0 and are never stored
        wp[g] = pts + tiled_index(Rw, c.N, (wok[g] ? g0 + g : 0) * J, i, p);
    }
#pragma unroll
    for (uint32_t x = 0; x < NX; x++) {
        xok[x] = s0 + x / 2 < S;
        xp[x] = baby + tiled_index(Rx, c.N, (xok[x] ? s0 + x / 2 : 0) * J * 2 + (x & 1), i, p);
    }
    auto issue = [&](uint32_t j) {
        if (j < J) {
            const uint32_t st = j % MAC_DEPTH;
#pragma unroll
            for (uint32_t g = 0; g < MAC_GT; g++) cp_async8(&ring[st][g][tid], wp[g] + (size_t)j * 64);
#pragma unroll
            for (uint32_t x = 0; x < NX; x++) cp_async8(&ring[st][MAC_GT + x][tid], xp[x] + (size_t)j * 128);
        }
        cp_async_commit();
    };
#pragma unroll
    for (uint32_t j = 0; j < MAC_DEPTH - 1; j++) issue(j);
    for (uint32_t j = 0; j < J; j++) {
        cp_async_wait<MAC_DEPTH - 2>();           // step j has landed
        const uint32_t st = j % MAC_DEPTH;
        Split w[MAC_GT], x[NX];
#pragma unroll
        for (uint32_t g = 0; g < MAC_GT; g++) w[g] = split25(ring[st][g][tid]);
#pragma unroll
        for (uint32_t k = 0; k < NX; k++) x[k] = split25(ring[st][MAC_GT + k][tid]);
        issue(j + MAC_DEPTH - 1);                 // refills the slot read in the previous step
#pragma unroll
        for (uint32_t g = 0; g < MAC_GT; g++)
#pragma unroll
            for (uint32_t k = 0; k < NX; k++) {
                LL[g][k] += (u64)x[k].l * w[g].l;
                HH[g][k] += (u64)x[k].h * w[g].h;
                MM[g][k] += (u64)x[k].s * w[g].s;
            }
    }
#pragma unroll
    for (uint32_t g = 0; g < MAC_GT; g++)
#pragma unroll
        for (uint32_t k = 0; k < NX; k++)
            if (wok[g] && xok[k]) {
                const u64 mid = MM[g][k] - LL[g][k] - HH[g][k];
                const u128 t = (u128)LL[g][k] + ((u128)mid << 25) + ((u128)HH[g][k] << 50);
                acc[((size_t)(g0 + g) * S + s0 + k / 2) * ctl + (k & 1) * lN + off] = barrett112((u64)(t >> 64), (u64)t, q, mu);
            }
}

}  // namespace

void launch_mac_tile(const ckks_ctx *c, const u64 *baby, const u64 *pts, u64 *acc, uint32_t J, uint32_t S, uint32_t G, uint32_t level,
                     cudaStream_t s) {
    const uint32_t stiles = (S + MAC_ST - 1) / MAC_ST, gtiles = (G + MAC_GT - 1) / MAC_GT;
    mac_tile_kernel<<<dim3(stiles * gtiles, c->N / MAC_THREADS, level), MAC_THREADS, 0, s>>>(c->dev, baby, pts, acc, J, S, G, level);
    count_launches();
}

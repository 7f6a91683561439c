// Pointwise (coefficient-wise) kernels on evaluation-domain limbs: ciphertext x
// plaintext multiply-accumulate, addition, tensor product, Galois automorphism.
// All are streaming kernels bound by HBM bandwidth: 128-bit loads and stores,
// one pass over each operand.
#include "common.cuh"

namespace {

constexpr uint32_t THREADS = 256;
constexpr uint32_t MAC_MAX = 32;   // ciphertexts per launch

struct MacArgs {
    const u64 *ct[MAC_MAX];
    u64 *acc[MAC_MAX];
};

// acc[s][c][i][k] (+)= ct[s][c][i][k] * pt[i][k]; one thread owns two adjacent coefficients of one (c, i).
template <bool INIT>
__global__ void __launch_bounds__(THREADS) mac_kernel(DevTables c, MacArgs a, uint32_t ncts, const u64 *pt, uint32_t level) {
    const uint32_t half = c.N / 2;
    const uint32_t x = blockIdx.x * THREADS + threadIdx.x;   // pair index inside the limb
    const uint32_t limb = blockIdx.y, comp = blockIdx.z;
    if (x >= half) return;
    const u64 q = c.mod[limb], mu = c.mu[limb];
    const ulonglong2 p = reinterpret_cast<const ulonglong2 *>(pt + (size_t)limb * c.N)[x];
    const size_t off = ((size_t)comp * level + limb) * half + x;
    for (uint32_t s = 0; s < ncts; s++) {
        ulonglong2 v = reinterpret_cast<const ulonglong2 *>(a.ct[s])[off];
        ulonglong2 r;
        r.x = mul_mod(v.x, p.x, q, mu);
        r.y = mul_mod(v.y, p.y, q, mu);
        ulonglong2 *dst = reinterpret_cast<ulonglong2 *>(a.acc[s]) + off;
        if (!INIT) {
            ulonglong2 o = *dst;
            r.x = add_mod(r.x, o.x, q);
            r.y = add_mod(r.y, o.y, q);
        }
        *dst = r;
    }
}

__global__ void __launch_bounds__(THREADS) add_kernel(DevTables c, const u64 *a, const u64 *b, u64 *out, uint32_t level) {
    const uint32_t half = c.N / 2;
    const uint32_t x = blockIdx.x * THREADS + threadIdx.x;
    if (x >= half) return;
    const u64 q = c.mod[blockIdx.y % level];
    const size_t off = (size_t)blockIdx.y * half + x;
    ulonglong2 u = reinterpret_cast<const ulonglong2 *>(a)[off], v = reinterpret_cast<const ulonglong2 *>(b)[off];
    reinterpret_cast<ulonglong2 *>(out)[off] = make_ulonglong2(add_mod(u.x, v.x, q), add_mod(u.y, v.y, q));
}

// out[y][p] = in[y][pi(p)], 2 bitrev(pi(p)) + 1 = g (2 bitrev(p) + 1) mod 2N
__global__ void __launch_bounds__(THREADS) automorphism_kernel(DevTables c, const u64 *in, u64 *out, u64 g) {
    const uint32_t p = blockIdx.x * THREADS + threadIdx.x;
    if (p >= c.N) return;
    const u64 e = (g * (2ull * bitrev_n(p, c.log_n) + 1)) & (2ull * c.N - 1);
    const uint32_t src = bitrev_n((uint32_t)((e - 1) >> 1), c.log_n);
    out[(size_t)blockIdx.y * c.N + p] = in[(size_t)blockIdx.y * c.N + src];
}

// (a0 b0, a0 b1 + a1 b0) -> e01 [2][level][N];  a1 b1 -> e2 [level][N]
__global__ void __launch_bounds__(THREADS) tensor_kernel(DevTables c, const u64 *a, const u64 *b, u64 *e01, u64 *e2, uint32_t level) {
    const uint32_t k = blockIdx.x * THREADS + threadIdx.x;
    if (k >= c.N) return;
    const uint32_t limb = blockIdx.y;
    const u64 q = c.mod[limb], mu = c.mu[limb];
    const size_t o0 = (size_t)limb * c.N + k, o1 = o0 + (size_t)level * c.N;
    const u64 a0 = a[o0], a1 = a[o1], b0 = b[o0], b1 = b[o1];
    u64 hi = 0, lo = 0;
    mac128(hi, lo, a0, b1);
    mac128(hi, lo, a1, b0);
    const u64 r0 = mul_mod(a0, b0, q, mu), r1 = barrett112(hi, lo, q, mu), r2 = mul_mod(a1, b1, q, mu);
    e01[o0] = r0;
    e01[o1] = r1;
    e2[o0] = r2;
}

// out = in * v (MUL) or in + v on component 0 (the constant polynomial v, a signed integer, has the value v mod q in
// every position of the evaluation domain); blockIdx.y = component * level + limb
template <bool MUL>
__global__ void __launch_bounds__(THREADS) const_kernel(DevTables c, const u64 *in, long long v, u64 *out, uint32_t level) {
    const uint32_t half = c.N / 2;
    const uint32_t x = blockIdx.x * THREADS + threadIdx.x;
    if (x >= half) return;
    const uint32_t limb = blockIdx.y % level;
    const u64 q = c.mod[limb], mu = c.mu[limb];
    const u64 m = (u64)(v < 0 ? -v : v) % q;
    u64 r = (v < 0 && m) ? q - m : m;
    if (!MUL && blockIdx.y >= level) r = 0;
    const size_t off = (size_t)blockIdx.y * half + x;
    const ulonglong2 u = reinterpret_cast<const ulonglong2 *>(in)[off];
    reinterpret_cast<ulonglong2 *>(out)[off] =
        MUL ? make_ulonglong2(mul_mod(u.x, r, q, mu), mul_mod(u.y, r, q, mu)) : make_ulonglong2(add_mod(u.x, r, q), add_mod(u.y, r, q));
}

// e (+)= sum_{i < n} tensor(a_i, b_i): lazy 128-bit sums (n <= TS_MAX pairs per launch: 2 n products stay below
// 2^112), one Barrett step per component, then the previous partial sum is added unless INIT
template <bool INIT>
__global__ void __launch_bounds__(THREADS) tensor_sum_kernel(DevTables c, TensorSumArgs args, uint32_t n, u64 *e01, u64 *e2, uint32_t level) {
    const uint32_t k = blockIdx.x * THREADS + threadIdx.x;
    if (k >= c.N) return;
    const uint32_t limb = blockIdx.y;
    const u64 q = c.mod[limb], mu = c.mu[limb];
    const size_t o0 = (size_t)limb * c.N + k, o1 = o0 + (size_t)level * c.N;
    u64 h0 = 0, l0 = 0, h1 = 0, l1 = 0, h2 = 0, l2 = 0;
    for (uint32_t i = 0; i < n; i++) {
        const u64 a0 = args.a[i][o0], a1 = args.a[i][o1], b0 = args.b[i][o0], b1 = args.b[i][o1];
        mac128(h0, l0, a0, b0);
        mac128(h1, l1, a0, b1);
        mac128(h1, l1, a1, b0);
        mac128(h2, l2, a1, b1);
    }
    u64 r0 = barrett112(h0, l0, q, mu), r1 = barrett112(h1, l1, q, mu), r2 = barrett112(h2, l2, q, mu);
    if (!INIT) { r0 = add_mod(r0, e01[o0], q); r1 = add_mod(r1, e01[o1], q); r2 = add_mod(r2, e2[o0], q); }
    e01[o0] = r0;
    e01[o1] = r1;
    e2[o0] = r2;
}

}  // namespace

// out[x] = 1.0 where lo <= x / B < hi and t0 <= x % Ti < t1, else 0.0 (slot masks of the attention layout's conversions)
__global__ void __launch_bounds__(THREADS) slot_mask_kernel(double *out, uint32_t n, uint32_t B, uint32_t lo, uint32_t hi, uint32_t Ti, uint32_t t0,
                                                            uint32_t t1) {
    const uint32_t x = blockIdx.x * THREADS + threadIdx.x;
    if (x >= n) return;
    const uint32_t blk = x / B, t = x % Ti;
    out[x] = (blk >= lo && blk < hi && t >= t0 && t < t1) ? 1.0 : 0.0;
}

void launch_slot_mask(const ckks_ctx *c, double *out, uint32_t B, uint32_t lo, uint32_t hi, uint32_t Ti, uint32_t t0, uint32_t t1, cudaStream_t s) {
    slot_mask_kernel<<<(c->n + THREADS - 1) / THREADS, THREADS, 0, s>>>(out, c->n, B, lo, hi, Ti, t0, t1);
    count_launches();
}

void launch_const(const ckks_ctx *c, const u64 *in, long long v, bool mul, u64 *out, uint32_t ncomp, uint32_t level, cudaStream_t s) {
    dim3 grid((c->N / 2 + THREADS - 1) / THREADS, ncomp * level);
    if (mul) const_kernel<true><<<grid, THREADS, 0, s>>>(c->dev, in, v, out, level);
    else const_kernel<false><<<grid, THREADS, 0, s>>>(c->dev, in, v, out, level);
    count_launches();
}

void launch_tensor_sum(const ckks_ctx *c, const u64 *const *a, const u64 *const *b, uint32_t n, u64 *e01, u64 *e2, uint32_t level,
                       cudaStream_t s) {
    dim3 grid((c->N + THREADS - 1) / THREADS, level);
    for (uint32_t i0 = 0; i0 < n; i0 += TS_MAX) {
        TensorSumArgs args;
        const uint32_t m = n - i0 < TS_MAX ? n - i0 : TS_MAX;
        for (uint32_t i = 0; i < m; i++) { args.a[i] = a[i0 + i]; args.b[i] = b[i0 + i]; }
        if (i0 == 0) tensor_sum_kernel<true><<<grid, THREADS, 0, s>>>(c->dev, args, m, e01, e2, level);
        else tensor_sum_kernel<false><<<grid, THREADS, 0, s>>>(c->dev, args, m, e01, e2, level);
        count_launches();
    }
}

void launch_mul_plain_acc(const ckks_ctx *c, const u64 *const *cts, u64 *const *accs, uint32_t ncts, const u64 *pt,
                          uint32_t level, bool init, cudaStream_t s) {
    dim3 grid((c->N / 2 + THREADS - 1) / THREADS, level, 2);
    for (uint32_t s0 = 0; s0 < ncts; s0 += MAC_MAX) {
        MacArgs a;
        uint32_t n = ncts - s0 < MAC_MAX ? ncts - s0 : MAC_MAX;
        for (uint32_t i = 0; i < n; i++) { a.ct[i] = cts[s0 + i]; a.acc[i] = accs[s0 + i]; }
        if (init) { mac_kernel<true><<<grid, THREADS, 0, s>>>(c->dev, a, n, pt, level); count_launches(); }
        else { mac_kernel<false><<<grid, THREADS, 0, s>>>(c->dev, a, n, pt, level); count_launches(); }
    }
}

void launch_add(const ckks_ctx *c, const u64 *a, const u64 *b, u64 *out, uint32_t ncomp, uint32_t level, cudaStream_t s) {
    dim3 grid((c->N / 2 + THREADS - 1) / THREADS, ncomp * level);
    add_kernel<<<grid, THREADS, 0, s>>>(c->dev, a, b, out, level); count_launches();
}

void launch_automorphism(const ckks_ctx *c, const u64 *in, u64 *out, uint32_t nlimbs, u64 galois, cudaStream_t s) {
    dim3 grid((c->N + THREADS - 1) / THREADS, nlimbs);
    automorphism_kernel<<<grid, THREADS, 0, s>>>(c->dev, in, out, galois); count_launches();
}

void launch_tensor(const ckks_ctx *c, const u64 *a, const u64 *b, u64 *e01, u64 *e2, uint32_t level, cudaStream_t s) {
    dim3 grid((c->N + THREADS - 1) / THREADS, level);
    tensor_kernel<<<grid, THREADS, 0, s>>>(c->dev, a, b, e01, e2, level); count_launches();
}

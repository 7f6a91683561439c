// Context: parameter validation, host-side table construction, upload.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>

#include "common.cuh"

namespace {

u64 h_mul(u64 a, u64 b, u64 q) { return (u64)((u128)a * b % q); }
u64 h_pow(u64 a, u64 e, u64 q) {
    u64 r = 1;
    a %= q;
    for (; e; e >>= 1) {
        if (e & 1) r = h_mul(r, a, q);
        a = h_mul(a, a, q);
    }
    return r;
}
u64 h_inv(u64 a, u64 q) { return h_pow(a, q - 2, q); }
u64 h_shoup(u64 w, u64 q) { return (u64)(((u128)w << 64) / q); }
ulonglong2 h_pair(u64 w, u64 q) { return make_ulonglong2(w, h_shoup(w, q)); }

bool h_is_prime(u64 n) {
    static const u64 bases[] = {2, 3, 5, 7, 11, 13, 17, 19, 23, 29, 31, 37};
    if (n < 2) return false;
    for (u64 b : bases) {
        if (n % b == 0) return n == b;
    }
    u64 d = n - 1;
    int s = 0;
    while (!(d & 1)) { d >>= 1; s++; }
    for (u64 a : bases) {
        u64 x = h_pow(a, d, n);
        if (x == 1 || x == n - 1) continue;
        bool comp = true;
        for (int i = 1; i < s && comp; i++) {
            x = h_mul(x, x, n);
            if (x == n - 1) comp = false;
        }
        if (comp) return false;
    }
    return true;
}

uint32_t h_bitrev(uint32_t x, uint32_t bits) {
    uint32_t r = 0;
    for (uint32_t i = 0; i < bits; i++) { r = (r << 1) | ((x >> i) & 1); }
    return r;
}

// Smallest primitive 2N-th root of unity mod q: scan the odd powers of any one of them.
u64 h_min_root(u64 q, u64 N) {
    u64 r = 0;
    for (u64 x = 2;; x++) {
        r = h_pow(x, (q - 1) / (2 * N), q);
        if (h_pow(r, N, q) == q - 1) break;
    }
    u64 r2 = h_mul(r, r, q), cur = r, best = r;
    for (u64 k = 0; k < N; k++) {
        best = std::min(best, cur);
        cur = h_mul(cur, r2, q);
    }
    return best;
}

template <class V>
int upload(ckks_ctx *c, const std::vector<V> &v, const V **dst) {
    void *p = nullptr;
    size_t bytes = std::max<size_t>(v.size(), 1) * sizeof(V);
    cudaError_t e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) { c->cuda_error = cudaGetErrorString(e); return CKKS_ERR_CUDA; }
    c->allocs.push_back(p);
    if (!v.empty()) {
        e = cudaMemcpy(p, v.data(), v.size() * sizeof(V), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) { c->cuda_error = cudaGetErrorString(e); return CKKS_ERR_CUDA; }
    }
    *dst = (const V *)p;
    return CKKS_OK;
}

}  // namespace

unsigned long long g_kernel_launches = 0;
extern "C" uint64_t ckks_kernel_launches(void) { return g_kernel_launches; }

extern "C" const char *ckks_status_string(int32_t s) {
    switch (s) {
        case CKKS_OK: return "ok";
        case CKKS_ERR_ARG: return "bad argument";
        case CKKS_ERR_LEVEL: return "bad or mismatched level";
        case CKKS_ERR_SCALE: return "scale mismatch";
        case CKKS_ERR_NO_KEY: return "switching key for a needed Galois element is missing";
        case CKKS_ERR_WORKSPACE: return "workspace missing or too small";
        case CKKS_ERR_RANGE: return "encode: scaled value out of range";
        case CKKS_ERR_UNSUPPORTED: return "unsupported parameters";
        case CKKS_ERR_CUDA: return "CUDA runtime error";
        case CKKS_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

extern "C" const char *ckks_last_cuda_error(const ckks_ctx *ctx) { return ctx ? ctx->cuda_error.c_str() : ""; }

extern "C" void ckks_context_destroy(ckks_ctx *ctx) {
    if (!ctx) return;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(ctx->device);
    for (void *p : ctx->allocs) cudaFree(p);
    for (cudaStream_t s : ctx->lane_stream)
        if (s) cudaStreamDestroy(s);
    for (cudaEvent_t e : ctx->lane_event)
        if (e) cudaEventDestroy(e);
    cudaSetDevice(prev);
    delete ctx;
}

extern "C" int32_t ckks_context_set_option(ckks_ctx *ctx, int32_t option, int64_t value) {
    if (!ctx) return CKKS_ERR_ARG;
    switch (option) {
        case CKKS_OPT_NTT_FP_SHARE:
            if (value < 0 || value > 8) return CKKS_ERR_ARG;
            ctx->ntt_fp_share = (uint32_t)value;
            return CKKS_OK;
        case CKKS_OPT_CONV_KERNEL:
            if (value != CKKS_CONV_FP64 && value != CKKS_CONV_TENSOR) return CKKS_ERR_ARG;
            ctx->conv_kernel = (int)value;
            return CKKS_OK;
        case CKKS_OPT_MAC_KERNEL:
            if (value != CKKS_MAC_MMA && value != CKKS_MAC_MMA_ASYNC && value != CKKS_MAC_MMA_SPLIT && value != CKKS_MAC_MMA_HALF &&
                value != CKKS_MAC_TCGEN05)
                return CKKS_ERR_ARG;
            ctx->mac_kernel = (int)value;
            return CKKS_OK;
        case CKKS_OPT_NTT_BULK_STORE:
            if (value != 0 && value != 1) return CKKS_ERR_ARG;
            ctx->ntt_bulk_store = (int)value;
            return CKKS_OK;
        case CKKS_OPT_WAIT_CYCLES:
            if (value < 0) return CKKS_ERR_ARG;
            ctx->wait_cycles = (long long)value;
            return CKKS_OK;
        case CKKS_OPT_LANES:
            if (value < 1 || value > 4) return CKKS_ERR_ARG;
            ctx->lanes = (int)value;
            return CKKS_OK;
        default: return CKKS_ERR_ARG;
    }
}

extern "C" int64_t ckks_context_get_option(const ckks_ctx *ctx, int32_t option) {
    if (!ctx) return -1;
    switch (option) {
        case CKKS_OPT_NTT_FP_SHARE: return ctx->ntt_fp_share;
        case CKKS_OPT_CONV_KERNEL: return ctx->conv_kernel;
        case CKKS_OPT_MAC_KERNEL: return ctx->mac_kernel;
        case CKKS_OPT_WAIT_CYCLES: return ctx->wait_cycles;
        case CKKS_OPT_NTT_BULK_STORE: return ctx->ntt_bulk_store;
        case CKKS_OPT_LANES: return ctx->lanes;
        case CKKS_OPT_STATIC_SCRATCH_BYTES: return (int64_t)CKKS_STATIC_SCRATCH_BYTES;
        default: return -1;
    }
}

extern "C" uint64_t ckks_galois_element(const ckks_ctx *ctx, int64_t r) {
    if (!ctx) return 0;
    int64_t n = (int64_t)ctx->n;
    r %= n;
    if (r < 0) r += n;
    return ctx->pow5[(size_t)r];
}

extern "C" int32_t ckks_context_create(const ckks_params *prm, ckks_ctx **out) {
    if (!prm || !out || !prm->q || (prm->num_p && !prm->p)) return CKKS_ERR_ARG;
    *out = nullptr;
    if (prm->log_n < 10 || prm->log_n > 16) return CKKS_ERR_UNSUPPORTED;
    if (prm->num_q == 0 || prm->dnum == 0 || prm->dnum > prm->num_q || prm->num_q > 64 || prm->num_p > 64) return CKKS_ERR_UNSUPPORTED;
    const uint32_t L = prm->num_q, K = prm->num_p, T = L + K, N = 1u << prm->log_n, n = N / 2;
    const uint32_t alpha = (L + prm->dnum - 1) / prm->dnum;
    if (K < alpha) return CKKS_ERR_UNSUPPORTED;
    std::vector<u64> mod(T);
    for (uint32_t t = 0; t < T; t++) mod[t] = t < L ? prm->q[t] : prm->p[t - L];
    for (uint32_t t = 0; t < T; t++) {
        u64 m = mod[t];
        if (m <= (1ull << 49) || m >= (1ull << 50) || m % (2ull * N) != 1 || !h_is_prime(m)) return CKKS_ERR_UNSUPPORTED;
        for (uint32_t s = 0; s < t; s++)
            if (mod[s] == m) return CKKS_ERR_UNSUPPORTED;
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || prm->device < 0 || prm->device >= ndev) return CKKS_ERR_CUDA;

    ckks_ctx *c = new ckks_ctx();
    c->log_n = prm->log_n; c->N = N; c->n = n; c->L = L; c->K = K; c->dnum = prm->dnum; c->alpha = alpha; c->T = T;
    c->device = prm->device;
    c->mod = mod;
    c->pow5.resize(n);
    c->pow5[0] = 1;
    for (uint32_t j = 1; j < n; j++) c->pow5[j] = c->pow5[j - 1] * 5 % (2ull * N);

    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(c->device);

    // ---- per-prime scalars and twiddles
    std::vector<u64> mu(T), mu64(T);
    std::vector<double2> modd(T);
    std::vector<ulonglong2> ninv(T), twf((size_t)T * N), twi((size_t)T * N);
    const bool fp = prm->log_n == 16;
    std::vector<double> twdf(fp ? (size_t)T * N : 0), twdi(fp ? (size_t)T * N : 0);
    std::vector<double2> ninvd((size_t)2 * T);
    for (uint32_t t = 0; t < T; t++) {
        u64 m = mod[t];
        mu[t] = (u64)((((u128)1) << 112) / m);
        mu64[t] = (u64)((((u128)1) << 64) / m);
        modd[t] = make_double2((double)m, 1.0 / (double)m);
        ninv[t] = h_pair(h_inv(N % m, m), m);
        auto centred_pair = [&](u64 v) {
            const double d = v > m / 2 ? -(double)(m - v) : (double)v;
            return make_double2(d, d * (1.0 / (double)m));
        };
        ninvd[2 * t] = centred_pair(ninv[t].x);
        u64 psi = h_min_root(m, N), psi_inv = h_inv(psi, m);
        std::vector<u64> pw(N), pwi(N);
        pw[0] = pwi[0] = 1;
        for (uint32_t j = 1; j < N; j++) { pw[j] = h_mul(pw[j - 1], psi, m); pwi[j] = h_mul(pwi[j - 1], psi_inv, m); }
        for (uint32_t i = 0; i < N; i++) {
            uint32_t r = h_bitrev(i, prm->log_n);
            twf[(size_t)t * N + i] = h_pair(pw[r], m);
            twi[(size_t)t * N + i] = h_pair(pwi[r], m);
            if (fp) {
                // centred representatives: |w| <= q/2 halves the quotient estimate's error and doubles the input range
                twdf[(size_t)t * N + i] = pw[r] > m / 2 ? -(double)(m - pw[r]) : (double)pw[r];
                twdi[(size_t)t * N + i] = pwi[r] > m / 2 ? -(double)(m - pwi[r]) : (double)pwi[r];
                if (i == 1) ninvd[2 * t + 1] = centred_pair(h_mul(pwi[r], ninv[t].x, m));     // the inverse's last twiddle times N^-1
            }
        }
    }

    // ---- ModUp constants for every level
    const uint32_t dn = prm->dnum;
    std::vector<ulonglong2> up_inv((size_t)(L + 1) * dn * alpha, make_ulonglong2(0, 0));
    std::vector<u64> up_mod((size_t)(L + 1) * dn * alpha * T, 0);
    std::vector<double2> up_mod_d(up_mod.size(), make_double2(0.0, 0.0));
    for (uint32_t lvl = 1; lvl <= L; lvl++)
        for (uint32_t j = 0; j * alpha < lvl; j++) {
            uint32_t lo = j * alpha, hi = std::min(lo + alpha, lvl);
            for (uint32_t a = lo; a < hi; a++) {
                u64 qa = mod[a], h = 1;
                for (uint32_t b = lo; b < hi; b++)
                    if (b != a) h = h_mul(h, mod[b] % qa, qa);
                size_t base = ((size_t)lvl * dn + j) * alpha + (a - lo);
                up_inv[base] = h_pair(h_inv(h, qa), qa);
                for (uint32_t t = 0; t < T; t++) {
                    u64 mt = mod[t], v = 1;
                    for (uint32_t b = lo; b < hi; b++)
                        if (b != a) v = h_mul(v, mod[b] % mt, mt);
                    up_mod[base * T + t] = v;
                    up_mod_d[base * T + t] = make_double2((double)v, (double)v / (double)mt);
                }
            }
        }

    // ---- ModDown constants
    std::vector<ulonglong2> dn_inv(K), dn_pinv(L);
    std::vector<double2> dn_pinv_d(L);
    std::vector<double> dn_pmod_d(L);
    std::vector<u64> dn_mod((size_t)L * K);
    std::vector<double2> dn_mod_d((size_t)L * K);
    for (uint32_t a = 0; a < K; a++) {
        u64 pa = mod[L + a], h = 1;
        for (uint32_t b = 0; b < K; b++)
            if (b != a) h = h_mul(h, mod[L + b] % pa, pa);
        dn_inv[a] = h_pair(h_inv(h, pa), pa);
    }
    for (uint32_t i = 0; i < L; i++) {
        u64 q = mod[i], Pm = 1;
        for (uint32_t a = 0; a < K; a++) {
            u64 v = 1;
            for (uint32_t b = 0; b < K; b++)
                if (b != a) v = h_mul(v, mod[L + b] % q, q);
            dn_mod[(size_t)i * K + a] = v;
            dn_mod_d[(size_t)i * K + a] = make_double2((double)v, (double)v / (double)q);
            Pm = h_mul(Pm, mod[L + a] % q, q);
        }
        dn_pinv[i] = h_pair(h_inv(Pm, q), q);
        dn_pinv_d[i] = make_double2((double)dn_pinv[i].x, (double)dn_pinv[i].x / (double)q);
        dn_pmod_d[i] = (double)Pm;
    }

    // ---- The inverse transform can deliver the conversions' first factor directly: its last stage multiplies by
    // N^-1 anyway, so with N^-1 qhat^-1 (and the last twiddle times that) in its place the coefficient-domain output is
    // y = [d qhat^-1] instead of d.  Pairs {constant, constant / prime}, centred; index [level][limb][2] and [k][2].
    std::vector<double2> isc_up(fp ? (size_t)(L + 1) * L * 2 : 0), isc_dn(fp ? (size_t)K * 2 : 0);
    if (fp) {
        auto centred_pair_mod = [&](u64 v, u64 m) {
            const double dd = v > m / 2 ? -(double)(m - v) : (double)v;
            return make_double2(dd, dd * (1.0 / (double)m));
        };
        auto last_tw = [&](uint32_t t) {     // the inverse transform's last twiddle (index 1 of the inverse table)
            return twi[(size_t)t * N + 1].x;
        };
        for (uint32_t l = 1; l <= L; l++)
            for (uint32_t x = 0; x < l; x++) {
                const uint32_t j = x / alpha, a = x % alpha;
                const u64 m = mod[x], h = up_inv[((size_t)l * dn + j) * alpha + a].x;
                const u64 nh = h_mul(ninv[x].x, h, m);
                isc_up[((size_t)l * L + x) * 2] = centred_pair_mod(nh, m);
                isc_up[((size_t)l * L + x) * 2 + 1] = centred_pair_mod(h_mul(last_tw(x), nh, m), m);
            }
        for (uint32_t a = 0; a < K; a++) {
            const u64 m = mod[L + a], nh = h_mul(ninv[L + a].x, dn_inv[a].x, m);
            isc_dn[(size_t)a * 2] = centred_pair_mod(nh, m);
            isc_dn[(size_t)a * 2 + 1] = centred_pair_mod(h_mul(last_tw(L + a), nh, m), m);
        }
    }

    // ---- Byte matrices for the tensor-core basis conversion.  Row k = 8 a + b of the k-dimension is byte b of source
    // a's centred-lift word (b = 7: the "negative" flag); column (x, d) collects the byte products of weight 2^(8 d):
    // byte d - b of the constant C[a][x] for b < 7, and byte d of (-q_a C[a][x]) mod t for the flag, so that the
    // 13 diagonal sums recombine to sum_a centre(v_a) C[a][x] modulo t.
    const uint32_t conv_groups = (alpha <= 8 && K <= 8) ? (L + K + 7) / 8 : 0;
    const size_t gwords = 13 * 2 * 64;
    auto fill_bmat = [&](uint32_t *out, uint32_t nsrc, uint32_t ntgt, auto &&konst) {
        for (uint32_t gr = 0; gr < conv_groups; gr++)
            for (uint32_t d = 0; d < 13; d++)
                for (uint32_t ks = 0; ks < 2; ks++)
                    for (uint32_t lane = 0; lane < 32; lane++)
                        for (uint32_t half = 0; half < 2; half++) {
                            const uint32_t n = lane >> 2, t = lane & 3, x = gr * 8 + n, a = ks * 4 + half * 2 + (t >> 1), bb = (t & 1) * 4;
                            uint32_t word = 0;
                            if (x < ntgt && a < nsrc) {
                                u64 C, Kn;
                                konst(a, x, C, Kn);
                                for (uint32_t i = 0; i < 4; i++) {
                                    const uint32_t b = bb + i;
                                    uint32_t byte = 0;
                                    if (b < 7) { if (d >= b && d - b <= 6) byte = (uint32_t)(C >> (8 * (d - b))) & 255u; }
                                    else if (d <= 6) byte = (uint32_t)(Kn >> (8 * d)) & 255u;
                                    word |= byte << (8 * i);
                                }
                            }
                            out[((size_t)(gr * 13 + d) * 2 + ks) * 64 + lane * 2 + half] = word;
                        }
    };
    std::vector<uint32_t> up_bmat((size_t)(L + 1) * dn * conv_groups * gwords, 0), dn_bmat((size_t)conv_groups * gwords, 0);
    std::vector<double2> two52(T);
    for (uint32_t t = 0; t < T; t++) {
        const u64 v = (u64)(((u128)1 << 52) % mod[t]);
        two52[t] = make_double2((double)v, (double)v / (double)mod[t]);
    }
    if (conv_groups) {
        for (uint32_t lvl = 1; lvl <= L; lvl++)
            for (uint32_t j = 0; j * alpha < lvl; j++) {
                const uint32_t lo = j * alpha, hi = std::min(lo + alpha, lvl), nd = hi - lo, nt = lvl + K;
                fill_bmat(up_bmat.data() + ((size_t)lvl * dn + j) * conv_groups * gwords, nd, nt - nd, [&](uint32_t a, uint32_t x, u64 &C, u64 &Kn) {
                    const uint32_t xp = x < lo ? x : x + nd, t = xp < lvl ? xp : L + (xp - lvl);
                    C = up_mod[(((size_t)lvl * dn + j) * alpha + a) * T + t];
                    const u64 m = h_mul(mod[lo + a] % mod[t], C, mod[t]);
                    Kn = m ? mod[t] - m : 0;
                });
            }
        fill_bmat(dn_bmat.data(), K, L, [&](uint32_t a, uint32_t x, u64 &C, u64 &Kn) {
            C = dn_mod[(size_t)x * K + a];
            const u64 m = h_mul(mod[L + a] % mod[x], C, mod[x]);
            Kn = m ? mod[x] - m : 0;
        });
    }

    // ---- Rescale constants
    std::vector<ulonglong2> rs((size_t)L * L, make_ulonglong2(0, 0));
    for (uint32_t last = 0; last < L; last++)
        for (uint32_t i = 0; i < L; i++)
            if (i != last) rs[(size_t)last * L + i] = h_pair(h_inv(mod[last] % mod[i], mod[i]), mod[i]);

    // ---- Encode tables: input permutation and fp64 twiddles from the host libm
    std::vector<uint32_t> enc_src(n);
    std::vector<double2> om(n), ze(n);
    for (uint32_t j = 0; j < n; j++) {
        uint32_t e = (uint32_t)((c->pow5[j] - 1) / 4);
        enc_src[h_bitrev(e, prm->log_n - 1)] = j;
    }
    for (uint32_t t = 0; t < n; t++) {
        om[t] = make_double2(cos(2.0 * M_PI * (double)t / (double)n), sin(2.0 * M_PI * (double)t / (double)n));
        ze[t] = make_double2(cos(2.0 * M_PI * (double)t / (double)(2.0 * N)), sin(2.0 * M_PI * (double)t / (double)(2.0 * N)));
    }

    // the twiddles of the encoder's first pass (stages m = 2 .. min(n, 1024)) laid out stage by stage, so that a CTA
    // fetches them once into shared memory with contiguous loads
    const uint32_t enc_ch = std::min<uint32_t>(n, 1024);
    std::vector<double2> om_st(enc_ch, make_double2(0.0, 0.0));
    for (uint32_t half = 1; half < enc_ch; half <<= 1)
        for (uint32_t j = 0; j < half; j++) om_st[half + j] = om[(size_t)j * (n / (2 * half))];

    // the second pass's twiddles (stages m = 2 ch .. n on strips of columns) by stage and row, so that a strip's 16
    // columns of a row are 16 consecutive entries
    std::vector<double2> om_st2(n, make_double2(0.0, 0.0));
    for (uint32_t hr = 1; hr < n / enc_ch; hr <<= 1)
        for (uint32_t jr = 0; jr < hr; jr++)
            for (uint32_t col = 0; col < enc_ch; col++)
                om_st2[(size_t)(hr + jr) * enc_ch + col] = om[((size_t)jr * enc_ch + col) * (n / (2 * hr * enc_ch))];

    DevTables &d = c->dev;
    d.conv_groups = conv_groups; d.log_n = prm->log_n; d.N = N; d.L = L; d.K = K; d.alpha = alpha; d.T = T; d.dnum = prm->dnum;
    int rc = CKKS_OK;
    std::vector<int> flag(2, 0);
    const int *flag_dev = nullptr;
    if ((rc = upload(c, mod, &d.mod)) || (rc = upload(c, mu, &d.mu)) || (rc = upload(c, mu64, &d.mu64)) || (rc = upload(c, modd, &d.modd)) || (rc = upload(c, twf, &d.tw_fwd)) ||
        (rc = upload(c, twi, &d.tw_inv)) || (rc = upload(c, twdf, &d.twd_fwd)) || (rc = upload(c, twdi, &d.twd_inv)) || (rc = upload(c, ninvd, &d.n_inv_d)) || (rc = upload(c, isc_up, &d.inv_scale_up)) || (rc = upload(c, isc_dn, &d.inv_scale_dn)) || (rc = upload(c, ninv, &d.n_inv)) || (rc = upload(c, up_inv, &d.up_hat_inv)) ||
        (rc = upload(c, up_mod, &d.up_hat_mod)) || (rc = upload(c, up_mod_d, &d.up_hat_mod_d)) || (rc = upload(c, dn_mod_d, &d.dn_hat_mod_d)) || (rc = upload(c, dn_inv, &d.dn_hat_inv)) ||
        (rc = upload(c, dn_mod, &d.dn_hat_mod)) || (rc = upload(c, dn_pinv, &d.dn_p_inv)) || (rc = upload(c, dn_pinv_d, &d.dn_p_inv_d)) || (rc = upload(c, dn_pmod_d, &d.dn_p_mod_d)) || (rc = upload(c, up_bmat, &d.up_bmat)) || (rc = upload(c, dn_bmat, &d.dn_bmat)) || (rc = upload(c, two52, &d.two52_d)) || (rc = upload(c, rs, &d.rs_inv)) ||
        (rc = upload(c, enc_src, &d.enc_src)) || (rc = upload(c, om, &d.enc_omega)) || (rc = upload(c, om_st, &d.enc_omega_st)) || (rc = upload(c, om_st2, &d.enc_omega_st2)) || (rc = upload(c, ze, &d.enc_zeta)) ||
        (rc = upload(c, flag, &flag_dev))) {
        cudaSetDevice(prev);
        ckks_context_destroy(c);
        return rc;
    }
    d.range_flag = const_cast<int *>(flag_dev);
    bool lanes_ok = true;
    for (cudaStream_t &ls : c->lane_stream) lanes_ok = lanes_ok && cudaStreamCreateWithFlags(&ls, cudaStreamNonBlocking) == cudaSuccess;
    for (cudaEvent_t &le : c->lane_event) lanes_ok = lanes_ok && cudaEventCreateWithFlags(&le, cudaEventDisableTiming) == cudaSuccess;
    if (!lanes_ok) {
        cudaSetDevice(prev);
        ckks_context_destroy(c);
        return CKKS_ERR_CUDA;
    }
    cudaSetDevice(prev);
    *out = c;
    return CKKS_OK;
}

// C ABI layer: argument validation on the host, then the kernel sequences.
#include <math.h>

#include <algorithm>
#include <set>

#include "common.cuh"

namespace {

struct DeviceGuard {
    int prev = 0;
    explicit DeviceGuard(int dev) { cudaGetDevice(&prev); cudaSetDevice(dev); }
    ~DeviceGuard() { cudaSetDevice(prev); }
};

int finish(ckks_ctx *c) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { c->cuda_error = cudaGetErrorString(e); return CKKS_ERR_CUDA; }
    return CKKS_OK;
}

bool scales_agree(double a, double b) { return fabs(a - b) <= ldexp(fmax(fabs(a), fabs(b)), -30); }
bool level_ok(const ckks_ctx *c, uint32_t level) { return level >= 1 && level <= c->L; }
bool ct_ok(const ckks_ct *ct) { return ct && ct->data; }
size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

size_t ks_bytes(const ckks_ctx *c, uint32_t level) { return ks_workspace_limbs(c, level) * c->N * sizeof(u64); }
// hoisted rotations: one set of digits, nbh rotations' worth of inner-product and ModDown buffers side by side
size_t hoisted_bytes(const ckks_ctx *c, uint32_t level, uint32_t nbh) {
    const size_t beta = (level + c->alpha - 1) / c->alpha, nt = level + c->K;
    return (level + beta * nt + (size_t)nbh * (2 * nt + 2 * level)) * c->N * sizeof(u64);
}
constexpr uint32_t MRB_CHUNK = 16;      // products key-switched side by side by ckks_mul_relin_batch
size_t rescale_bytes(const ckks_ctx *c, uint32_t level, uint32_t ncomp) { return (size_t)ncomp * level * c->N * sizeof(u64); }

// ---- projection plan -------------------------------------------------------
struct Block { uint32_t start, size; };
struct ProjPlan {
    uint32_t F, T, B, S;
    std::vector<Block> ins, outs;
    std::vector<int64_t> rots;
    uint32_t gmax;   // largest giant-step count over block pairs
};

int split_blocks(uint32_t d, uint32_t F, std::vector<Block> &out) {
    for (uint32_t s = 0; s < d;) {
        uint32_t m = std::min(F, d - s);
        if (F % m) return CKKS_ERR_UNSUPPORTED;
        out.push_back({s, m});
        s += m;
    }
    return CKKS_OK;
}

int make_plan(const ckks_ctx *c, const ckks_proj_desc *d, ProjPlan &p) {
    if (!d || !d->d_in || !d->d_out || !d->tokens_per_shard || !d->nshards || !d->baby) return CKKS_ERR_ARG;
    if (c->n % d->tokens_per_shard) return CKKS_ERR_UNSUPPORTED;
    p.T = d->tokens_per_shard; p.F = c->n / p.T; p.B = d->baby; p.S = d->nshards;
    int rc;
    if ((rc = split_blocks(d->d_in, p.F, p.ins)) || (rc = split_blocks(d->d_out, p.F, p.outs))) return rc;
    std::set<int64_t> rots;
    for (uint32_t b = 1; b < p.B; b++) rots.insert((int64_t)b * p.T);
    p.gmax = 0;
    for (const Block &o : p.outs) {
        int64_t fold = -1;
        for (const Block &i : p.ins) {
            uint32_t nd = std::min(i.size, o.size);
            if (nd % p.B) return CKKS_ERR_UNSUPPORTED;
            p.gmax = std::max(p.gmax, nd / p.B);
            for (uint32_t g = 1; g < nd / p.B; g++) rots.insert((int64_t)g * p.B * p.T);
            int64_t f = i.size > o.size ? i.size / o.size : 1;
            if (fold >= 0 && fold != f) return CKKS_ERR_UNSUPPORTED;
            fold = f;
            for (uint32_t x = o.size; x < i.size; x *= 2) rots.insert((int64_t)x * p.T);
        }
    }
    p.rots.assign(rots.begin(), rots.end());
    return CKKS_OK;
}

struct ProjWs { size_t baby, xin, pts, ptt, slots, enc, acc, total, tmp, ks, ksx, rs, bytes; uint32_t gg, gacc, eg; bool per_block, ib_outer; };

constexpr uint32_t BABY_ROTS = 4;            // baby-step rotations per key-switch pass (N = 2^16)
constexpr uint32_t MAC_GT = 4;               // giants per register tile of the fallback multiply-accumulate kernel
constexpr uint32_t ENC_PTS = 128;            // plaintexts per encode call of the tensor-core path (its scratch is 13.25 MiB each)

ProjWs proj_layout(const ckks_ctx *c, const ProjPlan &p, uint32_t level, bool lazy, uint32_t nmat = 1) {
    const size_t ct = (size_t)2 * level * c->N * sizeof(u64), pt = (size_t)level * c->N * sizeof(u64);
    const size_t nib = p.ins.size();
    ProjWs w;
    // giant steps are processed in groups of gg: their plaintexts are encoded in one batch and
    // multiply-accumulated in one launch (about 16 * B plaintexts live at a time).  With the tensor-core kernel a
    // group is 16 giants and the input blocks are taken one after the other (accumulating launches), so its 16-row
    // tiles are full whatever the number of input blocks; the fallback kernel takes all blocks at once.
    w.per_block = mac_mma_supported(c, p.B);
    if (w.per_block) w.gg = std::max<uint32_t>(1, std::min<uint32_t>(p.gmax, 16));
    else w.gg = std::max<uint32_t>(1, std::min<uint32_t>(p.gmax, 16 / (uint32_t)nib ? 16 / (uint32_t)nib : 1));
    w.gg = (w.gg + MAC_GT - 1) / MAC_GT * MAC_GT;
    // Several input blocks and one output block (a down-shaped projection): the input blocks are taken in the outer
    // loop, so that only one block's baby ciphertexts are resident (B per shard instead of nib * B) and the key-switch
    // buffers serve one block's batch; the accumulators of all giant steps then stay live across the blocks.
    w.ib_outer = w.per_block && nib > 1 && p.outs.size() == 1 && nmat == 1;
    w.gacc = w.ib_outer ? (p.gmax + w.gg - 1) / w.gg * w.gg : w.gg;
    const size_t nbb = w.ib_outer ? 1 : nib;                // input blocks whose baby ciphertexts are resident together
    const size_t npt = (size_t)w.gg * (w.per_block ? 1 : nib) * p.B;
    // the tensor-core path encodes a group's plaintexts a few giants at a time straight into the tiled buffer, so the
    // encoder's scratch (slot values, FFT buffer, coefficients, the words between the two NTT passes) serves ENC_PTS plaintexts
    w.eg = w.per_block ? std::max<uint32_t>(1, std::min<uint32_t>(w.gg, ENC_PTS / p.B)) : w.gg;
    const size_t nenc = w.per_block ? (size_t)w.eg * p.B : npt;
    const size_t knt = level + c->K, kbeta = (level + c->alpha - 1) / c->alpha;
    // all shards' key switches run side by side; the baby steps take BABY_ROTS rotations per pass, which needs that
    // many inner-product and conversion buffers per input ciphertext
    const size_t ks_sz = align256(ks_bytes(c, level) * p.S * nbb + (size_t)(BABY_ROTS - 1) * p.S * nbb * (2 * knt + 2 * level) * c->N * sizeof(u64));
    // lazy giant steps: coefficient copies and extended digits of IP_TERMS giant steps of every shard
    const size_t ksx_sz = lazy ? align256((size_t)IP_TERMS * p.S * (level + kbeta * (level + c->K)) * c->N * sizeof(u64)) : 0;
    size_t off = 0;
    w.baby = off;  off += align256(ct * p.S * nbb * p.B);   // tiled: rows (shard * J + j) * 2 + component
    w.xin = off;   off += align256(ct * p.S * nbb);         // the inputs of the resident blocks side by side, plain layout
    w.acc = off;   off += align256(ct * p.S * w.gacc);
    w.total = off; off += align256(ct * p.S);
    w.tmp = off;   off += align256(ct);
    w.rs = off;    off += align256(rescale_bytes(c, level, 2));
    const size_t shared = off;
    w.ptt = off;   off += align256(pt * npt);               // encoded plaintexts of a group, tiled: rows g * J + j
    w.pts = off;   off += align256(pt * nenc);              // plain layout: the encoder's words between its two NTT passes
    w.slots = off; off += align256(nenc * c->n * sizeof(double));
    w.enc = off;   off += align256(encode_workspace_bytes(c, (uint32_t)nenc));
    // With the input blocks in the outer loop no key switch runs between a block's first encode and its last
    // multiply-accumulate and nothing of a key switch outlives its phase (the baby steps of a block; the giant steps at
    // the end), so the key-switch buffers share their bytes with the plaintext buffers.  In the other order the running
    // sum of the lazy giant steps lives in a key-switch buffer across the groups, so they stay apart.
    if (w.ib_outer) {
        w.ks = shared; w.ksx = shared + ks_sz;
        off = std::max(off, shared + ks_sz + ksx_sz);
    } else {
        w.ks = off;    off += ks_sz;
        w.ksx = off;   off += ksx_sz;
    }
    w.bytes = off;
    return w;
}

const ckks_evk *find_key(const ckks_evk *keys, uint32_t nkeys, u64 g) {
    for (uint32_t i = 0; i < nkeys; i++)
        if (keys[i].galois == g && keys[i].data) return &keys[i];
    return nullptr;
}

}  // namespace

extern "C" size_t ckks_workspace_bytes(const ckks_ctx *c, int32_t op, uint32_t level, uint32_t count) {
    if (!c || !level_ok(c, level)) return 0;
    const size_t limb = (size_t)c->N * sizeof(u64);
    switch (op) {
        case CKKS_OP_ENCODE: return encode_workspace_bytes(c, count ? count : 1);
        case CKKS_OP_MUL_RELIN: return ks_bytes(c, level) + (size_t)level * limb;
        case CKKS_OP_ROTATE: return ks_bytes(c, level);
        case CKKS_OP_ROTATE_HOISTED: return hoisted_bytes(c, level, std::min<uint32_t>(count ? count : 1, KS_MULTI));
        case CKKS_OP_RESCALE: return rescale_bytes(c, level, 2);
        // per product of a chunk (at most MRB_CHUNK): the staged result, e_2 and a key-switch workspace
        // per ciphertext of a chunk: staged input, staged output and a key-switch workspace
        case CKKS_OP_ROTATE_BATCH:
            return (size_t)std::min<uint32_t>(count ? count : 1, MRB_CHUNK) * ((size_t)4 * level * limb + ks_bytes(c, level));
        // a chunk of staged inputs with their key-switch workspaces
        case CKKS_OP_ROTATE_SUM:
            return (size_t)std::min<uint32_t>(count ? count : 1, MRB_CHUNK) * ((size_t)2 * level * limb + ks_bytes(c, level));
        case CKKS_OP_MUL_RELIN_BATCH:
            return (size_t)std::min<uint32_t>(count ? count : 1, MRB_CHUNK) * ((size_t)3 * level * limb + ks_bytes(c, level));
        // two running ciphertexts, the truncated copy of x, then the Mult and rescale scratch
        case CKKS_OP_POLY_EVAL: return 3 * (size_t)2 * level * limb + ks_bytes(c, level) + (size_t)level * limb + rescale_bytes(c, level, 2);
        // the powers x^2..x^degree, two truncated operands, the product, the accumulator and a term, then the scratch
        case CKKS_OP_POLY_EVAL_TREE:
            return ((size_t)(count > 1 ? count - 1 : 1) + 5) * 2 * level * limb + ks_bytes(c, level) + (size_t)level * limb + rescale_bytes(c, level, 2);
        default: return 0;
    }
}

extern "C" int32_t ckks_ntt(ckks_ctx *c, uint64_t *polys, uint32_t batch, uint32_t first, uint32_t nlimbs, void *stream) {
    if (!c || !polys || !batch || !nlimbs) return CKKS_ERR_ARG;
    if ((uint64_t)first + nlimbs > c->T) return CKKS_ERR_LEVEL;
    DeviceGuard g(c->device);
    launch_ntt(c, (u64 *)polys, batch * nlimbs, plain_map(first, nlimbs), false, (cudaStream_t)stream);
    return finish(c);
}

extern "C" int32_t ckks_intt(ckks_ctx *c, uint64_t *polys, uint32_t batch, uint32_t first, uint32_t nlimbs, void *stream) {
    if (!c || !polys || !batch || !nlimbs) return CKKS_ERR_ARG;
    if ((uint64_t)first + nlimbs > c->T) return CKKS_ERR_LEVEL;
    DeviceGuard g(c->device);
    launch_ntt(c, (u64 *)polys, batch * nlimbs, plain_map(first, nlimbs), true, (cudaStream_t)stream);
    return finish(c);
}

extern "C" int32_t ckks_ntt_butterfly_probe(ckks_ctx *c, uint32_t iters, uint64_t *scratch, size_t scratch_words, uint64_t *butterflies,
                                            void *stream) {
    if (!c || !scratch || !iters || !butterflies) return CKKS_ERR_ARG;
    if (c->log_n != 16) return CKKS_ERR_UNSUPPORTED;
    DeviceGuard g(c->device);
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
    if (scratch_words < (size_t)sms * 4 * 256) return CKKS_ERR_WORKSPACE;
    *butterflies = launch_butterfly_probe(c, iters, (u64 *)scratch, (cudaStream_t)stream);
    return finish(c);
}

extern "C" int32_t ckks_encode(ckks_ctx *c, const double *re, const double *im, uint32_t batch, double scale, uint32_t level,
                               uint64_t *out, void *ws, size_t ws_bytes, void *stream) {
    if (!c || !re || !out || !batch || !(scale > 0.0) || !isfinite(scale)) return CKKS_ERR_ARG;
    if (!level_ok(c, level)) return CKKS_ERR_LEVEL;
    if (!ws || ws_bytes < encode_workspace_bytes(c, batch)) return CKKS_ERR_WORKSPACE;
    DeviceGuard g(c->device);
    launch_encode(c, re, im, batch, scale, level, (u64 *)out, ws, (cudaStream_t)stream);
    return finish(c);
}

extern "C" int32_t ckks_encode_range_flag(ckks_ctx *c, void *stream) {
    if (!c) return CKKS_ERR_ARG;
    DeviceGuard g(c->device);
    int flag = 0;
    cudaError_t e = cudaMemcpyAsync(&flag, c->dev.range_flag, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e == cudaSuccess && flag) e = cudaMemsetAsync(c->dev.range_flag, 0, sizeof(int), (cudaStream_t)stream);
    if (e != cudaSuccess) { c->cuda_error = cudaGetErrorString(e); return CKKS_ERR_CUDA; }
    return flag ? CKKS_ERR_RANGE : CKKS_OK;
}

extern "C" int32_t ckks_device_status(ckks_ctx *c, void *stream) {
    if (!c) return CKKS_ERR_ARG;
    DeviceGuard g(c->device);
    int flag = 0;
    cudaError_t e = cudaMemcpyAsync(&flag, c->dev.range_flag + 1, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e == cudaSuccess && flag) e = cudaMemsetAsync(c->dev.range_flag + 1, 0, sizeof(int), (cudaStream_t)stream);
    if (e != cudaSuccess) { c->cuda_error = cudaGetErrorString(e); return CKKS_ERR_CUDA; }
    return flag ? CKKS_ERR_TIMEOUT : CKKS_OK;
}

extern "C" int32_t ckks_mul_plain_acc(ckks_ctx *c, const ckks_ct *cts, uint32_t ncts, const ckks_pt *pt, ckks_ct *accs,
                                      int32_t init, void *stream) {
    if (!c || !cts || !ncts || !pt || !pt->data || !accs) return CKKS_ERR_ARG;
    const uint32_t level = pt->level;
    if (!level_ok(c, level)) return CKKS_ERR_LEVEL;
    for (uint32_t s = 0; s < ncts; s++) {
        if (!cts[s].data || !accs[s].data || cts[s].ncomp != 2) return CKKS_ERR_ARG;
        if (cts[s].level != level) return CKKS_ERR_LEVEL;
        if (!init) {
            if (accs[s].ncomp != 2) return CKKS_ERR_ARG;
            if (accs[s].level != level) return CKKS_ERR_LEVEL;
            if (!scales_agree(cts[s].scale * pt->scale, accs[s].scale)) return CKKS_ERR_SCALE;
        }
    }
    DeviceGuard g(c->device);
    std::vector<const u64 *> cp(ncts);
    std::vector<u64 *> ap(ncts);
    for (uint32_t s = 0; s < ncts; s++) { cp[s] = (const u64 *)cts[s].data; ap[s] = (u64 *)accs[s].data; }
    launch_mul_plain_acc(c, cp.data(), ap.data(), ncts, (const u64 *)pt->data, level, init != 0, (cudaStream_t)stream);
    int rc = finish(c);
    if (rc == CKKS_OK && init)
        for (uint32_t s = 0; s < ncts; s++) { accs[s].level = level; accs[s].ncomp = 2; accs[s].scale = cts[s].scale * pt->scale; }
    return rc;
}

extern "C" int32_t ckks_add(ckks_ctx *c, const ckks_ct *a, const ckks_ct *b, ckks_ct *out, void *stream) {
    if (!c || !ct_ok(a) || !ct_ok(b) || !ct_ok(out) || a->ncomp != b->ncomp || !a->ncomp) return CKKS_ERR_ARG;
    if (!level_ok(c, a->level) || a->level != b->level) return CKKS_ERR_LEVEL;
    if (!scales_agree(a->scale, b->scale)) return CKKS_ERR_SCALE;
    DeviceGuard g(c->device);
    launch_add(c, (const u64 *)a->data, (const u64 *)b->data, (u64 *)out->data, a->ncomp, a->level, (cudaStream_t)stream);
    int rc = finish(c);
    if (rc == CKKS_OK) { out->level = a->level; out->ncomp = a->ncomp; out->scale = a->scale; }
    return rc;
}

extern "C" int32_t ckks_mul_relin(ckks_ctx *c, const ckks_ct *a, const ckks_ct *b, const ckks_evk *rlk, ckks_ct *out, void *ws,
                                  size_t ws_bytes, void *stream) {
    if (!c || !ct_ok(a) || !ct_ok(b) || !ct_ok(out) || a->ncomp != 2 || b->ncomp != 2) return CKKS_ERR_ARG;
    if (!level_ok(c, a->level) || a->level != b->level) return CKKS_ERR_LEVEL;
    if (!rlk || !rlk->data || rlk->galois != 0) return CKKS_ERR_NO_KEY;
    const uint32_t level = a->level;
    if (!ws || ws_bytes < ckks_workspace_bytes(c, CKKS_OP_MUL_RELIN, level, 0)) return CKKS_ERR_WORKSPACE;
    DeviceGuard g(c->device);
    cudaStream_t s = (cudaStream_t)stream;
    u64 *e2 = (u64 *)ws;
    KsWorkspace w = ks_carve(c, level, e2 + (size_t)level * c->N);
    u64 *o = (u64 *)out->data;
    launch_tensor(c, (const u64 *)a->data, (const u64 *)b->data, o, e2, level, s);
    ks_modup(c, e2, level, w, s);
    ks_inner_moddown(c, (const u64 *)rlk->data, level, 1, w, o, o + (size_t)level * c->N, 1, o, s);
    int rc = finish(c);
    if (rc == CKKS_OK) { out->level = level; out->ncomp = 2; out->scale = a->scale * b->scale; }
    return rc;
}

static int rotate_checks(const ckks_ctx *c, const ckks_ct *in, const ckks_evk *keys, uint32_t nrot, const ckks_ct *outs,
                         const void *ws, size_t ws_bytes) {
    if (!c || !ct_ok(in) || !keys || !outs || !nrot || in->ncomp != 2) return CKKS_ERR_ARG;
    if (!level_ok(c, in->level)) return CKKS_ERR_LEVEL;
    for (uint32_t r = 0; r < nrot; r++) {
        if (!outs[r].data || outs[r].data == in->data) return CKKS_ERR_ARG;
        if (!keys[r].data || !(keys[r].galois & 1) || keys[r].galois >= 2ull * c->N) return CKKS_ERR_NO_KEY;
    }
    if (!ws || ws_bytes < ks_bytes(c, in->level)) return CKKS_ERR_WORKSPACE;
    return CKKS_OK;
}

extern "C" int32_t ckks_mul_relin_batch(ckks_ctx *c, const ckks_ct *a, const ckks_ct *b, uint32_t n, const ckks_evk *rlk, ckks_ct *out,
                                        void *ws, size_t ws_bytes, void *stream) {
    if (!c || !a || !b || !out || !n) return CKKS_ERR_ARG;
    for (uint32_t i = 0; i < n; i++)
        if (!ct_ok(&a[i]) || !ct_ok(&b[i]) || !ct_ok(&out[i]) || a[i].ncomp != 2 || b[i].ncomp != 2) return CKKS_ERR_ARG;
    const uint32_t level = a[0].level;
    if (!level_ok(c, level)) return CKKS_ERR_LEVEL;
    for (uint32_t i = 0; i < n; i++)
        if (a[i].level != level || b[i].level != level) return CKKS_ERR_LEVEL;
    if (!rlk || !rlk->data || rlk->galois != 0) return CKKS_ERR_NO_KEY;
    if (!ws || ws_bytes < ckks_workspace_bytes(c, CKKS_OP_MUL_RELIN_BATCH, level, n)) return CKKS_ERR_WORKSPACE;
    DeviceGuard g(c->device);
    cudaStream_t s = (cudaStream_t)stream;
    const size_t N = c->N, ctl = (size_t)2 * level * N, ptl = (size_t)level * N;
    for (uint32_t i0 = 0; i0 < n; i0 += MRB_CHUNK) {
        const uint32_t m = std::min(MRB_CHUNK, n - i0);
        u64 *stage = (u64 *)ws, *e2 = stage + (size_t)m * ctl;
        KsWorkspace w = ks_carve(c, level, e2 + (size_t)m * ptl, m);
        for (uint32_t i = 0; i < m; i++)
            launch_tensor(c, (const u64 *)a[i0 + i].data, (const u64 *)b[i0 + i].data, stage + (size_t)i * ctl, e2 + (size_t)i * ptl, level, s);
        // the m key switches run side by side: one ModUp, one inner product, one ModDown over the whole chunk
        ks_modup(c, e2, level, w, s, m, ptl);
        ks_inner_moddown(c, (const u64 *)rlk->data, level, 1, w, stage, stage + ptl, 1, stage, s, m, ctl, ctl, false);
        for (uint32_t i = 0; i < m; i++)
            cudaMemcpyAsync(out[i0 + i].data, stage + (size_t)i * ctl, ctl * sizeof(u64), cudaMemcpyDeviceToDevice, s);
    }
    int rc = finish(c);
    if (rc == CKKS_OK)
        for (uint32_t i = 0; i < n; i++) { out[i].level = level; out[i].ncomp = 2; out[i].scale = a[i].scale * b[i].scale; }
    return rc;
}

extern "C" int32_t ckks_mul_relin_sum(ckks_ctx *c, const ckks_ct *a, const ckks_ct *b, uint32_t n, const ckks_evk *rlk, ckks_ct *out,
                                      void *ws, size_t ws_bytes, void *stream) {
    if (!c || !a || !b || !n || !ct_ok(out)) return CKKS_ERR_ARG;
    for (uint32_t i = 0; i < n; i++)
        if (!ct_ok(&a[i]) || !ct_ok(&b[i]) || a[i].ncomp != 2 || b[i].ncomp != 2) return CKKS_ERR_ARG;
    const uint32_t level = a[0].level;
    if (!level_ok(c, level)) return CKKS_ERR_LEVEL;
    for (uint32_t i = 0; i < n; i++) {
        if (a[i].level != level || b[i].level != level) return CKKS_ERR_LEVEL;
        if (!scales_agree(a[i].scale, a[0].scale) || !scales_agree(b[i].scale, b[0].scale)) return CKKS_ERR_SCALE;
        if (a[i].data == out->data || b[i].data == out->data) return CKKS_ERR_ARG;       // out is written before the last read
    }
    if (!rlk || !rlk->data || rlk->galois != 0) return CKKS_ERR_NO_KEY;
    if (!ws || ws_bytes < ckks_workspace_bytes(c, CKKS_OP_MUL_RELIN, level, 0)) return CKKS_ERR_WORKSPACE;
    DeviceGuard g(c->device);
    cudaStream_t s = (cudaStream_t)stream;
    u64 *e2 = (u64 *)ws;
    KsWorkspace w = ks_carve(c, level, e2 + (size_t)level * c->N);
    u64 *o = (u64 *)out->data;
    std::vector<const u64 *> pa(n), pb(n);
    for (uint32_t i = 0; i < n; i++) { pa[i] = (const u64 *)a[i].data; pb[i] = (const u64 *)b[i].data; }
    launch_tensor_sum(c, pa.data(), pb.data(), n, o, e2, level, s);
    ks_modup(c, e2, level, w, s);
    ks_inner_moddown(c, (const u64 *)rlk->data, level, 1, w, o, o + (size_t)level * c->N, 1, o, s);
    int rc = finish(c);
    if (rc == CKKS_OK) { out->level = level; out->ncomp = 2; out->scale = a[0].scale * b[0].scale; }
    return rc;
}

static bool const_value(double c, double scale, long long *v) {
    const double x = c * scale;
    if (!(fabs(x) < 4611686018427387904.0)) return false;      // 2^62; also rejects NaN
    *v = llrint(x);                                            // round half to even in the default rounding mode
    return true;
}

extern "C" int32_t ckks_mul_const(ckks_ctx *c, const ckks_ct *in, double cv, double cscale, ckks_ct *out, void *stream) {
    if (!c || !ct_ok(in) || !ct_ok(out) || !in->ncomp || in->ncomp > 3 || !(cscale >= 0.0) || !isfinite(cscale)) return CKKS_ERR_ARG;
    if (!level_ok(c, in->level)) return CKKS_ERR_LEVEL;
    const double cs = cscale > 0.0 ? cscale : (double)c->mod[in->level - 1];
    long long v;
    if (!const_value(cv, cs, &v)) return CKKS_ERR_RANGE;
    DeviceGuard g(c->device);
    launch_const(c, (const u64 *)in->data, v, true, (u64 *)out->data, in->ncomp, in->level, (cudaStream_t)stream);
    int rc = finish(c);
    if (rc == CKKS_OK) { out->level = in->level; out->ncomp = in->ncomp; out->scale = in->scale * cs; }
    return rc;
}

extern "C" int32_t ckks_add_const(ckks_ctx *c, const ckks_ct *in, double cv, ckks_ct *out, void *stream) {
    if (!c || !ct_ok(in) || !ct_ok(out) || !in->ncomp || in->ncomp > 3) return CKKS_ERR_ARG;
    if (!level_ok(c, in->level)) return CKKS_ERR_LEVEL;
    long long v;
    if (!const_value(cv, in->scale, &v)) return CKKS_ERR_RANGE;
    DeviceGuard g(c->device);
    launch_const(c, (const u64 *)in->data, v, false, (u64 *)out->data, in->ncomp, in->level, (cudaStream_t)stream);
    int rc = finish(c);
    if (rc == CKKS_OK) { out->level = in->level; out->ncomp = in->ncomp; out->scale = in->scale; }
    return rc;
}

extern "C" int32_t ckks_poly_eval(ckks_ctx *c, const ckks_ct *x, const double *coeffs, uint32_t degree, const ckks_evk *rlk, ckks_ct *out,
                                  void *ws, size_t ws_bytes, void *stream) {
    if (!c || !ct_ok(x) || !ct_ok(out) || x->ncomp != 2 || !coeffs || degree < 1) return CKKS_ERR_ARG;
    const uint32_t level = x->level;
    if (!level_ok(c, level) || level < degree + 1) return CKKS_ERR_LEVEL;
    if (degree > 1 && (!rlk || !rlk->data || rlk->galois != 0)) return CKKS_ERR_NO_KEY;
    if (!ws || ws_bytes < ckks_workspace_bytes(c, CKKS_OP_POLY_EVAL, level, 0)) return CKKS_ERR_WORKSPACE;
    // every constant is fixed (and range-checked) before anything is launched; the scales follow the documented order
    std::vector<long long> vs(degree + 1);
    std::vector<double> scales(degree + 1);
    {
        const double cs = (double)c->mod[level - 1];
        if (!const_value(coeffs[degree], cs, &vs[degree])) return CKKS_ERR_RANGE;
        double rs = x->scale * cs;
        rs = rs / (double)c->mod[level - 1];
        uint32_t lvl = level - 1;
        if (!const_value(coeffs[degree - 1], rs, &vs[degree - 1])) return CKKS_ERR_RANGE;
        scales[degree - 1] = rs;
        for (uint32_t k = degree - 1; k-- > 0;) {
            rs = rs * x->scale;
            rs = rs / (double)c->mod[lvl - 1];
            lvl--;
            if (!const_value(coeffs[k], rs, &vs[k])) return CKKS_ERR_RANGE;
            scales[k] = rs;
        }
    }
    DeviceGuard g(c->device);
    cudaStream_t s = (cudaStream_t)stream;
    const size_t N = c->N, ctw = (size_t)2 * level * N;
    u64 *ra = (u64 *)ws, *rb = ra + ctw, *xt = rb + ctw, *e2 = xt + ctw;
    u64 *ksw = e2 + (size_t)level * N;
    u64 *rsw = (u64 *)((char *)ksw + ks_bytes(c, level));
    const u64 *xd = (const u64 *)x->data;
    // r = x * c_d; rescale; + c_{d-1}
    launch_const(c, xd, vs[degree], true, ra, 2, level, s);
    launch_rescale(c, ra, rb, 2, level, rsw, s);
    uint32_t lvl = level - 1;
    launch_const(c, rb, vs[degree - 1], false, rb, 2, lvl, s);
    u64 *cur = rb, *other = ra;
    for (uint32_t k = degree - 1; k-- > 0;) {
        // x truncated to lvl limbs per component
        for (uint32_t comp = 0; comp < 2; comp++)
            cudaMemcpyAsync(xt + (size_t)comp * lvl * N, xd + (size_t)comp * level * N, (size_t)lvl * N * sizeof(u64), cudaMemcpyDeviceToDevice, s);
        KsWorkspace w = ks_carve(c, lvl, ksw);
        launch_tensor(c, cur, xt, other, e2, lvl, s);
        ks_modup(c, e2, lvl, w, s);
        ks_inner_moddown(c, (const u64 *)rlk->data, lvl, 1, w, other, other + (size_t)lvl * N, 1, other, s);
        launch_rescale(c, other, cur, 2, lvl, rsw, s);
        lvl--;
        launch_const(c, cur, vs[k], false, cur, 2, lvl, s);
    }
    cudaMemcpyAsync(out->data, cur, (size_t)2 * lvl * N * sizeof(u64), cudaMemcpyDeviceToDevice, s);
    int rc = finish(c);
    if (rc == CKKS_OK) { out->level = lvl; out->ncomp = 2; out->scale = scales[0]; }
    return rc;
}

extern "C" int32_t ckks_poly_eval_tree(ckks_ctx *c, const ckks_ct *x, const double *coeffs, uint32_t degree, const ckks_evk *rlk,
                                       ckks_ct *out, void *ws, size_t ws_bytes, void *stream) {
    if (!c || !ct_ok(x) || !ct_ok(out) || x->ncomp != 2 || !coeffs || degree < 2) return CKKS_ERR_ARG;
    const uint32_t level = x->level;
    uint32_t depth = 0;
    while ((1u << depth) < degree) depth++;
    if (!level_ok(c, level) || level < depth + 2) return CKKS_ERR_LEVEL;
    if (!rlk || !rlk->data || rlk->galois != 0) return CKKS_ERR_NO_KEY;
    if (!ws || ws_bytes < ckks_workspace_bytes(c, CKKS_OP_POLY_EVAL_TREE, level, degree)) return CKKS_ERR_WORKSPACE;
    // levels and scales of the powers, the combination's constants: all fixed and range-checked before the first launch
    std::vector<uint32_t> lvl(degree + 1);
    std::vector<double> sc(degree + 1);
    lvl[1] = level; sc[1] = x->scale;
    for (uint32_t k = 2; k <= degree; k++) {
        const uint32_t a = k / 2, b = k - a, lv = std::min(lvl[a], lvl[b]);
        sc[k] = sc[a] * sc[b] / (double)c->mod[lv - 1];
        lvl[k] = lv - 1;
    }
    const uint32_t Lt = lvl[degree];
    const double T = x->scale * (double)c->mod[Lt - 1], so = T / (double)c->mod[Lt - 1];
    std::vector<long long> vs(degree + 1, 0);
    bool any = false;
    for (uint32_t k = 1; k <= degree; k++) {
        if (coeffs[k] == 0.0) continue;
        any = true;
        if (!const_value(coeffs[k], T / sc[k], &vs[k])) return CKKS_ERR_RANGE;
    }
    if (!any) return CKKS_ERR_ARG;
    if (!const_value(coeffs[0], so, &vs[0])) return CKKS_ERR_RANGE;

    DeviceGuard g(c->device);
    cudaStream_t s = (cudaStream_t)stream;
    const size_t N = c->N, ctw = (size_t)2 * level * N;
    u64 *pw = (u64 *)ws;                                        // x^k at pw + (k - 2) * ctw, k >= 2
    u64 *ta = pw + (size_t)(degree - 1) * ctw, *tb = ta + ctw, *prod = tb + ctw, *acc = prod + ctw, *term = acc + ctw;
    u64 *e2 = term + ctw, *ksw = e2 + (size_t)level * N;
    u64 *rsw = (u64 *)((char *)ksw + ks_bytes(c, level));
    const u64 *xd = (const u64 *)x->data;
    auto power = [&](uint32_t k) { return k == 1 ? xd : pw + (size_t)(k - 2) * ctw; };
    // [2][from][N] -> [2][to][N], to <= from
    auto truncate = [&](const u64 *src, uint32_t from, uint32_t to, u64 *dst) {
        for (uint32_t comp = 0; comp < 2; comp++)
            cudaMemcpyAsync(dst + (size_t)comp * to * N, src + (size_t)comp * from * N, (size_t)to * N * sizeof(u64), cudaMemcpyDeviceToDevice, s);
    };
    for (uint32_t k = 2; k <= degree; k++) {
        const uint32_t a = k / 2, b = k - a, lv = std::min(lvl[a], lvl[b]);
        const u64 *pa = power(a), *pb = power(b);
        if (lvl[a] != lv) { truncate(pa, lvl[a], lv, ta); pa = ta; }
        if (lvl[b] != lv) { truncate(pb, lvl[b], lv, tb); pb = tb; }
        KsWorkspace w = ks_carve(c, lv, ksw);
        launch_tensor(c, pa, pb, prod, e2, lv, s);
        ks_modup(c, e2, lv, w, s);
        ks_inner_moddown(c, (const u64 *)rlk->data, lv, 1, w, prod, prod + (size_t)lv * N, 1, prod, s);
        launch_rescale(c, prod, pw + (size_t)(k - 2) * ctw, 2, lv, rsw, s);
    }
    bool first = true;
    for (uint32_t k = 1; k <= degree; k++) {
        if (coeffs[k] == 0.0) continue;
        const u64 *pk = power(k);
        if (lvl[k] != Lt) { truncate(pk, lvl[k], Lt, ta); pk = ta; }
        launch_const(c, pk, vs[k], true, first ? acc : term, 2, Lt, s);
        if (!first) launch_add(c, acc, term, acc, 2, Lt, s);
        first = false;
    }
    launch_rescale(c, acc, (u64 *)out->data, 2, Lt, rsw, s);
    launch_const(c, (const u64 *)out->data, vs[0], false, (u64 *)out->data, 2, Lt - 1, s);
    int rc = finish(c);
    if (rc == CKKS_OK) { out->level = Lt - 1; out->ncomp = 2; out->scale = so; }
    return rc;
}

// ---- Baby-step / giant-step polynomial evaluation: a composition of the entry points above
static bool bsgs_shape_ok(uint32_t degree, uint32_t m) { return m >= 2 && !(m & (m - 1)) && m <= degree; }
static size_t bsgs_scratch_bytes(const ckks_ctx *c, uint32_t level) {
    return align256(std::max(ckks_workspace_bytes(c, CKKS_OP_MUL_RELIN, level, 0), ckks_workspace_bytes(c, CKKS_OP_RESCALE, level, 0)));
}
static uint32_t bsgs_buffers(uint32_t degree, uint32_t m) {
    const uint32_t G = degree / m + 1;
    return (m - 1) + (G > 2 ? G - 2 : 0) + 2 * (G - 1) + 6;      // baby powers, giant powers, blocks and truncated giants, temporaries
}

extern "C" size_t ckks_poly_eval_bsgs_workspace_bytes(const ckks_ctx *c, uint32_t level, uint32_t degree, uint32_t m) {
    if (!c || !level_ok(c, level) || !bsgs_shape_ok(degree, m)) return 0;
    return (size_t)bsgs_buffers(degree, m) * align256((size_t)2 * level * c->N * sizeof(u64)) + bsgs_scratch_bytes(c, level);
}

extern "C" int32_t ckks_poly_eval_bsgs(ckks_ctx *c, const ckks_ct *x, const double *coeffs, uint32_t degree, uint32_t m, const ckks_evk *rlk,
                                       ckks_ct *out, void *ws, size_t ws_bytes, void *stream) {
    if (!c || !ct_ok(x) || !ct_ok(out) || x->ncomp != 2 || !coeffs || !bsgs_shape_ok(degree, m)) return CKKS_ERR_ARG;
    const uint32_t level = x->level, G = degree / m + 1;
    if (!level_ok(c, level)) return CKKS_ERR_LEVEL;
    if (!rlk || !rlk->data || rlk->galois != 0) return CKKS_ERR_NO_KEY;
    // levels of the powers (operands k / 2 and k - k / 2, one level per product)
    std::vector<uint32_t> lb(m + 1), lg(G);
    lb[1] = level;
    for (uint32_t k = 2; k <= m; k++) {
        const uint32_t lv = std::min(lb[k / 2], lb[k - k / 2]);
        if (lv < 2) return CKKS_ERR_LEVEL;
        lb[k] = lv - 1;
    }
    lg[1] = lb[m];
    for (uint32_t i = 2; i < G; i++) {
        const uint32_t lv = std::min(lg[i / 2], lg[i - i / 2]);
        if (lv < 2) return CKKS_ERR_LEVEL;
        lg[i] = lv - 1;
    }
    const uint32_t Lb = lb[m - 1], Lc = std::min(lg[G - 1], Lb - 1);
    if (Lb < 2 || Lc < 2) return CKKS_ERR_LEVEL;
    if (!ws || ws_bytes < ckks_poly_eval_bsgs_workspace_bytes(c, level, degree, m)) return CKKS_ERR_WORKSPACE;
    auto coef = [&](uint32_t k) { return k <= degree ? coeffs[k] : 0.0; };
    auto q = [&](uint32_t l) { return (double)c->mod[l - 1]; };

    const size_t N = c->N, ctb = align256((size_t)2 * level * N * sizeof(u64)), scratch = bsgs_scratch_bytes(c, level);
    char *base = (char *)ws;
    uint32_t next = 0;
    auto buffer = [&]() { return ckks_ct{(uint64_t *)(base + (size_t)(next++) * ctb), level, 2, 0.0}; };
    std::vector<ckks_ct> pw(m + 1), gp(G);
    pw[1] = *x;
    for (uint32_t k = 2; k <= m; k++) pw[k] = buffer();
    for (uint32_t i = 2; i < G; i++) gp[i] = buffer();
    std::vector<ckks_ct> blk(G), gpt(G);
    for (uint32_t i = 1; i < G; i++) { blk[i] = buffer(); gpt[i] = buffer(); }
    ckks_ct ta = buffer(), tb = buffer(), prod = buffer(), acc = buffer(), term = buffer(), S = buffer();
    void *sw = base + (size_t)bsgs_buffers(degree, m) * ctb;
    cudaStream_t s = (cudaStream_t)stream;
    DeviceGuard guard(c->device);
    // src cut down to `to` limbs per component (a copy into dst), or src itself if it has that many
    auto at_level = [&](const ckks_ct &src, uint32_t to, ckks_ct &dst) -> ckks_ct {
        if (src.level == to) return src;
        for (uint32_t comp = 0; comp < 2; comp++)
            cudaMemcpyAsync(dst.data + (size_t)comp * to * N, src.data + (size_t)comp * src.level * N, (size_t)to * N * sizeof(u64),
                            cudaMemcpyDeviceToDevice, s);
        dst.level = to; dst.ncomp = 2; dst.scale = src.scale;
        return dst;
    };
    int rc;
    auto powers = [&](std::vector<ckks_ct> &p, uint32_t top) -> int {
        for (uint32_t k = 2; k <= top; k++) {
            const uint32_t a = k / 2, b = k - a, lv = std::min(p[a].level, p[b].level);
            const ckks_ct pa = at_level(p[a], lv, ta), pb = at_level(p[b], lv, tb);
            int r;
            if ((r = ckks_mul_relin(c, &pa, &pb, rlk, &prod, sw, scratch, stream))) return r;
            if ((r = ckks_rescale(c, &prod, &p[k], sw, scratch, stream))) return r;
        }
        return CKKS_OK;
    };
    if ((rc = powers(pw, m))) return rc;
    gp[1] = pw[m];
    if ((rc = powers(gp, G - 1))) return rc;
    const double Tp = x->scale * q(Lc);
    // the blocks B_i, i >= 1, encoded so that B_i y^i has scale Tp; constant-only blocks are kept for later
    std::vector<ckks_ct> A, B;
    std::vector<uint32_t> const_only;
    for (uint32_t i = 1; i < G; i++) {
        const double Ti = (Tp / gp[i].scale) * q(Lb);
        bool first = true;
        for (uint32_t j = 1; j < m; j++) {
            if (coef(i * m + j) == 0.0) continue;
            const ckks_ct pj = at_level(pw[j], Lb, ta);
            ckks_ct &dst = first ? acc : term;
            if ((rc = ckks_mul_const(c, &pj, coef(i * m + j), Ti / pw[j].scale, &dst, stream))) return rc;
            if (!first && (rc = ckks_add(c, &acc, &term, &acc, stream))) return rc;
            first = false;
        }
        if (first) {
            if (coef(i * m) != 0.0) const_only.push_back(i);
            continue;
        }
        acc.scale = Ti;
        if ((rc = ckks_rescale(c, &acc, &prod, sw, scratch, stream))) return rc;
        if ((rc = ckks_add_const(c, &prod, coef(i * m), &prod, stream))) return rc;
        ckks_ct a = at_level(prod, Lc, blk[i]);
        if (a.data == prod.data) {       // already at the common level: keep a copy, prod is reused
            cudaMemcpyAsync(blk[i].data, prod.data, (size_t)2 * Lc * N * sizeof(u64), cudaMemcpyDeviceToDevice, s);
            blk[i].level = Lc; blk[i].ncomp = 2;
            a = blk[i];
        }
        ckks_ct b = at_level(gp[i], Lc, gpt[i]);
        a.scale = 1.0; b.scale = Tp;      // the products agree in scale (Tp up to rounding); the factors need not
        A.push_back(a); B.push_back(b);
    }
    bool have = false;
    if (!A.empty()) {
        if ((rc = ckks_mul_relin_sum(c, A.data(), B.data(), (uint32_t)A.size(), rlk, &S, sw, scratch, stream))) return rc;
        have = true;
    }
    auto add_in = [&](const ckks_ct &src, double cv, double cs) -> int {
        const ckks_ct p = at_level(src, Lc, ta);
        ckks_ct &dst = have ? term : S;
        int r;
        if ((r = ckks_mul_const(c, &p, cv, cs, &dst, stream))) return r;
        dst.scale = Tp;
        if (have && (r = ckks_add(c, &S, &term, &S, stream))) return r;
        have = true;
        return CKKS_OK;
    };
    S.scale = Tp;
    for (uint32_t j = 1; j < m; j++)
        if (coef(j) != 0.0 && (rc = add_in(pw[j], coef(j), Tp / pw[j].scale))) return rc;
    for (uint32_t i : const_only)
        if ((rc = add_in(gp[i], coef(i * m), Tp / gp[i].scale))) return rc;
    if (!have) return CKKS_ERR_ARG;
    S.scale = Tp;
    if ((rc = ckks_rescale(c, &S, out, sw, scratch, stream))) return rc;
    return ckks_add_const(c, out, coef(0), out, stream);
}

// ---- Softmax by doubling (Algorithm 1): a composition of the entry points above on buffers carved from the workspace
static uint32_t log2_ceil(uint32_t x) { uint32_t d = 0; while ((1u << d) < x) d++; return d; }
static size_t softmax_scratch_bytes(const ckks_ctx *c, const ckks_softmax_desc *d, uint32_t level) {
    const uint32_t deg = std::max(d->exp_degree, d->rsqrt_degree);
    size_t b = std::max(ckks_workspace_bytes(c, CKKS_OP_POLY_EVAL_TREE, level, deg),
                        std::max(ckks_workspace_bytes(c, CKKS_OP_MUL_RELIN, level, 0), ckks_workspace_bytes(c, CKKS_OP_RESCALE, level, 0)));
    if (d->exp_m) b = std::max(b, ckks_poly_eval_bsgs_workspace_bytes(c, level, d->exp_degree, d->exp_m));
    if (d->rsqrt_m && d->rounds) b = std::max(b, ckks_poly_eval_bsgs_workspace_bytes(c, level, d->rsqrt_degree, d->rsqrt_m));
    return align256(b);
}
static bool softmax_desc_ok(const ckks_ctx *c, const ckks_softmax_desc *d) {
    return d && d->exp_coeffs && d->exp_degree >= 2 && (d->rounds == 0 || (d->rsqrt_coeffs && d->rsqrt_degree >= 2)) && d->row_len >= 2 &&
           !(d->row_len & (d->row_len - 1)) && c->n % d->row_len == 0 && (!d->exp_m || bsgs_shape_ok(d->exp_degree, d->exp_m)) &&
           (!d->rsqrt_m || !d->rounds || bsgs_shape_ok(d->rsqrt_degree, d->rsqrt_m));
}

// The same polynomial of n ciphertexts: independent chains, spread over the context's lanes with a workspace each.
extern "C" size_t ckks_poly_eval_bsgs_batch_workspace_bytes(const ckks_ctx *c, uint32_t level, uint32_t degree, uint32_t m, uint32_t n) {
    const size_t one = ckks_poly_eval_bsgs_workspace_bytes(c, level, degree, m);
    return one ? align256(one) * std::min<uint32_t>(std::max<uint32_t>(n, 1), lane_count(c)) : 0;
}

extern "C" int32_t ckks_poly_eval_bsgs_batch(ckks_ctx *c, const ckks_ct *x, uint32_t n, const double *coeffs, uint32_t degree, uint32_t m,
                                             const ckks_evk *rlk, ckks_ct *out, void *ws, size_t ws_bytes, void *stream) {
    if (!c || !x || !out || !n) return CKKS_ERR_ARG;
    for (uint32_t i = 0; i < n; i++)
        if (!ct_ok(&x[i]) || !ct_ok(&out[i]) || x[i].level != x[0].level) return x && ct_ok(&x[i]) && ct_ok(&out[i]) ? CKKS_ERR_LEVEL : CKKS_ERR_ARG;
    const size_t one = align256(ckks_poly_eval_bsgs_workspace_bytes(c, x[0].level, degree, m));
    if (!one) return CKKS_ERR_ARG;
    const Lanes lanes(c, stream);
    const uint32_t nl = std::min<uint32_t>(n, lanes.n);
    if (!ws || ws_bytes < one * nl) return CKKS_ERR_WORKSPACE;
    int rc = CKKS_OK;
    lanes.fork();
    for (uint32_t i = 0; i < n && !rc; i++)
        rc = ckks_poly_eval_bsgs(c, &x[i], coeffs, degree, m, rlk, &out[i], (char *)ws + (size_t)(i % nl) * one, one, lanes.at(i % nl));
    lanes.join();
    return rc;
}

extern "C" size_t ckks_softmax_workspace_bytes(const ckks_ctx *c, const ckks_softmax_desc *d, uint32_t level) {
    if (!c || !softmax_desc_ok(c, d) || !level_ok(c, level)) return 0;
    return 4 * align256((size_t)2 * level * c->N * sizeof(u64)) + softmax_scratch_bytes(c, d, level);
}

extern "C" int32_t ckks_softmax(ckks_ctx *c, const ckks_softmax_desc *d, const ckks_ct *in, const ckks_evk *rlk, const ckks_evk *keys,
                                uint32_t nkeys, ckks_ct *out, void *ws, size_t ws_bytes, void *stream) {
    if (!c || !softmax_desc_ok(c, d) || !ct_ok(in) || !ct_ok(out) || in->ncomp != 2) return CKKS_ERR_ARG;
    const uint32_t level = in->level;
    const uint32_t de = log2_ceil(d->exp_degree), dr = d->rounds ? log2_ceil(d->rsqrt_degree) : 0;
    if (!level_ok(c, level)) return CKKS_ERR_LEVEL;
    if (!d->exp_m && !d->rsqrt_m && level < (de + 1) + d->rounds * (dr + 4) + 1) return CKKS_ERR_LEVEL;    // else the steps report it
    if (!rlk || !rlk->data || rlk->galois != 0) return CKKS_ERR_NO_KEY;
    const uint32_t stride = c->n / d->row_len;
    std::vector<const ckks_evk *> rk;
    for (uint32_t i = 1; i < d->row_len && d->rounds; i *= 2) {
        const ckks_evk *k = keys ? find_key(keys, nkeys, ckks_galois_element(c, (int64_t)stride * i)) : nullptr;
        if (!k) return CKKS_ERR_NO_KEY;
        rk.push_back(k);
    }
    if (!ws || ws_bytes < ckks_softmax_workspace_bytes(c, d, level)) return CKKS_ERR_WORKSPACE;
    const size_t ctb = align256((size_t)2 * level * c->N * sizeof(u64)), scratch = softmax_scratch_bytes(c, d, level);
    char *base = (char *)ws;
    ckks_ct U{(uint64_t *)base, level, 2, 0.0}, A{(uint64_t *)(base + ctb), level, 2, 0.0}, B{(uint64_t *)(base + 2 * ctb), level, 2, 0.0},
        S{(uint64_t *)(base + 3 * ctb), level, 2, 0.0};
    void *sw = base + 4 * ctb;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t N = c->N;
    int rc;
    // z = x - shift;  u = p_exp(z)
    if ((rc = ckks_add_const(c, in, -d->shift, &A, stream))) return rc;
    auto poly = [&](const ckks_ct *x, const double *co, uint32_t deg, uint32_t bm, ckks_ct *o) {
        return bm ? ckks_poly_eval_bsgs(c, x, co, deg, bm, rlk, o, sw, scratch, stream) : ckks_poly_eval_tree(c, x, co, deg, rlk, o, sw, scratch, stream);
    };
    if ((rc = poly(&A, d->exp_coeffs, d->exp_degree, d->exp_m, &U))) return rc;
    for (uint32_t j = 0; j < d->rounds; j++) {
        // s = row sums of u^2
        if ((rc = ckks_mul_relin(c, &U, &U, rlk, &A, sw, scratch, stream))) return rc;
        if ((rc = ckks_rescale(c, &A, &S, sw, scratch, stream))) return rc;
        for (const ckks_evk *k : rk) {
            if ((rc = ckks_rotate(c, &S, k, &A, sw, scratch, stream))) return rc;
            if ((rc = ckks_add(c, &S, &A, &S, stream))) return rc;
        }
        // lambda = p_rsqrt_j(s);  u = (lambda u)^2
        if ((rc = poly(&S, d->rsqrt_coeffs + (size_t)j * (d->rsqrt_degree + 1), d->rsqrt_degree, d->rsqrt_m, &B))) return rc;
        {
            DeviceGuard g(c->device);       // u truncated to lambda's level
            for (uint32_t comp = 0; comp < 2; comp++)
                cudaMemcpyAsync((u64 *)A.data + (size_t)comp * B.level * N, (const u64 *)U.data + (size_t)comp * U.level * N,
                                (size_t)B.level * N * sizeof(u64), cudaMemcpyDeviceToDevice, s);
            A.level = B.level; A.ncomp = 2; A.scale = U.scale;
        }
        if ((rc = ckks_mul_relin(c, &B, &A, rlk, &S, sw, scratch, stream))) return rc;
        if ((rc = ckks_rescale(c, &S, &A, sw, scratch, stream))) return rc;
        if ((rc = ckks_mul_relin(c, &A, &A, rlk, &S, sw, scratch, stream))) return rc;
        if ((rc = ckks_rescale(c, &S, &U, sw, scratch, stream))) return rc;
    }
    {
        DeviceGuard g(c->device);
        cudaMemcpyAsync(out->data, U.data, (size_t)2 * U.level * N * sizeof(u64), cudaMemcpyDeviceToDevice, s);
    }
    rc = finish(c);
    if (rc == CKKS_OK) { out->level = U.level; out->ncomp = 2; out->scale = U.scale; }
    return rc;
}

extern "C" int32_t ckks_rotate(ckks_ctx *c, const ckks_ct *in, const ckks_evk *key, ckks_ct *out, void *ws, size_t ws_bytes,
                               void *stream) {
    int rc = rotate_checks(c, in, key, 1, out, ws, ws_bytes);
    if (rc) return rc;
    DeviceGuard g(c->device);
    cudaStream_t s = (cudaStream_t)stream;
    const uint32_t level = in->level;
    KsWorkspace w = ks_carve(c, level, ws);
    const u64 *c0 = (const u64 *)in->data, *c1 = c0 + (size_t)level * c->N;
    ks_modup(c, c1, level, w, s);
    ks_inner_moddown(c, (const u64 *)key->data, level, key->galois, w, c0, nullptr, key->galois, (u64 *)out->data, s);
    rc = finish(c);
    if (rc == CKKS_OK) { out->level = level; out->ncomp = 2; out->scale = in->scale; }
    return rc;
}

extern "C" int32_t ckks_rotate_batch(ckks_ctx *c, const ckks_ct *in, uint32_t n, const ckks_evk *key, ckks_ct *out, void *ws,
                                     size_t ws_bytes, void *stream) {
    if (!c || !in || !out || !n) return CKKS_ERR_ARG;
    for (uint32_t i = 0; i < n; i++)
        if (!ct_ok(&in[i]) || !ct_ok(&out[i]) || in[i].ncomp != 2) return CKKS_ERR_ARG;
    const uint32_t level = in[0].level;
    if (!level_ok(c, level)) return CKKS_ERR_LEVEL;
    for (uint32_t i = 0; i < n; i++)
        if (in[i].level != level) return CKKS_ERR_LEVEL;
    if (!key || !key->data || key->galois == 0) return CKKS_ERR_NO_KEY;
    if (!ws || ws_bytes < ckks_workspace_bytes(c, CKKS_OP_ROTATE_BATCH, level, n)) return CKKS_ERR_WORKSPACE;
    DeviceGuard g(c->device);
    cudaStream_t s = (cudaStream_t)stream;
    const size_t N = c->N, ctl = (size_t)2 * level * N, ptl = (size_t)level * N;
    for (uint32_t i0 = 0; i0 < n; i0 += MRB_CHUNK) {
        const uint32_t m = std::min(MRB_CHUNK, n - i0);
        u64 *xin = (u64 *)ws, *xout = xin + (size_t)m * ctl;
        KsWorkspace w = ks_carve(c, level, xout + (size_t)m * ctl, m);
        for (uint32_t i = 0; i < m; i++)
            cudaMemcpyAsync(xin + (size_t)i * ctl, in[i0 + i].data, ctl * sizeof(u64), cudaMemcpyDeviceToDevice, s);
        ks_modup(c, xin + ptl, level, w, s, m, ctl);
        ks_inner_moddown(c, (const u64 *)key->data, level, key->galois, w, xin, nullptr, key->galois, xout, s, m, ctl, ctl, false);
        for (uint32_t i = 0; i < m; i++)
            cudaMemcpyAsync(out[i0 + i].data, xout + (size_t)i * ctl, ctl * sizeof(u64), cudaMemcpyDeviceToDevice, s);
    }
    int rc = finish(c);
    if (rc == CKKS_OK)
        for (uint32_t i = 0; i < n; i++) { out[i].level = level; out[i].ncomp = 2; out[i].scale = in[i].scale; }
    return rc;
}

extern "C" int32_t ckks_rotate_sum(ckks_ctx *c, const ckks_ct *in, const ckks_evk *keys, uint32_t n, ckks_ct *out, void *ws, size_t ws_bytes,
                                   void *stream) {
    if (!c || !in || !keys || !out || !n || !ct_ok(out)) return CKKS_ERR_ARG;
    for (uint32_t i = 0; i < n; i++)
        if (!ct_ok(&in[i]) || in[i].ncomp != 2) return CKKS_ERR_ARG;
    const uint32_t level = in[0].level;
    if (!level_ok(c, level)) return CKKS_ERR_LEVEL;
    for (uint32_t i = 0; i < n; i++) {
        if (in[i].level != level) return CKKS_ERR_LEVEL;
        if (!scales_agree(in[i].scale, in[0].scale)) return CKKS_ERR_SCALE;
        if (!keys[i].data || keys[i].galois == 0) return CKKS_ERR_NO_KEY;
    }
    if (!ws || ws_bytes < ckks_workspace_bytes(c, CKKS_OP_ROTATE_SUM, level, n)) return CKKS_ERR_WORKSPACE;
    DeviceGuard g(c->device);
    cudaStream_t s = (cudaStream_t)stream;
    const size_t N = c->N, ctl = (size_t)2 * level * N, ptl = (size_t)level * N;
    const uint32_t beta = (level + c->alpha - 1) / c->alpha, nt = level + c->K;
    const uint32_t mmax = std::min(MRB_CHUNK, n);
    u64 *xin = (u64 *)ws;
    KsWorkspace w = ks_carve(c, level, xin + (size_t)mmax * ctl, mmax);
    for (uint32_t i0 = 0; i0 < n; i0 += MRB_CHUNK) {
        const uint32_t m = std::min(MRB_CHUNK, n - i0);
        for (uint32_t i = 0; i < m; i++)
            cudaMemcpyAsync(xin + (size_t)i * ctl, in[i0 + i].data, ctl * sizeof(u64), cudaMemcpyDeviceToDevice, s);
        ks_modup(c, xin + ptl, level, w, s, m, ctl);
        // every term has its own digits, key and first component; all of them add into entry 0 of the inner-product
        // buffer, the first components multiplied by P so that the one ModDown returns them unchanged
        for (uint32_t t0 = 0; t0 < m; t0 += IP_TERMS) {
            const uint32_t nterm = std::min(IP_TERMS, m - t0);
            IpTerms tm{};
            for (uint32_t t = 0; t < nterm; t++) {
                tm.evk[t] = (const u64 *)keys[i0 + t0 + t].data;
                tm.galois[t] = keys[i0 + t0 + t].galois;
                tm.c0[t] = xin + (size_t)(t0 + t) * ctl;
            }
            KsWorkspace wt = w;
            wt.ext = w.ext + (size_t)t0 * beta * nt * N;
            ks_inner_terms(c, level, wt, (size_t)beta * nt * N, tm, nterm, 0, s, 1, i0 + t0 > 0);
        }
    }
    ks_moddown(c, level, w, nullptr, nullptr, 1, (u64 *)out->data, s);
    int rc = finish(c);
    if (rc == CKKS_OK) { out->level = level; out->ncomp = 2; out->scale = in[0].scale; }
    return rc;
}

extern "C" int32_t ckks_rotate_hoisted(ckks_ctx *c, const ckks_ct *in, const ckks_evk *keys, uint32_t nrot, ckks_ct *outs,
                                       void *ws, size_t ws_bytes, void *stream) {
    int rc = rotate_checks(c, in, keys, nrot, outs, ws, ws_bytes);
    if (rc) return rc;
    DeviceGuard g(c->device);
    cudaStream_t s = (cudaStream_t)stream;
    const uint32_t level = in->level;
    // as many rotations side by side as the workspace allows (one is always possible)
    uint32_t nbh = std::min<uint32_t>(nrot, KS_MULTI);
    while (nbh > 1 && hoisted_bytes(c, level, nbh) > ws_bytes) nbh--;
    const size_t beta = (level + c->alpha - 1) / c->alpha, nt = level + c->K, N = c->N;
    KsWorkspace w;
    w.dcoef = (u64 *)ws;
    w.ext = w.dcoef + (size_t)level * N;
    w.u = w.ext + beta * nt * N;
    w.conv = w.u + (size_t)nbh * 2 * nt * N;
    const u64 *c0 = (const u64 *)in->data, *c1 = c0 + (size_t)level * N;
    ks_modup(c, c1, level, w, s);
    for (uint32_t r0 = 0; r0 < nrot; r0 += nbh) {
        const uint32_t nb = std::min(nbh, nrot - r0);
        KsMulti m{};
        for (uint32_t b = 0; b < nb; b++) { m.evk[b] = (const u64 *)keys[r0 + b].data; m.galois[b] = keys[r0 + b].galois; m.out[b] = (u64 *)outs[r0 + b].data; }
        ks_inner_moddown(c, nullptr, level, 1, w, c0, nullptr, 1, nullptr, s, nb, 0, 0, false, TiledOut(), &m);
    }
    rc = finish(c);
    if (rc == CKKS_OK)
        for (uint32_t r = 0; r < nrot; r++) { outs[r].level = level; outs[r].ncomp = 2; outs[r].scale = in->scale; }
    return rc;
}

extern "C" int32_t ckks_rescale(ckks_ctx *c, const ckks_ct *in, ckks_ct *out, void *ws, size_t ws_bytes, void *stream) {
    if (!c || !ct_ok(in) || !out || !in->ncomp || in->ncomp > 3) return CKKS_ERR_ARG;
    if (!level_ok(c, in->level) || in->level < 2) return CKKS_ERR_LEVEL;
    if (!out->data || (in->ncomp > 1 && in->data == out->data)) return CKKS_ERR_ARG;
    if (!ws || ws_bytes < rescale_bytes(c, in->level, in->ncomp)) return CKKS_ERR_WORKSPACE;
    DeviceGuard g(c->device);
    launch_rescale(c, (const u64 *)in->data, (u64 *)out->data, in->ncomp, in->level, (u64 *)ws, (cudaStream_t)stream);
    int rc = finish(c);
    if (rc == CKKS_OK) {
        const double ql = (double)c->mod[in->level - 1];
        out->ncomp = in->ncomp; out->scale = in->scale / ql; out->level = in->level - 1;
    }
    return rc;
}

extern "C" int32_t ckks_linear_proj_rotations(const ckks_ctx *c, const ckks_proj_desc *d, int64_t *rots, uint32_t cap) {
    if (!c) return CKKS_ERR_ARG;
    ProjPlan p;
    int rc = make_plan(c, d, p);
    if (rc) return rc;
    for (uint32_t i = 0; i < p.rots.size() && i < cap && rots; i++) rots[i] = p.rots[i];
    return (int32_t)p.rots.size();
}

extern "C" size_t ckks_linear_proj_workspace_bytes(const ckks_ctx *c, const ckks_proj_desc *d, uint32_t level) {
    if (!c || !level_ok(c, level) || level < 2) return 0;
    ProjPlan p;
    if (make_plan(c, d, p)) return 0;
    return proj_layout(c, p, level, (d->flags & CKKS_PROJ_LAZY_MODDOWN) != 0).bytes;
}

// nmat projections of the same inputs (descriptors agreeing in d_in, tokens_per_shard, nshards, baby): the inputs'
// ModUp and baby-step rotations are done once, then every matrix runs its giant steps.  out: the outputs of matrix 0
// (nshards * its output blocks), then those of matrix 1, and so on.
static int32_t run_projections(ckks_ctx *c, const ckks_proj_desc *descs, uint32_t nmat, const ckks_ct *in, const double *const *Ws,
                               const ckks_evk *keys, uint32_t nkeys, ckks_ct *out, void *ws, size_t ws_bytes, void *stream) {
    if (!c || !descs || !nmat || !in || !Ws || !keys || !out) return CKKS_ERR_ARG;
    std::vector<ProjPlan> plans(nmat);
    ProjPlan merged;
    int rc;
    for (uint32_t m = 0; m < nmat; m++) {
        if (!Ws[m]) return CKKS_ERR_ARG;
        if ((rc = make_plan(c, &descs[m], plans[m]))) return rc;
        if (descs[m].d_in != descs[0].d_in || descs[m].tokens_per_shard != descs[0].tokens_per_shard || descs[m].nshards != descs[0].nshards ||
            descs[m].baby != descs[0].baby)
            return CKKS_ERR_ARG;
        if (descs[m].flags & ~CKKS_PROJ_LAZY_MODDOWN) return CKKS_ERR_ARG;
    }
    merged = plans[0];
    for (uint32_t m = 1; m < nmat; m++) merged.gmax = std::max(merged.gmax, plans[m].gmax);
    const ProjPlan &p0 = plans[0];
    const uint32_t nib = (uint32_t)p0.ins.size(), S = p0.S, B = p0.B, T = p0.T, N = c->N;
    const uint32_t level = in[0].level;
    if (!level_ok(c, level) || level < 2) return CKKS_ERR_LEVEL;
    for (uint32_t x = 0; x < S * nib; x++) {
        if (!in[x].data || in[x].ncomp != 2) return CKKS_ERR_ARG;
        if (in[x].level != level) return CKKS_ERR_LEVEL;
        if (!scales_agree(in[x].scale, in[0].scale)) return CKKS_ERR_SCALE;
    }
    uint32_t nout = 0;
    for (uint32_t m = 0; m < nmat; m++) {
        for (uint32_t x = 0; x < S * plans[m].outs.size(); x++)
            if (!out[nout + x].data) return CKKS_ERR_ARG;
        nout += S * (uint32_t)plans[m].outs.size();
        for (int64_t r : plans[m].rots)
            if (!find_key(keys, nkeys, ckks_galois_element(c, r))) return CKKS_ERR_NO_KEY;
    }
    bool any_lazy = false;
    for (uint32_t m = 0; m < nmat; m++) any_lazy = any_lazy || (descs[m].flags & CKKS_PROJ_LAZY_MODDOWN) != 0;
    const ProjWs L = proj_layout(c, merged, level, any_lazy, nmat);
    if (!ws || ws_bytes < L.bytes) return CKKS_ERR_WORKSPACE;

    DeviceGuard g(c->device);
    cudaStream_t s = (cudaStream_t)stream;
    char *base = (char *)ws;
    const size_t ctl = (size_t)2 * level * N, ptl = (size_t)level * N;
    u64 *baby = (u64 *)(base + L.baby), *pts = (u64 *)(base + L.pts), *acc = (u64 *)(base + L.acc);
    u64 *xin = (u64 *)(base + L.xin), *ptt = (u64 *)(base + L.ptt);
    u64 *total = (u64 *)(base + L.total), *rsw = (u64 *)(base + L.rs);
    double *slots = (double *)(base + L.slots);
    void *encw = base + L.enc;
    // baby row ((sh*nbb + ib)*B + b)*2 + comp = component comp of rho^(b T)(x_{sh,ib}), tiled layout: one ModUp for all
    // input ciphertexts of the block set at once, then every baby rotation is applied to all of them in one batch (the
    // key is read once per rotation, not once per shard) and written straight into the tiled buffer.  The block set is
    // all input blocks, or one block at a time (L.ib_outer): its inputs are then the ciphertexts ib, ib + nib, ..
    const uint32_t nbb = L.ib_outer ? 1 : nib;
    const uint32_t Jall = nbb * B, Rx = 2 * S * Jall;
    if (!L.ib_outer)
        for (uint32_t x = 0; x < S * nib; x++)
            cudaMemcpyAsync(xin + (size_t)x * ctl, in[x].data, ctl * sizeof(u64), cudaMemcpyDeviceToDevice, s);
    KsWorkspace kw = ks_carve(c, level, base + L.ks, S * nbb);
    // lazy giant steps: digits of IP_TERMS x S accumulators side by side; the running sum and the ModDown use kw's buffers
    const uint32_t kbeta = (level + c->alpha - 1) / c->alpha, knt = level + c->K;
    KsWorkspace kx = kw;
    kx.dcoef = (u64 *)(base + L.ksx);
    kx.ext = kx.dcoef + (size_t)IP_TERMS * S * level * N;
    auto baby_steps = [&](uint32_t ib0) {
        const u64 *xb = xin;                                           // first ciphertext of the set
        const size_t xs = ctl;                                         // from one ciphertext of the set to the next
        const uint32_t nx = S * nbb;
        if (L.ib_outer)
            for (uint32_t sh = 0; sh < S; sh++)
                cudaMemcpyAsync(xin + (size_t)sh * ctl, in[sh * nib + ib0].data, ctl * sizeof(u64), cudaMemcpyDeviceToDevice, s);
        for (uint32_t comp = 0; comp < 2; comp++)
            launch_to_tiled(c, xb + comp * ptl, xs, nx, baby, Rx, comp, 2 * B, level, s);
        if (B <= 1) return;
        ks_modup(c, xb + ptl, level, kw, s, nx, xs);
        // N = 2^16: BABY_ROTS rotations of all inputs per pass (the digits of a limb are fetched once for all of them and
        // the launches are four times larger); the inner-product and conversion buffers follow the digits
        const uint32_t rots = c->log_n == 16 ? BABY_ROTS : 1;       // the grouped ModDown tail exists for N = 2^16 only
        KsWorkspace kb = kw;
        kb.u = kw.ext + (size_t)nx * kbeta * knt * N;
        kb.conv = kb.u + (size_t)rots * nx * 2 * knt * N;
        for (uint32_t b = 1; b < B; b += rots) {
            const uint32_t nr = std::min(rots, B - b);
            TiledOut to;
            to.R = Rx; to.row0 = 2 * b; to.row_stride = 2 * B;
            if (rots == 1) {
                const u64 ge = ckks_galois_element(c, (int64_t)b * T);
                ks_inner_moddown(c, (const u64 *)find_key(keys, nkeys, ge)->data, level, ge, kw, xb, nullptr, ge, baby, s, nx, xs, 0,
                                 false, to);
                continue;
            }
            KsMulti m{};
            m.group = nx; m.rot_rows = 2;
            for (uint32_t r = 0; r < nr; r++) {
                m.galois[r] = ckks_galois_element(c, (int64_t)(b + r) * T);
                m.evk[r] = (const u64 *)find_key(keys, nkeys, m.galois[r])->data;
            }
            ks_inner_moddown(c, nullptr, level, 1, kb, xb, nullptr, 1, baby, s, nr * nx, xs, 0, false, to, &m);
        }
    };
    if (!L.ib_outer) baby_steps(0);

    ckks_ct *out_m = out;
    for (uint32_t m = 0; m < nmat; m++) {
        const ProjPlan &p = plans[m];
        const ckks_proj_desc *d = &descs[m];
        const double *W = Ws[m];
        const uint32_t nob = (uint32_t)p.outs.size();
        const double pt_scale = d->pt_scale > 0.0 ? d->pt_scale : (double)c->mod[level - 1];
        for (uint32_t ob = 0; ob < nob; ob++) {
            const Block &o = p.outs[ob];
            uint32_t gcount = 0, fold = 1;
            const bool lazy = (d->flags & CKKS_PROJ_LAZY_MODDOWN) != 0;
            bool u_live = false;        // the inner-product buffer holds a running sum of giant steps
            for (const Block &i : p.ins) {
                gcount = std::max(gcount, std::min(i.size, o.size) / B);
                if (i.size > o.size) fold = i.size / o.size;
            }
            // the giant steps of a group of accumulators accg (giants g0 .. g0 + ng - 1, all shards)
            auto giant_steps = [&](u64 *acc, uint32_t g0, uint32_t ng) {
                for (uint32_t gl = 0; gl < ng && !lazy; gl++) {
                    const uint32_t gi = g0 + gl;
                    u64 *ag = acc + (size_t)gl * S * ctl;
                    if (gi == 0) {
                        cudaMemcpyAsync(total, ag, (size_t)S * ctl * sizeof(u64), cudaMemcpyDeviceToDevice, s);
                        continue;
                    }
                    const u64 ge = ckks_galois_element(c, (int64_t)gi * B * T);
                    const u64 *key = (const u64 *)find_key(keys, nkeys, ge)->data;
                    // total[sh] += rotate(acc_g[sh]) for all shards in one batch
                    ks_modup(c, ag + ptl, level, kw, s, S, ctl);
                    ks_inner_moddown(c, key, level, ge, kw, ag, nullptr, ge, total, s, S, ctl, ctl, true);
                }
                // lazy: the key-switched parts of up to IP_TERMS giant steps (all shards) are extended in one batch and
                // added to the running sum in the key-switching basis in one pass, their first components with them
                for (uint32_t gl = 0; gl < ng && lazy;) {
                    if (g0 + gl == 0) {
                        cudaMemcpyAsync(total, acc, (size_t)S * ctl * sizeof(u64), cudaMemcpyDeviceToDevice, s);
                        gl++;
                        continue;
                    }
                    const uint32_t nterm = std::min(IP_TERMS, ng - gl);
                    u64 *ag = acc + (size_t)gl * S * ctl;
                    ks_modup(c, ag + ptl, level, kx, s, nterm * S, ctl);
                    IpTerms tm{};
                    for (uint32_t t = 0; t < nterm; t++) {
                        const u64 ge = ckks_galois_element(c, (int64_t)(g0 + gl + t) * B * T);
                        tm.evk[t] = (const u64 *)find_key(keys, nkeys, ge)->data;
                        tm.galois[t] = ge;
                        tm.c0[t] = ag + (size_t)t * S * ctl;
                    }
                    ks_inner_terms(c, level, kx, (size_t)S * kbeta * knt * N, tm, nterm, ctl, s, S, u_live);
                    u_live = true;
                    gl += nterm;
                }
            };
            // the diagonals of giants g0 .. g0 + ngi - 1 of a block pair, encoded into rows 0 .. ngi B - 1 of the tiled buffer
            auto encode_group = [&](const Block &i, uint32_t g0, uint32_t ngi) {
                for (uint32_t e0 = 0; e0 < ngi; e0 += L.eg) {
                    const uint32_t ne = std::min(L.eg, ngi - e0);
                    for (uint32_t gl = 0; gl < ne; gl++)
                        launch_extract_diagonals(c, W, d->d_out, i.start, i.size, o.start, o.size, p.F, T, (g0 + e0 + gl) * B, B,
                                                 (g0 + e0 + gl) * B, slots + (size_t)gl * B * c->n, s);
                    TiledOut to;
                    to.R = ngi * B; to.row0 = e0 * B; to.row_stride = 1;
                    launch_encode(c, slots, nullptr, ne * B, pt_scale, level, pts, encw, s, to, ptt);
                }
            };
            if (L.ib_outer) {
                // one input block at a time: its baby steps, then its share of every giant step's accumulator (block 0 is a
                // full block, so its launch initialises every accumulator it reaches); the giant steps follow at the end
                for (uint32_t ib = 0; ib < nib; ib++) {
                    const Block &i = p.ins[ib];
                    const uint32_t cnt = std::min(i.size, o.size) / B;
                    baby_steps(ib);
                    for (uint32_t g0 = 0; g0 < cnt; g0 += L.gg) {
                        const uint32_t ngi = std::min(L.gg, cnt - g0);
                        u64 *accg = acc + (size_t)g0 * S * ctl;
                        const bool covered = ib > 0 || ngi == std::min(L.gg, gcount - g0);
                        if (ib == 0 && !covered) cudaMemsetAsync(accg, 0, (size_t)std::min(L.gg, gcount - g0) * S * ctl * sizeof(u64), s);
                        encode_group(i, g0, ngi);
                        launch_mac_mma(c, baby, ptt, accg, B, S, ngi, level, s, B, 0, ib > 0 || !covered);
                    }
                }
                for (uint32_t g0 = 0; g0 < gcount; g0 += L.gg) giant_steps(acc + (size_t)g0 * S * ctl, g0, std::min(L.gg, gcount - g0));
            } else
            for (uint32_t g0 = 0; g0 < gcount; g0 += L.gg) {
                const uint32_t ng = std::min(L.gg, gcount - g0);
                const uint32_t J = nib * B;
                if (L.per_block) {
                    // one input block at a time: encode its ng x B diagonals, multiply-accumulate them with that block's
                    // baby rows into the group's accumulators.  A block that has run out of diagonals takes part with
                    // fewer giants; the accumulators are then cleared first so that every launch can accumulate.
                    bool full0 = g0 + ng <= std::min(p.ins[0].size, o.size) / B;
                    if (!full0) cudaMemsetAsync(acc, 0, (size_t)ng * S * ctl * sizeof(u64), s);
                    for (uint32_t ib = 0; ib < nib; ib++) {
                        const Block &i = p.ins[ib];
                        const uint32_t cnt = std::min(i.size, o.size) / B;
                        if (g0 >= cnt) continue;
                        const uint32_t ngi = std::min(ng, cnt - g0);
                        encode_group(i, g0, ngi);
                        launch_mac_mma(c, baby, ptt, acc, B, S, ngi, level, s, J, ib * B, !full0 || ib > 0);
                    }
                } else {
                // plaintexts of the group: pts[(gl * nib + ib) * B + b]; a block pair that has run out of diagonals
                // contributes zero plaintexts
                bool ragged = false;
                for (uint32_t gl = 0; gl < ng; gl++)
                    for (uint32_t ib = 0; ib < nib; ib++)
                        if (g0 + gl >= std::min(p.ins[ib].size, o.size) / B) ragged = true;
                if (ragged) cudaMemsetAsync(ptt, 0, (size_t)ng * J * ptl * sizeof(u64), s);
                for (uint32_t gl = 0; gl < ng; gl++)
                    for (uint32_t ib = 0; ib < nib; ib++) {
                        const Block &i = p.ins[ib];
                        const uint32_t gi = g0 + gl;
                        if (gi >= std::min(i.size, o.size) / B) continue;
                        const size_t idx = ((size_t)gl * nib + ib) * B;
                        launch_extract_diagonals(c, W, d->d_out, i.start, i.size, o.start, o.size, p.F, T, gi * B, B, gi * B,
                                                 slots + idx * c->n, s);
                        if (ragged) {
                            TiledOut to;
                            to.R = ng * J; to.row0 = (uint32_t)idx; to.row_stride = 1;
                            launch_encode(c, slots + idx * c->n, nullptr, B, pt_scale, level, pts + idx * ptl, encw, s, to, ptt);
                        }
                    }
                if (!ragged) {
                    TiledOut to;
                    to.R = ng * J; to.row0 = 0; to.row_stride = 1;
                    launch_encode(c, slots, nullptr, ng * J, pt_scale, level, pts, encw, s, to, ptt);
                }
                if (!launch_mac_mma(c, baby, ptt, acc, J, S, ng, level, s)) launch_mac_tile(c, baby, ptt, acc, J, S, ng, level, s);
                }
                giant_steps(acc, g0, ng);
            }
            if (u_live) ks_moddown(c, level, kw, total, total + ptl, 1, total, s, S, ctl, ctl, false);
            for (uint32_t f = o.size; fold > 1; f *= 2, fold /= 2) {
                const u64 ge = ckks_galois_element(c, (int64_t)f * T);
                const u64 *key = (const u64 *)find_key(keys, nkeys, ge)->data;
                // total += rotate(total): the rotated copy goes to the (now free) accumulator buffer first
                ks_modup(c, total + ptl, level, kw, s, S, ctl);
                ks_inner_moddown(c, key, level, ge, kw, total, nullptr, ge, acc, s, S, ctl, ctl, false);
                for (uint32_t sh = 0; sh < S; sh++)
                    launch_add(c, total + (size_t)sh * ctl, acc + (size_t)sh * ctl, total + (size_t)sh * ctl, 2, level, s);
            }
            for (uint32_t sh = 0; sh < S; sh++)
                launch_rescale(c, total + (size_t)sh * ctl, (u64 *)out_m[sh * nob + ob].data, 2, level, rsw, s);
        }
        out_m += S * nob;
    }
    rc = finish(c);
    if (rc == CKKS_OK) {
        out_m = out;
        for (uint32_t m = 0; m < nmat; m++) {
            const uint32_t nob = (uint32_t)plans[m].outs.size();
            const double pt_scale = descs[m].pt_scale > 0.0 ? descs[m].pt_scale : (double)c->mod[level - 1];
            for (uint32_t x = 0; x < S * nob; x++) {
                out_m[x].level = level - 1; out_m[x].ncomp = 2;
                out_m[x].scale = in[0].scale * pt_scale / (double)c->mod[level - 1];
            }
            out_m += S * nob;
        }
    }
    return rc;
}

extern "C" int32_t ckks_linear_proj(ckks_ctx *c, const ckks_proj_desc *d, const ckks_ct *in, const double *W, const ckks_evk *keys,
                                    uint32_t nkeys, ckks_ct *out, void *ws, size_t ws_bytes, void *stream) {
    if (!d || !W) return CKKS_ERR_ARG;
    return run_projections(c, d, 1, in, &W, keys, nkeys, out, ws, ws_bytes, stream);
}

extern "C" int32_t ckks_linear_proj_multi(ckks_ctx *c, const ckks_proj_desc *descs, uint32_t nmat, const ckks_ct *in, const double *const *W,
                                          const ckks_evk *keys, uint32_t nkeys, ckks_ct *out, void *ws, size_t ws_bytes, void *stream) {
    return run_projections(c, descs, nmat, in, W, keys, nkeys, out, ws, ws_bytes, stream);
}

extern "C" size_t ckks_linear_proj_multi_workspace_bytes(const ckks_ctx *c, const ckks_proj_desc *descs, uint32_t nmat, uint32_t level) {
    if (!c || !descs || !nmat || !level_ok(c, level) || level < 2) return 0;
    ProjPlan merged;
    if (make_plan(c, &descs[0], merged)) return 0;
    bool lazy = (descs[0].flags & CKKS_PROJ_LAZY_MODDOWN) != 0;
    for (uint32_t m = 1; m < nmat; m++) {
        ProjPlan p;
        if (make_plan(c, &descs[m], p)) return 0;
        merged.gmax = std::max(merged.gmax, p.gmax);
        lazy = lazy || (descs[m].flags & CKKS_PROJ_LAZY_MODDOWN) != 0;
    }
    return proj_layout(c, merged, level, lazy, nmat).bytes;
}

// Attention in the diagonal-block layout: compositions of the entry points of api.cu on buffers carved from the caller's
// workspace.  No kernels of its own.
//
// Layout.  Every operand and every score ciphertext uses the slot index
//     slot = ((e * tokens + i) * heads + h) * R + r,      R = n / (diag_block * tokens * heads),
// i a token position, h a head, e < diag_block one of the score diagonals a ciphertext holds side by side, r trailing
// copies.  One ciphertext per channel d: the query operand repeats Q[i, h, d] in every block e, the key and value
// operands hold token (i + e) mod tokens in block e.  A left rotation by g * diag_block token positions (that many times
// heads * R slots) of a key operand is cyclic over the flattened (e, i) index, so
//     S_g = sum_d q[d] * rot_g(k[d])
// holds in slot (e, i, h) the score of query i against one key token, and over g < tokens / diag_block and e every key
// token occurs exactly once: the score row of (i, h) is the set of slots (e, i, h) of all S_g.  Softmax needs nothing
// else (its row sums are ciphertext additions over g and a rotate-and-add ladder over e, which is cyclic because e is
// the slowest index), and the probabilities meet the value operands, rotated the same way, slot by slot.
#include <algorithm>
#include <vector>

#include "common.cuh"

namespace {

struct AttnPlan {
    uint32_t E, Tk, H, R, G, Gb;
    std::vector<int64_t> tok, lad, neg;      // rotations in slots (neg: the query operands' right rotations of the split)
};

bool pow2(uint32_t x) { return x && !(x & (x - 1)); }

int make_attn_plan(const ckks_ctx *c, const ckks_attn_desc *d, AttnPlan &p) {
    if (!d || !d->tokens || !d->heads || !d->diag_block) return CKKS_ERR_ARG;
    if (!pow2(d->tokens) || !pow2(d->diag_block) || d->tokens % d->diag_block) return CKKS_ERR_UNSUPPORTED;
    const uint64_t block = (uint64_t)d->diag_block * d->tokens * d->heads;
    if (block > c->n || c->n % block) return CKKS_ERR_UNSUPPORTED;
    p.E = d->diag_block; p.Tk = d->tokens; p.H = d->heads; p.R = (uint32_t)(c->n / block); p.G = p.Tk / p.E;
    for (uint32_t g = 1; g < p.G; g++) p.tok.push_back((int64_t)g * p.E * p.H * p.R);
    for (uint32_t k = 1; k < p.E; k *= 2) p.lad.push_back((int64_t)p.Tk * p.H * p.R * k);
    p.Gb = d->group_baby ? d->group_baby : 1;
    if (!pow2(p.Gb) || p.G % p.Gb) return CKKS_ERR_UNSUPPORTED;
    if (p.Gb > 1)
        for (uint32_t g1 = 1; g1 < p.G / p.Gb; g1++) p.neg.push_back(-p.tok[g1 * p.Gb - 1]);
    return CKKS_OK;
}

const ckks_evk *find_key(const ckks_ctx *c, const ckks_evk *keys, uint32_t nkeys, int64_t rot) {
    const uint64_t g = ckks_galois_element(c, rot);
    for (uint32_t i = 0; i < nkeys; i++)
        if (keys[i].galois == g && keys[i].data) return &keys[i];
    return nullptr;
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
size_t ct_bytes(const ckks_ctx *c, uint32_t level) { return align256((size_t)2 * level * c->N * sizeof(uint64_t)); }
size_t scratch_bytes(const ckks_ctx *c, uint32_t level, uint32_t nrot) {
    return align256(std::max({ckks_workspace_bytes(c, CKKS_OP_MUL_RELIN, level, 0), ckks_workspace_bytes(c, CKKS_OP_RESCALE, level, 0),
                              ckks_workspace_bytes(c, CKKS_OP_ROTATE_HOISTED, level, nrot ? nrot : 1),
                              ckks_workspace_bytes(c, CKKS_OP_ROTATE, level, 0)}));
}

// s += rotate(s, r) for the ladder rotations in ascending order; tmp: a ciphertext buffer
int block_ladder(ckks_ctx *c, const AttnPlan &p, const ckks_evk *keys, uint32_t nkeys, ckks_ct *s, ckks_ct *tmp, void *sw, size_t sw_bytes,
                 void *stream) {
    for (int64_t r : p.lad) {
        int rc;
        if ((rc = ckks_rotate(c, s, find_key(c, keys, nkeys, r), tmp, sw, sw_bytes, stream))) return rc;
        if ((rc = ckks_add(c, s, tmp, s, stream))) return rc;
    }
    return CKKS_OK;
}

int check_cts(const ckks_ctx *c, const ckks_ct *cts, uint32_t n, uint32_t *level, bool same_scale) {
    if (!cts || !n) return CKKS_ERR_ARG;
    for (uint32_t i = 0; i < n; i++)
        if (!cts[i].data || cts[i].ncomp != 2) return CKKS_ERR_ARG;
    *level = cts[0].level;
    if (*level < 1 || *level > c->L) return CKKS_ERR_LEVEL;
    for (uint32_t i = 0; i < n; i++) {
        if (cts[i].level != *level) return CKKS_ERR_LEVEL;
        if (same_scale && fabs(cts[i].scale - cts[0].scale) > ldexp(fabs(cts[0].scale), -30)) return CKKS_ERR_SCALE;
    }
    return CKKS_OK;
}

bool rlk_ok(const ckks_evk *rlk) { return rlk && rlk->data && rlk->galois == 0; }

uint32_t log2_ceil(uint32_t x) { uint32_t d = 0; while ((1u << d) < x) d++; return d; }

}  // namespace

extern "C" int32_t ckks_attention_rotations(const ckks_ctx *c, const ckks_attn_desc *d, int64_t *rots, uint32_t cap) {
    if (!c) return CKKS_ERR_ARG;
    AttnPlan p;
    int rc = make_attn_plan(c, d, p);
    if (rc) return rc;
    uint32_t k = 0;
    for (int64_t r : p.tok) { if (rots && k < cap) rots[k] = r; k++; }
    for (int64_t r : p.lad) { if (rots && k < cap) rots[k] = r; k++; }
    for (int64_t r : p.neg) { if (rots && k < cap) rots[k] = r; k++; }
    return (int32_t)k;
}

// ---- scores -------------------------------------------------------------------------------------------------------
// workspace: [pass groups][dim] rotated key operands, one product, the scratch of the calls
extern "C" size_t ckks_attention_scores_workspace_bytes(const ckks_ctx *c, const ckks_attn_desc *d, uint32_t level, uint32_t dim) {
    AttnPlan p;
    if (!c || !dim || level < 2 || level > c->L || make_attn_plan(c, d, p)) return 0;
    // the split holds Gb - 1 rotated key sets, G / Gb - 1 rotated query sets, a product and a rescaled product
    if (p.Gb > 1) return (size_t)(p.Gb + p.G / p.Gb - 2) * dim * ct_bytes(c, level) + 2 * ct_bytes(c, level) + scratch_bytes(c, level, p.G - 1);
    return (size_t)(p.G - 1) * dim * ct_bytes(c, level) + ct_bytes(c, level) + scratch_bytes(c, level, p.G - 1);
}

// scores with the groups split into Gb baby and G / Gb giant steps
static int scores_split(ckks_ctx *c, const AttnPlan &p, const ckks_ct *q, const ckks_ct *k, uint32_t dim, uint32_t level, const ckks_evk *rlk,
                        const ckks_evk *keys, uint32_t nkeys, ckks_ct *scores, void *ws, size_t ws_bytes, void *stream) {
    const uint32_t Gb = p.Gb, Gg = p.G / p.Gb;
    const size_t ctb = ct_bytes(c, level);
    char *base = (char *)ws;
    char *kr = base, *qr = base + (size_t)(Gb - 1) * dim * ctb;         // [Gb - 1][dim], [Gg - 1][dim] ciphertexts
    char *rest = qr + (size_t)(Gg - 1) * dim * ctb;
    ckks_ct prod{(uint64_t *)rest, level, 2, 0.0}, resc{(uint64_t *)(rest + ctb), level - 1, 2, 0.0};
    void *sw = rest + 2 * ctb;
    const size_t sw_bytes = ws_bytes - (size_t)((char *)sw - base);
    int rc;
    std::vector<ckks_evk> bk, gk;
    for (uint32_t g0 = 1; g0 < Gb; g0++) bk.push_back(*find_key(c, keys, nkeys, p.tok[g0 - 1]));
    for (int64_t r : p.neg) gk.push_back(*find_key(c, keys, nkeys, r));
    std::vector<ckks_ct> outs(std::max(Gb, Gg));
    for (uint32_t dd = 0; dd < dim; dd++) {
        for (uint32_t x = 0; x + 1 < Gb; x++) outs[x] = ckks_ct{(uint64_t *)(kr + ((size_t)x * dim + dd) * ctb), level, 2, 0.0};
        if (Gb > 1 && (rc = ckks_rotate_hoisted(c, &k[dd], bk.data(), Gb - 1, outs.data(), sw, sw_bytes, stream))) return rc;
        for (uint32_t y = 0; y + 1 < Gg; y++) outs[y] = ckks_ct{(uint64_t *)(qr + ((size_t)y * dim + dd) * ctb), level, 2, 0.0};
        if (Gg > 1 && (rc = ckks_rotate_hoisted(c, &q[dd], gk.data(), Gg - 1, outs.data(), sw, sw_bytes, stream))) return rc;
    }
    std::vector<ckks_ct> a(dim), b(dim);
    for (uint32_t g = 0; g < p.G; g++) {
        const uint32_t g1 = g / Gb, g0 = g % Gb;
        for (uint32_t dd = 0; dd < dim; dd++) {
            a[dd] = g1 ? ckks_ct{(uint64_t *)(qr + ((size_t)(g1 - 1) * dim + dd) * ctb), level, 2, q[dd].scale} : q[dd];
            b[dd] = g0 ? ckks_ct{(uint64_t *)(kr + ((size_t)(g0 - 1) * dim + dd) * ctb), level, 2, k[dd].scale} : k[dd];
        }
        if ((rc = ckks_mul_relin_sum(c, a.data(), b.data(), dim, rlk, &prod, sw, sw_bytes, stream))) return rc;
        if (!g1) {
            if ((rc = ckks_rescale(c, &prod, &scores[g], sw, sw_bytes, stream))) return rc;
            continue;
        }
        if ((rc = ckks_rescale(c, &prod, &resc, sw, sw_bytes, stream))) return rc;
        if ((rc = ckks_rotate(c, &resc, find_key(c, keys, nkeys, p.tok[g1 * Gb - 1]), &scores[g], sw, sw_bytes, stream))) return rc;
    }
    return CKKS_OK;
}

extern "C" int32_t ckks_attention_scores(ckks_ctx *c, const ckks_attn_desc *d, const ckks_ct *q, const ckks_ct *k, uint32_t dim,
                                         const ckks_evk *rlk, const ckks_evk *keys, uint32_t nkeys, ckks_ct *scores, void *ws, size_t ws_bytes,
                                         void *stream) {
    if (!c || !scores) return CKKS_ERR_ARG;
    AttnPlan p;
    int rc = make_attn_plan(c, d, p);
    if (rc) return rc;
    uint32_t level, lk;
    if ((rc = check_cts(c, q, dim, &level, true)) || (rc = check_cts(c, k, dim, &lk, true))) return rc;
    if (lk != level || level < 2) return CKKS_ERR_LEVEL;
    if (!rlk_ok(rlk)) return CKKS_ERR_NO_KEY;
    for (int64_t r : p.tok)
        if (!keys || !find_key(c, keys, nkeys, r)) return CKKS_ERR_NO_KEY;
    for (int64_t r : p.neg)
        if (!find_key(c, keys, nkeys, r)) return CKKS_ERR_NO_KEY;
    for (uint32_t g = 0; g < p.G; g++)
        if (!scores[g].data) return CKKS_ERR_ARG;
    if (p.Gb > 1) {
        if (!ws || ws_bytes < ckks_attention_scores_workspace_bytes(c, d, level, dim)) return CKKS_ERR_WORKSPACE;
        return scores_split(c, p, q, k, dim, level, rlk, keys, nkeys, scores, ws, ws_bytes, stream);
    }
    // as many groups per pass as the workspace holds (one at least)
    const size_t ctb = ct_bytes(c, level), fixed = ctb + scratch_bytes(c, level, p.G - 1);
    uint32_t per_pass = p.G > 1 ? (uint32_t)std::min<size_t>(p.G - 1, ws_bytes > fixed ? (ws_bytes - fixed) / ((size_t)dim * ctb) : 0) : 0;
    if (!ws || ws_bytes < fixed || (p.G > 1 && per_pass == 0)) return CKKS_ERR_WORKSPACE;
    char *base = (char *)ws;
    char *rk = base;                                                     // [per_pass][dim] ciphertexts
    ckks_ct prod{(uint64_t *)(base + (size_t)per_pass * dim * ctb), level, 2, 0.0};
    void *sw = base + (size_t)per_pass * dim * ctb + ctb;
    const size_t sw_bytes = ws_bytes - ((size_t)per_pass * dim * ctb + ctb);
    // group 0: the key operands as they are
    if ((rc = ckks_mul_relin_sum(c, q, k, dim, rlk, &prod, sw, sw_bytes, stream))) return rc;
    if ((rc = ckks_rescale(c, &prod, &scores[0], sw, sw_bytes, stream))) return rc;
    std::vector<ckks_evk> pk(per_pass);
    std::vector<ckks_ct> outs(per_pass), kr(dim);
    for (uint32_t g0 = 1; g0 < p.G; g0 += per_pass) {
        const uint32_t ng = std::min(per_pass, p.G - g0);
        for (uint32_t x = 0; x < ng; x++) pk[x] = *find_key(c, keys, nkeys, p.tok[g0 - 1 + x]);
        // every key operand is extended once and rotated to the pass's groups off the shared digits
        for (uint32_t dd = 0; dd < dim; dd++) {
            for (uint32_t x = 0; x < ng; x++) outs[x] = ckks_ct{(uint64_t *)(rk + ((size_t)x * dim + dd) * ctb), level, 2, 0.0};
            if ((rc = ckks_rotate_hoisted(c, &k[dd], pk.data(), ng, outs.data(), sw, sw_bytes, stream))) return rc;
        }
        for (uint32_t x = 0; x < ng; x++) {
            for (uint32_t dd = 0; dd < dim; dd++) kr[dd] = ckks_ct{(uint64_t *)(rk + ((size_t)x * dim + dd) * ctb), level, 2, k[dd].scale};
            if ((rc = ckks_mul_relin_sum(c, q, kr.data(), dim, rlk, &prod, sw, sw_bytes, stream))) return rc;
            if ((rc = ckks_rescale(c, &prod, &scores[g0 + x], sw, sw_bytes, stream))) return rc;
        }
    }
    return CKKS_OK;
}

// ---- Softmax over rows spread across the groups ---------------------------------------------------------------------
static bool rows_desc_ok(const ckks_softmax_desc *s) {
    return s && s->exp_coeffs && s->exp_degree >= 2 && (s->rounds == 0 || (s->rsqrt_coeffs && s->rsqrt_degree >= 2));
}
static size_t rows_scratch(const ckks_ctx *c, const ckks_softmax_desc *s, uint32_t level) {
    return align256(std::max({ckks_workspace_bytes(c, CKKS_OP_POLY_EVAL_TREE, level, std::max(s->exp_degree, s->rsqrt_degree)),
                              ckks_workspace_bytes(c, CKKS_OP_MUL_RELIN, level, 0), ckks_workspace_bytes(c, CKKS_OP_RESCALE, level, 0),
                              ckks_workspace_bytes(c, CKKS_OP_ROTATE, level, 0)}));
}

// workspace: the groups' running ciphertexts u_g, four temporaries, the scratch of the calls
extern "C" size_t ckks_softmax_rows_workspace_bytes(const ckks_ctx *c, const ckks_attn_desc *d, const ckks_softmax_desc *s, uint32_t level) {
    AttnPlan p;
    if (!c || level < 1 || level > c->L || !rows_desc_ok(s) || make_attn_plan(c, d, p)) return 0;
    return (size_t)(p.G + 4) * ct_bytes(c, level) + rows_scratch(c, s, level);
}

extern "C" int32_t ckks_softmax_rows(ckks_ctx *c, const ckks_attn_desc *d, const ckks_softmax_desc *s, const ckks_ct *in, const ckks_evk *rlk,
                                     const ckks_evk *keys, uint32_t nkeys, ckks_ct *out, void *ws, size_t ws_bytes, void *stream) {
    if (!c || !out || !rows_desc_ok(s)) return CKKS_ERR_ARG;
    AttnPlan p;
    int rc = make_attn_plan(c, d, p);
    if (rc) return rc;
    uint32_t level;
    if ((rc = check_cts(c, in, p.G, &level, true))) return rc;
    const uint32_t de = log2_ceil(s->exp_degree), dr = s->rounds ? log2_ceil(s->rsqrt_degree) : 0;
    if (level < (de + 1) + s->rounds * (dr + 4) + 1) return CKKS_ERR_LEVEL;
    if (!rlk_ok(rlk)) return CKKS_ERR_NO_KEY;
    for (int64_t r : p.lad)
        if (s->rounds && (!keys || !find_key(c, keys, nkeys, r))) return CKKS_ERR_NO_KEY;
    for (uint32_t g = 0; g < p.G; g++)
        if (!out[g].data) return CKKS_ERR_ARG;
    if (!ws || ws_bytes < ckks_softmax_rows_workspace_bytes(c, d, s, level)) return CKKS_ERR_WORKSPACE;
    const size_t ctb = ct_bytes(c, level), N = c->N;
    char *base = (char *)ws;
    std::vector<ckks_ct> u(p.G);
    for (uint32_t g = 0; g < p.G; g++) u[g] = ckks_ct{(uint64_t *)(base + (size_t)g * ctb), level, 2, 0.0};
    ckks_ct A{(uint64_t *)(base + (size_t)p.G * ctb), level, 2, 0.0}, B{(uint64_t *)(base + (size_t)(p.G + 1) * ctb), level, 2, 0.0},
        T{(uint64_t *)(base + (size_t)(p.G + 2) * ctb), level, 2, 0.0}, X{(uint64_t *)(base + (size_t)(p.G + 3) * ctb), level, 2, 0.0};
    void *sw = base + (size_t)(p.G + 4) * ctb;
    const size_t sw_bytes = rows_scratch(c, s, level);
    cudaStream_t st = (cudaStream_t)stream;
    for (uint32_t g = 0; g < p.G; g++) {
        if ((rc = ckks_add_const(c, &in[g], -s->shift, &A, stream))) return rc;
        if ((rc = ckks_poly_eval_tree(c, &A, s->exp_coeffs, s->exp_degree, rlk, &u[g], sw, sw_bytes, stream))) return rc;
    }
    for (uint32_t j = 0; j < s->rounds; j++) {
        // t = row sums of u^2: one relinearisation for the sum over the groups, then the ladder over the blocks
        if ((rc = ckks_mul_relin_sum(c, u.data(), u.data(), p.G, rlk, &A, sw, sw_bytes, stream))) return rc;
        if ((rc = ckks_rescale(c, &A, &T, sw, sw_bytes, stream))) return rc;
        if ((rc = block_ladder(c, p, keys, nkeys, &T, &A, sw, sw_bytes, stream))) return rc;
        // lambda = p_rsqrt_j(t), once for all groups
        if ((rc = ckks_poly_eval_tree(c, &T, s->rsqrt_coeffs + (size_t)j * (s->rsqrt_degree + 1), s->rsqrt_degree, rlk, &B, sw, sw_bytes, stream)))
            return rc;
        for (uint32_t g = 0; g < p.G; g++) {
            // u_g truncated to lambda's level
            int prev = 0;
            cudaGetDevice(&prev);
            cudaSetDevice(c->device);
            for (uint32_t comp = 0; comp < 2; comp++)
                cudaMemcpyAsync(X.data + (size_t)comp * B.level * N, u[g].data + (size_t)comp * u[g].level * N, (size_t)B.level * N * sizeof(uint64_t),
                                cudaMemcpyDeviceToDevice, st);
            cudaSetDevice(prev);
            X.level = B.level; X.ncomp = 2; X.scale = u[g].scale;
            if ((rc = ckks_mul_relin(c, &B, &X, rlk, &A, sw, sw_bytes, stream))) return rc;
            if ((rc = ckks_rescale(c, &A, &X, sw, sw_bytes, stream))) return rc;
            if ((rc = ckks_mul_relin(c, &X, &X, rlk, &A, sw, sw_bytes, stream))) return rc;
            if ((rc = ckks_rescale(c, &A, &u[g], sw, sw_bytes, stream))) return rc;
        }
    }
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(c->device);
    for (uint32_t g = 0; g < p.G; g++)
        cudaMemcpyAsync(out[g].data, u[g].data, (size_t)2 * u[g].level * N * sizeof(uint64_t), cudaMemcpyDeviceToDevice, st);
    cudaError_t e = cudaGetLastError();
    cudaSetDevice(prev);
    if (e != cudaSuccess) { c->cuda_error = cudaGetErrorString(e); return CKKS_ERR_CUDA; }
    for (uint32_t g = 0; g < p.G; g++) { out[g].level = u[g].level; out[g].ncomp = 2; out[g].scale = u[g].scale; }
    return CKKS_OK;
}

// ---- probability x value ------------------------------------------------------------------------------------------
// The ladder over the blocks runs for VAL_CHUNK output channels at a time (ckks_rotate_batch: their key switches side by side).
constexpr uint32_t VAL_CHUNK = 16;
static size_t values_scratch(const ckks_ctx *c, uint32_t level, uint32_t nrot) {
    return std::max(scratch_bytes(c, level, nrot), align256(ckks_workspace_bytes(c, CKKS_OP_ROTATE_BATCH, level - 1, VAL_CHUNK)));
}
// workspace: the truncated value operand and its rotated copies, a product, the rotated outputs of a chunk, the scratch of the calls
extern "C" size_t ckks_attention_values_workspace_bytes(const ckks_ctx *c, const ckks_attn_desc *d, uint32_t level) {
    AttnPlan p;
    if (!c || level < 2 || level > c->L || make_attn_plan(c, d, p)) return 0;
    return (size_t)(p.G + 1) * ct_bytes(c, level) + (size_t)VAL_CHUNK * ct_bytes(c, level - 1) + values_scratch(c, level, p.G - 1);
}

extern "C" int32_t ckks_attention_values(ckks_ctx *c, const ckks_attn_desc *d, const ckks_ct *probs, const ckks_ct *v, uint32_t dim_v,
                                         const ckks_evk *rlk, const ckks_evk *keys, uint32_t nkeys, ckks_ct *out, void *ws, size_t ws_bytes,
                                         void *stream) {
    if (!c || !out) return CKKS_ERR_ARG;
    AttnPlan p;
    int rc = make_attn_plan(c, d, p);
    if (rc) return rc;
    uint32_t lp, lv;
    if ((rc = check_cts(c, probs, p.G, &lp, true)) || (rc = check_cts(c, v, dim_v, &lv, true))) return rc;
    if (lv < lp || lp < 2) return CKKS_ERR_LEVEL;
    if (!rlk_ok(rlk)) return CKKS_ERR_NO_KEY;
    for (int64_t r : p.tok)
        if (!keys || !find_key(c, keys, nkeys, r)) return CKKS_ERR_NO_KEY;
    for (int64_t r : p.lad)
        if (!keys || !find_key(c, keys, nkeys, r)) return CKKS_ERR_NO_KEY;
    for (uint32_t dd = 0; dd < dim_v; dd++)
        if (!out[dd].data) return CKKS_ERR_ARG;
    if (!ws || ws_bytes < ckks_attention_values_workspace_bytes(c, d, lp)) return CKKS_ERR_WORKSPACE;
    const size_t ctb = ct_bytes(c, lp), N = c->N;
    char *base = (char *)ws;
    std::vector<ckks_ct> vr(p.G);
    for (uint32_t g = 0; g < p.G; g++) vr[g] = ckks_ct{(uint64_t *)(base + (size_t)g * ctb), lp, 2, v[0].scale};
    ckks_ct prod{(uint64_t *)(base + (size_t)p.G * ctb), lp, 2, 0.0};
    const size_t ctb1 = ct_bytes(c, lp - 1);
    char *rot = base + (size_t)(p.G + 1) * ctb;                          // [VAL_CHUNK] rotated outputs of the ladder
    void *sw = rot + (size_t)VAL_CHUNK * ctb1;
    const size_t sw_bytes = values_scratch(c, lp, p.G - 1);
    std::vector<ckks_evk> pk;
    for (int64_t r : p.tok) pk.push_back(*find_key(c, keys, nkeys, r));
    cudaStream_t st = (cudaStream_t)stream;
    std::vector<ckks_ct> tmp(VAL_CHUNK);
    for (uint32_t d0 = 0; d0 < dim_v; d0 += VAL_CHUNK) {
        const uint32_t nd = std::min(VAL_CHUNK, dim_v - d0);
        for (uint32_t dd = d0; dd < d0 + nd; dd++) {
            int prev = 0;
            cudaGetDevice(&prev);
            cudaSetDevice(c->device);
            for (uint32_t comp = 0; comp < 2; comp++)
                cudaMemcpyAsync(vr[0].data + (size_t)comp * lp * N, v[dd].data + (size_t)comp * lv * N, (size_t)lp * N * sizeof(uint64_t),
                                cudaMemcpyDeviceToDevice, st);
            cudaSetDevice(prev);
            if (p.G > 1 && (rc = ckks_rotate_hoisted(c, &vr[0], pk.data(), p.G - 1, vr.data() + 1, sw, sw_bytes, stream))) return rc;
            for (uint32_t g = 0; g < p.G; g++) vr[g].scale = v[dd].scale;
            if ((rc = ckks_mul_relin_sum(c, probs, vr.data(), p.G, rlk, &prod, sw, sw_bytes, stream))) return rc;
            if ((rc = ckks_rescale(c, &prod, &out[dd], sw, sw_bytes, stream))) return rc;
        }
        // the ladder over the blocks, a rotation of the whole chunk at a time: out += rotate(out, r), r ascending
        for (int64_t r : p.lad) {
            for (uint32_t x = 0; x < nd; x++) tmp[x] = ckks_ct{(uint64_t *)(rot + (size_t)x * ctb1), lp - 1, 2, 0.0};
            if ((rc = ckks_rotate_batch(c, &out[d0], nd, find_key(c, keys, nkeys, r), tmp.data(), sw, sw_bytes, stream))) return rc;
            for (uint32_t x = 0; x < nd; x++)
                if ((rc = ckks_add(c, &out[d0 + x], &tmp[x], &out[d0 + x], stream))) return rc;
        }
    }
    return CKKS_OK;
}

// ---- the three steps in a row -------------------------------------------------------------------------------------
extern "C" size_t ckks_attention_workspace_bytes(const ckks_ctx *c, const ckks_attn_desc *d, const ckks_softmax_desc *s, uint32_t level, uint32_t dim) {
    AttnPlan p;
    if (!c || level < 3 || level > c->L || !dim || !rows_desc_ok(s) || make_attn_plan(c, d, p)) return 0;
    const size_t held = (size_t)2 * p.G * ct_bytes(c, level - 1);        // scores and probabilities
    const size_t steps = std::max({ckks_attention_scores_workspace_bytes(c, d, level, dim), ckks_softmax_rows_workspace_bytes(c, d, s, level - 1),
                                   ckks_attention_values_workspace_bytes(c, d, level - 1)});
    return held + steps;
}

extern "C" int32_t ckks_attention(ckks_ctx *c, const ckks_attn_desc *d, const ckks_softmax_desc *s, const ckks_ct *q, const ckks_ct *k, uint32_t dim,
                                  const ckks_ct *v, uint32_t dim_v, const ckks_evk *rlk, const ckks_evk *keys, uint32_t nkeys, ckks_ct *out,
                                  void *ws, size_t ws_bytes, void *stream) {
    if (!c || !q || !dim) return CKKS_ERR_ARG;
    AttnPlan p;
    int rc = make_attn_plan(c, d, p);
    if (rc) return rc;
    if (!rows_desc_ok(s)) return CKKS_ERR_ARG;
    const uint32_t level = q[0].level;
    if (level < 3 || level > c->L) return CKKS_ERR_LEVEL;
    const size_t need = ckks_attention_workspace_bytes(c, d, s, level, dim);
    if (!ws || !need || ws_bytes < need) return CKKS_ERR_WORKSPACE;
    const size_t ctb = ct_bytes(c, level - 1);
    char *base = (char *)ws;
    std::vector<ckks_ct> S(p.G), P(p.G);
    for (uint32_t g = 0; g < p.G; g++) {
        S[g] = ckks_ct{(uint64_t *)(base + (size_t)g * ctb), level - 1, 2, 0.0};
        P[g] = ckks_ct{(uint64_t *)(base + (size_t)(p.G + g) * ctb), level - 1, 2, 0.0};
    }
    void *sw = base + (size_t)2 * p.G * ctb;
    const size_t sw_bytes = ws_bytes - (size_t)2 * p.G * ctb;
    if ((rc = ckks_attention_scores(c, d, q, k, dim, rlk, keys, nkeys, S.data(), sw, sw_bytes, stream))) return rc;
    if ((rc = ckks_softmax_rows(c, d, s, S.data(), rlk, keys, nkeys, P.data(), sw, sw_bytes, stream))) return rc;
    return ckks_attention_values(c, d, P.data(), v, dim_v, rlk, keys, nkeys, out, sw, sw_bytes, stream);
}

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
    uint32_t E, Tk, H, R, G, Gb, Ti;
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
    // tokens kept innermost in the slot index: the products, rotations and ladders above are the same for every value (a
    // group step is diag_block tokens = diag_block * heads * R slots either way); only the conversions below use it
    p.Ti = d->token_inner ? d->token_inner : 1;
    if (p.E % p.Ti) return CKKS_ERR_UNSUPPORTED;
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
    if (p.Gb > 1)
        return (size_t)(p.Gb + p.G / p.Gb - 2) * dim * ct_bytes(c, level) + 2 * ct_bytes(c, level) + lane_count(c) * scratch_bytes(c, level, p.G - 1);
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
    const size_t sw_bytes = scratch_bytes(c, level, p.G - 1);
    int rc = CKKS_OK;
    std::vector<ckks_evk> bk, gk;
    for (uint32_t g0 = 1; g0 < Gb; g0++) bk.push_back(*find_key(c, keys, nkeys, p.tok[g0 - 1]));
    for (int64_t r : p.neg) gk.push_back(*find_key(c, keys, nkeys, r));
    std::vector<ckks_ct> outs(std::max(Gb, Gg));
    // the channels' rotations are independent: spread over the lanes, each with its own scratch
    const Lanes lanes(c, stream);
    lanes.fork();
    for (uint32_t dd = 0; dd < dim && !rc; dd++) {
        void *lw = (char *)sw + (dd % lanes.n) * sw_bytes, *ls = lanes.at(dd);
        for (uint32_t x = 0; x + 1 < Gb; x++) outs[x] = ckks_ct{(uint64_t *)(kr + ((size_t)x * dim + dd) * ctb), level, 2, 0.0};
        if (Gb > 1) rc = ckks_rotate_hoisted(c, &k[dd], bk.data(), Gb - 1, outs.data(), lw, sw_bytes, ls);
        for (uint32_t y = 0; y + 1 < Gg; y++) outs[y] = ckks_ct{(uint64_t *)(qr + ((size_t)y * dim + dd) * ctb), level, 2, 0.0};
        if (!rc && Gg > 1) rc = ckks_rotate_hoisted(c, &q[dd], gk.data(), Gg - 1, outs.data(), lw, sw_bytes, ls);
    }
    lanes.join();
    if (rc) return rc;
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
    // the groups' running ciphertexts u_g, the row sums and lambda, then per lane two temporaries and the scratch of the calls
    return (size_t)(p.G + 2) * ct_bytes(c, level) + lane_count(c) * (2 * ct_bytes(c, level) + rows_scratch(c, s, level));
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
    ckks_ct B{(uint64_t *)(base + (size_t)p.G * ctb), level, 2, 0.0}, T{(uint64_t *)(base + (size_t)(p.G + 1) * ctb), level, 2, 0.0};
    const Lanes lanes(c, stream);
    const size_t sw_bytes = rows_scratch(c, s, level), lane_bytes = 2 * ctb + sw_bytes;
    char *lane0 = base + (size_t)(p.G + 2) * ctb;
    // lane l: temporaries A and X, then the scratch
    auto lane_A = [&](uint32_t l) { return ckks_ct{(uint64_t *)(lane0 + l * lane_bytes), level, 2, 0.0}; };
    auto lane_X = [&](uint32_t l) { return ckks_ct{(uint64_t *)(lane0 + l * lane_bytes + ctb), level, 2, 0.0}; };
    auto lane_sw = [&](uint32_t l) { return (void *)(lane0 + l * lane_bytes + 2 * ctb); };
    cudaStream_t st = (cudaStream_t)stream;
    // the groups' exponentials are independent: spread over the lanes
    lanes.fork();
    for (uint32_t g = 0; g < p.G && !rc; g++) {
        const uint32_t l = g % lanes.n;
        ckks_ct A = lane_A(l);
        if ((rc = ckks_add_const(c, &in[g], -s->shift, &A, lanes.at(g)))) break;
        rc = ckks_poly_eval_tree(c, &A, s->exp_coeffs, s->exp_degree, rlk, &u[g], lane_sw(l), sw_bytes, lanes.at(g));
    }
    lanes.join();
    if (rc) return rc;
    for (uint32_t j = 0; j < s->rounds; j++) {
        ckks_ct A = lane_A(0);
        void *sw = lane_sw(0);
        // t = row sums of u^2: one relinearisation for the sum over the groups, then the ladder over the blocks
        if ((rc = ckks_mul_relin_sum(c, u.data(), u.data(), p.G, rlk, &A, sw, sw_bytes, stream))) return rc;
        if ((rc = ckks_rescale(c, &A, &T, sw, sw_bytes, stream))) return rc;
        if ((rc = block_ladder(c, p, keys, nkeys, &T, &A, sw, sw_bytes, stream))) return rc;
        // lambda = p_rsqrt_j(t), once for all groups
        if ((rc = ckks_poly_eval_tree(c, &T, s->rsqrt_coeffs + (size_t)j * (s->rsqrt_degree + 1), s->rsqrt_degree, rlk, &B, sw, sw_bytes, stream)))
            return rc;
        // u_g = rescale(rescale(lambda u_g)^2): independent over the groups
        lanes.fork();
        for (uint32_t g = 0; g < p.G && !rc; g++) {
            const uint32_t l = g % lanes.n;
            ckks_ct Al = lane_A(l), X = lane_X(l);
            void *ls = lanes.at(g), *lw = lane_sw(l);
            // u_g truncated to lambda's level
            int prev = 0;
            cudaGetDevice(&prev);
            cudaSetDevice(c->device);
            for (uint32_t comp = 0; comp < 2; comp++)
                cudaMemcpyAsync(X.data + (size_t)comp * B.level * N, u[g].data + (size_t)comp * u[g].level * N, (size_t)B.level * N * sizeof(uint64_t),
                                cudaMemcpyDeviceToDevice, (cudaStream_t)ls);
            cudaSetDevice(prev);
            X.level = B.level; X.ncomp = 2; X.scale = u[g].scale;
            if ((rc = ckks_mul_relin(c, &B, &X, rlk, &Al, lw, sw_bytes, ls))) break;
            if ((rc = ckks_rescale(c, &Al, &X, lw, sw_bytes, ls))) break;
            if ((rc = ckks_mul_relin(c, &X, &X, rlk, &Al, lw, sw_bytes, ls))) break;
            rc = ckks_rescale(c, &Al, &u[g], lw, sw_bytes, ls);
        }
        lanes.join();
        if (rc) return rc;
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
    // per lane: the truncated value operand with its rotated copies, a product, the scratch of the calls; then a ladder chunk
    return lane_count(c) * ((size_t)(p.G + 1) * ct_bytes(c, level) + values_scratch(c, level, p.G - 1)) + (size_t)VAL_CHUNK * ct_bytes(c, level - 1);
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
    const size_t ctb = ct_bytes(c, lp), ctb1 = ct_bytes(c, lp - 1), N = c->N;
    char *base = (char *)ws;
    const Lanes lanes(c, stream);
    const size_t sw_bytes = values_scratch(c, lp, p.G - 1), lane_bytes = (size_t)(p.G + 1) * ctb + sw_bytes;
    char *rot = base + lanes.n * lane_bytes;                           // [VAL_CHUNK] rotated outputs of the ladder
    std::vector<ckks_evk> pk;
    for (int64_t r : p.tok) pk.push_back(*find_key(c, keys, nkeys, r));
    // the channels are independent up to the ladder: spread over the lanes, each with its own buffers
    lanes.fork();
    std::vector<ckks_ct> vr(p.G);
    for (uint32_t dd = 0; dd < dim_v; dd++) {
        char *lb = base + (dd % lanes.n) * lane_bytes;
        void *ls = lanes.at(dd);
        for (uint32_t g = 0; g < p.G; g++) vr[g] = ckks_ct{(uint64_t *)(lb + (size_t)g * ctb), lp, 2, v[dd].scale};
        ckks_ct prod{(uint64_t *)(lb + (size_t)p.G * ctb), lp, 2, 0.0};
        void *sw = lb + (size_t)(p.G + 1) * ctb;
        int prev = 0;
        cudaGetDevice(&prev);
        cudaSetDevice(c->device);
        for (uint32_t comp = 0; comp < 2; comp++)
            cudaMemcpyAsync(vr[0].data + (size_t)comp * lp * N, v[dd].data + (size_t)comp * lv * N, (size_t)lp * N * sizeof(uint64_t),
                            cudaMemcpyDeviceToDevice, (cudaStream_t)ls);
        cudaSetDevice(prev);
        if (p.G > 1 && (rc = ckks_rotate_hoisted(c, &vr[0], pk.data(), p.G - 1, vr.data() + 1, sw, sw_bytes, ls))) break;
        for (uint32_t g = 0; g < p.G; g++) vr[g].scale = v[dd].scale;
        if ((rc = ckks_mul_relin_sum(c, probs, vr.data(), p.G, rlk, &prod, sw, sw_bytes, ls))) break;
        if ((rc = ckks_rescale(c, &prod, &out[dd], sw, sw_bytes, ls))) break;
    }
    lanes.join();
    if (rc) return rc;
    // the ladder over the blocks, a rotation of a whole chunk of channels at a time: out += rotate(out, r), r ascending
    void *sw = base;                                                   // lane 0's buffers are free again
    std::vector<ckks_ct> tmp(VAL_CHUNK);
    for (uint32_t d0 = 0; d0 < dim_v; d0 += VAL_CHUNK) {
        const uint32_t nd = std::min(VAL_CHUNK, dim_v - d0);
        for (int64_t r : p.lad) {
            for (uint32_t x = 0; x < nd; x++) tmp[x] = ckks_ct{(uint64_t *)(rot + (size_t)x * ctb1), lp - 1, 2, 0.0};
            if ((rc = ckks_rotate_batch(c, &out[d0], nd, find_key(c, keys, nkeys, r), tmp.data(), sw, lane_bytes, stream))) return rc;
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

// ---- conversion between the projections' token-shard layout and the attention operands ---------------------------------
// Shard ciphertext c (c < P = tokens / token_inner) holds, in slot (d * heads + h) * token_inner + t, channel d of token
// c * token_inner + t and head h (the feature-major layout with the features in channel-major order).  The operands keep
// token_inner tokens innermost:  slot = ((e * P + pos) * heads + h) * token_inner + t,  so that a channel's share of a
// shard (B = heads * token_inner slots) moves as one block:
//   gathered[d] = rotate( rescale( sum_c rotate(in[c], -c B) * mask(block c + d) ), d B )     (one rotation per input and output)
//   query:      q[d] = ladder(gathered[d])                               (every block alike)
//   key, value: k0 = gathered[d] + rotate(gathered[d], -P B);  k[d] = rescale( sum_e [ rotate(k0, sA_e) * mask(block e,
//               t < token_inner - b) + rotate(k0, sB_e) * mask(block e, t >= token_inner - b) ] ),  e = a token_inner + b,
//               sA_e = a B + b - e P B,  sB_e = (a + 1) B + b - token_inner - e P B  (the token of the next position)
//   back:       out[c] = rotate( rescale( sum_d rotate(o[d], -d B) * mask(block c + d) ), c B )
// Masks are encoded at the scale of their level's last prime, so every rescale returns the input's scale.  The token shifts
// of a ciphertext run off one ModUp (ckks_rotate_hoisted).  Needs diag_block * tokens * heads = n (no trailing copies).
namespace {

struct PackPlan {
    uint32_t E, P, B, Ti;
    std::vector<int64_t> move, dbl, shA, shB;       // shB[e] = 0 where block e needs no second part (sA of block 0 is 0 too)
};

int make_pack_plan(const ckks_ctx *c, const ckks_attn_desc *d, uint32_t dim, bool back, AttnPlan &ap, PackPlan &p) {
    int rc = make_attn_plan(c, d, ap);
    if (rc) return rc;
    if (ap.R != 1 || !dim) return CKKS_ERR_UNSUPPORTED;
    p.E = ap.E; p.Ti = ap.Ti; p.P = ap.Tk / ap.Ti; p.B = ap.H * ap.Ti;
    if ((uint64_t)dim * p.B > c->n) return CKKS_ERR_UNSUPPORTED;
    // block moves: every input x is rotated by -x B, every output y by y B (pack: inputs = shards, outputs = channels)
    const uint32_t nin = back ? dim : p.P, nout = back ? p.P : dim;
    for (uint32_t x = 1; x < nin; x++) p.move.push_back(-(int64_t)x * p.B);
    for (uint32_t y = 1; y < nout; y++) p.move.push_back((int64_t)y * p.B);
    if (p.E > 1) p.dbl.push_back(-(int64_t)p.P * p.B);
    for (uint32_t e = 0; e < p.E; e++) {
        const int64_t a = e / p.Ti, b = e % p.Ti, back_e = (int64_t)e * p.P * p.B;
        p.shA.push_back(a * p.B + b - back_e);
        p.shB.push_back(b ? (a + 1) * p.B + b - p.Ti - back_e : 0);
    }
    return CKKS_OK;
}

int list_rots(const std::vector<int64_t> &v, int64_t *rots, uint32_t cap, uint32_t &k) {
    for (int64_t r : v) { if (r) { if (rots && k < cap) rots[k] = r; k++; } }
    return 0;
}

size_t pt_bytes(const ckks_ctx *c, uint32_t level) { return align256((size_t)level * c->N * sizeof(uint64_t)); }
size_t mask_scratch(const ckks_ctx *c, uint32_t level) {
    return align256((size_t)c->n * sizeof(double)) + align256(ckks_workspace_bytes(c, CKKS_OP_ENCODE, level, 1));
}

// pt = encode(mask) at `level` with the scale of that level's last prime; scratch: mask_scratch bytes
int encode_mask(ckks_ctx *c, uint32_t level, uint32_t B, uint32_t lo, uint32_t hi, uint32_t Ti, uint32_t t0, uint32_t t1, ckks_pt *pt, void *scratch,
                void *stream) {
    double *slots = (double *)scratch;
    void *ew = (char *)scratch + align256((size_t)c->n * sizeof(double));
    {
        int prev = 0;
        cudaGetDevice(&prev);
        cudaSetDevice(c->device);
        launch_slot_mask(c, slots, B, lo, hi, Ti, t0, t1, (cudaStream_t)stream);
        cudaSetDevice(prev);
    }
    pt->level = level;
    pt->scale = (double)c->mod[level - 1];
    return ckks_encode(c, slots, nullptr, 1, pt->scale, level, pt->data, ew, ckks_workspace_bytes(c, CKKS_OP_ENCODE, level, 1), stream);
}

// outs[x] = rotate(in, rots[x]) for the non-zero rotations, in chunks of 16 off one ModUp each; outs[x] = in's descriptor for a zero rotation
int rotate_many(ckks_ctx *c, const ckks_ct *in, const std::vector<int64_t> &rots, const ckks_evk *keys, uint32_t nkeys, ckks_ct *outs, void *sw,
                size_t sw_bytes, void *stream) {
    std::vector<ckks_evk> ks;
    std::vector<ckks_ct> os;
    for (size_t x = 0; x < rots.size(); x++) {
        if (rots[x] % (int64_t)c->n == 0) { outs[x] = *in; continue; }
        ks.push_back(*find_key(c, keys, nkeys, rots[x]));
        os.push_back(outs[x]);
    }
    if (ks.empty()) return CKKS_OK;
    int rc = ckks_rotate_hoisted(c, in, ks.data(), (uint32_t)ks.size(), os.data(), sw, sw_bytes, stream);
    if (rc) return rc;
    size_t y = 0;
    for (size_t x = 0; x < rots.size(); x++)
        if (rots[x] % (int64_t)c->n != 0) outs[x] = os[y++];
    return CKKS_OK;
}

bool have_keys(const ckks_ctx *c, const std::vector<int64_t> &v, const ckks_evk *keys, uint32_t nkeys) {
    for (int64_t r : v)
        if (r % (int64_t)c->n != 0 && (!keys || !find_key(c, keys, nkeys, r))) return false;
    return true;
}

struct PackWs { size_t rot, acc, tmp, gat, pts, mask, sw, sw_bytes, lane, lane_bytes, bytes; uint32_t nrot; };

// kind 0 / 1: pack; kind 2: back
PackWs pack_layout(const ckks_ctx *c, const PackPlan &p, int kind, uint32_t level, uint32_t dim) {
    PackWs w;
    const uint32_t nin = kind == 2 ? dim : p.P, nout = kind == 2 ? p.P : dim;
    w.nrot = std::max<uint32_t>({nin, 2 * p.E, 16});            // rotated inputs; later the token shifts or a ladder's chunk
    size_t off = 0;
    w.rot = off;  off += (size_t)w.nrot * ct_bytes(c, level);
    w.acc = off;  off += (size_t)nout * ct_bytes(c, level);
    w.tmp = off;  off += ct_bytes(c, level);
    w.gat = off;  off += kind == 1 ? (size_t)dim * ct_bytes(c, level - 1) : 0;                                  // gathered[d]
    w.pts = off;  off += (size_t)(kind == 1 ? 2 * p.E : 1) * pt_bytes(c, level);
    w.mask = off; off += mask_scratch(c, level);
    w.sw = off;
    w.sw_bytes = align256(std::max({ckks_workspace_bytes(c, CKKS_OP_ROTATE_HOISTED, level, 16), ckks_workspace_bytes(c, CKKS_OP_RESCALE, level, 0),
                                    ckks_workspace_bytes(c, CKKS_OP_ROTATE, level, 0), ckks_workspace_bytes(c, CKKS_OP_ROTATE_BATCH, level, 16)}));
    off += w.sw_bytes;
    // key, value: per lane the rotated copies of the token shifts, k0, a sum and the scratch of the calls
    w.lane = off;
    w.lane_bytes = (size_t)2 * p.E * ct_bytes(c, level - 1) + 2 * ct_bytes(c, level - 1) + w.sw_bytes;
    if (kind == 1) off += lane_count(c) * w.lane_bytes;
    w.bytes = off;
    return w;
}

}  // namespace

extern "C" int32_t ckks_attention_pack_rotations(const ckks_ctx *c, const ckks_attn_desc *d, int32_t kind, uint32_t dim, int64_t *rots, uint32_t cap) {
    if (!c || kind < 0 || kind > 2) return CKKS_ERR_ARG;
    AttnPlan ap;
    PackPlan p;
    int rc = make_pack_plan(c, d, dim, kind == 2, ap, p);
    if (rc) return rc;
    uint32_t k = 0;
    list_rots(p.move, rots, cap, k);
    if (kind == 0) list_rots(ap.lad, rots, cap, k);
    if (kind == 1) { list_rots(p.dbl, rots, cap, k); list_rots(p.shA, rots, cap, k); list_rots(p.shB, rots, cap, k); }
    return (int32_t)k;
}

extern "C" size_t ckks_attention_pack_workspace_bytes(const ckks_ctx *c, const ckks_attn_desc *d, int32_t kind, uint32_t level, uint32_t dim) {
    AttnPlan ap;
    PackPlan p;
    if (!c || kind < 0 || kind > 2 || level < 3 || level > c->L || make_pack_plan(c, d, dim, kind == 2, ap, p)) return 0;
    return pack_layout(c, p, kind, level, dim).bytes;
}

extern "C" int32_t ckks_attention_pack(ckks_ctx *c, const ckks_attn_desc *d, int32_t kind, const ckks_ct *in, uint32_t dim, const ckks_evk *keys,
                                       uint32_t nkeys, ckks_ct *out, void *ws, size_t ws_bytes, void *stream) {
    if (!c || !out || kind < 0 || kind > 2) return CKKS_ERR_ARG;
    AttnPlan ap;
    PackPlan p;
    int rc = make_pack_plan(c, d, dim, kind == 2, ap, p);
    if (rc) return rc;
    const uint32_t nin = kind == 2 ? dim : p.P, nout = kind == 2 ? p.P : dim;
    uint32_t level;
    if ((rc = check_cts(c, in, nin, &level, true))) return rc;
    if (level < 3) return CKKS_ERR_LEVEL;
    for (uint32_t x = 0; x < nout; x++)
        if (!out[x].data) return CKKS_ERR_ARG;
    if (!have_keys(c, p.move, keys, nkeys)) return CKKS_ERR_NO_KEY;
    if (kind == 0 && !have_keys(c, ap.lad, keys, nkeys)) return CKKS_ERR_NO_KEY;
    if (kind == 1 && (!have_keys(c, p.dbl, keys, nkeys) || !have_keys(c, p.shA, keys, nkeys) || !have_keys(c, p.shB, keys, nkeys))) return CKKS_ERR_NO_KEY;
    const PackWs L = pack_layout(c, p, kind, level, dim);
    if (!ws || ws_bytes < L.bytes) return CKKS_ERR_WORKSPACE;
    char *base = (char *)ws;
    const size_t ctb = ct_bytes(c, level), ctb1 = ct_bytes(c, level - 1);
    void *sw = base + L.sw;
    // First step, the same in both directions: a transpose between the ciphertext index and the block index.  Input x is
    // rotated by -x B (its block y then sits at block x + y), output y collects block x + y of every rotated input under a
    // 0/1 mask, is rescaled and rotated by y B, so that input x's share lands in block x.  Blocks count cyclically.
    const uint32_t nblk = c->n / p.B;
    std::vector<ckks_ct> xp(nin), acc(nout);
    xp[0] = in[0];
    for (uint32_t x = 1; x < nin; x++) {
        xp[x] = ckks_ct{(uint64_t *)(base + L.rot + (size_t)x * ctb), level, 2, 0.0};
        if ((rc = ckks_rotate(c, &in[x], find_key(c, keys, nkeys, -(int64_t)x * p.B), &xp[x], sw, L.sw_bytes, stream))) return rc;
    }
    ckks_pt pt{(uint64_t *)(base + L.pts), level, 0.0};
    {
        int prev = 0;
        cudaGetDevice(&prev);
        cudaSetDevice(c->device);
        cudaMemsetAsync(base + L.acc, 0, (size_t)nout * ctb, (cudaStream_t)stream);
        cudaSetDevice(prev);
    }
    for (uint32_t y = 0; y < nout; y++) acc[y] = ckks_ct{(uint64_t *)(base + L.acc + (size_t)y * ctb), level, 2, in[0].scale * (double)c->mod[level - 1]};
    std::vector<ckks_ct> mc, ma;
    for (uint32_t j = 0; j < std::min(nin + nout - 1, nblk); j++) {
        mc.clear(); ma.clear();
        for (uint32_t x = 0; x < nin; x++)
            for (uint32_t y = 0; y < nout; y++)
                if ((x + y) % nblk == j) { mc.push_back(xp[x]); ma.push_back(acc[y]); }
        if (mc.empty()) continue;
        if ((rc = encode_mask(c, level, p.B, j, j + 1, p.Ti, 0, p.Ti, &pt, base + L.mask, stream))) return rc;
        if ((rc = ckks_mul_plain_acc(c, mc.data(), (uint32_t)mc.size(), &pt, ma.data(), 0, stream))) return rc;
    }
    // rescaled and rotated into place: straight to the outputs, or (key, value) to the buffer the token shifts read
    ckks_ct tmp{(uint64_t *)(base + L.tmp), level - 1, 2, 0.0};
    std::vector<ckks_ct> moved(nout);
    for (uint32_t y = 0; y < nout; y++) {
        moved[y] = (kind == 1 && p.E > 1) ? ckks_ct{(uint64_t *)(base + L.gat + (size_t)y * ctb1), level - 1, 2, 0.0} : out[y];
        if (y == 0) {
            if ((rc = ckks_rescale(c, &acc[0], &moved[0], sw, L.sw_bytes, stream))) return rc;
            continue;
        }
        if ((rc = ckks_rescale(c, &acc[y], &tmp, sw, L.sw_bytes, stream))) return rc;
        if ((rc = ckks_rotate(c, &tmp, find_key(c, keys, nkeys, (int64_t)y * p.B), &moved[y], sw, L.sw_bytes, stream))) return rc;
    }
    if (kind != 1 || p.E == 1) {
        for (uint32_t y = 0; y < nout; y++) out[y] = moved[y];
        if (kind != 0) return CKKS_OK;
        // query: the ladder over the blocks, 16 channels at a time
        std::vector<ckks_ct> tmp(16);
        for (uint32_t d0 = 0; d0 < dim; d0 += 16) {
            const uint32_t nd = std::min<uint32_t>(16, dim - d0);
            for (int64_t r : ap.lad) {
                for (uint32_t x = 0; x < nd; x++) tmp[x] = ckks_ct{(uint64_t *)(base + L.rot + (size_t)x * ctb), level - 1, 2, 0.0};
                if ((rc = ckks_rotate_batch(c, &out[d0], nd, find_key(c, keys, nkeys, r), tmp.data(), sw, L.sw_bytes, stream))) return rc;
                for (uint32_t x = 0; x < nd; x++)
                    if ((rc = ckks_add(c, &out[d0 + x], &tmp[x], &out[d0 + x], stream))) return rc;
            }
        }
        return CKKS_OK;
    }
    // key, value: the token shifts, one level down
    const uint32_t l1 = level - 1;
    std::vector<ckks_pt> mA(p.E), mB(p.E);
    for (uint32_t e = 0; e < p.E; e++) {
        const uint32_t b = e % p.Ti;
        mA[e] = ckks_pt{(uint64_t *)(base + L.pts + (size_t)(2 * e) * pt_bytes(c, level)), l1, 0.0};
        mB[e] = ckks_pt{(uint64_t *)(base + L.pts + (size_t)(2 * e + 1) * pt_bytes(c, level)), l1, 0.0};
        if ((rc = encode_mask(c, l1, p.B, e * p.P, (e + 1) * p.P, p.Ti, 0, p.Ti - b, &mA[e], base + L.mask, stream))) return rc;
        if (b && (rc = encode_mask(c, l1, p.B, e * p.P, (e + 1) * p.P, p.Ti, p.Ti - b, p.Ti, &mB[e], base + L.mask, stream))) return rc;
    }
    std::vector<int64_t> sr;
    for (uint32_t e = 0; e < p.E; e++) { sr.push_back(p.shA[e]); if (e % p.Ti) sr.push_back(p.shB[e]); }
    std::vector<ckks_ct> so(sr.size());
    // the copy of block 0 in block 1, k0 = moved + rotate(moved, -P B), in place and 16 channels at a time (one key)
    {
        std::vector<ckks_ct> tmp16(16);
        for (uint32_t d0 = 0; d0 < dim; d0 += 16) {
            const uint32_t nd = std::min<uint32_t>(16, dim - d0);
            for (uint32_t x = 0; x < nd; x++) tmp16[x] = ckks_ct{(uint64_t *)(base + L.rot + (size_t)x * ctb), l1, 2, 0.0};
            if ((rc = ckks_rotate_batch(c, &moved[d0], nd, find_key(c, keys, nkeys, p.dbl[0]), tmp16.data(), sw, L.sw_bytes, stream))) return rc;
            for (uint32_t x = 0; x < nd; x++)
                if ((rc = ckks_add(c, &moved[d0 + x], &tmp16[x], &moved[d0 + x], stream))) return rc;
        }
    }
    // the channels are independent: spread over the lanes, each with its own buffers
    const Lanes lanes(c, stream);
    lanes.fork();
    for (uint32_t dd = 0; dd < dim && !rc; dd++) {
        char *lb = base + L.lane + (dd % lanes.n) * L.lane_bytes;
        void *ls = lanes.at(dd), *lw = lb + (size_t)(2 * p.E + 2) * ctb1;
        ckks_ct sum{(uint64_t *)(lb + (size_t)(2 * p.E + 1) * ctb1), l1, 2, 0.0};
        ckks_ct k0 = moved[dd];
        for (size_t x = 0; x < sr.size(); x++) so[x] = ckks_ct{(uint64_t *)(lb + x * ctb1), l1, 2, 0.0};
        if ((rc = rotate_many(c, &k0, sr, keys, nkeys, so.data(), lw, L.sw_bytes, ls))) break;
        size_t x = 0;
        for (uint32_t e = 0; e < p.E && !rc; e++) {
            rc = ckks_mul_plain_acc(c, &so[x++], 1, &mA[e], &sum, e == 0, ls);
            if (!rc && e % p.Ti) rc = ckks_mul_plain_acc(c, &so[x++], 1, &mB[e], &sum, 0, ls);
        }
        if (!rc) rc = ckks_rescale(c, &sum, &out[dd], lw, L.sw_bytes, ls);
    }
    lanes.join();
    return rc;
}

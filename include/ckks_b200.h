/*
 * ckks_b200 -- CKKS RNS primitive layer for NVIDIA B200 (sm_100a), C ABI.
 *
 * The operations are the ones the paper's server-side evaluation is built
 * from (Section 2.1, "The CKKS Computation Model": Encode, Add, PCMult, Mult,
 * Rot_k, KeySwitch, Rescale) plus the diagonal matrix-vector product of
 * Eq. 5 evaluated baby-step/giant-step over the feature-major token-shard
 * layout (Sections 1 and 3: feature-major cross-layer state; plaintexts
 * organised by logical diagonal and reused across token-shard inputs).  The
 * paper fixes what is called and with which shapes; the arithmetic is the
 * full-RNS form of the scheme it cites.
 *
 * General rules
 *   - Every function returns a status (0 = CKKS_OK, negative = error) and
 *     never throws.  Arguments are validated on the host before any launch:
 *     a failing call launches nothing and writes nothing.
 *   - The caller owns every device buffer: inputs, outputs, keys, workspace.
 *     The library allocates device memory only in ckks_context_create (its
 *     tables) and frees it in ckks_context_destroy.  Calls enqueue work on the
 *     given stream (a cudaStream_t passed as void*, NULL = default stream) and
 *     return without synchronising.
 *   - The library never sees a secret key.
 *   - "Host" / "device" is stated for every pointer.  Descriptor structs
 *     (ckks_ct, ckks_pt, ckks_evk, ckks_proj_desc) live in host memory and hold
 *     device pointers.
 *
 * Data layout
 *   N ring degree, n = N/2 slots.  Prime index space: 0..L-1 are the ciphertext
 *   primes q_0..q_{L-1}, L..L+K-1 the special primes p_0..p_{K-1}.  All primes
 *   must lie in (2^49, 2^50) and be 1 mod 2N.  A limb is N uint64 residues in
 *   [0, prime).  Every stored polynomial is in the evaluation domain in
 *   bit-reversed order: limb[p] = a(psi^(2*bitrev(p)+1)), psi = the smallest
 *   primitive 2N-th root of unity modulo the limb's prime.
 *     ciphertext      [ncomp][level][N]      limbs q_0..q_{level-1}
 *     plaintext       [level][N]
 *     switching key   [dnum][2][L+K][N]      component 0 = b, 1 = a
 *   "level" counts limbs; rescale drops q_{level-1}.  Digit j of the hybrid
 *   key switch covers limbs j*alpha .. min((j+1)*alpha, level)-1 with
 *   alpha = ceil(L/dnum); K >= alpha is required.
 *   Slot j of a plaintext sits at the root zeta^(5^j), zeta = exp(2 pi i / 2N),
 *   so the Galois element 5^r is a left rotation by r slots (Eq. 5's rho^r).
 */
#ifndef CKKS_B200_H
#define CKKS_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    CKKS_OK = 0,
    CKKS_ERR_ARG = -1,         /* null pointer, zero count, bad enum                       */
    CKKS_ERR_LEVEL = -2,       /* level 0, level > L, operand levels differ                */
    CKKS_ERR_SCALE = -3,       /* scales that must agree differ by more than 2^-30 relative */
    CKKS_ERR_NO_KEY = -4,      /* a needed Galois element is not among the supplied keys   */
    CKKS_ERR_WORKSPACE = -5,   /* workspace missing or smaller than ckks_workspace_bytes   */
    CKKS_ERR_RANGE = -6,       /* encode: a scaled value does not fit 2^62                 */
    CKKS_ERR_UNSUPPORTED = -7, /* parameters outside what the kernels implement            */
    CKKS_ERR_CUDA = -8,        /* a CUDA runtime call failed (see ckks_last_cuda_error)    */
    CKKS_ERR_TIMEOUT = -9      /* a bounded device-side wait gave up (see ckks_device_status) */
};

/* Operation selectors for ckks_workspace_bytes. */
enum {
    CKKS_OP_ENCODE = 1, CKKS_OP_MUL_RELIN = 2, CKKS_OP_ROTATE = 3,
    CKKS_OP_ROTATE_HOISTED = 4, CKKS_OP_RESCALE = 5, CKKS_OP_LINEAR_PROJ = 6, CKKS_OP_POLY_EVAL = 7,
    CKKS_OP_POLY_EVAL_TREE = 8 /* count = degree */, CKKS_OP_MUL_RELIN_BATCH = 9 /* count = products */, CKKS_OP_ROTATE_BATCH = 10 /* count = ciphertexts */, CKKS_OP_ROTATE_SUM = 11 /* count = ciphertexts */
};

typedef struct ckks_ctx ckks_ctx; /* opaque */

/* All fields host-side.  q[num_q], p[num_p] host arrays. */
typedef struct {
    uint32_t log_n;       /* 10..16                                             */
    uint32_t num_q;       /* L                                                  */
    uint32_t num_p;       /* K  (>= ceil(L/dnum))                               */
    uint32_t dnum;        /* number of key-switch digits                        */
    const uint64_t *q;    /* host                                               */
    const uint64_t *p;    /* host                                               */
    int32_t device;       /* CUDA device ordinal the tables are placed on       */
} ckks_params;

typedef struct { uint64_t *data; /* device */ uint32_t level, ncomp; double scale; } ckks_ct;
typedef struct { uint64_t *data; /* device */ uint32_t level; double scale; } ckks_pt;
typedef struct { const uint64_t *data; /* device */ uint64_t galois; /* 0 for a relinearisation key */ } ckks_evk;

/*
 * Shape of one projection Y = X W (Eq. 5 per block, baby-step/giant-step).
 * Tokens are split into nshards shards of tokens_per_shard (T) tokens; one
 * ciphertext holds F = n/T features of one shard, slot = f*T + t.  d_in and
 * d_out are cut into blocks of F features; a trailing block smaller than F
 * must divide F and is stored repeated F/m times.  For an (input block m_in,
 * output block m_out) pair the min(m_in, m_out) generalised diagonals
 * d_k[r] = W^T[r mod m_out, (r + k) mod m_in] are used; `baby` (B) must divide
 * that count; when m_out < m_in the result is folded by log2(m_in/m_out)
 * rotate-and-add steps.  pt_scale is the scale the weights are encoded at
 * (0 selects q_{level-1}, so that the final rescale restores the input scale).
 * flags: 0, or CKKS_PROJ_LAZY_MODDOWN: the rotated giant-step accumulators of an output ciphertext are summed in the
 * key-switching basis Q_level P and divided by P once (ckks_rotate_sum's function) instead of once per rotation.
 * The two settings are different integer functions with the same plaintext result; after the final rescale their
 * residues differ by at most one unit.
 */
#define CKKS_PROJ_LAZY_MODDOWN 1u
typedef struct {
    uint32_t d_in, d_out, tokens_per_shard, nshards, baby, flags;
    double pt_scale;
} ckks_proj_desc;

/* ---- context ----------------------------------------------------------- */

/* Builds the tables (twiddles, conversion constants, permutation helpers) on
 * params->device.  *out receives the context.  Errors: ARG, UNSUPPORTED
 * (log_n, prime size, prime not 1 mod 2N, duplicates, K < alpha), CUDA. */
int32_t ckks_context_create(const ckks_params *params, ckks_ctx **out);
void ckks_context_destroy(ckks_ctx *ctx);

const char *ckks_status_string(int32_t status);
/* Text of the last CUDA error seen by this context ("" if none).  Host string owned by the context. */
const char *ckks_last_cuda_error(const ckks_ctx *ctx);

/* Options of a context: host-side state, read whenever a call is made (set them between calls, not while another
 * thread is inside one).  None of them changes a result: every kernel variant is bit-identical.
 *   CKKS_OPT_NTT_FP_SHARE   N = 2^16 transform: of every 8 limbs, how many run on the FP64 pipe (0..8, default 8).
 *   CKKS_OPT_CONV_KERNEL    ModUp / ModDown basis conversions: CKKS_CONV_FP64 (default) or CKKS_CONV_TENSOR.
 *   CKKS_OPT_MAC_KERNEL     the projection's multiply-accumulate: CKKS_MAC_MMA (default: mma.sync, 8 coefficients per
 *                           CTA, a warp per coefficient), CKKS_MAC_MMA_ASYNC (the same joined by mbarriers instead of
 *                           CTA-wide barriers), CKKS_MAC_MMA_SPLIT (two warps per coefficient), CKKS_MAC_MMA_HALF (4
 *                           coefficients per CTA), CKKS_MAC_TCGEN05 (tcgen05.mma with TMEM accumulators, baby <= 64).
 *   CKKS_OPT_WAIT_CYCLES    bound, in SM clock cycles, of every device-side wait on an mbarrier (default 2 * 10^9,
 *                           about a second).  A wait that runs out makes its kernel drain its copies and return, and
 *                           sets the sticky flag ckks_device_status reports; 0 makes every wait that is not already
 *                           satisfied give up at once (used to test that path).
 *   CKKS_OPT_NTT_BULK_STORE N = 2^16 transforms: 1 (default) = in the forward transform's last pass every thread stages its
 *                           16 results in shared memory and a 128-byte bulk copy writes them out, and in the inverse
 *                           transform's first pass every thread's 16 inputs arrive by a 128-byte bulk copy (a bounded wait
 *                           on an mbarrier, see CKKS_OPT_WAIT_CYCLES); 0 = 32-byte global stores and loads.
 *   CKKS_OPT_LANES          1..4 (default 4): streams over which the attention entry points spread their independent
 *                           single-ciphertext chains (per channel, per score group).  Lane 0 is the caller's stream, the
 *                           others belong to the context; they are forked from and joined to the caller's stream by events
 *                           inside the call, so the call still behaves as work on the caller's stream.  The workspace sizes
 *                           of those calls depend on it: set it before asking for them.  Results do not depend on it.
 *                           The lanes' streams and events belong to the context: two host threads must not run attention
 *                           entry points on the same context at the same time (use a context per thread).
 *   CKKS_OPT_STATIC_SCRATCH_BYTES  (read only) CKKS_STATIC_SCRATCH_BYTES of the loaded library.
 * set returns CKKS_ERR_ARG for an unknown option or a value outside its range; get returns -1 for an unknown option. */
enum { CKKS_OPT_NTT_FP_SHARE = 1, CKKS_OPT_CONV_KERNEL = 2, CKKS_OPT_MAC_KERNEL = 3, CKKS_OPT_WAIT_CYCLES = 4,
       CKKS_OPT_STATIC_SCRATCH_BYTES = 5, CKKS_OPT_NTT_BULK_STORE = 6, CKKS_OPT_LANES = 7 };
enum { CKKS_CONV_FP64 = 0, CKKS_CONV_TENSOR = 1 };
enum { CKKS_MAC_MMA = 82, CKKS_MAC_MMA_ASYNC = 83, CKKS_MAC_MMA_SPLIT = 81, CKKS_MAC_MMA_HALF = 42, CKKS_MAC_TCGEN05 = 100 };
int32_t ckks_context_set_option(ckks_ctx *ctx, int32_t option, int64_t value);
int64_t ckks_context_get_option(const ckks_ctx *ctx, int32_t option);

/* Bytes of caller-provided device workspace `op` needs at this level.  `count`
 * is the batch size for CKKS_OP_ENCODE, the number of rotations for
 * CKKS_OP_ROTATE_HOISTED, the degree for CKKS_OP_POLY_EVAL_TREE and the number
 * of products / ciphertexts for CKKS_OP_MUL_RELIN_BATCH / CKKS_OP_ROTATE_BATCH / CKKS_OP_ROTATE_SUM; ignored
 * otherwise.  For CKKS_OP_LINEAR_PROJ use ckks_linear_proj_workspace_bytes.
 * Returns 0 for an unknown op. */
size_t ckks_workspace_bytes(const ckks_ctx *ctx, int32_t op, uint32_t level, uint32_t count);

/* Number of kernels this library has launched since it was loaded (all contexts).  Not thread safe. */
uint64_t ckks_kernel_launches(void);

/* 5^r mod 2N with r taken mod n: Galois element of a left rotation by r slots. */
uint64_t ckks_galois_element(const ckks_ctx *ctx, int64_t left_rot_slots);

/* ---- NTT --------------------------------------------------------------- */

/* Forward / inverse negacyclic NTT, in place, of `batch * nlimbs` limbs laid
 * out [batch][nlimbs][N] (device); limb i of every batch entry is taken
 * modulo prime first_prime + i (prime index space above).  Forward: natural-
 * order coefficients in, bit-reversed evaluations out; inverse undoes it
 * (including N^-1).  Inputs must be canonical residues.  Errors: ARG, LEVEL
 * (prime range outside 0..L+K-1). */
int32_t ckks_ntt(ckks_ctx *ctx, uint64_t *polys, uint32_t batch, uint32_t first_prime, uint32_t nlimbs, void *stream);
int32_t ckks_intt(ckks_ctx *ctx, uint64_t *polys, uint32_t batch, uint32_t first_prime, uint32_t nlimbs, void *stream);

/* Measurement aid (the paper has no counterpart): runs the forward butterflies of the N = 2^16 transform on
 * registers only -- `iters` groups of 4 stages (32 butterflies) per thread, with the transform's own range
 * reductions and twiddle fetches, on a grid of three 256-thread CTAs per SM -- so that a caller can time the
 * launch and compare the transform's butterflies per second with what the arithmetic alone sustains.
 * scratch: device, at least SMs * 1024 words, never written in practice.  *butterflies (host) receives the
 * number of butterflies of the launch.  CKKS_ERR_UNSUPPORTED unless log_n = 16. */
int32_t ckks_ntt_butterfly_probe(ckks_ctx *ctx, uint32_t iters, uint64_t *scratch, size_t scratch_words, uint64_t *butterflies,
                                 void *stream);

/* ---- Encode (Section 2.1, Encode) ----------------------------------------
 * re, im: device, [batch][n] fp64 slot values (im may be NULL = real input).
 * out: device, [batch][level][N].  Steps: slot permutation e_j = (5^j mod 2N
 * - 1)/4, unnormalised inverse DFT of size n by radix-2 butterflies with every
 * product and sum rounded on its own (no FMA), twist by conj(zeta^k), multiply
 * by scale/n, round half to even, reduce modulo each prime, NTT.  A scaled
 * value of magnitude >= 2^62 sets a sticky range flag (the coefficient is
 * encoded as 0); read it with ckks_encode_range_flag.
 * Errors: ARG, LEVEL, WORKSPACE. */
int32_t ckks_encode(ckks_ctx *ctx, const double *re, const double *im, uint32_t batch, double scale,
                    uint32_t level, uint64_t *out, void *ws, size_t ws_bytes, void *stream);
/* Synchronises `stream`, returns CKKS_ERR_RANGE if any encode since the last
 * query overflowed (and clears the flag), else CKKS_OK. */
int32_t ckks_encode_range_flag(ckks_ctx *ctx, void *stream);

/* Synchronises `stream`; returns CKKS_ERR_TIMEOUT if a bounded device-side wait (the mbarrier hand-offs of the
 * projection's multiply-accumulate variants CKKS_MAC_MMA_ASYNC and CKKS_MAC_TCGEN05) gave up since the last query
 * (and clears the flag), else CKKS_OK.  After a timeout the outputs of the call that hit it are undefined. */
int32_t ckks_device_status(ckks_ctx *ctx, void *stream);

/* ---- PCMult + Add (Section 2.1) -------------------------------------------
 * accs[s] (+)= cts[s] * pt for s < ncts, both components, all limbs.  cts,
 * accs: host arrays of descriptors.  init = 1: accs[s] = cts[s]*pt and
 * accs[s].scale/level/ncomp are set; init = 0: requires cts[s].scale *
 * pt->scale == accs[s].scale within 2^-30 relative.  Levels must all agree.
 * accs[s] may not alias cts[s'].  Errors: ARG, LEVEL, SCALE. */
int32_t ckks_mul_plain_acc(ckks_ctx *ctx, const ckks_ct *cts, uint32_t ncts, const ckks_pt *pt,
                           ckks_ct *accs, int32_t init, void *stream);

/* Add (Section 2.1): out = a + b, same level, ncomp, scale (2^-30 relative).  out may alias a or b. */
int32_t ckks_add(ckks_ctx *ctx, const ckks_ct *a, const ckks_ct *b, ckks_ct *out, void *stream);

/* ---- Mult with relinearisation (Section 2.1, Mult + KeySwitch) -------------
 * out = (a0 b0 + k0, a0 b1 + a1 b0 + k1), (k0, k1) = KeySwitch(a1 b1, rlk).
 * out->scale = a->scale * b->scale; no rescale inside.  rlk->galois must be 0.
 * out may alias a or b.  Errors: ARG, LEVEL, NO_KEY, WORKSPACE. */
int32_t ckks_mul_relin(ckks_ctx *ctx, const ckks_ct *a, const ckks_ct *b, const ckks_evk *rlk, ckks_ct *out,
                       void *ws, size_t ws_bytes, void *stream);

/* n independent products out[i] = Mult+relin(a[i], b[i]) in one call: the key switches of up to 16 products run side by
 * side (one batched ModUp, inner product and ModDown), which fills the GPU where a single ciphertext does not.
 * Every out[i] is bit-identical to ckks_mul_relin(a[i], b[i]).  a, b, out: host arrays of n ciphertexts at one
 * level; out[i] may be a[i] or b[i].  Workspace: ckks_workspace_bytes(CKKS_OP_MUL_RELIN_BATCH, level, n). */
int32_t ckks_mul_relin_batch(ckks_ctx *ctx, const ckks_ct *a, const ckks_ct *b, uint32_t n, const ckks_evk *rlk, ckks_ct *out,
                             void *ws, size_t ws_bytes, void *stream);

/* Sum of n products with one relinearisation (Section 4: the attention products add up many ciphertext x
 * ciphertext terms): e = sum_i a_i (x) b_i component-wise modulo each prime, then as ckks_mul_relin from the
 * key switch on.  a, b: host arrays of n two-component ciphertexts, all at one level; the a_i share a scale,
 * the b_i share a scale; out.scale = a_0.scale * b_0.scale.  n = 1 gives ckks_mul_relin's result bit for bit; for
 * n > 1 the integers differ from the sum of n ckks_mul_relin results (one rounding of the key switch instead of n)
 * while the plaintext is the same.  out must not alias an input.  Workspace: CKKS_OP_MUL_RELIN.
 * Errors: as ckks_mul_relin; CKKS_ERR_SCALE if the a_i (or the b_i) disagree in scale. */
int32_t ckks_mul_relin_sum(ckks_ctx *ctx, const ckks_ct *a, const ckks_ct *b, uint32_t n, const ckks_evk *rlk, ckks_ct *out,
                           void *ws, size_t ws_bytes, void *stream);

/* ---- Constants and polynomials (Section 2.1 Add / Mult with a constant-slot plaintext; Section 3: the
 * element-wise polynomials that replace the non-linear layers) -------------------------------------------
 * A plaintext holding the same real value c in every slot is the constant polynomial v = round(c * scale)
 * (round half to even); its evaluation-domain image is v in every position, so no encode is needed.
 *   ckks_mul_const: out = in * v with v = round(c * cscale) on all components; out.scale = in.scale * cscale.
 *                   cscale = 0 selects q_{level-1}, so that a following rescale restores in.scale.
 *   ckks_add_const: out = in with v = round(c * in.scale) added to component 0; scale and level unchanged.
 * out may be in.  CKKS_ERR_RANGE if |c * scale| >= 2^62.
 *   ckks_poly_eval: sum_k coeffs[k] x^k (coeffs: host, degree + 1 doubles, degree >= 1) by Horner's rule:
 *                   r = x * round(c_d q_{l-1}); rescale; r += c_{d-1};  then for k = d-2 .. 0:
 *                   r = Mult+relin(r, x truncated to r's level); rescale; r += c_k   (constants at r's scale).
 *                   x must have ncomp = 2 and level l >= degree + 1; out is written at level l - degree with the
 *                   scale obtained by multiplying by x.scale and dividing by the dropped prime at every step, in
 *                   that order.  Workspace: ckks_workspace_bytes(CKKS_OP_POLY_EVAL, l, 0).  A scale close to the
 *                   primes (2^50) keeps the precision; errors as ckks_mul_relin, plus CKKS_ERR_RANGE. */
int32_t ckks_mul_const(ckks_ctx *ctx, const ckks_ct *in, double c, double cscale, ckks_ct *out, void *stream);
int32_t ckks_add_const(ckks_ctx *ctx, const ckks_ct *in, double c, ckks_ct *out, void *stream);
int32_t ckks_poly_eval(ckks_ctx *ctx, const ckks_ct *x, const double *coeffs, uint32_t degree, const ckks_evk *rlk, ckks_ct *out,
                       void *ws, size_t ws_bytes, void *stream);
/* The same polynomial in depth ceil(log2 degree) + 1 (degree >= 2, level >= depth + 1): powers x^k = x^(k/2) *
 * x^(k - k/2) for k = 2..degree (Mult + relinearisation, rescale; operands truncated to the lower of their levels),
 * then, at the level Lt of x^degree and the scale T = x.scale * q_{Lt-1}, acc = sum over k >= 1 with coeffs[k] != 0, in
 * increasing k, of x^k * round(coeffs[k] * (T / scale(x^k))), a rescale, and round(coeffs[0] * scale) added last.
 * out is written at level Lt - 1 with scale T / q_{Lt-1}.  Workspace: ckks_workspace_bytes(CKKS_OP_POLY_EVAL_TREE,
 * level, degree).  CKKS_ERR_ARG if all non-constant coefficients are zero. */
int32_t ckks_poly_eval_tree(ckks_ctx *ctx, const ckks_ct *x, const double *coeffs, uint32_t degree, const ckks_evk *rlk, ckks_ct *out,
                            void *ws, size_t ws_bytes, void *stream);

/* The same polynomial by baby steps and giant steps: blocks of m coefficients (m a power of two, 2 <= m <= degree) over
 * the baby powers x .. x^(m-1), times the giant powers (x^m)^i, i < G = degree / m + 1, the giant-step sum relinearised
 * once (ckks_mul_relin_sum): about m + 2 degree / m products instead of degree - 1, at most one level more than
 * ckks_poly_eval_tree.  The powers are formed as ckks_poly_eval_tree forms them; blocks are encoded so that every
 * product lands on the scale x.scale * q at the common level Lc = min(level of x^(m (G-1)), level of x^(m-1) - 1); the
 * result has level Lc - 1 and scale x.scale * q_{Lc-1} / q_{Lc-1}.  Workspace: ckks_poly_eval_bsgs_workspace_bytes.
 * Errors as ckks_poly_eval_tree; CKKS_ERR_ARG for an m that is not a power of two in [2, degree]. */
int32_t ckks_poly_eval_bsgs(ckks_ctx *ctx, const ckks_ct *x, const double *coeffs, uint32_t degree, uint32_t m, const ckks_evk *rlk,
                            ckks_ct *out, void *ws, size_t ws_bytes, void *stream);
size_t ckks_poly_eval_bsgs_workspace_bytes(const ckks_ctx *ctx, uint32_t level, uint32_t degree, uint32_t m);
/* The same polynomial of n ciphertexts at one level (an activation function over a layer's ciphertexts): every out[i] is
 * bit-identical to ckks_poly_eval_bsgs(x[i]); the n independent chains are spread over the context's lanes
 * (CKKS_OPT_LANES), each with a workspace of its own.  Errors as ckks_poly_eval_bsgs. */
int32_t ckks_poly_eval_bsgs_batch(ckks_ctx *ctx, const ckks_ct *x, uint32_t n, const double *coeffs, uint32_t degree, uint32_t m,
                                  const ckks_evk *rlk, ckks_ct *out, void *ws, size_t ws_bytes, void *stream);
size_t ckks_poly_eval_bsgs_batch_workspace_bytes(const ckks_ctx *ctx, uint32_t level, uint32_t degree, uint32_t m, uint32_t n);

/* ---- Softmax by doubling with a public shift (Algorithm 1) --------------------
 * One ciphertext of score rows: row r holds its row_len scores (a power of two dividing n) in slots
 * i * (n / row_len) + r, so that rotations by (n / row_len) 2^i, i < log2 row_len, leave a row's sum in every one of its
 * slots (keys for these rotations must be among `keys`).  exp_coeffs (host, exp_degree + 1 values, degree >= 2): the
 * polynomial p_exp(z / 2^rounds) written as a polynomial in z = x - shift; rsqrt_coeffs (host, rounds x
 * (rsqrt_degree + 1) values): round j's inverse-square-root polynomial.  Steps, all on the device:
 *   z = x - shift;  u = p_exp(z);  per round: s = row sums of u^2;  lambda = p_rsqrt_j(s);  u = (lambda u)^2,
 * every product followed by a rescale, both polynomials evaluated as ckks_poly_eval_tree does, or, where exp_m /
 * rsqrt_m is not 0, as ckks_poly_eval_bsgs does with blocks of that size.  No bootstrapping: with the power tree
 * the input needs (d_e + 1) + rounds * (d_r + 4) limbs more than the output keeps, d = ceil(log2 degree).  Scores should
 * be encrypted at a scale near the primes.  out: level and scale as they come out.  Workspace:
 * ckks_softmax_workspace_bytes.  Errors: ARG, LEVEL, NO_KEY, RANGE (a constant beyond 2^62), WORKSPACE. */
typedef struct {
    double shift;
    uint32_t rounds, row_len, exp_degree, rsqrt_degree;
    const double *exp_coeffs;   /* host */
    const double *rsqrt_coeffs; /* host */
    uint32_t exp_m, rsqrt_m;    /* 0: power tree; else the block size of ckks_poly_eval_bsgs */
} ckks_softmax_desc;
int32_t ckks_softmax(ckks_ctx *ctx, const ckks_softmax_desc *desc, const ckks_ct *in, const ckks_evk *rlk, const ckks_evk *keys,
                     uint32_t nkeys, ckks_ct *out, void *ws, size_t ws_bytes, void *stream);
size_t ckks_softmax_workspace_bytes(const ckks_ctx *ctx, const ckks_softmax_desc *desc, uint32_t level);

/* ---- Attention in a diagonal-block layout (Section 2.2: QK^T and PV multiply two encrypted operands; Section 4 names a
 * layout in which QK^T yields score diagonals that Softmax and PV consume without repacking, and does not define it) ----
 * The layout built here.  Every operand and score ciphertext uses the slot index
 *     slot = ((e * tokens + i) * heads + h) * R + r,     R = n / (diag_block * tokens * heads),
 * i a token position, h a head, e < diag_block, r trailing copies (tokens and diag_block powers of two, diag_block
 * dividing tokens, diag_block * tokens * heads dividing n).  Operands are one ciphertext per channel d:
 *     q[d]: Q[i, h, d] in every block e;      k[d], v[d]: token (i + e) mod tokens in block e.
 * (The 1/sqrt(dim) factor and, for grouped-query attention, the repetition of key/value heads are the caller's: they
 * are part of the projections that produce the operands.  No causal mask is applied.)
 *   ckks_attention_scores: S_g = rescale(sum_d q[d] * rot_g(k[d])) for g < groups = tokens / diag_block, rot_g the left
 *     rotation by g * diag_block * heads * R slots (cyclic over the flattened (e, i) index), the sum over d relinearised
 *     once (ckks_mul_relin_sum).  Slot (e, i, h) of S_g is the score of query i, head h against one key token; over all
 *     g and e every key token occurs exactly once, so the score row of (i, h) is the set of slots (e, i, h) of the S_g.
 *     scores: host array of `groups` descriptors with buffers for level - 1 limbs.  Every rotated operand is bit-identical
 *     to ckks_rotate's.  Workspace: ckks_attention_scores_workspace_bytes holds all rotated operands at once
 *     ((groups - 1) * dim ciphertexts); any workspace that holds one group's is accepted and the groups are then taken in passes.
 *     desc->group_baby = Gb > 1 (a power of two dividing groups) splits the groups g = g1 Gb + g0 into baby and giant steps:
 *     S_g = rot_{g1 Gb}( rescale( sum_d rot_{-g1 Gb}(q[d]) * rot_{g0}(k[d]) ) ), the same slot values (a rotation is a ring
 *     automorphism and a query operand rotated to the right is the query operand of cyclically shifted tokens) from other
 *     integers: per channel Gb - 1 key and groups / Gb - 1 query rotations instead of groups - 1 key rotations, and one
 *     rotation per group with g1 > 0 after its rescale.  The workspace then holds all rotated operands
 *     ((Gb + groups / Gb - 2) * dim ciphertexts) and is needed in full.  group_baby 0 or 1: no split.
 *   ckks_softmax_rows: Algorithm 1 on rows spread that way.  Per group u_g = p_exp(S_g - shift); per round
 *     t = rescale(sum_g u_g^2) (one relinearisation), t += rot(t, tokens * heads * R * 2^k) for k < log2 diag_block (cyclic
 *     over e: the row sum in every slot of the row), lambda = p_rsqrt_j(t) once for all groups, u_g = rescale(rescale(lambda
 *     u_g)^2).  desc->row_len, exp_m and rsqrt_m are ignored (both polynomials as ckks_poly_eval_tree).  in, out: host
 *     arrays of `groups` descriptors; out buffers sized for the input level.
 *   ckks_attention_values: out[d] = ladder(rescale(sum_g P_g * rot_g(v[d] truncated to P's level))), the same ladder
 *     over e: slot (e, i, h) of out[d] holds sum over all key tokens of probability x value, in every block e (the query
 *     operand's layout).  out: dim_v descriptors with buffers for P's level - 1.
 *   ckks_attention: the three in a row (scores at level - 1, then the Softmax's levels, then one more).
 * desc->token_inner = T' > 1 (dividing diag_block) keeps T' consecutive tokens innermost in the slot index,
 *     slot = ((((e * P + pos) * heads + h) * T' + t) * R + r,   token i = pos * T' + t,   P = tokens / T',
 * which is the order the projections' token-shard layout has (T' tokens per shard).  Operands are defined as above in terms
 * of (e, i, h); the four calls are the same for every T' (a group step is diag_block tokens = diag_block * heads * R slots
 * either way, the ladder steps tokens * heads * R * 2^k).  token_inner 0 or 1: a token's heads side by side.
 * keys must hold the rotations ckks_attention_rotations lists (token rotations first, then the ladder, then, with
 * group_baby > 1, the query operands' right rotations as negative numbers).
 * Errors: ARG, LEVEL, SCALE, NO_KEY, WORKSPACE, UNSUPPORTED (shape rules above), RANGE (a polynomial constant). */
typedef struct { uint32_t tokens, heads, diag_block, group_baby, token_inner; } ckks_attn_desc;
int32_t ckks_attention_rotations(const ckks_ctx *ctx, const ckks_attn_desc *desc, int64_t *rots, uint32_t cap);
int32_t ckks_attention_scores(ckks_ctx *ctx, const ckks_attn_desc *desc, const ckks_ct *q, const ckks_ct *k, uint32_t dim,
                              const ckks_evk *rlk, const ckks_evk *keys, uint32_t nkeys, ckks_ct *scores, void *ws, size_t ws_bytes, void *stream);
size_t ckks_attention_scores_workspace_bytes(const ckks_ctx *ctx, const ckks_attn_desc *desc, uint32_t level, uint32_t dim);
int32_t ckks_attention_values(ckks_ctx *ctx, const ckks_attn_desc *desc, const ckks_ct *probs, const ckks_ct *v, uint32_t dim_v,
                              const ckks_evk *rlk, const ckks_evk *keys, uint32_t nkeys, ckks_ct *out, void *ws, size_t ws_bytes, void *stream);
size_t ckks_attention_values_workspace_bytes(const ckks_ctx *ctx, const ckks_attn_desc *desc, uint32_t level);

int32_t ckks_softmax_rows(ckks_ctx *ctx, const ckks_attn_desc *desc, const ckks_softmax_desc *sm, const ckks_ct *in, const ckks_evk *rlk,
                          const ckks_evk *keys, uint32_t nkeys, ckks_ct *out, void *ws, size_t ws_bytes, void *stream);
size_t ckks_softmax_rows_workspace_bytes(const ckks_ctx *ctx, const ckks_attn_desc *desc, const ckks_softmax_desc *sm, uint32_t level);
int32_t ckks_attention(ckks_ctx *ctx, const ckks_attn_desc *desc, const ckks_softmax_desc *sm, const ckks_ct *q, const ckks_ct *k, uint32_t dim,
                       const ckks_ct *v, uint32_t dim_v, const ckks_evk *rlk, const ckks_evk *keys, uint32_t nkeys, ckks_ct *out,
                       void *ws, size_t ws_bytes, void *stream);
size_t ckks_attention_workspace_bytes(const ckks_ctx *ctx, const ckks_attn_desc *desc, const ckks_softmax_desc *sm, uint32_t level, uint32_t dim);

/* Conversion between the projections' token-shard layout and the attention operands (Section 6.2 names an adaptation of
 * the Q/K/V inputs before the attention products and a conversion after them; neither is defined in the text).  Needs
 * diag_block * tokens * heads = n and token_inner = the shards' tokens per ciphertext.  A shard ciphertext c < P holds, in
 * slot (d * heads + h) * T' + t, channel d of token c T' + t and head h (the feature-major layout with the features in
 * channel-major order, which is the caller's choice of the projection's output columns); B = heads * T' slots.
 *   Both directions start with a transpose between the ciphertext index and the block index:
 *       moved[y] = rot( rescale( sum_x rot(in[x], -x B) * mask(block x + y) ), y B ),
 *   one rotation per input and per output ciphertext, blocks counted cyclically over the n / B blocks.
 *   kind CKKS_ATTN_QUERY:     in: P shards -> out[d], d < dim, at level - 1: ladder(moved[d]): every block e alike.
 *   kind CKKS_ATTN_KEY_VALUE: in: P shards -> out[d] at level - 2 (level - 1 if diag_block = 1): with k0 = moved[d] and its
 *       copy in block 1, rescale( sum_e [ rot(k0, sA_e) * mask(block e, t < T' - b) + rot(k0, sB_e) * mask(block e, t >= T' - b) ] ),
 *       e = a T' + b, sA_e = a B + b - e P B, sB_e = (a + 1) B + b - T' - e P B: block e holds token i + e.
 *   kind CKKS_ATTN_TO_SHARDS: in: dim outputs in the query operand's layout -> out[c] = moved[c], c < P, at level - 1.
 * Masks are 0/1 plaintexts encoded at the scale of their level's last prime, so every rescale returns the input's scale;
 * every rotated ciphertext is bit-identical to ckks_rotate's (the token shifts of an operand share one ModUp).  out: host
 * array of descriptors with buffers for level - 1 limbs.  ckks_attention_pack_rotations lists the rotations a kind needs
 * (negative = to the right); returns their number.  Errors: ARG, LEVEL (level < 3), SCALE, NO_KEY, WORKSPACE, UNSUPPORTED. */
enum { CKKS_ATTN_QUERY = 0, CKKS_ATTN_KEY_VALUE = 1, CKKS_ATTN_TO_SHARDS = 2 };
int32_t ckks_attention_pack_rotations(const ckks_ctx *ctx, const ckks_attn_desc *desc, int32_t kind, uint32_t dim, int64_t *rots, uint32_t cap);
int32_t ckks_attention_pack(ckks_ctx *ctx, const ckks_attn_desc *desc, int32_t kind, const ckks_ct *in, uint32_t dim, const ckks_evk *keys,
                            uint32_t nkeys, ckks_ct *out, void *ws, size_t ws_bytes, void *stream);
size_t ckks_attention_pack_workspace_bytes(const ckks_ctx *ctx, const ckks_attn_desc *desc, int32_t kind, uint32_t level, uint32_t dim);

/* ---- Rot_k (Section 2.1, Rot + KeySwitch) ----------------------------------
 * Plain: apply sigma_g (g = key->galois) to both components, key-switch the
 * permuted c1: out = (sigma c0 + k0, k1).  Key switch = iNTT, centred ModUp
 * per digit, NTT, inner product with the key over the active limbs, centred
 * ModDown.  out must not alias in.  Errors: ARG, LEVEL, NO_KEY (galois 0 or
 * even), WORKSPACE. */
int32_t ckks_rotate(ckks_ctx *ctx, const ckks_ct *in, const ckks_evk *key, ckks_ct *out,
                    void *ws, size_t ws_bytes, void *stream);

/* The same rotation of n ciphertexts (one key) in one call: the key switches of up to 16 ciphertexts run side by
 * side and the key is read once per chunk.  Every out[i] is bit-identical to ckks_rotate(in[i], key).  in, out: host
 * arrays of n two-component ciphertexts at one level; out[i] may be in[i].  Workspace:
 * ckks_workspace_bytes(CKKS_OP_ROTATE_BATCH, level, n). */
int32_t ckks_rotate_batch(ckks_ctx *ctx, const ckks_ct *in, uint32_t n, const ckks_evk *key, ckks_ct *out, void *ws, size_t ws_bytes,
                          void *stream);

/* out = sum_i rotate(in[i], keys[i]) with the sum taken before the division by P ("lazy" ModDown, Section 2.1's key
 * switch): U = sum_i <ModUp(c1_i) read through sigma_{g_i}, key_i> over the limbs of Q_level P, then
 * out = (sum_i sigma_{g_i}(c0_i) + ModDown(U_0), ModDown(U_1)).  One division rounding instead of n, and one ModDown's
 * worth of transforms; n = 1 is ckks_rotate bit for bit.  in: host array of n two-component ciphertexts at one level
 * and scale; keys: host array of n rotation keys (keys[i] for in[i]); out may be any in[i].  Workspace:
 * ckks_workspace_bytes(CKKS_OP_ROTATE_SUM, level, n).  Errors: ARG, LEVEL, SCALE, NO_KEY, WORKSPACE. */
int32_t ckks_rotate_sum(ckks_ctx *ctx, const ckks_ct *in, const ckks_evk *keys, uint32_t n, ckks_ct *out, void *ws, size_t ws_bytes,
                        void *stream);

/* Hoisted: one iNTT + ModUp + NTT of c1 shared by nrot rotations; rotation r
 * permutes the extended digits by sigma_{g_r}, takes the inner product with
 * keys[r], ModDown, adds sigma(c0).  Every outs[r] is bit-identical to
 * ckks_rotate(in, keys[r]): the centred basis conversion is an odd function, so
 * it commutes with the signed permutation sigma.  keys, outs: host arrays of
 * nrot descriptors.  With the workspace ckks_workspace_bytes(CKKS_OP_ROTATE_HOISTED, level, nrot) asks
 * for, up to 16 rotations run side by side; any workspace of at least the CKKS_OP_ROTATE size is accepted.
 * Errors as ckks_rotate. */
int32_t ckks_rotate_hoisted(ckks_ctx *ctx, const ckks_ct *in, const ckks_evk *keys, uint32_t nrot, ckks_ct *outs,
                            void *ws, size_t ws_bytes, void *stream);

/* ---- Rescale (Section 2.1) --------------------------------------------------
 * Drops limb level-1 with exact rounding: out_i = (c_i - [centred c_last]) *
 * q_last^-1 mod q_i.  out->level = level-1, out->scale = in->scale / q_last.
 * out may alias in (the result is packed [ncomp][level-1][N]) only if ncomp
 * == 1; otherwise it must not overlap.  Errors: ARG, LEVEL (level < 2), WORKSPACE. */
int32_t ckks_rescale(ckks_ctx *ctx, const ckks_ct *in, ckks_ct *out, void *ws, size_t ws_bytes, void *stream);

/* ---- Rescale with built-in scratch ---------------------------------------------
 * (No counterpart in the paper: an addition for callers that cannot allocate.)
 * Same result as ckks_rescale, bit for bit, but needs no workspace argument and allocates nothing: its scratch
 * is a fixed array of CKKS_STATIC_SCRATCH_BYTES inside the library image, present on every GPU that loads the
 * library until the process exits.  Meant for callers that have no way to get device memory when the call is
 * made -- inside a stream capture, behind a frozen memory pool, or in an application that only lends this
 * library fixed buffers.
 *   - in, out: as for ckks_rescale (host descriptors, device data; out must not overlap in unless ncomp == 1).
 *   - Inputs with ncomp * level * N * 8 > CKKS_STATIC_SCRATCH_BYTES are refused with CKKS_ERR_WORKSPACE (the
 *     reason is readable through ckks_last_cuda_error); use ckks_rescale for those.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress); make that first
 *     call outside any stream capture.  Later calls only launch kernels.
 *   - All calls on a device share the one array and it keeps the previous call's contents.  Nothing in it needs
 *     clearing between calls, but two calls whose kernels can overlap on the GPU (different streams without an
 *     ordering between them) race on it: serialise them.
 * Errors: ARG, LEVEL, WORKSPACE (too large), UNSUPPORTED (device ordinal >= 64), CUDA. */
#define CKKS_STATIC_SCRATCH_BYTES (8u << 20)
int32_t ckks_rescale_static(ckks_ctx *ctx, const ckks_ct *in, ckks_ct *out, void *stream);

/* ---- Linear projection (Eq. 5, baby-step/giant-step) -----------------------
 * in: host array of nshards * n_in_blocks descriptors (index shard * n_in_blocks
 * + block), all at one level and scale.  W: device, row-major [d_in][d_out]
 * fp64.  keys: host array of nkeys rotation keys; every rotation the schedule
 * uses (ckks_linear_proj_rotations) must be present.  out: host array of
 * nshards * n_out_blocks descriptors with device buffers for level-1 limbs;
 * level and scale are set.  Schedule: hoisted baby rotations b*T (b < B) of
 * every input ciphertext; for each giant step g the pre-rotated diagonals are
 * extracted from W, encoded at pt_scale and multiply-accumulated over b and
 * over input blocks; the sum is rotated by g*B*T with the plain rotation and
 * added up; optional fold; one rescale per output ciphertext.
 * Errors: ARG, LEVEL, SCALE, NO_KEY, WORKSPACE, UNSUPPORTED (shape rules above). */
int32_t ckks_linear_proj(ckks_ctx *ctx, const ckks_proj_desc *desc, const ckks_ct *in, const double *W,
                         const ckks_evk *keys, uint32_t nkeys, ckks_ct *out,
                         void *ws, size_t ws_bytes, void *stream);
size_t ckks_linear_proj_workspace_bytes(const ckks_ctx *ctx, const ckks_proj_desc *desc, uint32_t level);

/*
 * Several projections of the same inputs in one call (the query/key/value or the gate/up matrices of a
 * transformer layer, Section 4: the activations are shared): descs[0..nmat-1] must agree in d_in,
 * tokens_per_shard, nshards and baby; W[m] is the device matrix of descs[m].  The extension of the inputs to the
 * key-switching basis and their baby-step rotations are computed once and used by every matrix; each matrix then
 * runs its own giant steps.  out: host array holding the outputs of matrix 0 (nshards * its output blocks, ordered
 * as in ckks_linear_proj), then those of matrix 1, and so on; every output is bit-identical to what a separate
 * ckks_linear_proj call returns.  Keys for the rotations of every matrix must be present.  Errors as
 * ckks_linear_proj; CKKS_ERR_ARG if the descriptors do not share their input shape.
 */
int32_t ckks_linear_proj_multi(ckks_ctx *ctx, const ckks_proj_desc *descs, uint32_t nmat, const ckks_ct *in, const double *const *W,
                               const ckks_evk *keys, uint32_t nkeys, ckks_ct *out, void *ws, size_t ws_bytes, void *stream);
size_t ckks_linear_proj_multi_workspace_bytes(const ckks_ctx *ctx, const ckks_proj_desc *descs, uint32_t nmat, uint32_t level);
/* Writes up to cap left-rotation amounts (in slots) the schedule needs into
 * rots (host) and returns how many there are; <0 on a shape error. */
int32_t ckks_linear_proj_rotations(const ckks_ctx *ctx, const ckks_proj_desc *desc, int64_t *rots, uint32_t cap);

#ifdef __cplusplus
}
#endif
#endif /* CKKS_B200_H */

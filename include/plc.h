/*
 * plc.h -- C ABI of libplc: predictive delta coding of a transformer KV cache on one B200.
 *
 * For every (session, layer, K-or-V, head, position) the library predicts the d-vector from the
 * next-token distribution, subtracts the prediction, quantises the residual with a uniform step and
 * entropy-codes it; the decoder inverts each step exactly at the quantised level.  A small second
 * path finds shared session prefixes (longest common prefix and the trie metric).
 *
 * Conventions
 *   - C linkage, no exceptions.  Every function returns a plc_status (0 = PLC_OK).
 *   - Every pointer named *_dev is DEVICE memory owned by the caller and must stay valid until the
 *     work enqueued on the given stream has completed.  Everything else is host memory.
 *   - All work is enqueued on the caller's cudaStream_t (passed as void*; NULL = default stream).
 *     Calls on one plc_ctx must be stream-ordered with respect to each other: the context's scratch
 *     (top-K results, encoder staging) is shared between calls.
 *   - The library allocates only inside plc_create / plc_reserve / plc_destroy (and inside
 *     plc_encode / plc_decode / plc_append_step when the reserved scratch is too small).
 *   - Problems found on the host (shapes, alignment) are returned at once and nothing is launched.
 *     Problems found on the device (output capacity, damaged streams) are OR-ed into a device status
 *     word that plc_sync_status reads; kernels never read or write outside the stated extents.
 *   - Floating-point inputs are IEEE binary16 ("f16").  NaN logits are not supported.
 *
 * Notation: S sessions, n positions per session, L layers, H KV heads, d head dimension
 * (32, 64, 128 or 256), V vocabulary, K candidates, W = 2*L*H streams per position.
 * Table id t = (layer*2 + kv)*H + head, kv = 0 for keys and 1 for values.
 */
#ifndef PLC_H
#define PLC_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t plc_status;
enum {
    PLC_OK = 0,
    PLC_E_INVALID = 1,   /* null pointer, non-positive size, value out of range */
    PLC_E_SHAPE = 2,     /* unsupported d, K > V, K > 1024, chunk_pos < 1 ... */
    PLC_E_ALIGN = 3,     /* a pointer or stride that must be 16-byte aligned is not */
    PLC_E_CAPACITY = 4,  /* payload buffer too small; *total_bytes_dev holds the size needed */
    PLC_E_CORRUPT = 5,   /* a chunk does not decode to its end state / runs past its bytes */
    PLC_E_STATE = 6,     /* call not valid in the object's current state */
    PLC_E_CUDA = 7       /* a CUDA runtime call failed (allocation, launch) */
};

enum { PLC_PRED_TOPK = 0, PLC_PRED_DENSE = 1, PLC_PRED_LINEAR = 2 };
enum { PLC_OUT_F32 = 0, PLC_OUT_F16 = 1 };

/* Codec parameters.  delta: quantiser step (>= 2^-12).  sigma_floor: added in quadrature to the
 * mixture's standard deviation before the scale class is taken (0 = none).  chunk_pos: positions
 * per independently coded chunk.  variant: PLC_PRED_TOPK (Sec. 7.1 of the paper, top-k
 * approximation), PLC_PRED_DENSE (Def. 5, sum over the whole vocabulary as a bf16 contraction) or
 * PLC_PRED_LINEAR (Sec. 7.1, linear-embedding approximation; contexts made by plc_create_linear). */
typedef struct {
    int32_t n_layers, n_kv_heads, head_dim, vocab, top_k;
    float delta, sigma_floor;
    int32_t chunk_pos;
    int32_t variant;
    int32_t out_dtype;   /* dtype plc_decode writes: PLC_OUT_F32 or PLC_OUT_F16 */
    /* Surprisal-adaptive quantiser (Def. 7 of the paper), used by plc_encode_adaptive /
     * plc_decode_adaptive: adaptive_b0 > 0 turns it on; a position of surprisal h_i = -log2 P(x_i | x_<i)
     * gets b_i = min(adaptive_b0 + adaptive_extra, max(1, floor(adaptive_b0 * h_i / adaptive_hbar)))
     * bits, i.e. the step delta * 2^(adaptive_b0 - b_i).  0 <= adaptive_extra <= 12, adaptive_b0 <= 16. */
    int32_t adaptive_b0, adaptive_extra;
    float adaptive_hbar;
    /* Zero-rate rule (Thm. 3 / Cor. 6 of the paper: a position whose residual variance per component
     * does not exceed the target distortion D needs no bits).  zero_rate_D > 0 turns it on: a
     * (stream, position) whose scale class q = round(4 log2(sigma^2 / step^2)) satisfies
     * q <= floor(4 log2(zero_rate_D / step^2) - 1/2) -- which implies sigma^2 <= zero_rate_D, sigma^2
     * being the mixture variance plus sigma_floor^2 -- puts nothing in the stream and decodes to the
     * prediction itself (symbols 0); the step/2 error bound does not hold there, the expected squared
     * error per component is at most zero_rate_D if KV follows the predictor's distribution.  With
     * the adaptive step the comparison uses the position's own step.  0 = off.  Works with every
     * variant and with plc_append_step. */
    float zero_rate_D;
} plc_config;

/* A KV tensor indexed [layer][kv][session][head][position][d]; strides in ELEMENTS, the d
 * components of one vector are contiguous and every vector starts on a 16-byte boundary. */
typedef struct {
    void* base_dev;
    int64_t stride_layer, stride_kv, stride_session, stride_head, stride_pos;
} plc_kv_view;

/* Coded output.  Chunk c of stream (session s, table t) has index slot
 *     slot = (((s*L + layer)*2 + kv)*H + head) * max_chunks + c
 * chunk_offset_dev[slot] = byte offset of the chunk in payload_dev (multiple of 16),
 * chunk_bytes_dev[slot]  = its exact size (0 = no such chunk).  Chunks are placed in the order in
 * which they are finished, so offsets differ from run to run; the bytes of each chunk do not.
 * *total_bytes_dev = bytes of payload_dev in use (with padding); the caller zeroes it before the
 * first plc_encode into a buffer and may keep it to append more chunks behind the ones present.
 * It must be a multiple of 16 whenever an encoder runs (the library only ever adds multiples of 16);
 * otherwise the chunks of that call are not written and the status word reports PLC_E_ALIGN. */
typedef struct {
    uint8_t* payload_dev;
    uint64_t payload_capacity;
    uint64_t* chunk_offset_dev;
    uint32_t* chunk_bytes_dev;
    uint64_t* total_bytes_dev;
    int32_t max_chunks;
} plc_streams;

/* Optional per-(session, position, table) exports of the coder's intermediate values, written by
 * plc_encode / plc_decode when the pointers are non-NULL: sym [S][n][W][d] int32 (quantised
 * residual), q [S][n][W] int32 (scale class), mu [S][n][W][d] float (prediction). */
typedef struct {
    int32_t* sym_dev;
    int32_t* q_dev;
    float* mu_dev;
    int32_t* bits_dev;   /* [S][n] int32: b_i of the adaptive quantiser (adaptive calls only) */
    int32_t count_ideal_bits;   /* non-zero (plc_encode and variants): add the code length the coder's model
                                 * assigns to everything coded to plc_stats.ideal_bits */
} plc_debug_buffers;

typedef struct {
    uint64_t payload_bytes;   /* sum of exact chunk sizes written since the counters were last reset */
    uint64_t n_chunks;
    uint64_t n_escapes;       /* components whose magnitude left the 63-symbol alphabet */
    uint64_t coded_vectors;   /* (stream, position) pairs covered by the chunks written */
    uint64_t skipped_vectors; /* of those, pairs the zero-rate rule left out of the stream */
    double ideal_bits;        /* sum over the coded components of log2(2^15 / f) + raw bit-plane bits + 32 per
                               * escape: the ideal -log2 P code length under the coder's own model (Prop. 2's
                               * "standard source coding" rate); only encodes that asked for it contribute
                               * (plc_debug_buffers.count_ideal_bits).  8 * payload_bytes exceeds it by the
                               * coder's state flush (128 bytes per chunk) and rounding only. */
} plc_stats;

/* State of a batch of B sessions that grow by one position per plc_append_step (lock step).
 * open_sym_dev [2][B][W][chunk_pos][d] int32 and open_q_dev [2][B][W][chunk_pos] int32 hold the
 * symbols and classes of positions that are not coded yet, in two buffers: chunk c uses buffer
 * c mod 2, so that the chunk completed last can be coded while the next one fills.  steps counts the
 * positions appended so far (host side).  The index in `streams` is [B][W][max_chunks] (the caller
 * zeroes it); chunk c holds positions [c*chunk_pos, ...). */
typedef struct {
    int32_t B;
    int32_t steps;
    int32_t* open_sym_dev;
    int32_t* open_q_dev;
    plc_streams streams;
} plc_session_batch;

typedef struct plc_ctx plc_ctx;

/* Creates a context for one parameter set and one candidate table.
 * T_dev: [L][2][H][V][d] f16, the stand-in for F_M(t_<i, t) of Def. 5 (one d-vector per layer, K/V,
 * head and candidate token); 16-byte aligned; must outlive the context (it is not copied).
 * Synchronises the device once (it pre-computes the squared norm of every row of T).
 * Errors: PLC_E_INVALID / PLC_E_SHAPE / PLC_E_ALIGN on bad arguments, PLC_E_CUDA. */
plc_status plc_create(plc_ctx** out, const plc_config* cfg, const void* T_dev);

/* Linear-embedding predictor (Sec. 7.1 of the paper: the KV function taken as affine in the token
 * embedding, so that the expectation over the next token moves inside it):
 *     KV^ = c + A * Ebar,   Ebar = sum_v P(v) E(v)   over the whole vocabulary,
 *     sigma_mix^2 = sum_v P(v) ||c + A E(v)||^2 / d - ||KV^||^2 / d          (Thm. 2 with F := c + A E).
 * E_dev [V][d_model], A_dev [L][2][H][d][d_model], c_dev [L][2][H][d], all f16, 16-byte aligned, not
 * copied (they must outlive the context).  d_model: a multiple of 64, at most 16384.
 * Arithmetic: P, E, A and Ebar are rounded to bfloat16 and contracted on the tensor cores with
 * binary32 accumulation; c is added in binary32. */
typedef struct {
    const void* E_dev;
    const void* A_dev;
    const void* c_dev;
    int32_t d_model;
} plc_linear_model;

/* Creates a context whose predictor is the linear-embedding model; cfg->variant must be
 * PLC_PRED_LINEAR (top_k is ignored by encode / decode, adaptive_b0 must be 0).  Builds, once, the
 * bf16 transpose of E and the table of candidate norms ||c + A E(v)||^2 / d of every layer (L
 * contractions of V x 2Hd x d_model), allocating and freeing its temporaries; synchronises the device.
 * plc_encode / plc_decode then work as for the other variants; plc_append_step returns PLC_E_STATE.
 * Errors: PLC_E_INVALID / PLC_E_SHAPE / PLC_E_ALIGN on bad arguments, PLC_E_CUDA. */
plc_status plc_create_linear(plc_ctx** out, const plc_config* cfg, const plc_linear_model* model);
plc_status plc_destroy(plc_ctx* ctx);

/* Grows the context's scratch so that calls over up to max_positions = S*n positions allocate
 * nothing (top-K results: 8*K bytes per position; encoder staging: fixed per device). */
plc_status plc_reserve(plc_ctx* ctx, int64_t max_positions);

/* Top-K softmax of N rows of logits (Sec. 5.1: P(t | t_<i) = softmax; Sec. 7.1: renormalised top-k;
 * Thm. 4(a): Z_k).  logits_dev [N][V] f16.  tokens_dev [N] int32 or NULL.
 * Outputs, each optional (NULL = skip): idx_dev [N][K] int32 ordered by (logit descending, index
 * ascending); w_dev [N][K] float, exp(l_k - l_max) / sum over the K; lse_dev [N] natural
 * log-sum-exp over V; zk_dev [N] sum of the K probabilities; logp2_dev [N] log2 P(tokens[i])
 * (needs tokens_dev; the edge weight of the probabilistic language trie, Def. 1).  A call with idx_dev,
 * w_dev and zk_dev all NULL does not determine the K largest at all (one pass for the maximum, one for
 * the sum): the cheap way to get the trie's edge weights for plc_prefix_dedup. */
plc_status plc_topk_softmax(plc_ctx* ctx, const void* logits_dev, const int32_t* tokens_dev, int64_t N,
                            int32_t* idx_dev, float* w_dev, float* lse_dev, float* zk_dev, float* logp2_dev,
                            void* stream);

/* Layer 1 (Def. 2; Sec. 7.3 best-match lookup = deepest stored ancestor).
 * tokens_dev [S][token_stride] int32, lens_dev [S], logp2_dev [S][token_stride] float.
 * lcp_dev [S][S] int32: length of the longest common prefix.  dT_dev [S][S] float:
 * d_T(a,b) = -sum_{j<lcp(a,b)} logp2[a][j] (0 for an empty common prefix).  parent_dev [S]: the
 * earlier session with the longest common prefix (ties: smallest index; none or length 0: -1).
 * shared_len_dev [S]: that length -- the pos_begin of plc_encode (Prop. 2: the shared prefix costs
 * zero bits, only the tail is coded).  All four outputs are written in full. */
plc_status plc_prefix_dedup(plc_ctx* ctx, const int32_t* tokens_dev, const int32_t* lens_dev, const float* logp2_dev,
                            int32_t S, int64_t token_stride, int32_t* lcp_dev, float* dT_dev, int32_t* parent_dev,
                            int32_t* shared_len_dev, void* stream);

/* Semantic prefix clusters (Def. 3 of the paper) on the matrices plc_prefix_dedup wrote.  Reading
 * taken: with d_T = -log2 P(s ^ s') a longer shared prefix gives a larger d_T, and
 * d_T(a,c) >= min(d_T(a,b), d_T(b,c)); the relation whose maximal subsets are unique is therefore
 * "the shared prefix carries at least delta bits", d_T(a,b) >= delta (compared in binary32, the
 * precision of dT_dev), which makes the clusters the cut of the trie at cost delta.  Every session
 * belongs to its own cluster.  Outputs, each [S] int32: cluster_dev = smallest member index (the
 * cluster's label), centroid_dev = the member with the largest P(s) = 2^-dT[s][s] (Def. 3's
 * argmax; ties: smallest index), begin_dev = lcp(s, centroid), the first position of s that the
 * centroid's cache does not cover (0 for the centroid itself): the pos_begin from which Cor. 3
 * charges for the tail.  delta >= 0. */
plc_status plc_prefix_clusters(plc_ctx* ctx, const int32_t* lcp_dev, const float* dT_dev, int32_t S, float delta,
                               int32_t* cluster_dev, int32_t* centroid_dev, int32_t* begin_dev, void* stream);

/* Trie-based prefix index of Sec. 7.3 (host side; all pointers are HOST memory): stored session
 * prefixes with insert, best-match lookup and evict, each one walk along a root-to-node path.
 * epsilon > 0 prunes the trie at nodes whose probability P(prefix) = prod_j P(x_j | x_<j) (Def. 1)
 * is below epsilon: a prefix is kept only down to its deepest node with P >= epsilon.
 *   insert: id must be new (PLC_E_STATE otherwise); logp2[j] = log2 P(tokens[j] | tokens[<j]);
 *           *stored_len (optional) = number of tokens kept.
 *   best_match: follows the query until it leaves all stored paths and reports the deepest stored
 *           ancestor: *lcp its depth, *dT = -log2 P of that common prefix (Def. 2), *id one stored
 *           prefix passing through it (the lexicographically smallest stored continuation, then the
 *           smallest id); *id = -1 when nothing is stored.
 *   evict: removes a stored prefix and the nodes no other prefix uses (PLC_E_INVALID if unknown). */
typedef struct plc_trie plc_trie;
plc_status plc_trie_create(plc_trie** out, float epsilon);
plc_status plc_trie_destroy(plc_trie* trie);
plc_status plc_trie_insert(plc_trie* trie, int32_t id, const int32_t* tokens, const float* logp2, int32_t len,
                           int32_t* stored_len);
plc_status plc_trie_best_match(const plc_trie* trie, const int32_t* tokens, int32_t len, int32_t* id, int32_t* lcp,
                               float* dT);
plc_status plc_trie_evict(plc_trie* trie, int32_t id);
plc_status plc_trie_stats(const plc_trie* trie, int64_t* n_nodes, int64_t* n_prefixes);

/* Integration point 1 of Sec. 7.2: before KV_i is written, predict it, subtract (Def. 6), quantise
 * and code the residual -- for every position in [pos_begin[s], pos_end[s]) of every session and
 * every stream.  logits_dev [S][n][V] f16, logits[s][i] being the distribution over token i.
 * pos_begin_dev / pos_end_dev [S] int32 or NULL (= 0 / n).  The index entries of all S*W*max_chunks
 * slots are rewritten (0 bytes for chunks that do not exist); out->max_chunks >= ceil(n/chunk_pos).
 * Chunk c of a session covers positions pos_begin + c*chunk_pos ... .
 * Device-side error: PLC_E_CAPACITY (nothing is written past payload_capacity). */
plc_status plc_encode(plc_ctx* ctx, const plc_kv_view* kv, const void* logits_dev, int32_t S, int32_t n,
                      const int32_t* pos_begin_dev, const int32_t* pos_end_dev, const plc_streams* out,
                      const plc_debug_buffers* dbg, void* stream);

/* Integration point 2 of Sec. 7.2: recompute the prediction identically, decode the residual, add
 * back (Prop. 3, "Correctness").  Writes cfg.out_dtype vectors into kv_out for the coded positions
 * only.  Device-side error: PLC_E_CORRUPT (reads never leave a chunk's bytes; a damaged chunk
 * yields garbage values for that chunk and sets the status). */
plc_status plc_decode(plc_ctx* ctx, const plc_streams* in, const void* logits_dev, int32_t S, int32_t n,
                      const int32_t* pos_begin_dev, const int32_t* pos_end_dev, const plc_kv_view* kv_out,
                      const plc_debug_buffers* dbg, void* stream);

/* The same two calls with the surprisal-adaptive step of Def. 7 (cfg.adaptive_b0 > 0, top-K variant).
 * tokens_dev [S][n] int32: the token at every position; both directions need it, because the step
 * of position i depends on the surprisal of the token that actually occurred there.  Calling these
 * with adaptive_b0 = 0, or plc_encode / plc_decode / plc_append_step with adaptive_b0 > 0, returns
 * PLC_E_STATE. */
plc_status plc_encode_adaptive(plc_ctx* ctx, const plc_kv_view* kv, const void* logits_dev, const int32_t* tokens_dev,
                               int32_t S, int32_t n, const int32_t* pos_begin_dev, const int32_t* pos_end_dev,
                               const plc_streams* out, const plc_debug_buffers* dbg, void* stream);
plc_status plc_decode_adaptive(plc_ctx* ctx, const plc_streams* in, const void* logits_dev, const int32_t* tokens_dev,
                               int32_t S, int32_t n, const int32_t* pos_begin_dev, const int32_t* pos_end_dev,
                               const plc_kv_view* kv_out, const plc_debug_buffers* dbg, void* stream);

/* Prop. 3 of the paper, step 3, with a rotated fixed-rate quantiser in place of the entropy-coded one
 * ("any per-vector quantizer" may follow the residual; the paper names TurboQuant and gives no details
 * of it, so this is the generic member of that family): for every coded (stream, position)
 *     x = eps * (KV - KV^),   y = H x  (Sylvester-Hadamard matrix of order d, scaled by d^(-1/2)),
 *     s = max |y|,   c_k = clamp(floor((y_k / s + 1) 2^bits / 2), 0, 2^bits - 1),
 * and back  y^_k = s ((c_k + 1/2) 2 / 2^bits - 1),  KV' = KV^ + eps * H y^,  so that
 * ||KV' - KV||_2 <= sqrt(d) s / 2^bits  (Prop. 3, "Correctness": the error on KV is the error on R).
 * eps_j = -1 where bit j of sign_bits is set, else +1: the caller draws these d random signs once and
 * passes the same ones to both directions.  KV^ is the top-k prediction of the context (PLC_PRED_TOPK,
 * adaptive_b0 = 0; PLC_E_STATE otherwise).
 * Records: fixed size, plc_rotq_record_bytes = 4 + d*bits/8 bytes (1 <= bits <= 8 and at most 256
 * bytes: PLC_E_SHAPE otherwise); the record of (session s, table t, position i) starts at byte
 * ((s*W + t)*n + i) * record_bytes of records_dev (4-byte aligned): the scale s as binary32, then for
 * g < d/32 and p < bits one 32-bit word whose bit l is bit p of the code of component
 * 8 (l mod d/8) + (d/32) (l div d/8) + g.  Positions outside [pos_begin, pos_end) are not touched.
 * Errors: PLC_E_CAPACITY if records_capacity < S*W*n*record_bytes (nothing is launched), and as for
 * plc_encode / plc_decode. */
typedef struct {
    int32_t bits;
    uint32_t sign_bits[8];
} plc_rotq_params;
plc_status plc_rotq_record_bytes(const plc_ctx* ctx, int32_t bits, uint64_t* bytes);
plc_status plc_encode_rotq(plc_ctx* ctx, const plc_kv_view* kv, const void* logits_dev, int32_t S, int32_t n,
                           const int32_t* pos_begin_dev, const int32_t* pos_end_dev, const plc_rotq_params* params,
                           void* records_dev, uint64_t records_capacity, void* stream);
plc_status plc_decode_rotq(plc_ctx* ctx, const void* records_dev, uint64_t records_capacity, const void* logits_dev,
                           int32_t S, int32_t n, const int32_t* pos_begin_dev, const int32_t* pos_end_dev,
                           const plc_rotq_params* params, const plc_kv_view* kv_out, void* stream);

/* Decode-time append (integration point 1 for one new token per session).  kv_step_dev
 * [L][2][B][H][d] f16, logits_step_dev [B][V] f16.  The new position's symbols and class go to the
 * open chunk (a LIFO coder cannot be extended in place, so a stream grows chunk by chunk).  A chunk
 * that has reached chunk_pos positions is coded into sb->streams over the following chunk_pos steps,
 * 1/chunk_pos of the B*W streams per step (stream i = table*B + session in slice
 * floor(i*chunk_pos / (B*W)) is coded by the step at which steps mod chunk_pos equals the slice
 * number), so that every step costs the same: chunk c of every stream is in sb->streams once
 * steps >= (c+2)*chunk_pos - 1, or after plc_append_flush.  sb->steps is advanced. */
plc_status plc_append_step(plc_ctx* ctx, plc_session_batch* sb, const void* kv_step_dev, const void* logits_step_dev,
                           void* stream);
/* Codes what is not coded yet (the remaining slices of the chunk completed last and the partly
 * filled open chunk, if any) so that all sb->steps positions are decodable with
 * plc_decode(S = B, n = steps).  No further plc_append_step is allowed afterwards. */
plc_status plc_append_flush(plc_ctx* ctx, plc_session_batch* sb, void* stream);
/* Bytes of open_sym_dev / open_q_dev for B sessions (both buffers). */
plc_status plc_append_sizes(const plc_ctx* ctx, int32_t B, uint64_t* open_sym_bytes, uint64_t* open_q_bytes);

/* Entropy-codes one chunk per stream from symbols and classes that are already on the device,
 * without allocating anything.  (The paper has no counterpart for this call: it exists for callers
 * that are not allowed to allocate device memory at the point where they seal a chunk -- code that
 * runs inside a serving loop with a frozen memory pool, inside a memory-budgeted plugin, or after
 * start-up in a process whose allocator is locked down -- and that therefore cannot own a plc_ctx,
 * whose creation allocates.)  The bitstream is exactly the one plc_append_step / plc_append_flush
 * write for the same symbols and classes.
 *   sym_dev [n_streams][chunk_capacity][head_dim] int32, q_dev [n_streams][chunk_capacity] int32:
 *   the first n_pos positions of every stream are coded (the layout of one buffer of
 *   plc_session_batch's open chunks, with n_streams = B*W); classes outside [-24, 135] are clamped
 *   and reported.
 *   Chunk `chunk_index` of stream i goes to index slot i*out->max_chunks + chunk_index.
 *   status_dev: one device word, an OUTPUT: 0, or a bit-or of 1 (payload capacity exceeded; nothing
 *   is written past it and *total_bytes_dev holds the size needed), 4 (a class was out of range) and
 *   16 (*total_bytes_dev was not a multiple of 16: the chunk is not written).
 * Limits: n_pos * head_dim <= 4096 components per chunk (PLC_E_SHAPE beyond that); head_dim in
 * {32, 64, 128, 256}.  All working memory is one static device array of about 8 MiB that every GPU
 * using the library holds until the process exits.  Every call on a device shares that array, so
 * two calls whose kernels could overlap on the GPU (different streams, no ordering) race with each
 * other: order them.  The first call on each device looks up the array's device address (with that
 * device current); make that first call before starting any stream capture. */
plc_status plc_rans_encode_static(const int32_t* sym_dev, const int32_t* q_dev, int32_t n_streams, int32_t n_pos,
                                  int32_t head_dim, int32_t chunk_capacity, int32_t chunk_index,
                                  const plc_streams* out, uint32_t* status_dev, void* stream);

/* Waits for the stream and returns the device status word's most severe code; clears it.
 * PLC_E_ALIGN here means that *total_bytes_dev was not a multiple of 16 when an encoder reserved a
 * chunk's place (the chunk is then not written). */
plc_status plc_sync_status(plc_ctx* ctx, void* stream);
/* The same word read without waiting for any enqueued work (a 4-byte copy on a stream of the
 * context's own) and without clearing it: *bits receives the raw word (1 capacity, 2 corrupt,
 * 8 a bounded wait inside a kernel ran out, 16 unaligned byte cursor), the return value its most
 * severe code.  Work still running may set further bits afterwards. */
plc_status plc_poll_status(plc_ctx* ctx, uint32_t* bits);
/* Waits for the stream, copies the counters, optionally clears them. */
plc_status plc_get_stats(plc_ctx* ctx, plc_stats* out, int32_t reset, void* stream);

/* The two 32-bit constants (theta, rho) from which the frequency table of table id qp in [-24,15]
 * is built with integer arithmetic, and the table itself (f[64], c[65]); host-side, no GPU work. */
plc_status plc_table_constants(int32_t qp, uint32_t* theta, uint32_t* rho);
plc_status plc_build_table(int32_t qp, uint32_t* f, uint32_t* c);
/* With profiling on, plc_encode / plc_decode record CUDA events on the caller's stream directly
 * around their fused predict+code kernel (the top-K kernel that precedes it is outside);
 * plc_last_kernel_ms waits for the most recent such launch (which = 0 encode, 1 decode, 2 the dense
 * variant's tensor-core contraction of the last layer) and returns its duration.  PLC_E_STATE if
 * no such launch was recorded. */
plc_status plc_set_profiling(plc_ctx* ctx, int32_t on);
/* Work-queue layout the most recent top-K plc_encode / plc_decode of this context used: *n_queues
 * queues of (table, session, chunk) items, each served by *sms_per_queue SMs (one queue for the whole
 * GPU when the tables in flight fit in L2, else about one table's worth of chunks per queue).  For
 * tests and benchmarks that must state which path they ran.  PLC_E_STATE before the first such call. */
plc_status plc_last_schedule(const plc_ctx* ctx, int32_t* n_queues, int32_t* sms_per_queue);
plc_status plc_last_kernel_ms(plc_ctx* ctx, int32_t which, float* ms);
/* Every profiled launch since the last reset keeps its event pair (up to 4096 per kind; further
 * launches overwrite the newest).  Waits for them and returns their mean duration and their number
 * (each optional); reset != 0 then empties the log of that kind.  Meant to be called outside a
 * timed region: it synchronises with the recorded events. */
plc_status plc_kernel_ms(plc_ctx* ctx, int32_t which, float* mean_ms, int32_t* launches, int32_t reset);
/* Number of kernels this library has launched in this process (for benchmarks). */
uint64_t plc_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* PLC_H */

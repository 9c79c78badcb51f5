// C ABI of libplc (see include/plc.h): argument checks, context scratch, kernel launches.
#include <atomic>
#include <new>
#include <vector>

#include "plc_common.cuh"
#include <cmath>

namespace plc {
static std::atomic<unsigned long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }
}  // namespace plc

using namespace plc;

struct plc_ctx {
    plc_config cfg;
    const __half* T;
    float* rownorm2;
    int2* pairs;
    uint8_t* cand;                  // [positions] candidate lists + headers of the two-kernel selection
    int* step_exp;                  // [positions] adaptive step exponents
    long long pairs_cap;            // positions
    uint16_t* staging;
    unsigned long long staging_words_per_warp;
    unsigned int* ticket;
    unsigned int* status;
    unsigned int* status_host;      // pinned word plc_poll_status copies into
    cudaStream_t poll_stream;       // non-blocking stream of plc_poll_status
    cudaStream_t side_stream;       // append path: the slice of a completed chunk is coded beside the step's own kernels
    cudaEvent_t side_ev[2];         // fork / join of the side stream
    unsigned int* side_ticket;      // work counter of the side stream's launches
    Counters* counters;
    uint8_t* dense_scratch;         // dense variant: P, Tb, n2b, mu, s1; linear variant: P, Ebar, s1, A_layer, mu
    size_t dense_bytes;
    const __half* lin_E;            // linear variant (Sec. 7.1): caller's E [V][dm], A [L][2H*d][dm], c [L][2H*d]
    const __half* lin_A;
    const __half* lin_c;
    int lin_dm;
    uint8_t* lin_model;             // linear: E transposed (bf16) and the candidate-norm table of every (layer, table);
                                    // dense: the candidate-norm table alone
    size_t lin_off[2];
    int last_nq, last_g;            // work-queue layout of the most recent top-K encode / decode launch
    int profiling;                  // record events around the codec kernels
    // Event pairs (start, stop) of the profiled launches since the last reset, per kind: 0 encode
    // kernel, 1 decode kernel, 2 tensor-core contraction.  Events are created on demand and reused.
    std::vector<cudaEvent_t> prof_ev[3];
    int prof_used[3];               // pairs in use
};

namespace {
constexpr int kMaxProfPairs = 4096;

// Next event pair of a kind (the newest pair is reused once the log is full); null when profiling is off.
cudaEvent_t* prof_pair(plc_ctx* c, int which) {
    if (!c->profiling) return nullptr;
    std::vector<cudaEvent_t>& v = c->prof_ev[which];
    if (c->prof_used[which] == kMaxProfPairs) c->prof_used[which] -= 1;
    const int i = c->prof_used[which];
    while ((int)v.size() < 2 * (i + 1)) {
        cudaEvent_t e = nullptr;
        if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
        v.push_back(e);
    }
    c->prof_used[which] = i + 1;
    return &v[2 * i];
}
}  // namespace

namespace {

plc_status status_code(unsigned int w) {
    if (w & kStTimeout) return PLC_E_CUDA;
    if (w & kStCorrupt) return PLC_E_CORRUPT;
    if (w & kStCursor) return PLC_E_ALIGN;
    if (w & kStCapacity) return PLC_E_CAPACITY;
    return PLC_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
bool valid_d(int d) { return d == 32 || d == 64 || d == 128 || d == 256; }

plc_status check_view(const plc_kv_view* v, int d, int elem_bytes) {
    if (!v || !v->base_dev) return PLC_E_INVALID;
    if (!aligned16(v->base_dev)) return PLC_E_ALIGN;
    const int64_t per16 = 16 / elem_bytes;
    const int64_t st[5] = {v->stride_layer, v->stride_kv, v->stride_session, v->stride_head, v->stride_pos};
    for (int i = 0; i < 5; ++i)
        if (st[i] % per16) return PLC_E_ALIGN;
    (void)d;
    return PLC_OK;
}

plc_status check_streams(const plc_streams* s, int need_chunks) {
    if (!s || !s->payload_dev || !s->chunk_offset_dev || !s->chunk_bytes_dev || !s->total_bytes_dev) return PLC_E_INVALID;
    if (!aligned16(s->payload_dev)) return PLC_E_ALIGN;
    if (s->max_chunks < need_chunks || s->max_chunks < 1) return PLC_E_SHAPE;
    return PLC_OK;
}

int padded_k(const plc_config& cfg) {
    const int rows = 256 / cfg.head_dim;      // rows of T that one warp-wide 16-byte-per-lane load fetches
    return (cfg.top_k + rows - 1) / rows * rows;
}

// Scratch of the two-kernel selection: headers first (16 bytes per row), then the lists.
size_t cand_word_bytes(const plc_config& cfg) { return cfg.vocab <= 65536 ? 4 : 8; }
size_t cand_bytes(const plc_config& cfg, long long positions) {
    return (size_t)positions * (16 + (size_t)kTopkListCap * cand_word_bytes(cfg)) + 16;   // + the redo counter
}
void set_cand(const plc_ctx* c, TopkArgs& a, long long positions);

plc_status ensure_pairs(plc_ctx* c, long long positions) {
    if (positions <= c->pairs_cap) return PLC_OK;
    if (c->pairs) cudaFree(c->pairs);
    if (c->step_exp) cudaFree(c->step_exp);
    if (c->cand) cudaFree(c->cand);
    c->pairs = nullptr; c->step_exp = nullptr; c->cand = nullptr; c->pairs_cap = 0;
    if (cudaMalloc(&c->pairs, sizeof(int2) * (size_t)positions * padded_k(c->cfg)) != cudaSuccess) return PLC_E_CUDA;
    if (cudaMalloc(&c->step_exp, sizeof(int) * (size_t)positions) != cudaSuccess) return PLC_E_CUDA;
    if (cudaMalloc(&c->cand, cand_bytes(c->cfg, positions)) != cudaSuccess) return PLC_E_CUDA;
    c->pairs_cap = positions;
    return PLC_OK;
}

void set_cand(const plc_ctx* c, TopkArgs& a, long long positions) {
    a.cand_hdr = reinterpret_cast<float4*>(c->cand);
    a.cand = c->cand + (size_t)positions * 16;
    a.redo = reinterpret_cast<unsigned int*>(c->cand + (size_t)positions * (16 + (size_t)kTopkListCap * cand_word_bytes(c->cfg)));
}

CodecArgs base_args(const plc_ctx* c) {
    CodecArgs a{};
    a.sh.L = c->cfg.n_layers; a.sh.H = c->cfg.n_kv_heads; a.sh.d = c->cfg.head_dim; a.sh.V = c->cfg.vocab;
    a.sh.K = c->cfg.top_k; a.sh.Kp = padded_k(c->cfg); a.sh.chunk_pos = c->cfg.chunk_pos; a.sh.out_dtype = c->cfg.out_dtype;
    a.sh.delta = c->cfg.delta; a.sh.sigma_floor = c->cfg.sigma_floor;
    a.sh.inv_delta = 1.0f / c->cfg.delta;
    a.sh.inv_delta2 = (float)(1.0 / ((double)c->cfg.delta * (double)c->cfg.delta));
    // zero-rate rule (Thm. 3): skip iff q <= floor(4 log2(D / delta^2) - 1/2), which implies sigma^2 <= D
    a.sh.zero_q = c->cfg.zero_rate_D > 0.0f
        ? (int)floor(4.0 * log2((double)c->cfg.zero_rate_D / ((double)c->cfg.delta * (double)c->cfg.delta)) - 0.5)
        : kZeroOff;
    a.T = c->T; a.rownorm2 = c->rownorm2; a.pairs = c->pairs;
    a.staging = c->staging; a.staging_words_per_warp = c->staging_words_per_warp;
    a.ticket = c->ticket; a.status = c->status; a.counters = c->counters;
    return a;
}

DenseShape dense_shape(const plc_ctx* c, long long rows) {
    DenseShape sh;
    sh.rows = rows; sh.V = c->cfg.vocab; sh.d = c->cfg.head_dim; sh.tables = 2 * c->cfg.n_kv_heads;
    sh.ldv = (sh.V + 63) / 64 * 64;
    sh.ncols = sh.tables * sh.d; sh.ncols_pad = (sh.ncols + 255) / 256 * 256;
    sh.nt_all = c->cfg.n_layers * sh.tables; sh.nt_all_pad = (sh.nt_all + 255) / 256 * 256;
    return sh;
}

LinearShape linear_shape(const plc_config& cfg, int dm, long long rows) {
    LinearShape sh;
    sh.rows = rows; sh.V = cfg.vocab; sh.d = cfg.head_dim; sh.dm = dm; sh.tables = 2 * cfg.n_kv_heads; sh.L = cfg.n_layers;
    sh.ldv = (sh.V + 63) / 64 * 64;
    sh.ncols = sh.tables * sh.d; sh.ncols_pad = (sh.ncols + 255) / 256 * 256;
    sh.nt_all = sh.L * sh.tables; sh.nt_all_pad = (sh.nt_all + 255) / 256 * 256;
    return sh;
}

plc_status ensure_scratch(plc_ctx* c, size_t need) {
    if (need <= c->dense_bytes) return PLC_OK;
    if (c->dense_scratch) cudaFree(c->dense_scratch);
    c->dense_scratch = nullptr; c->dense_bytes = 0;
    if (cudaMalloc(&c->dense_scratch, need) != cudaSuccess) return PLC_E_CUDA;
    c->dense_bytes = need;
    return PLC_OK;
}

plc_status ensure_dense(plc_ctx* c, const DenseShape& sh, size_t* off) {
    const size_t need = dense_scratch_bytes(sh, off);
    if (need <= c->dense_bytes) return PLC_OK;
    if (c->dense_scratch) cudaFree(c->dense_scratch);
    c->dense_scratch = nullptr; c->dense_bytes = 0;
    if (cudaMalloc(&c->dense_scratch, need) != cudaSuccess) return PLC_E_CUDA;
    c->dense_bytes = need;
    return PLC_OK;
}

StreamsDev to_dev(const plc_streams* s) {
    StreamsDev d;
    d.payload = s->payload_dev; d.capacity = s->payload_capacity;
    d.chunk_offset = reinterpret_cast<unsigned long long*>(s->chunk_offset_dev);
    d.chunk_bytes = s->chunk_bytes_dev;
    d.total_bytes = reinterpret_cast<unsigned long long*>(s->total_bytes_dev);
    d.max_chunks = s->max_chunks;
    return d;
}

KvView to_dev(const plc_kv_view* v) {
    return KvView{v->base_dev, v->stride_layer, v->stride_kv, v->stride_session, v->stride_head, v->stride_pos};
}

}  // namespace

extern "C" {

static plc_status create_common(plc_ctx** out, const plc_config* cfg, const void* T_dev, const plc_linear_model* lin);

plc_status plc_create(plc_ctx** out, const plc_config* cfg, const void* T_dev) {
    if (!out || !cfg || !T_dev) return PLC_E_INVALID;
    if (cfg->variant != PLC_PRED_TOPK && cfg->variant != PLC_PRED_DENSE) return PLC_E_INVALID;
    return create_common(out, cfg, T_dev, nullptr);
}

plc_status plc_create_linear(plc_ctx** out, const plc_config* cfg, const plc_linear_model* model) {
    if (!out || !cfg || !model || !model->E_dev || !model->A_dev || !model->c_dev) return PLC_E_INVALID;
    if (cfg->variant != PLC_PRED_LINEAR) return PLC_E_INVALID;
    if (model->d_model < 64 || model->d_model % 64 || model->d_model > 16384) return PLC_E_SHAPE;
    if ((long long)cfg->n_layers * 2 * cfg->n_kv_heads > 65536) return PLC_E_SHAPE;
    if (!aligned16(model->E_dev) || !aligned16(model->A_dev) || !aligned16(model->c_dev)) return PLC_E_ALIGN;
    return create_common(out, cfg, nullptr, model);
}

static plc_status create_common(plc_ctx** out, const plc_config* cfg, const void* T_dev, const plc_linear_model* lin) {
    *out = nullptr;
    if (cfg->n_layers < 1 || cfg->n_kv_heads < 1 || cfg->vocab < 1) return PLC_E_INVALID;
    if (!valid_d(cfg->head_dim) || cfg->top_k < 1 || cfg->top_k > cfg->vocab || cfg->top_k > 1024) return PLC_E_SHAPE;
    if (cfg->chunk_pos < 1 || cfg->chunk_pos > 4096) return PLC_E_SHAPE;
    if (!(cfg->delta >= 1.0f / 4096.0f) || !(cfg->delta < 65536.0f) || !(cfg->sigma_floor >= 0.0f)) return PLC_E_INVALID;
    if (cfg->out_dtype != PLC_OUT_F32 && cfg->out_dtype != PLC_OUT_F16) return PLC_E_INVALID;
    if (cfg->adaptive_b0 < 0 || cfg->adaptive_b0 > 16 || cfg->adaptive_extra < 0 || cfg->adaptive_extra > 12) return PLC_E_INVALID;
    if (cfg->adaptive_b0 > 0 && !(cfg->adaptive_hbar > 0.0f)) return PLC_E_INVALID;
    if (!(cfg->zero_rate_D >= 0.0f) || !(cfg->zero_rate_D < 1e30f)) return PLC_E_INVALID;
    if (cfg->adaptive_b0 > 0 && cfg->variant != PLC_PRED_TOPK) return PLC_E_STATE;
    if (cfg->variant != PLC_PRED_TOPK && 2 * cfg->n_kv_heads > 256) return PLC_E_SHAPE;
    if (T_dev && !aligned16(T_dev)) return PLC_E_ALIGN;
    plc_ctx* c = new (std::nothrow) plc_ctx();
    if (!c) return PLC_E_CUDA;
    c->cfg = *cfg;
    c->T = static_cast<const __half*>(T_dev);
    const long long rows = (long long)cfg->n_layers * 2 * cfg->n_kv_heads * cfg->vocab;
    c->staging_words_per_warp = 4ull * cfg->chunk_pos * cfg->head_dim + 64;
    const int warps = codec_grid_warps(0);
    bool ok = (!T_dev || cudaMalloc(&c->rownorm2, sizeof(float) * (size_t)rows) == cudaSuccess) &&
              cudaMalloc(&c->staging, sizeof(uint16_t) * c->staging_words_per_warp * warps) == cudaSuccess &&
              cudaMalloc(&c->ticket, sizeof(unsigned int) * kTicketWords) == cudaSuccess &&
              cudaMalloc(&c->status, sizeof(unsigned int)) == cudaSuccess &&
              cudaMallocHost(&c->status_host, sizeof(unsigned int)) == cudaSuccess &&
              cudaStreamCreateWithFlags(&c->poll_stream, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&c->side_stream, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&c->side_ev[0], cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&c->side_ev[1], cudaEventDisableTiming) == cudaSuccess &&
              cudaMalloc(&c->side_ticket, sizeof(unsigned int)) == cudaSuccess &&
              cudaMalloc(&c->counters, sizeof(Counters)) == cudaSuccess;
    if (ok) ok = cudaMemset(c->status, 0, sizeof(unsigned int)) == cudaSuccess &&
                 cudaMemset(c->counters, 0, sizeof(Counters)) == cudaSuccess;
    if (ok && T_dev) ok = launch_rownorm(c->T, c->rownorm2, rows, cfg->head_dim, 0) == cudaSuccess &&
                          cudaDeviceSynchronize() == cudaSuccess;
    if (ok && T_dev && cfg->variant == PLC_PRED_DENSE) {     // candidate norms of every layer, once
        const DenseShape sh = dense_shape(c, 0);
        ok = (long long)cfg->n_layers * 2 * cfg->n_kv_heads <= 65536 &&
             cudaMalloc(&c->lin_model, dense_model_bytes(sh)) == cudaSuccess &&
             dense_prepare(c->T, cfg->n_layers, sh, c->lin_model, 0) == cudaSuccess && cudaDeviceSynchronize() == cudaSuccess;
    }
    if (ok && lin) {
        c->lin_E = static_cast<const __half*>(lin->E_dev); c->lin_A = static_cast<const __half*>(lin->A_dev);
        c->lin_c = static_cast<const __half*>(lin->c_dev); c->lin_dm = lin->d_model;
        const LinearShape sh = linear_shape(*cfg, lin->d_model, 0);
        const size_t bytes = linear_model_bytes(sh, c->lin_off);
        ok = cudaMalloc(&c->lin_model, bytes) == cudaSuccess &&
             linear_prepare(c->lin_E, c->lin_A, c->lin_c, sh, c->lin_model, c->lin_off, c->status, 0) == cudaSuccess;
    }
    if (!ok) { plc_destroy(c); return PLC_E_CUDA; }
    *out = c;
    return PLC_OK;
}

plc_status plc_destroy(plc_ctx* c) {
    if (!c) return PLC_E_INVALID;
    cudaFree(c->rownorm2); cudaFree(c->pairs); cudaFree(c->cand); cudaFree(c->step_exp); cudaFree(c->staging);
    cudaFree(c->ticket); cudaFree(c->status); cudaFree(c->counters); cudaFree(c->dense_scratch); cudaFree(c->lin_model);
    for (int k = 0; k < 3; ++k)
        for (cudaEvent_t e : c->prof_ev[k]) cudaEventDestroy(e);
    if (c->status_host) cudaFreeHost(c->status_host);
    if (c->poll_stream) cudaStreamDestroy(c->poll_stream);
    if (c->side_stream) cudaStreamDestroy(c->side_stream);
    for (int i = 0; i < 2; ++i) if (c->side_ev[i]) cudaEventDestroy(c->side_ev[i]);
    cudaFree(c->side_ticket);
    delete c;
    return PLC_OK;
}

plc_status plc_reserve(plc_ctx* c, int64_t max_positions) {
    if (!c || max_positions < 0) return PLC_E_INVALID;
    return ensure_pairs(c, max_positions);
}

plc_status plc_topk_softmax(plc_ctx* c, const void* logits_dev, const int32_t* tokens_dev, int64_t N, int32_t* idx_dev,
                            float* w_dev, float* lse_dev, float* zk_dev, float* logp2_dev, void* stream) {
    if (!c || !logits_dev || N < 0) return PLC_E_INVALID;
    if (logp2_dev && !tokens_dev) return PLC_E_INVALID;
    TopkArgs a{};
    a.logits = static_cast<const __half*>(logits_dev); a.tokens = tokens_dev; a.N = N;
    a.V = c->cfg.vocab; a.K = c->cfg.top_k;
    a.idx = idx_dev; a.w = w_dev; a.lse = lse_dev; a.zk = zk_dev; a.logp2 = logp2_dev;
    a.n_per_session = 1; a.status = c->status;
    if (idx_dev || w_dev || zk_dev) {                    // the selection uses the context's scratch
        plc_status rc = ensure_pairs(c, N);
        if (rc) return rc;
        set_cand(c, a, c->pairs_cap);
    }
    return launch_topk(a, static_cast<cudaStream_t>(stream)) == cudaSuccess ? PLC_OK : PLC_E_CUDA;
}

plc_status plc_prefix_dedup(plc_ctx* c, const int32_t* tokens_dev, const int32_t* lens_dev, const float* logp2_dev,
                            int32_t S, int64_t token_stride, int32_t* lcp_dev, float* dT_dev, int32_t* parent_dev,
                            int32_t* shared_len_dev, void* stream) {
    if (!c || !tokens_dev || !lens_dev || !logp2_dev || !lcp_dev || !dT_dev || !parent_dev || !shared_len_dev)
        return PLC_E_INVALID;
    if (S < 0 || token_stride < 0) return PLC_E_INVALID;
    return launch_prefix_dedup(tokens_dev, lens_dev, logp2_dev, S, token_stride, lcp_dev, dT_dev, parent_dev,
                               shared_len_dev, static_cast<cudaStream_t>(stream)) == cudaSuccess ? PLC_OK : PLC_E_CUDA;
}

plc_status plc_prefix_clusters(plc_ctx* c, const int32_t* lcp_dev, const float* dT_dev, int32_t S, float delta,
                               int32_t* cluster_dev, int32_t* centroid_dev, int32_t* begin_dev, void* stream) {
    if (!c || !lcp_dev || !dT_dev || !cluster_dev || !centroid_dev || !begin_dev) return PLC_E_INVALID;
    if (S < 0 || !(delta >= 0.0f)) return PLC_E_INVALID;
    return launch_prefix_clusters(lcp_dev, dT_dev, S, delta, cluster_dev, centroid_dev, begin_dev,
                                  static_cast<cudaStream_t>(stream)) == cudaSuccess ? PLC_OK : PLC_E_CUDA;
}

static plc_status run_topk_for(plc_ctx* c, const void* logits_dev, int S, int n, const int32_t* pb, const int32_t* pe,
                               cudaStream_t st, const int32_t* tokens = nullptr, int32_t* bits_out = nullptr) {
    plc_status rc = ensure_pairs(c, (long long)S * n);
    if (rc) return rc;
    TopkArgs a{};
    a.logits = static_cast<const __half*>(logits_dev); a.N = (long long)S * n; a.V = c->cfg.vocab; a.K = c->cfg.top_k;
    a.pairs = c->pairs; a.Kp = padded_k(c->cfg); a.n_per_session = n; a.pos_begin = pb; a.pos_end = pe;
    set_cand(c, a, c->pairs_cap); a.status = c->status;
    if (tokens) {
        a.tokens = tokens; a.step_exp = c->step_exp; a.bits_out = bits_out;
        a.b0 = c->cfg.adaptive_b0; a.extra = c->cfg.adaptive_extra; a.hbar = c->cfg.adaptive_hbar;
    }
    return launch_topk(a, st) == cudaSuccess ? PLC_OK : PLC_E_CUDA;
}

// Dense variant: softmax once, then per layer the bf16 contraction and the coding of its 2H tables.
static plc_status run_dense(plc_ctx* c, CodecArgs a, const void* logits_dev, bool encode, cudaStream_t st) {
    const DenseShape sh = dense_shape(c, (long long)a.S * a.n);
    if (sh.tables > 256) return PLC_E_SHAPE;              // one norm column per table, at most 256 per launch
    size_t off[5];
    plc_status rc = ensure_dense(c, sh, off);
    if (rc) return rc;
    if (dense_begin(static_cast<const __half*>(logits_dev), sh, c->lin_model, c->dense_scratch, off, c->status, st) != cudaSuccess)
        return PLC_E_CUDA;
    a.mu_dense = reinterpret_cast<const float*>(c->dense_scratch + off[3]);
    a.mu_ld = sh.ncols; a.s1_ld = sh.nt_all;
    const size_t layer_elems = (size_t)sh.tables * sh.V * sh.d;
    for (int l = 0; l < c->cfg.n_layers; ++l) {
        cudaEvent_t* pg = prof_pair(c, 2);
        if (dense_layer(c->T + l * layer_elems, sh, c->dense_scratch, off, c->status, st, pg ? pg[0] : nullptr,
                        pg ? pg[1] : nullptr) != cudaSuccess) return PLC_E_CUDA;
        a.dense_layer = l;
        a.s1_dense = reinterpret_cast<const float*>(c->dense_scratch + off[4]) + (size_t)l * sh.tables;
        cudaEvent_t* pk = prof_pair(c, encode ? 0 : 1);
        if (pk) cudaEventRecord(pk[0], st);
        if ((encode ? launch_encode(a, st) : launch_decode(a, st)) != cudaSuccess) return PLC_E_CUDA;
        if (pk) cudaEventRecord(pk[1], st);
    }
    return PLC_OK;
}

// Linear-embedding variant (Sec. 7.1): Ebar and the variance term once, then per layer mu = Ebar A^T and the coding.
static plc_status run_linear(plc_ctx* c, CodecArgs a, const void* logits_dev, bool encode, cudaStream_t st) {
    const LinearShape sh = linear_shape(c->cfg, c->lin_dm, (long long)a.S * a.n);
    size_t off[6];
    plc_status rc = ensure_scratch(c, linear_scratch_bytes(sh, off));
    if (rc) return rc;
    if (linear_begin(static_cast<const __half*>(logits_dev), sh, c->lin_model, c->lin_off, c->dense_scratch, off, c->status, st) !=
        cudaSuccess) return PLC_E_CUDA;
    a.mu_dense = reinterpret_cast<const float*>(c->dense_scratch + off[5]);
    a.mu_ld = sh.ncols; a.s1_ld = sh.nt_all;
    for (int l = 0; l < c->cfg.n_layers; ++l) {
        cudaEvent_t* pg = prof_pair(c, 2);
        if (linear_layer(c->lin_A + (size_t)l * sh.ncols * sh.dm, sh, c->dense_scratch, off, c->status, st,
                         pg ? pg[0] : nullptr, pg ? pg[1] : nullptr) != cudaSuccess) return PLC_E_CUDA;
        a.dense_layer = l;
        a.s1_dense = reinterpret_cast<const float*>(c->dense_scratch + off[3]) + (size_t)l * sh.tables;
        a.mu_bias = c->lin_c + (size_t)l * sh.ncols;
        cudaEvent_t* pk = prof_pair(c, encode ? 0 : 1);
        if (pk) cudaEventRecord(pk[0], st);
        if ((encode ? launch_encode(a, st) : launch_decode(a, st)) != cudaSuccess) return PLC_E_CUDA;
        if (pk) cudaEventRecord(pk[1], st);
    }
    return PLC_OK;
}

// tokens_dev non-null <=> adaptive call
static plc_status encode_impl(plc_ctx* c, const plc_kv_view* kv, const void* logits_dev, const int32_t* tokens_dev,
                              int32_t S, int32_t n, const int32_t* pos_begin_dev, const int32_t* pos_end_dev,
                              const plc_streams* out, const plc_debug_buffers* dbg, void* stream) {
    if (!c || !logits_dev || S < 0 || n < 0) return PLC_E_INVALID;
    if ((c->cfg.adaptive_b0 > 0) != (tokens_dev != nullptr)) return PLC_E_STATE;
    plc_status rc = check_view(kv, c->cfg.head_dim, 2);
    if (rc) return rc;
    const int need = (n + c->cfg.chunk_pos - 1) / c->cfg.chunk_pos;
    rc = check_streams(out, need);
    if (rc) return rc;
    if (S == 0 || n == 0) return PLC_OK;
    const long long items = (long long)2 * c->cfg.n_layers * c->cfg.n_kv_heads * S * out->max_chunks;
    if (items >= (1ll << 32)) return PLC_E_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CodecArgs a = base_args(c);
    a.kv = to_dev(kv); a.S = S; a.n = n; a.pos_begin = pos_begin_dev; a.pos_end = pos_end_dev;
    a.st = to_dev(out);
    if (dbg) a.dbg = DebugDev{dbg->sym_dev, dbg->q_dev, dbg->mu_dev, dbg->count_ideal_bits};
    if (c->cfg.variant == PLC_PRED_DENSE) return run_dense(c, a, logits_dev, true, st);
    if (c->cfg.variant == PLC_PRED_LINEAR) return run_linear(c, a, logits_dev, true, st);
    rc = run_topk_for(c, logits_dev, S, n, pos_begin_dev, pos_end_dev, st, tokens_dev, dbg ? dbg->bits_dev : nullptr);
    if (rc) return rc;
    a.pairs = c->pairs;
    a.step_exp = tokens_dev ? c->step_exp : nullptr;
    codec_schedule(a, 2 * a.sh.L * a.sh.H, &c->last_nq, &c->last_g);
    cudaEvent_t* pk = prof_pair(c, 0);
    if (pk) cudaEventRecord(pk[0], st);
    cudaError_t e = launch_encode(a, st);
    if (pk) cudaEventRecord(pk[1], st);
    return e == cudaSuccess ? PLC_OK : PLC_E_CUDA;
}

plc_status plc_encode(plc_ctx* c, const plc_kv_view* kv, const void* logits_dev, int32_t S, int32_t n,
                      const int32_t* pos_begin_dev, const int32_t* pos_end_dev, const plc_streams* out,
                      const plc_debug_buffers* dbg, void* stream) {
    return encode_impl(c, kv, logits_dev, nullptr, S, n, pos_begin_dev, pos_end_dev, out, dbg, stream);
}

plc_status plc_encode_adaptive(plc_ctx* c, const plc_kv_view* kv, const void* logits_dev, const int32_t* tokens_dev,
                               int32_t S, int32_t n, const int32_t* pos_begin_dev, const int32_t* pos_end_dev,
                               const plc_streams* out, const plc_debug_buffers* dbg, void* stream) {
    if (!tokens_dev) return PLC_E_INVALID;
    return encode_impl(c, kv, logits_dev, tokens_dev, S, n, pos_begin_dev, pos_end_dev, out, dbg, stream);
}

static plc_status decode_impl(plc_ctx* c, const plc_streams* in, const void* logits_dev, const int32_t* tokens_dev,
                              int32_t S, int32_t n, const int32_t* pos_begin_dev, const int32_t* pos_end_dev,
                              const plc_kv_view* kv_out, const plc_debug_buffers* dbg, void* stream) {
    if (!c || !logits_dev || S < 0 || n < 0) return PLC_E_INVALID;
    if ((c->cfg.adaptive_b0 > 0) != (tokens_dev != nullptr)) return PLC_E_STATE;
    plc_status rc = check_view(kv_out, c->cfg.head_dim, c->cfg.out_dtype == PLC_OUT_F16 ? 2 : 4);
    if (rc) return rc;
    const int need = (n + c->cfg.chunk_pos - 1) / c->cfg.chunk_pos;
    rc = check_streams(in, need);
    if (rc) return rc;
    if (S == 0 || n == 0) return PLC_OK;
    const long long items = (long long)2 * c->cfg.n_layers * c->cfg.n_kv_heads * S * in->max_chunks;
    if (items >= (1ll << 32)) return PLC_E_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CodecArgs a = base_args(c);
    a.kv = to_dev(kv_out); a.S = S; a.n = n; a.pos_begin = pos_begin_dev; a.pos_end = pos_end_dev;
    a.st = to_dev(in);
    if (dbg) a.dbg = DebugDev{dbg->sym_dev, dbg->q_dev, dbg->mu_dev, dbg->count_ideal_bits};
    if (c->cfg.variant == PLC_PRED_DENSE) return run_dense(c, a, logits_dev, false, st);
    if (c->cfg.variant == PLC_PRED_LINEAR) return run_linear(c, a, logits_dev, false, st);
    rc = run_topk_for(c, logits_dev, S, n, pos_begin_dev, pos_end_dev, st, tokens_dev, dbg ? dbg->bits_dev : nullptr);
    if (rc) return rc;
    a.pairs = c->pairs;
    a.step_exp = tokens_dev ? c->step_exp : nullptr;
    codec_schedule(a, 2 * a.sh.L * a.sh.H, &c->last_nq, &c->last_g);
    cudaEvent_t* pk = prof_pair(c, 1);
    if (pk) cudaEventRecord(pk[0], st);
    cudaError_t e = launch_decode(a, st);
    if (pk) cudaEventRecord(pk[1], st);
    return e == cudaSuccess ? PLC_OK : PLC_E_CUDA;
}

plc_status plc_decode(plc_ctx* c, const plc_streams* in, const void* logits_dev, int32_t S, int32_t n,
                      const int32_t* pos_begin_dev, const int32_t* pos_end_dev, const plc_kv_view* kv_out,
                      const plc_debug_buffers* dbg, void* stream) {
    return decode_impl(c, in, logits_dev, nullptr, S, n, pos_begin_dev, pos_end_dev, kv_out, dbg, stream);
}

plc_status plc_decode_adaptive(plc_ctx* c, const plc_streams* in, const void* logits_dev, const int32_t* tokens_dev,
                               int32_t S, int32_t n, const int32_t* pos_begin_dev, const int32_t* pos_end_dev,
                               const plc_kv_view* kv_out, const plc_debug_buffers* dbg, void* stream) {
    if (!tokens_dev) return PLC_E_INVALID;
    return decode_impl(c, in, logits_dev, tokens_dev, S, n, pos_begin_dev, pos_end_dev, kv_out, dbg, stream);
}

static int rotq_words(const plc_ctx* c, int bits) { return 1 + c->cfg.head_dim / 32 * bits; }

plc_status plc_rotq_record_bytes(const plc_ctx* c, int32_t bits, uint64_t* bytes) {
    if (!c || !bytes) return PLC_E_INVALID;
    if (bits < 1 || bits > 8 || rotq_words(c, bits) > 64) return PLC_E_SHAPE;
    *bytes = 4ull * rotq_words(c, bits);
    return PLC_OK;
}

static plc_status rotq_impl(plc_ctx* c, const plc_kv_view* kv, int elem_bytes, const void* logits_dev, int32_t S, int32_t n,
                            const int32_t* pb, const int32_t* pe, const plc_rotq_params* p, const void* records_dev,
                            uint64_t capacity, bool encode, void* stream) {
    if (!c || !logits_dev || !p || !records_dev || S < 0 || n < 0) return PLC_E_INVALID;
    if (c->cfg.variant != PLC_PRED_TOPK || c->cfg.adaptive_b0 > 0) return PLC_E_STATE;
    if (p->bits < 1 || p->bits > 8 || rotq_words(c, p->bits) > 64) return PLC_E_SHAPE;
    if (reinterpret_cast<uintptr_t>(records_dev) & 3) return PLC_E_ALIGN;
    plc_status rc = check_view(kv, c->cfg.head_dim, elem_bytes);
    if (rc) return rc;
    const unsigned long long W = 2ull * c->cfg.n_layers * c->cfg.n_kv_heads;
    if (4ull * rotq_words(c, p->bits) * W * (unsigned long long)S * (unsigned long long)n > capacity) return PLC_E_CAPACITY;
    if (S == 0 || n == 0) return PLC_OK;
    const int mc = (n + c->cfg.chunk_pos - 1) / c->cfg.chunk_pos;
    if ((long long)W * S * mc >= (1ll << 32)) return PLC_E_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = run_topk_for(c, logits_dev, S, n, pb, pe, st);
    if (rc) return rc;
    CodecArgs a = base_args(c);
    a.kv = to_dev(kv); a.S = S; a.n = n; a.pos_begin = pb; a.pos_end = pe; a.pairs = c->pairs;
    a.st.max_chunks = mc;
    RotqArgs r{};
    r.bits = p->bits; r.rec_words = rotq_words(c, p->bits);
    for (int i = 0; i < 8; ++i) r.sign_bits[i] = p->sign_bits[i];
    r.records = static_cast<uint32_t*>(const_cast<void*>(records_dev));
    return launch_rotq(a, r, encode, st) == cudaSuccess ? PLC_OK : PLC_E_CUDA;
}

plc_status plc_encode_rotq(plc_ctx* c, const plc_kv_view* kv, const void* logits_dev, int32_t S, int32_t n,
                           const int32_t* pos_begin_dev, const int32_t* pos_end_dev, const plc_rotq_params* p,
                           void* records_dev, uint64_t records_capacity, void* stream) {
    return rotq_impl(c, kv, 2, logits_dev, S, n, pos_begin_dev, pos_end_dev, p, records_dev, records_capacity, true, stream);
}

plc_status plc_decode_rotq(plc_ctx* c, const void* records_dev, uint64_t records_capacity, const void* logits_dev,
                           int32_t S, int32_t n, const int32_t* pos_begin_dev, const int32_t* pos_end_dev,
                           const plc_rotq_params* p, const plc_kv_view* kv_out, void* stream) {
    return rotq_impl(c, kv_out, c && c->cfg.out_dtype == PLC_OUT_F16 ? 2 : 4, logits_dev, S, n, pos_begin_dev, pos_end_dev, p,
                     records_dev, records_capacity, false, stream);
}

plc_status plc_append_sizes(const plc_ctx* c, int32_t B, uint64_t* open_sym_bytes, uint64_t* open_q_bytes) {
    if (!c || B < 0 || !open_sym_bytes || !open_q_bytes) return PLC_E_INVALID;
    const uint64_t W = 2ull * c->cfg.n_layers * c->cfg.n_kv_heads;
    *open_q_bytes = 2ull * 4ull * B * W * c->cfg.chunk_pos;            // two buffers: chunk c fills buffer c mod 2
    *open_sym_bytes = *open_q_bytes * c->cfg.head_dim;
    return PLC_OK;
}

// Codes items [first, first + items) (item = table * B + session) of chunk `chunk_index`, whose `count`
// positions sit in open buffer chunk_index mod 2.
static plc_status seal(plc_ctx* c, plc_session_batch* sb, int chunk_index, int count, unsigned first, unsigned items,
                       cudaStream_t st, bool side = false) {
    if (items == 0 || count == 0) return PLC_OK;
    CodecArgs a = base_args(c);
    if (side) a.ticket = c->side_ticket;
    a.S = sb->B; a.n = 0;
    a.st = to_dev(&sb->streams);
    const size_t per_buf = (size_t)sb->B * 2 * c->cfg.n_layers * c->cfg.n_kv_heads * c->cfg.chunk_pos;
    a.open_sym = sb->open_sym_dev + (size_t)(chunk_index & 1) * per_buf * c->cfg.head_dim;
    a.open_q = sb->open_q_dev + (size_t)(chunk_index & 1) * per_buf;
    a.open_count = count; a.chunk_index = chunk_index; a.open_first = first; a.open_items = items;
    return launch_append_seal(a, st) == cudaSuccess ? PLC_OK : PLC_E_CUDA;
}

// Slice j of CP equal slices of the B*W streams.
static void seal_slice(long long n_streams, int CP, int j, unsigned* first, unsigned* items) {
    const long long lo = n_streams * j / CP, hi = n_streams * (j + 1) / CP;
    *first = (unsigned)lo; *items = (unsigned)(hi - lo);
}

plc_status plc_append_step(plc_ctx* c, plc_session_batch* sb, const void* kv_step_dev, const void* logits_step_dev,
                           void* stream) {
    if (!c || !sb || !kv_step_dev || !logits_step_dev || !sb->open_sym_dev || !sb->open_q_dev) return PLC_E_INVALID;
    if (c->cfg.variant != PLC_PRED_TOPK || c->cfg.adaptive_b0 > 0) return PLC_E_STATE;
    if (sb->B < 1 || sb->steps < 0) return PLC_E_INVALID;
    if (!aligned16(kv_step_dev)) return PLC_E_ALIGN;
    const int CP = c->cfg.chunk_pos;
    plc_status rc = check_streams(&sb->streams, sb->steps / CP + 1);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t d = c->cfg.head_dim, H = c->cfg.n_kv_heads, B = sb->B;
    const long long n_streams = (long long)B * 2 * c->cfg.n_layers * H;
    // The chunk completed last is coded a slice of the streams at a time, one slice per step, so that no
    // step carries the coding of all streams.  Slices 1 .. CP-1 read a buffer that this step does not
    // touch: they run on a stream of the context's own beside this step's kernels (forked from and
    // joined to the caller's stream, so the call stays stream-ordered for the caller).  Slice 0 reads
    // the position this very step writes and follows it on the caller's stream.
    const int after = sb->steps + 1, done = after / CP, phase = after % CP;
    unsigned first = 0, items = 0;
    if (done >= 1) seal_slice(n_streams, CP, phase, &first, &items);
    const bool beside = done >= 1 && phase != 0 && items > 0;
    if (beside) {
        if (cudaEventRecord(c->side_ev[0], st) != cudaSuccess || cudaStreamWaitEvent(c->side_stream, c->side_ev[0], 0) != cudaSuccess)
            return PLC_E_CUDA;
        rc = seal(c, sb, done - 1, CP, first, items, c->side_stream, true);
        if (rc) return rc;
        if (cudaEventRecord(c->side_ev[1], c->side_stream) != cudaSuccess) return PLC_E_CUDA;
    }
    rc = run_topk_for(c, logits_step_dev, sb->B, 1, nullptr, nullptr, st);
    if (rc) return rc;
    CodecArgs a = base_args(c);
    const size_t per_buf = (size_t)n_streams * CP;
    const int chunk = sb->steps / CP;
    a.kv = KvView{const_cast<void*>(kv_step_dev), 2 * B * H * d, B * H * d, H * d, d, 0};
    a.S = sb->B; a.n = 1;
    a.open_sym = sb->open_sym_dev + (size_t)(chunk & 1) * per_buf * d;
    a.open_q = sb->open_q_dev + (size_t)(chunk & 1) * per_buf;
    a.open_slot = sb->steps % CP;
    if (launch_append_quantise(a, st) != cudaSuccess) return PLC_E_CUDA;
    sb->steps = after;
    if (beside) return cudaStreamWaitEvent(st, c->side_ev[1], 0) == cudaSuccess ? PLC_OK : PLC_E_CUDA;
    if (done >= 1) return seal(c, sb, done - 1, CP, first, items, st);
    return PLC_OK;
}

plc_status plc_append_flush(plc_ctx* c, plc_session_batch* sb, void* stream) {
    if (!c || !sb || !sb->open_sym_dev || !sb->open_q_dev || sb->B < 1 || sb->steps < 0) return PLC_E_INVALID;
    const int CP = c->cfg.chunk_pos, rem = sb->steps % CP, done = sb->steps / CP;
    plc_status rc = check_streams(&sb->streams, done + (rem ? 1 : 0));
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const long long n_streams = (long long)sb->B * 2 * c->cfg.n_layers * c->cfg.n_kv_heads;
    if (done >= 1 && rem != CP - 1) {          // slices rem + 1 .. CP - 1 of the last complete chunk are still uncoded
        unsigned first, items, f2, i2;
        seal_slice(n_streams, CP, rem + 1, &first, &items);
        seal_slice(n_streams, CP, CP - 1, &f2, &i2);
        rc = seal(c, sb, done - 1, CP, first, f2 + i2 - first, st);
        if (rc) return rc;
    }
    return seal(c, sb, done, rem, 0u, (unsigned)n_streams, st);
}

plc_status plc_sync_status(plc_ctx* c, void* stream) {
    if (!c) return PLC_E_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned int w = 0;
    if (cudaMemcpyAsync(&w, c->status, sizeof(w), cudaMemcpyDeviceToHost, st) != cudaSuccess) return PLC_E_CUDA;
    if (cudaMemsetAsync(c->status, 0, sizeof(w), st) != cudaSuccess) return PLC_E_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return PLC_E_CUDA;
    return status_code(w);
}

plc_status plc_poll_status(plc_ctx* c, uint32_t* bits) {
    if (!c || !bits) return PLC_E_INVALID;
    // a copy on the context's own non-blocking stream: it does not wait for the work enqueued on the
    // caller's streams and reads the word as it stands now
    if (cudaMemcpyAsync(c->status_host, c->status, sizeof(unsigned int), cudaMemcpyDeviceToHost, c->poll_stream) != cudaSuccess)
        return PLC_E_CUDA;
    if (cudaStreamSynchronize(c->poll_stream) != cudaSuccess) return PLC_E_CUDA;
    *bits = *c->status_host;
    return status_code(*c->status_host);
}

plc_status plc_get_stats(plc_ctx* c, plc_stats* out, int32_t reset, void* stream) {
    if (!c || !out) return PLC_E_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Counters h{};
    if (cudaMemcpyAsync(&h, c->counters, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess) return PLC_E_CUDA;
    if (reset && cudaMemsetAsync(c->counters, 0, sizeof(h), st) != cudaSuccess) return PLC_E_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return PLC_E_CUDA;
    out->payload_bytes = h.payload_bytes; out->n_chunks = h.n_chunks; out->n_escapes = h.n_escapes;
    out->coded_vectors = h.coded_vectors; out->skipped_vectors = h.skipped_vectors;
    out->ideal_bits = h.ideal_bits;
    return PLC_OK;
}

plc_status plc_table_constants(int32_t qp, uint32_t* theta, uint32_t* rho) {
    if (qp < kQMin || qp > 15 || !theta || !rho) return PLC_E_INVALID;
    table_constants(qp, *theta, *rho);
    return PLC_OK;
}

plc_status plc_build_table(int32_t qp, uint32_t* f, uint32_t* cdf) {
    if (qp < kQMin || qp > 15 || !f || !cdf) return PLC_E_INVALID;
    build_freqs(qp, f);
    cdf[0] = 0;
    for (int i = 0; i < kNumSym; ++i) cdf[i + 1] = cdf[i] + f[i];
    return PLC_OK;
}

plc_status plc_last_schedule(const plc_ctx* c, int32_t* n_queues, int32_t* sms_per_queue) {
    if (!c || !n_queues || !sms_per_queue) return PLC_E_INVALID;
    if (c->last_nq < 1) return PLC_E_STATE;
    *n_queues = c->last_nq; *sms_per_queue = c->last_g;
    return PLC_OK;
}

plc_status plc_set_profiling(plc_ctx* c, int32_t on) {
    if (!c) return PLC_E_INVALID;
    c->profiling = on != 0;
    return PLC_OK;
}

plc_status plc_last_kernel_ms(plc_ctx* c, int32_t which, float* ms) {
    if (!c || !ms || which < 0 || which > 2) return PLC_E_INVALID;
    const int n = c->prof_used[which];
    if (n < 1) return PLC_E_STATE;
    cudaEvent_t* p = &c->prof_ev[which][2 * (n - 1)];
    if (cudaEventSynchronize(p[1]) != cudaSuccess) return PLC_E_CUDA;
    return cudaEventElapsedTime(ms, p[0], p[1]) == cudaSuccess ? PLC_OK : PLC_E_CUDA;
}

plc_status plc_kernel_ms(plc_ctx* c, int32_t which, float* mean_ms, int32_t* launches, int32_t reset) {
    if (!c || which < 0 || which > 2) return PLC_E_INVALID;
    const int n = c->prof_used[which];
    double sum = 0.0;
    for (int i = 0; i < n; ++i) {
        cudaEvent_t* p = &c->prof_ev[which][2 * i];
        float ms = 0.f;
        if (cudaEventSynchronize(p[1]) != cudaSuccess || cudaEventElapsedTime(&ms, p[0], p[1]) != cudaSuccess) return PLC_E_CUDA;
        sum += ms;
    }
    if (mean_ms) *mean_ms = n ? (float)(sum / n) : 0.f;
    if (launches) *launches = n;
    if (reset) c->prof_used[which] = 0;
    return PLC_OK;
}

uint64_t plc_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"

// Shared definitions of the libplc CUDA translation units (sm_100a only).
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "plc.h"

namespace plc {

constexpr int kProbBits = 15;
constexpr uint32_t kProbM = 1u << kProbBits;
constexpr uint32_t kRansL = 1u << 16;
constexpr int kNumSym = 64;        // zigzag(hi), hi in [-31,31] -> 0..62; 63 = escape
constexpr int kEsc = 63;
constexpr int kHiMax = 31;
constexpr int kQMin = -24;
constexpr int kQMax = 135;
constexpr int kNumTables = 40;     // table id qp in [-24, 15]
constexpr int kSymLimit = 1 << 30;
constexpr uint32_t kFull = 0xffffffffu;

// Bits of the device status word.
constexpr uint32_t kStCapacity = 1u, kStCorrupt = 2u, kStBadClass = 4u, kStTimeout = 8u, kStCursor = 16u;

// Device counters (plc_stats).
struct Counters {
    unsigned long long payload_bytes, n_chunks, n_escapes, coded_vectors, skipped_vectors;
    double ideal_bits;     // code length under the coder's model (only counted on request)
};

// Frequency-table entry used by the encoder: rcp = floor(2^32 / f) (2^32-1 for f = 1),
// fc = f | (c << 16).
struct EncEntry {
    uint32_t rcp, fc;
};

// Per-class tables as they sit in shared memory.
struct __align__(16) Tables {
    EncEntry enc[kNumTables][kNumSym];      // 20 KB
    uint16_t cum[kNumTables][kNumSym + 2];  // c[0..64], padded: 5280 B
};

// Two 32-bit constants per table id: theta = round(2^32 exp(-sqrt2/s')), rho = round(2^32
// exp(-sqrt2/(2 s'))), s' = 2^(qp/8).  Literal so that encoder and decoder builds agree bit for bit.
__host__ __device__ inline void table_constants(int qp, uint32_t& theta, uint32_t& rho) {
    constexpr uint32_t kC[kNumTables][2] = {
        {52418u, 15004422u},         {134053u, 23994893u},        {317125u, 36905875u},
        {698470u, 54771407u},        {1440801u, 78665070u},       {2798733u, 109637892u},
        {5145013u, 148652826u},      {8992185u, 196522626u},      {15004422u, 253857248u},
        {23994893u, 321025356u},     {36905875u, 398132550u},     {54771407u, 485016909u},
        {78665070u, 581260615u},     {109637892u, 686215099u},    {148652826u, 799036310u},
        {196522626u, 918726429u},    {253857248u, 1044178424u},   {321025356u, 1174220339u},
        {398132550u, 1307656790u},   {485016909u, 1443305845u},   {581260615u, 1580030169u},
        {686215099u, 1716761896u},   {799036310u, 1852521207u},   {918726429u, 1986428948u},
        {1044178424u, 2117713904u},  {1174220339u, 2245715466u},  {1307656790u, 2369882518u},
        {1443305845u, 2489769347u},  {1580030169u, 2605029347u},  {1716761896u, 2715407188u},
        {1852521207u, 2820730047u},  {1986428948u, 2920898384u},  {2117713904u, 3015876649u},
        {2245715466u, 3105684222u},  {2369882518u, 3190386796u},  {2489769347u, 3270088366u},
        {2605029347u, 3344923893u},  {2715407188u, 3415052718u},  {2820730047u, 3480652712u},
        {2920898384u, 3541915165u}};
    theta = kC[qp - kQMin][0];
    rho = kC[qp - kQMin][1];
}

// Discretised Laplace frequencies of table qp, integer recurrence:
// G0 = 2^32, G1 = rho, G(k+1) = (Gk theta) >> 32; f(0) = (G0-G1) >> 17, f(+-k) = (Gk-Gk+1) >> 18,
// f(ESC) = G32 >> 17, each at least 1; f(0) absorbs the difference to 2^15.
__host__ __device__ inline void build_freqs(int qp, uint32_t* f /*[64]*/) {
    uint32_t theta, rho;
    table_constants(qp, theta, rho);
    unsigned long long g = 1ull << 32, gn = rho;
    unsigned long long m = (g - gn) >> 17;
    f[0] = m < 1 ? 1u : (uint32_t)m;
    g = gn;
    for (int k = 1; k <= kHiMax; ++k) {
        gn = (g * (unsigned long long)theta) >> 32;
        m = (g - gn) >> 18;
        uint32_t fk = m < 1 ? 1u : (uint32_t)m;
        f[2 * k - 1] = fk;
        f[2 * k] = fk;
        g = gn;
    }
    m = g >> 17;
    f[kEsc] = m < 1 ? 1u : (uint32_t)m;
    long long sum = 0;
    for (int i = 0; i < kNumSym; ++i) sum += f[i];
    f[0] = (uint32_t)((long long)f[0] + ((long long)kProbM - sum));
}

// Scale class -> (number of bit planes s, table id qp).
__host__ __device__ inline void class_params(int q, int& s, int& qp) {
    if (q < 16) { s = 0; qp = q; }
    else { s = (q >> 3) - 1; qp = 8 + (q & 7); }
}

#ifdef __CUDACC__
// q = clamp(round(4 log2 v), kQMin, kQMax), decided on the binary32 exponent and four mantissa
// thresholds 2^((2i+1)/8); v <= 0 -> kQMin.
__device__ __forceinline__ int class_from_v(float v) {
    if (!(v > 0.0f)) return kQMin;
    uint32_t b = __float_as_uint(v);
    int e = (int)(b >> 23);
    if (e == 255) return kQMax;
    float m;
    if (e == 0) {                      // subnormal: far below the smallest class
        return kQMin;
    }
    m = __uint_as_float((b & 0x007fffffu) | 0x3f800000u);   // [1,2)
    int q = 4 * (e - 127);
    q += (m >= 1.09050773f) + (m >= 1.29683955f) + (m >= 1.54221083f) + (m >= 1.83400809f);
    return min(max(q, kQMin), kQMax);
}

__device__ __forceinline__ uint32_t lanemask_lt() {
    uint32_t m;
    asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
    return m;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}

// Fills the shared-memory tables; call with all threads of the block, then __syncthreads().
__device__ inline void build_tables_smem(Tables* t) {
    for (int id = threadIdx.x; id < kNumTables; id += blockDim.x) {
        uint32_t f[kNumSym];
        build_freqs(id + kQMin, f);
        uint32_t c = 0;
        for (int i = 0; i < kNumSym; ++i) {
            uint32_t fi = f[i];
            t->enc[id][i].rcp = fi == 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / fi);
            t->enc[id][i].fc = fi | (c << 16);
            t->cum[id][i] = (uint16_t)c;
            c += fi;
        }
        t->cum[id][kNumSym] = (uint16_t)c;       // 2^15 wraps to 0x8000: fits uint16
        t->cum[id][kNumSym + 1] = 0xffff;
    }
}
#endif

// Host-side launch counter shared by all translation units.
void count_launch(int n = 1);

// Internal launchers (one per .cu file).
struct TopkArgs {
    const __half* logits; const int32_t* tokens; int64_t N; int V, K;
    int2* pairs;            // [N][Kp] {idx, float bits of w}, or null; entries K..Kp-1 get {idx_0, 0}
    int Kp;
    int32_t* idx; float* w; float* lse; float* zk; float* logp2;   // optional user outputs
    // Adaptive step (needs tokens): step_exp[row] = b0 - b_i, bits_out[row] = b_i (both optional).
    int* step_exp; int* bits_out; int b0, extra; float hbar;
    // Rows are skipped (nothing written) when pos ranges are given and the row is outside them.
    int n_per_session; const int32_t* pos_begin; const int32_t* pos_end;
    // Optional scratch of the two-kernel selection: per row kTopkListCap order words (8 bytes each, 4 while
    // V <= 65536) and a header {l_max, sum of exp(l - l_max), number of candidates or -1}.  With it
    // the streaming kernel only collects the candidates of a row and a second kernel ranks them.
    void* cand; float4* cand_hdr;
    // Rows the shared-memory-staged kernel leaves to the general one carry -2 in their header and are
    // counted in *redo; a launch with redo_only set visits only those (and returns at once if none).
    unsigned int* redo; int redo_only;
    unsigned int* status;   // device status word (bounded waits report kStTimeout there), or null
};
constexpr int kTopkListCap = 256;
cudaError_t launch_topk(const TopkArgs& a, cudaStream_t st);

cudaError_t launch_prefix_dedup(const int32_t* tokens, const int32_t* lens, const float* logp2, int S, int64_t stride,
                                int32_t* lcp, float* dT, int32_t* parent, int32_t* shared_len, cudaStream_t st);

cudaError_t launch_prefix_clusters(const int32_t* lcp, const float* dT, int S, float delta, int32_t* cluster,
                                   int32_t* centroid, int32_t* begin, cudaStream_t st);

constexpr int kZeroOff = -1000000;

struct CodecShape {
    int L, H, d, V, K, Kp, chunk_pos, out_dtype;   // Kp: K rounded up to the rows one warp-wide load fetches
    float delta, sigma_floor;
    float inv_delta, inv_delta2;   // fl(1/delta), fl(1/(delta*delta)), rounded once on the host
    int zero_q;                    // zero-rate rule (Thm. 3): positions of class <= zero_q carry no symbols (kZeroOff = never)
};

struct KvView {
    void* base; int64_t sl, skv, ss, sh, sp;
};

struct StreamsDev {
    uint8_t* payload; unsigned long long capacity; unsigned long long* chunk_offset; uint32_t* chunk_bytes;
    unsigned long long* total_bytes; int max_chunks;
};

struct DebugDev {
    int32_t* sym; int32_t* q; float* mu;
    int ideal;             // non-zero: add every coded component's model code length to Counters::ideal_bits
};

struct CodecArgs {
    CodecShape sh;
    const __half* T; const float* rownorm2;        // [tables][V][d], [tables][V]
    const int2* pairs;                             // [S*n][Kp]
    const int* step_exp;                           // [S*n] adaptive step exponent, or null
    KvView kv;                                     // encode: input f16; decode: output
    int S, n; const int32_t* pos_begin; const int32_t* pos_end;
    StreamsDev st; DebugDev dbg;
    uint16_t* staging; unsigned long long staging_words_per_warp;   // encoder scratch
    unsigned int* ticket;                          // kTicketWords work counters (zeroed by the launcher)
    int sched_nq, sched_g;                         // gather kernels: work queues, SMs that share one (set by the launcher)
    unsigned int* status; Counters* counters;
    // dense variant: prediction read from buffers; one launch covers the 2*H tables of dense_layer
    const float* mu_dense; const float* s1_dense; long long mu_ld, s1_ld; int dense_layer;
    const __half* mu_bias;                         // optional [2*H][d] f16 added to mu (linear predictor's c), or null
    // append path: symbols come from / go to the open chunk
    int32_t* open_sym; int32_t* open_q; int open_slot; int open_count; int chunk_index;
    unsigned open_first, open_items;               // seal launch: the (table, session) items [open_first, open_first + open_items)
};
int codec_grid_warps(int device);
// Work-queue layout a gather launch over n_tables tables would use: nq queues, g SMs per queue.
void codec_schedule(const CodecArgs& a, int n_tables, int* nq, int* g);

// Rotated fixed-rate quantiser (Prop. 3 step 3): records of 1 + (d/32)*bits words per (stream, position),
// record of (session s, table t, position i) at word ((s*W + t)*n + i) * rec_words.
struct RotqArgs {
    int bits;
    uint32_t sign_bits[8];      // bit j set: component j is negated before and after the transform
    uint32_t* records;
    int rec_words;
};
cudaError_t launch_rotq(const CodecArgs& a, const RotqArgs& r, bool encode, cudaStream_t st);
constexpr int kTicketWords = 1024;               // one counter per work queue (at most one queue per SM)

// Dense (full-vocabulary) prediction, one layer at a time.
struct DenseShape {
    long long rows;        // S * n positions
    int V, d, tables;      // tables = 2 * H of one layer
    int ldv;               // V rounded up to 64 (row pitch of P and Tb, in elements)
    int ncols, ncols_pad;  // tables * d, rounded up to 256
    int nt_all, nt_all_pad;   // L * tables (one variance column per layer and table), rounded up to 256
};
size_t dense_scratch_bytes(const DenseShape& sh, size_t* off /*[5]: P, Tb, -, mu, s1*/);
size_t dense_model_bytes(const DenseShape& sh);
cudaError_t dense_prepare(const __half* T, int L, const DenseShape& sh, uint8_t* model, cudaStream_t st);
cudaError_t dense_begin(const __half* logits, const DenseShape& sh, const uint8_t* model, uint8_t* scratch, const size_t* off,
                        unsigned int* status, cudaStream_t st);
cudaError_t dense_softmax(const __half* logits, const DenseShape& sh, uint8_t* scratch, const size_t* off, cudaStream_t st);
// Linear-embedding predictor (Sec. 7.1).
struct LinearShape {
    long long rows;
    int V, d, dm, tables, L;   // tables = 2*H per layer, dm = d_model (multiple of 64)
    int ldv;                   // V rounded up to 64
    int ncols, ncols_pad;      // tables*d, rounded up to 256
    int nt_all, nt_all_pad;    // L*tables, rounded up to 256
};
size_t linear_model_bytes(const LinearShape& sh, size_t* off /*[2]*/);
size_t linear_scratch_bytes(const LinearShape& sh, size_t* off /*[6]*/);
cudaError_t linear_prepare(const __half* E, const __half* A, const __half* c, const LinearShape& sh, uint8_t* model,
                           const size_t* moff, unsigned int* status, cudaStream_t st);
cudaError_t linear_begin(const __half* logits, const LinearShape& sh, const uint8_t* model, const size_t* moff,
                         uint8_t* scratch, const size_t* off, unsigned int* status, cudaStream_t st);
cudaError_t linear_layer(const __half* A_layer, const LinearShape& sh, uint8_t* scratch, const size_t* off,
                         unsigned int* status, cudaStream_t st, cudaEvent_t ev0, cudaEvent_t ev1);
cudaError_t dense_layer(const __half* T_layer, const DenseShape& sh, uint8_t* scratch, const size_t* off,
                        unsigned int* status, cudaStream_t st, cudaEvent_t ev0, cudaEvent_t ev1);   // events bracket the contraction
cudaError_t launch_rownorm(const __half* T, float* out, long long rows, int d, cudaStream_t st);
cudaError_t launch_encode(const CodecArgs& a, cudaStream_t st);
cudaError_t launch_decode(const CodecArgs& a, cudaStream_t st);
cudaError_t launch_append_quantise(const CodecArgs& a, cudaStream_t st);   // predict + quantise into the open chunk
cudaError_t launch_append_seal(const CodecArgs& a, cudaStream_t st);       // code the open chunk

}  // namespace plc

// Fused predict / quantise / rANS kernels.
//
// One warp owns one (stream, chunk): it walks the chunk's positions (backwards when encoding,
// forwards when decoding), and for each position
//   1. gathers the K candidate rows of its table with 128-bit loads and accumulates the mixture
//      mu = sum_k w_k T[idx_k] in binary32 (each lane: 8 components of every ROWS-th row, then a
//      shuffle reduce-scatter so that lane l ends with its G = d/32 components),
//   2. derives the scale class from the mixture variance (precomputed row norms),
//   3. quantises the residual (encoder) or adds the decoded residual back (decoder),
//   4. runs one interleaved rANS step per owned component, the 32 lanes sharing one word stream.
// The encoder writes its words back to front into a per-warp staging area (global memory, reused
// from chunk to chunk so it stays in L2), then reserves the chunk's final place with one atomicAdd
// and copies it there.  Work items are handed out by an atomic ticket in table-major order so that
// the warps running at any time gather from few tables.
#include <algorithm>
#include <type_traits>

#include "plc_common.cuh"

namespace plc {
namespace {

#ifndef PLC_BLOCKS_PER_SM
#define PLC_BLOCKS_PER_SM 5
#endif
#ifndef PLC_GATHER_UNROLL
#define PLC_GATHER_UNROLL 8
#endif
#ifndef PLC_WARPS_PER_BLOCK
#define PLC_WARPS_PER_BLOCK 8
#endif
constexpr int kWarpsPerBlock = PLC_WARPS_PER_BLOCK;
constexpr int kThreads = kWarpsPerBlock * 32;
constexpr int kBlocksPerSM = PLC_BLOCKS_PER_SM;
constexpr int kGatherUnroll = PLC_GATHER_UNROLL;

template <int D>
struct Geo {
    static constexpr int R = D / 8;        // lanes that cover one row with 16-byte loads
    static constexpr int G = D / 32;       // components a lane owns
    static constexpr int ROWS = 32 / R;    // rows fetched by one warp-wide load
};

// Encoder tables are indexed by hi + 31 (hi in [-31, 31]; entry 63 = escape): the symbol's place in
// the alphabet (0, +1, -1, +2, ...) only matters for the cumulative counts, which are kept.
struct EncTables { EncEntry enc[kNumTables][kNumSym]; };
// Decoder tables: cum[] for the search, fc[] = f | (c << 16) for the state update.
struct DecTables { uint16_t cum[kNumTables][kNumSym + 2]; uint32_t fc[kNumTables][kNumSym]; };

__device__ inline void build_enc_tables(EncTables* t) {
    for (int id = threadIdx.x; id < kNumTables; id += blockDim.x) {
        uint32_t f[kNumSym];
        build_freqs(id + kQMin, f);
        uint32_t c = 0;
        for (int i = 0; i < kNumSym; ++i) {
            uint32_t fi = f[i];
            const int hi = (i & 1) ? (i + 1) / 2 : -(i / 2);            // alphabet order 0, +1, -1, +2, ...
            const int at = i == kEsc ? kEsc : hi + kHiMax;
            t->enc[id][at].rcp = fi == 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / fi);
            t->enc[id][at].fc = fi | (c << 16);
            c += fi;
        }
    }
}
__device__ inline void build_dec_tables(DecTables* t) {
    for (int id = threadIdx.x; id < kNumTables; id += blockDim.x) {
        uint32_t f[kNumSym];
        build_freqs(id + kQMin, f);
        uint32_t c = 0;
        for (int i = 0; i < kNumSym; ++i) {
            t->cum[id][i] = (uint16_t)c;
            t->fc[id][i] = f[i] | (c << 16);
            c += f[i];
        }
        t->cum[id][kNumSym] = (uint16_t)c;
        t->cum[id][kNumSym + 1] = 0xffff;
    }
}

// component owned by (lane, g): 8 (lane mod R) + G (lane div R) + g
template <int D>
__device__ __forceinline__ int first_comp(int lane) {
    return 8 * (lane % Geo<D>::R) + Geo<D>::G * (lane / Geo<D>::R);
}

// Sum of squares of the lane's G values, then over the warp; the same chain is used for the row
// norms and for ||mu||^2 so that a point-mass mixture has exactly zero variance.
template <int G>
__device__ __forceinline__ float warp_norm2(const float (&v)[G]) {
    float p = 0.f;
#pragma unroll
    for (int g = 0; g < G; ++g) p = __fmaf_rn(v[g], v[g], p);
    return warp_sum(p);
}

template <int D>
__global__ void __launch_bounds__(256) rownorm_kernel(const __half* __restrict__ T, float* __restrict__ out, long long rows) {
    constexpr int G = Geo<D>::G;
    const int lane = threadIdx.x & 31;
    const long long warp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long long nw = (long long)gridDim.x * (blockDim.x >> 5);
    const int c0 = first_comp<D>(lane);
    for (long long r = warp; r < rows; r += nw) {
        float v[G];
#pragma unroll
        for (int g = 0; g < G; ++g) v[g] = __half2float(T[r * D + c0 + g]);
        float s = warp_norm2<G>(v);
        if (lane == 0) out[r] = s;
    }
}

// Two binary32 fused multiply-adds in one instruction (sm_100 packed f32x2) on register pairs that
// stay packed across the gather loop; each half is an IEEE fma, so the result equals two scalar
// __fmaf_rn.
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1,%2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi) {
    asm("mov.b64 {%0,%1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void ffma2(unsigned long long& acc, unsigned long long a, unsigned long long b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}

// Mixture of one position for one table.  sp: the position's Kp {idx, w} entries in shared memory,
// Kp = K rounded up to a multiple of ROWS (the padding has weight 0 and a valid index).
template <int D>
__device__ __forceinline__ void predict(const char* __restrict__ col, const float* __restrict__ n2,
                                        const int2* sp, int Kp, int lane, float inv_d,
                                        float (&mu)[Geo<D>::G], float& sigma2) {
    constexpr int R = Geo<D>::R, G = Geo<D>::G, ROWS = Geo<D>::ROWS;
    const int h = lane / R;
    // variance term first: its row-norm loads are in flight while the rows are gathered
    float s1 = 0.f;
    for (int k = lane; k < Kp; k += 32) {
        const int2 pr = sp[k];
        s1 = __fmaf_rn(__int_as_float(pr.y), __ldg(n2 + pr.x), s1);
    }
    unsigned long long acc2[4] = {0ull, 0ull, 0ull, 0ull};   // four pairs of +0.f
    const int2* pl = sp + h;
    const int iters = Kp / ROWS;
#pragma unroll kGatherUnroll
    for (int it = 0; it < iters; ++it) {
        const int2 pr = pl[it * ROWS];
        const float w = __int_as_float(pr.y);
        const uint4 r = __ldg(reinterpret_cast<const uint4*>(col + (long long)pr.x * (D * 2)));
        const unsigned long long ww = pack2(w, w);
        const __half2* hp = reinterpret_cast<const __half2*>(&r);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f = __half22float2(hp[j]);
            ffma2(acc2[j], ww, pack2(f.x, f.y));
        }
    }
    float acc[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) unpack2(acc2[j], acc[2 * j], acc[2 * j + 1]);
    // reduce-scatter over the ROWS lanes that hold partial sums of the same 8 components
    int cnt = 8;
#pragma unroll
    for (int o = (ROWS / 2) * R; o >= R; o >>= 1) {
        const bool up = (h & (o / R)) != 0;
        const int half = cnt / 2;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (i < half) {
                float send = up ? acc[i] : acc[i + half];
                float keep = up ? acc[i + half] : acc[i];
                acc[i] = keep + __shfl_xor_sync(kFull, send, o);
            }
        }
        cnt = half;
    }
#pragma unroll
    for (int g = 0; g < G; ++g) mu[g] = acc[g];
    // variance: (sum_k w_k ||T_k||^2 - ||mu||^2) / d
    s1 = warp_sum(s1);
    float s2 = warp_norm2<G>(mu);
    sigma2 = fmaxf(0.f, (s1 - s2) * inv_d);
}

// The pairs of a position are brought into the warp's shared-memory slot with cp.async, one
// position ahead of their use and without passing through registers (two slots per warp).
__device__ __forceinline__ void prefetch_pairs(int2* sp, const int2* __restrict__ gp, int Kp, int lane) {
    if ((Kp & 1) == 0) {                            // two entries (16 bytes) per copy: the slots and the rows of `pairs` are 16-byte aligned
        for (int k = 2 * lane; k < Kp; k += 64) {
            const unsigned dst = (unsigned)__cvta_generic_to_shared(sp + k);
            asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gp + k) : "memory");
        }
    } else {
        for (int k = lane; k < Kp; k += 32) {
            const unsigned dst = (unsigned)__cvta_generic_to_shared(sp + k);
            asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst), "l"(gp + k) : "memory");
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}
// Waits for this lane's copies (all but the newest `pending` groups), then makes the whole warp's
// copies visible to every lane.
template <int PENDING>
__device__ __forceinline__ void pairs_ready() {
    asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory");
    __syncwarp();
}

__device__ __forceinline__ int scale_class(float sigma2, float floor2, float inv_delta2) {
    return class_from_v((sigma2 + floor2) * inv_delta2);
}

// Per-lane constants of the coder steps.
struct LaneCode {
    uint32_t lt;         // lanes below this one
    int sh;              // 16 * (lane & 1): which half of a bit-plane word lanes 0 / 1 store
    int hs;              // lane >> 4: which half of a bit-plane word this lane's bit sits in
    uint32_t bit;        // 1 << (lane & 15): this lane's bit in that half
    int lane;
};
__device__ __forceinline__ LaneCode lane_code(int lane) {
    LaneCode lc;
    lc.lt = lanemask_lt(); lc.sh = 16 * (lane & 1); lc.hs = lane >> 4; lc.bit = 1u << (lane & 15); lc.lane = lane;
    return lc;
}

// One encoder step for the warp: every lane codes `sym` with S raw bit planes (S is the same in
// all lanes).  Words are written back to front at stage[wp-1], stage[wp-2], ...; returns the new
// wp.  In decoder order a step is: 2S plane words, the refill words of the lanes that renormalise
// (lanes ascending), the raw high parts of escaped lanes (lanes ascending, low half first).
template <int SC>
__device__ __forceinline__ int encode_step(int sym, int s_dyn, const EncEntry* tbl, uint32_t& x, uint16_t* __restrict__ stage,
                                           int wp, const LaneCode& lc, unsigned& n_escapes) {
    const int S = SC >= 0 ? SC : s_dyn;                            // SC < 0: plane count known at run time only
    const int S2 = 2 * S;
    const int u = sym + (S ? (1 << (S - 1)) : 0);                  // |sym| <= 2^30, S <= 15: no overflow
    const int hi = u >> S;                                         // bits below S of u are the raw part
    const uint32_t at = (uint32_t)(hi + kHiMax);
    const bool esc = at > 2u * kHiMax;                             // |hi| > 31
    const EncEntry e = tbl[min(at, (uint32_t)kEsc)];
    const uint32_t f = e.fc & 0xffffu;
    const bool emit = x >= (f << 17);
    const uint32_t emask = __ballot_sync(kFull, emit);
    int base = wp - S2 - __popc(emask);
    if (__any_sync(kFull, esc)) {                  // rare: raw 32-bit hi of the escaped lanes
        const uint32_t xmask = __ballot_sync(kFull, esc);
        const int n_esc = __popc(xmask);
        base -= 2 * n_esc;
        if (esc) {
            const int at = base + S2 + __popc(emask) + 2 * __popc(xmask & lc.lt);
            stage[at] = (uint16_t)((uint32_t)hi & 0xffffu);
            stage[at + 1] = (uint16_t)((uint32_t)hi >> 16);
        }
        n_escapes += n_esc;
    }
    uint16_t* out = stage + base;
    if (emit) out[S2 + __popc(emask & lc.lt)] = (uint16_t)(x & 0xffffu);
    const uint32_t xe = emit ? x >> 16 : x;
    uint32_t q = __umulhi(xe, e.rcp);
    uint32_t r = xe - q * f;
    if (r >= f) { ++q; r -= f; }
    x = (q << kProbBits) + r + (e.fc >> 16);
    if (S > 0) {
        uint16_t* mine = out + lc.lane;            // lanes 0 and 1 store the two halves of every plane
#pragma unroll
        for (int b = 0; b < S; ++b) {
            const uint32_t plane = __ballot_sync(kFull, (u >> b) & 1);
            if (lc.lane < 2) mine[2 * b] = (uint16_t)(plane >> lc.sh);
        }
    }
    return base;
}

// All G components of one position, last component first, dispatched on the number of planes.
template <int G>
__device__ __forceinline__ int encode_position(const int (&sym)[G], int s, bool mixed, const EncEntry* tbl, uint32_t& x,
                                               uint16_t* __restrict__ stage, int wp, const LaneCode& lc, unsigned& n_escapes) {
#define PLC_ENC_CASE(S_, LABEL)                                                                            \
    LABEL:                                                                                                 \
        _Pragma("unroll") for (int g = G - 1; g >= 0; --g)                                                 \
            wp = encode_step<S_>(sym[g], s, tbl, x, stage, wp, lc, n_escapes);                             \
        break;
    // The plane counts that occur in practice get code of their own.  With a per-position step
    // (`mixed`) neighbouring positions differ in plane count, and jumping between a dozen
    // specialised bodies costs more in instruction fetch than they save: those take the loop.
    switch (mixed ? -1 : s) {
        PLC_ENC_CASE(0, case 0) PLC_ENC_CASE(1, case 1) PLC_ENC_CASE(2, case 2) PLC_ENC_CASE(3, case 3)
        PLC_ENC_CASE(4, case 4) PLC_ENC_CASE(5, case 5) PLC_ENC_CASE(6, case 6) PLC_ENC_CASE(7, case 7)
        PLC_ENC_CASE(-1, default)
    }
#undef PLC_ENC_CASE
    return wp;
}

// One decoder step for the warp; words[-1 .. nwords) are readable (words[-1] is the last half of
// the chunk's state block).  A read past the end is redirected to the chunk's last word; rp still
// advances, so the caller's final check rp == nwords reports it.
template <int SC>
__device__ __forceinline__ int decode_step(int s_dyn, const uint16_t* cum, const uint32_t* fcs, uint32_t& x,
                                           const uint16_t* __restrict__ words, int& rp, int last, const LaneCode& lc) {
    const int S = SC >= 0 ? SC : s_dyn;
    uint32_t lo = 0;
    if (S > 0) {
        const int S2 = 2 * S;
        uint32_t v = 0;
        if (lc.lane < S2) v = __ldg(words + min(rp + lc.lane, last));
#pragma unroll
        for (int b = 0; b < S; ++b) {
            const uint32_t hw = __shfl_sync(kFull, v, 2 * b + lc.hs);
            if (hw & lc.bit) lo |= 1u << b;
        }
        rp += S2;
    }
    const uint32_t slot = x & (kProbM - 1u);
    const uint16_t* cp = cum;
#pragma unroll
    for (int step = 32; step > 0; step >>= 1)
        if (cp[step] <= slot) cp += step;
    const int zz = (int)(cp - cum);
    const uint32_t fc = fcs[zz];
    x = (fc & 0xffffu) * (x >> kProbBits) + slot - (fc >> 16);
    const bool need = x < kRansL;
    const uint32_t nmask = __ballot_sync(kFull, need);
    if (need) x = (x << 16) | __ldg(words + min(rp + __popc(nmask & lc.lt), last));
    rp += __popc(nmask);
    const int t = (zz + 1) >> 1;
    int hi = (zz & 1) ? t : -t;
    if (__any_sync(kFull, zz == kEsc)) {
        const bool esc = zz == kEsc;
        const uint32_t xmask = __ballot_sync(kFull, esc);
        if (esc) {
            const int at = rp + 2 * __popc(xmask & lc.lt);
            hi = (int)((uint32_t)__ldg(words + min(at, last)) | ((uint32_t)__ldg(words + min(at + 1, last)) << 16));
        }
        rp += 2 * __popc(xmask);
    }
    return S ? (int)(((uint32_t)hi << S) + lo - (1u << (S - 1))) : hi;
}

template <int G>
__device__ __forceinline__ void decode_position(int (&sym)[G], int s, bool mixed, const uint16_t* cum, const uint32_t* fcs, uint32_t& x,
                                                const uint16_t* __restrict__ words, int& rp, int last, const LaneCode& lc) {
#define PLC_DEC_CASE(S_, LABEL)                                                                            \
    LABEL:                                                                                                 \
        _Pragma("unroll") for (int g = 0; g < G; ++g)                                                      \
            sym[g] = decode_step<S_>(s, cum, fcs, x, words, rp, last, lc);                                 \
        break;
    switch (mixed ? -1 : s) {
        PLC_DEC_CASE(0, case 0) PLC_DEC_CASE(1, case 1) PLC_DEC_CASE(2, case 2) PLC_DEC_CASE(3, case 3)
        PLC_DEC_CASE(4, case 4) PLC_DEC_CASE(5, case 5) PLC_DEC_CASE(6, case 6) PLC_DEC_CASE(7, case 7)
        PLC_DEC_CASE(-1, default)
    }
#undef PLC_DEC_CASE
}

// Lane 0's value for the whole warp, through a warp reduction: the result is provably the same in
// every lane, so everything derived from it (loop bounds, table addresses, branches) is kept out of
// the per-lane registers and needs no divergence handling.
__device__ __forceinline__ unsigned from_lane0(unsigned v, int lane) {
    return __reduce_or_sync(kFull, lane == 0 ? v : 0u);
}
__device__ __forceinline__ unsigned next_ticket(unsigned int* ticket, int lane) {
    unsigned t = 0;
    if (lane == 0) t = atomicAdd(ticket, 1u);
    return from_lane0(t, lane);
}

// Work queues of the gather kernels.  The tables are dealt round-robin to nq queues (queue k owns
// tables k, k + nq, ...), each queue lists its (table, session, chunk) items table-major, and the
// g SMs with the same smid / g serve one queue.  The warps resident on an SM therefore gather from
// one or two tables at a time, so candidate rows that several positions share are found in that
// SM's L1, and the number of tables in flight on the whole GPU stays near nq.  A warp whose queue
// is empty moves on to the next queue (and never returns), so the tail is balanced by stealing.
// Returns the item in table-major numbering (table * per_table + rest), or ~0u when all is taken.
__device__ __forceinline__ unsigned smid() {
    unsigned r;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(r));
    return r;
}
struct QueueCursor { int q, tried; };
__device__ __forceinline__ QueueCursor queue_of_this_sm(const CodecArgs& a) {
    QueueCursor qc;
    qc.q = (int)((smid() / (unsigned)a.sched_g) % (unsigned)a.sched_nq);   // fewer tables than SM groups: spread the groups evenly
    qc.tried = 0;
    return qc;
}
__device__ __forceinline__ unsigned next_queued(const CodecArgs& a, QueueCursor& qc, unsigned per_table, int n_tables, int lane) {
    unsigned item = ~0u;
    if (lane == 0) {
        while (qc.tried < a.sched_nq) {
            const unsigned nt = (unsigned)max(0, (n_tables - qc.q + a.sched_nq - 1) / a.sched_nq);
            const unsigned j = atomicAdd(a.ticket + qc.q, 1u);
            if (j < nt * per_table) {
                item = ((unsigned)qc.q + (unsigned)a.sched_nq * (j / per_table)) * per_table + j % per_table;
                break;
            }
            qc.q = qc.q + 1 == a.sched_nq ? 0 : qc.q + 1;
            ++qc.tried;
        }
    }
    return from_lane0(item, lane);
}

template <int G>
__device__ __forceinline__ void load_half_vec(const __half* p, float (&v)[G]) {
    if constexpr (G == 8) {
        uint4 r = *reinterpret_cast<const uint4*>(p);
        const __half2* hp = reinterpret_cast<const __half2*>(&r);
#pragma unroll
        for (int j = 0; j < 4; ++j) { float2 f = __half22float2(hp[j]); v[2 * j] = f.x; v[2 * j + 1] = f.y; }
    } else if constexpr (G == 4) {
        uint2 r = *reinterpret_cast<const uint2*>(p);
        const __half2* hp = reinterpret_cast<const __half2*>(&r);
#pragma unroll
        for (int j = 0; j < 2; ++j) { float2 f = __half22float2(hp[j]); v[2 * j] = f.x; v[2 * j + 1] = f.y; }
    } else if constexpr (G == 2) {
        float2 f = __half22float2(*reinterpret_cast<const __half2*>(p));
        v[0] = f.x; v[1] = f.y;
    } else {
        v[0] = __half2float(*p);
    }
}

// The same load without the conversion (the bits wait in (G+1)/2 registers), and the conversion.
template <int G>
__device__ __forceinline__ void load_half_raw(const __half* p, uint32_t (&raw)[(G + 1) / 2]) {
    if constexpr (G == 8) {
        const uint4 r = *reinterpret_cast<const uint4*>(p);
        raw[0] = r.x; raw[1] = r.y; raw[2] = r.z; raw[3] = r.w;
    } else if constexpr (G == 4) {
        const uint2 r = *reinterpret_cast<const uint2*>(p);
        raw[0] = r.x; raw[1] = r.y;
    } else if constexpr (G == 2) {
        raw[0] = *reinterpret_cast<const uint32_t*>(p);
    } else {
        raw[0] = (uint32_t)__half_as_ushort(*p);
    }
}
template <int G>
__device__ __forceinline__ void half_raw_to_float(const uint32_t (&raw)[(G + 1) / 2], float (&v)[G]) {
    if constexpr (G == 1) {
        v[0] = __half2float(__ushort_as_half((unsigned short)raw[0]));
    } else {
#pragma unroll
        for (int j = 0; j < G / 2; ++j) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&raw[j]));
            v[2 * j] = f.x; v[2 * j + 1] = f.y;
        }
    }
}

template <int G>
__device__ __forceinline__ void store_vec(void* base, long long elem, const float (&v)[G], int out_f16) {
    if (out_f16) {
        __half* p = reinterpret_cast<__half*>(base) + elem;
        if constexpr (G == 1) { *p = __float2half_rn(v[0]); }
        else {
            __half2 t[G / 2];
#pragma unroll
            for (int j = 0; j < G / 2; ++j) t[j] = __floats2half2_rn(v[2 * j], v[2 * j + 1]);
            if constexpr (G == 8) *reinterpret_cast<uint4*>(p) = *reinterpret_cast<uint4*>(t);
            else if constexpr (G == 4) *reinterpret_cast<uint2*>(p) = *reinterpret_cast<uint2*>(t);
            else *reinterpret_cast<__half2*>(p) = t[0];
        }
    } else {
        float* p = reinterpret_cast<float*>(base) + elem;
        if constexpr (G >= 4) {
#pragma unroll
            for (int j = 0; j < G / 4; ++j)
                reinterpret_cast<float4*>(p)[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
        } else if constexpr (G == 2) { *reinterpret_cast<float2*>(p) = make_float2(v[0], v[1]); }
        else { *p = v[0]; }
    }
}

struct Item {
    int t, s, c;        // table, session, chunk
    int p0, P;          // first position, positions in the chunk (0: no such chunk)
    long long slot;
};

__device__ __forceinline__ Item bulk_item(const CodecArgs& a, unsigned item, int t_first = 0) {
    Item it;
    const int MC = a.st.max_chunks;
    const unsigned per_table = (unsigned)a.S * (unsigned)MC;
    it.t = t_first + (int)(item / per_table);
    unsigned r = item % per_table;
    it.s = (int)(r / MC);
    it.c = (int)(r % MC);
    const int Wt = 2 * a.sh.L * a.sh.H;
    it.slot = ((long long)it.s * Wt + it.t) * MC + it.c;
    int b = a.pos_begin ? a.pos_begin[it.s] : 0, e = a.pos_end ? a.pos_end[it.s] : a.n;
    b = max(b, 0); e = min(e, a.n);
    long long p0 = (long long)b + (long long)it.c * a.sh.chunk_pos;
    it.p0 = (int)min(p0, (long long)a.n);
    it.P = p0 < e ? min(a.sh.chunk_pos, e - (int)p0) : 0;
    return it;
}

__device__ __forceinline__ long long kv_elem(const KvView& v, int t, int H, int s, int pos) {
    int layer = t / (2 * H), kv = (t / H) & 1, head = t % H;
    return layer * v.sl + kv * v.skv + s * v.ss + head * v.sh + (long long)pos * v.sp;
}

// Finishes an encoded chunk: reserves its place, writes states and words, index and counters.
__device__ __forceinline__ void commit_chunk(const CodecArgs& a, long long slot, uint32_t x, const uint16_t* stage,
                                             int wp, int cap_words, int lane, int P, unsigned n_escapes, int n_skipped = 0) {
    __syncwarp();
    const int n_words = cap_words - wp;
    const unsigned nbytes = 128u + 2u * (unsigned)n_words;
    unsigned long long off = 0;
    if (lane == 0) {
        off = atomicAdd(a.st.total_bytes, (unsigned long long)((nbytes + 15u) & ~15u));
        atomicAdd(&a.counters->payload_bytes, (unsigned long long)nbytes);
        atomicAdd(&a.counters->n_chunks, 1ull);
        atomicAdd(&a.counters->coded_vectors, (unsigned long long)P);
        if (n_skipped) atomicAdd(&a.counters->skipped_vectors, (unsigned long long)n_skipped);
    }
    off = __shfl_sync(kFull, off, 0);
    if (lane == 0 && n_escapes) atomicAdd(&a.counters->n_escapes, (unsigned long long)n_escapes);
    const bool fits = off + nbytes <= a.st.capacity;
    const bool aligned = (off & 15ull) == 0;             // the caller's byte cursor must be a multiple of 16
    if (lane == 0) {
        a.st.chunk_offset[slot] = off;
        a.st.chunk_bytes[slot] = nbytes;
        if (!fits) atomicOr(a.status, kStCapacity);
        if (!aligned) atomicOr(a.status, kStCursor);
    }
    if (!fits || !aligned) return;
    uint8_t* dst = a.st.payload + off;
    reinterpret_cast<uint32_t*>(dst)[lane] = x;
    uint16_t* dw = reinterpret_cast<uint16_t*>(dst + 128);
    for (int i = lane; i < n_words; i += 32) dw[i] = __ldcg(stage + wp + i);
}

// Quantiser decision in binary32: sym = rint((kv - mu) * fl(1/delta)), clamped to +-2^30.
__device__ __forceinline__ int quantise(float kv, float mu, float inv_delta) {
    float n = rintf(__fmul_rn(__fsub_rn(kv, mu), inv_delta));
    n = fminf(fmaxf(n, -(float)kSymLimit), (float)kSymLimit);
    return (int)n;
}

extern __shared__ __align__(16) int2 g_pair_smem[];   // per warp: two slots of Kp entries

// Prediction read from the dense variant's buffers: mu [row][tables_in_layer*D] and the variance
// term s1 [row][tables_in_layer] (sum_v p_v ||T_v||^2 / d); sigma2 = max(0, s1 - ||mu||^2 / d).
template <int D>
__device__ __forceinline__ void dense_fetch(const CodecArgs& a, long long row, int t_local, int c0,
                                            float (&m)[Geo<D>::G], float& s1) {
    constexpr int G = Geo<D>::G;
    const float* mp = a.mu_dense + row * a.mu_ld + (long long)t_local * D + c0;
#pragma unroll
    for (int g = 0; g < G; ++g) m[g] = __ldg(mp + g);
    s1 = __ldg(a.s1_dense + row * a.s1_ld + t_local);
}
template <int D>
__device__ __forceinline__ void dense_finish(const CodecArgs& a, int t_local, int c0, float inv_d, const float (&m)[Geo<D>::G],
                                             float s1, float (&mu)[Geo<D>::G], float& sigma2) {
    constexpr int G = Geo<D>::G;
#pragma unroll
    for (int g = 0; g < G; ++g) mu[g] = m[g];
    if (a.mu_bias) {
#pragma unroll
        for (int g = 0; g < G; ++g) mu[g] = __fadd_rn(mu[g], __half2float(a.mu_bias[t_local * D + c0 + g]));
    }
    const float s2 = warp_norm2<G>(mu);
    sigma2 = fmaxf(0.f, s1 - s2 * inv_d);
}

enum { kSrcGather = 0, kSrcOpen = 1, kSrcDense = 2 };

// ZR: the zero-rate rule (Thm. 3) is on; a separate instantiation keeps the plain coder's loop free of it.
// FLEX: the call exports intermediate values or statistics, or uses a per-position step; the plain
// instantiation carries none of those branches in its position loop.
template <int D, int SRC, bool ZR, bool FLEX>
__global__ void __launch_bounds__(kThreads, kBlocksPerSM) encode_kernel(const CodecArgs a) {
    constexpr int G = Geo<D>::G;
    constexpr bool FROM_OPEN = SRC == kSrcOpen;
    constexpr bool DENSE = SRC == kSrcDense;
    __shared__ EncTables tb;
    build_enc_tables(&tb);
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const LaneCode lc = lane_code(lane);
    const long long gw = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    uint16_t* stage = a.staging + gw * a.staging_words_per_warp;
    const int cap_words = (int)a.staging_words_per_warp;
    const int Wt = 2 * a.sh.L * a.sh.H, H = a.sh.H, Kp = a.sh.Kp;
    int2* sp0 = g_pair_smem + (threadIdx.x >> 5) * 2 * Kp;
    const int Wl = DENSE ? 2 * H : Wt;                       // tables this launch covers
    const unsigned total = FROM_OPEN ? a.open_items : (unsigned)Wl * a.S * a.st.max_chunks;
    const float inv_d = 1.0f / D, inv_delta = a.sh.inv_delta, inv_delta2 = a.sh.inv_delta2,
                floor2 = a.sh.sigma_floor * a.sh.sigma_floor;
    const int c0 = first_comp<D>(lane);

    constexpr bool QUEUED = SRC == kSrcGather;
    QueueCursor qc = QUEUED ? queue_of_this_sm(a) : QueueCursor{0, 0};
    const unsigned per_table = (unsigned)a.S * (unsigned)a.st.max_chunks;
    auto next = [&]() { return QUEUED ? next_queued(a, qc, per_table, Wl, lane) : next_ticket(a.ticket, lane); };
    for (unsigned item = next(); item < total; item = next()) {
        Item it;
        if (FROM_OPEN) {
            const unsigned oi = a.open_first + item;
            it.t = (int)(oi / a.S); it.s = (int)(oi % a.S); it.c = a.chunk_index;
            it.p0 = 0; it.P = a.open_count;
            it.slot = ((long long)it.s * Wt + it.t) * a.st.max_chunks + it.c;
        } else {
            it = bulk_item(a, item, DENSE ? a.dense_layer * Wl : 0);
        }
        if (it.P <= 0) {
            if (lane == 0 && !FROM_OPEN) { a.st.chunk_offset[it.slot] = 0; a.st.chunk_bytes[it.slot] = 0; }
            continue;
        }
        const char* col = reinterpret_cast<const char*>(a.T + (size_t)it.t * a.sh.V * D + 8 * (lane % Geo<D>::R));
        const float* n2 = a.rownorm2 + (size_t)it.t * a.sh.V;
        uint32_t x = kRansL;
        int wp = cap_words;
        unsigned n_escapes = 0;
        int n_skipped = 0;
        float ideal = 0.f;                                                         // this lane's share, if asked for
        const int2* gp = nullptr;
        const __half* kvp = nullptr;
        int buf = 0;
        if (!FROM_OPEN) {
            if (!DENSE) {
                gp = a.pairs + ((long long)it.s * a.n + it.p0 + it.P - 1) * Kp;  // last position first
                __syncwarp();                                                    // slot 0 is free again
                prefetch_pairs(sp0, gp, Kp, lane);
            }
            kvp = reinterpret_cast<const __half*>(a.kv.base) + kv_elem(a.kv, it.t, H, it.s, it.p0 + it.P - 1) + c0;
        }
        // dense source: the prediction of the next position is fetched while this one is coded
        float m_next[G] = {};
        float s1_next = 0.f;
        if (DENSE) dense_fetch<D>(a, (long long)it.s * a.n + it.p0 + it.P - 1, it.t - a.dense_layer * Wl, c0, m_next, s1_next);
        for (int p = it.P - 1; p >= 0; --p) {
            int sym[G];
            int q;
            bool skip;                                                             // zero-rate position (Thm. 3)
            if (FROM_OPEN) {
                const long long o = ((long long)it.s * Wt + it.t) * a.sh.chunk_pos + p;
                q = a.open_q[o];
                skip = ZR && q <= a.sh.zero_q;
#pragma unroll
                for (int g = 0; g < G; ++g) sym[g] = a.open_sym[o * D + c0 + g];
            } else {
                float mu[G], sigma2;
                uint32_t kv_raw[(G + 1) / 2];
                load_half_raw<G>(kvp, kv_raw);                                     // in flight during the prediction
                kvp -= a.kv.sp;
                if (DENSE) {
                    float m_cur[G];
#pragma unroll
                    for (int g = 0; g < G; ++g) m_cur[g] = m_next[g];
                    const float s1_cur = s1_next;
                    if (p > 0) dense_fetch<D>(a, (long long)it.s * a.n + it.p0 + p - 1, it.t - a.dense_layer * Wl, c0, m_next, s1_next);
                    dense_finish<D>(a, it.t - a.dense_layer * Wl, c0, inv_d, m_cur, s1_cur, mu, sigma2);
                } else {
                    const int2* sp = sp0 + buf * Kp;
                    if (p > 0) {                                                  // one position ahead
                        gp -= Kp;
                        prefetch_pairs(sp0 + (buf ^ 1) * Kp, gp, Kp, lane);
                        pairs_ready<1>();
                    } else {
                        pairs_ready<0>();
                    }
                    buf ^= 1;
                    predict<D>(col, n2, sp, Kp, lane, inv_d, mu, sigma2);
                }
                float inv_delta_p = inv_delta, inv_delta2_p = inv_delta2;
                int zero_q = ZR ? a.sh.zero_q : 0;
                if (FLEX && a.step_exp) {                                          // adaptive step delta * 2^e
                    const int e = __ldg(a.step_exp + (long long)it.s * a.n + it.p0 + p);
                    inv_delta_p = ldexpf(inv_delta, -e);
                    inv_delta2_p = ldexpf(inv_delta2, -2 * e);
                    if (ZR) zero_q -= 8 * e;                                       // same D against a step 2^e times larger
                }
                q = __reduce_max_sync(kFull, scale_class(sigma2, floor2, inv_delta2_p));   // same in all lanes
                skip = ZR && q <= zero_q;
                float kvv[G];
                half_raw_to_float<G>(kv_raw, kvv);
#pragma unroll
                for (int g = 0; g < G; ++g) sym[g] = quantise(kvv[g], mu[g], inv_delta_p);
                __syncwarp();                                                     // readers of this slot are done
                if (FLEX && (a.dbg.sym || a.dbg.q || a.dbg.mu)) {
                    const long long o = ((long long)it.s * a.n + it.p0 + p) * Wt + it.t;
                    if (a.dbg.q && lane == 0) a.dbg.q[o] = q;
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        if (a.dbg.sym) a.dbg.sym[o * D + c0 + g] = skip ? 0 : sym[g];
                        if (a.dbg.mu) a.dbg.mu[o * D + c0 + g] = mu[g];
                    }
                }
            }
            if (ZR && skip) { ++n_skipped; continue; }                             // nothing is coded
            int s, qp;
            class_params(q, s, qp);
            if (FLEX && a.dbg.ideal) {              // statistics only: log2(2^15 / f) + s raw bits (+ 32 per escape)
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const uint32_t at = (uint32_t)(((sym[g] + (s ? (1 << (s - 1)) : 0)) >> s) + kHiMax);
                    const uint32_t f = tb.enc[qp - kQMin][min(at, (uint32_t)kEsc)].fc & 0xffffu;
                    ideal += (float)(kProbBits + s) - log2f((float)f) + (at > 2u * kHiMax ? 32.f : 0.f);
                }
            }
            wp = encode_position<G>(sym, s, FLEX && a.step_exp != nullptr, tb.enc[qp - kQMin], x, stage, wp, lc, n_escapes);
        }
        if (FLEX && a.dbg.ideal) {
            ideal = warp_sum(ideal);
            if (lane == 0) atomicAdd(&a.counters->ideal_bits, (double)ideal);
        }
        commit_chunk(a, it.slot, x, stage, wp, cap_words, lane, it.P, n_escapes, n_skipped);
        __syncwarp();
    }
}

template <int D, bool DENSE, bool ZR, bool FLEX>
__global__ void __launch_bounds__(kThreads, kBlocksPerSM) decode_kernel(const CodecArgs a) {
    constexpr int G = Geo<D>::G;
    __shared__ DecTables tb;
    build_dec_tables(&tb);
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const LaneCode lc = lane_code(lane);
    const int Wt = 2 * a.sh.L * a.sh.H, H = a.sh.H, Kp = a.sh.Kp;
    int2* sp0 = g_pair_smem + (threadIdx.x >> 5) * 2 * Kp;
    const int Wl = DENSE ? 2 * H : Wt;
    const unsigned total = (unsigned)Wl * a.S * a.st.max_chunks;
    const float inv_d = 1.0f / D, delta = a.sh.delta, inv_delta2 = a.sh.inv_delta2,
                floor2 = a.sh.sigma_floor * a.sh.sigma_floor;
    const int c0 = first_comp<D>(lane);

    QueueCursor qc = DENSE ? QueueCursor{0, 0} : queue_of_this_sm(a);
    const unsigned per_table = (unsigned)a.S * (unsigned)a.st.max_chunks;
    auto next = [&]() { return DENSE ? next_ticket(a.ticket, lane) : next_queued(a, qc, per_table, Wl, lane); };
    for (unsigned item = next(); item < total; item = next()) {
        const Item it = bulk_item(a, item, DENSE ? a.dense_layer * Wl : 0);
        if (it.P <= 0) continue;
        const unsigned long long off = a.st.chunk_offset[it.slot];
        const unsigned nbytes = a.st.chunk_bytes[it.slot];
        if (nbytes < 128u || (nbytes & 1u) || (off & 15ull) || off + nbytes > a.st.capacity) {
            if (lane == 0) atomicOr(a.status, kStCorrupt);
            continue;
        }
        const uint8_t* src = a.st.payload + off;
        uint32_t x = reinterpret_cast<const uint32_t*>(src)[lane];
        bool bad = x < kRansL;
        const uint16_t* words = reinterpret_cast<const uint16_t*>(src + 128);
        const int nwords = (int)((nbytes - 128u) >> 1);
        const int last = nwords - 1;                 // -1 for a chunk of states only: words[-1] is inside the chunk
        int rp = 0;
        const char* col = reinterpret_cast<const char*>(a.T + (size_t)it.t * a.sh.V * D + 8 * (lane % Geo<D>::R));
        const float* n2 = a.rownorm2 + (size_t)it.t * a.sh.V;
        const int2* gp = a.pairs + ((long long)it.s * a.n + it.p0) * Kp;
        __syncwarp();
        if (!DENSE) prefetch_pairs(sp0, gp, Kp, lane);
        int buf = 0;
        long long kvo = kv_elem(a.kv, it.t, H, it.s, it.p0) + c0;
        float m_next[G] = {};
        float s1_next = 0.f;
        if (DENSE) dense_fetch<D>(a, (long long)it.s * a.n + it.p0, it.t - a.dense_layer * Wl, c0, m_next, s1_next);
        for (int p = 0; p < it.P; ++p) {
            float mu[G], sigma2;
            if (DENSE) {
                float m_cur[G];
#pragma unroll
                for (int g = 0; g < G; ++g) m_cur[g] = m_next[g];
                const float s1_cur = s1_next;
                if (p + 1 < it.P) dense_fetch<D>(a, (long long)it.s * a.n + it.p0 + p + 1, it.t - a.dense_layer * Wl, c0, m_next, s1_next);
                dense_finish<D>(a, it.t - a.dense_layer * Wl, c0, inv_d, m_cur, s1_cur, mu, sigma2);
            } else {
                const int2* sp = sp0 + buf * Kp;
                if (p + 1 < it.P) {
                    gp += Kp;
                    prefetch_pairs(sp0 + (buf ^ 1) * Kp, gp, Kp, lane);
                    pairs_ready<1>();
                } else {
                    pairs_ready<0>();
                }
                buf ^= 1;
                predict<D>(col, n2, sp, Kp, lane, inv_d, mu, sigma2);
            }
            float delta_p = delta, inv_delta2_p = inv_delta2;
            int zero_q = ZR ? a.sh.zero_q : 0;
            if (FLEX && a.step_exp) {
                const int e = __ldg(a.step_exp + (long long)it.s * a.n + it.p0 + p);
                delta_p = ldexpf(delta, e);
                inv_delta2_p = ldexpf(inv_delta2, -2 * e);
                if (ZR) zero_q -= 8 * e;
            }
            const int q = __reduce_max_sync(kFull, scale_class(sigma2, floor2, inv_delta2_p));   // same in all lanes
            __syncwarp();                                                         // readers of this slot are done
            int sym[G];
            float out[G];
            if (ZR && q <= zero_q) {                                              // zero-rate position: KV' = KV^
#pragma unroll
                for (int g = 0; g < G; ++g) { sym[g] = 0; out[g] = mu[g]; }
            } else {
                int s, qp;
                class_params(q, s, qp);
                decode_position<G>(sym, s, FLEX && a.step_exp != nullptr, tb.cum[qp - kQMin], tb.fc[qp - kQMin], x, words, rp, last, lc);
#pragma unroll
                for (int g = 0; g < G; ++g) out[g] = __fmaf_rn((float)sym[g], delta_p, mu[g]);
            }
            store_vec<G>(a.kv.base, kvo, out, a.sh.out_dtype);
            kvo += a.kv.sp;
            if (FLEX && (a.dbg.sym || a.dbg.q || a.dbg.mu)) {
                const long long o = ((long long)it.s * a.n + it.p0 + p) * Wt + it.t;
                if (a.dbg.q && lane == 0) a.dbg.q[o] = q;
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    if (a.dbg.sym) a.dbg.sym[o * D + c0 + g] = sym[g];
                    if (a.dbg.mu) a.dbg.mu[o * D + c0 + g] = mu[g];
                }
            }
        }
        bad = bad || x != kRansL || rp != nwords;
        if (__any_sync(kFull, bad) && lane == 0) atomicOr(a.status, kStCorrupt);
    }
}

// In-place orthonormal Walsh-Hadamard transform of a d-vector spread over the warp in the coder's
// ownership (lane l, register g  <->  component 8 (l mod R) + G (l div R) + g): every bit of the
// component index is either a bit of g (butterflies between registers) or a bit of the lane number
// (butterflies by shuffle), so log2(G) + 5 = log2(d) stages visit every bit once; the element whose
// bit is set receives partner - self.  Output index = input index (natural Hadamard order).
template <int D>
__device__ __forceinline__ void hadamard(float (&v)[Geo<D>::G], int lane) {
    constexpr int G = Geo<D>::G;
#pragma unroll
    for (int m = 1; m < G; m <<= 1) {
#pragma unroll
        for (int g = 0; g < G; ++g)
            if (!(g & m)) { const float a = v[g], b = v[g | m]; v[g] = a + b; v[g | m] = a - b; }
    }
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) {
        const bool up = (lane & m) != 0;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float p = __shfl_xor_sync(kFull, v[g], m);
            v[g] = up ? p - v[g] : v[g] + p;
        }
    }
    constexpr float norm = D == 32 ? 0.17677669529663687f : D == 64 ? 0.125f : D == 128 ? 0.08838834764831845f : 0.0625f;   // d^(-1/2)
#pragma unroll
    for (int g = 0; g < G; ++g) v[g] *= norm;
}

// Rotated fixed-rate quantiser (Prop. 3 step 3: a per-vector quantiser on the residual R = KV - KV^):
// x = eps * R, y = H x (orthonormal Hadamard), s = max |y|, b-bit mid-rise codes on [-s, s]; the
// record is s followed by one ballot word per (register, code bit).  ENC: KV -> records;
// otherwise records -> KV' = KV^ + eps * H y^.  One warp per (stream, chunk of positions).
template <int D, bool ENC>
__global__ void __launch_bounds__(kThreads, kBlocksPerSM) rotq_kernel(const CodecArgs a, const RotqArgs rq) {
    constexpr int G = Geo<D>::G;
    const int lane = threadIdx.x & 31;
    const int Wt = 2 * a.sh.L * a.sh.H, H = a.sh.H, Kp = a.sh.Kp, B = rq.bits;
    int2* sp0 = g_pair_smem + (threadIdx.x >> 5) * 2 * Kp;
    const unsigned total = (unsigned)Wt * a.S * a.st.max_chunks;
    const float inv_d = 1.0f / D, half_levels = 0.5f * (float)(1 << B), cell = 2.0f / (float)(1 << B);
    const int c0 = first_comp<D>(lane);
    float sgn[G];
#pragma unroll
    for (int g = 0; g < G; ++g) sgn[g] = (rq.sign_bits[(c0 + g) >> 5] >> ((c0 + g) & 31)) & 1u ? -1.0f : 1.0f;
    QueueCursor qc = queue_of_this_sm(a);
    const unsigned per_table = (unsigned)a.S * (unsigned)a.st.max_chunks;
    for (unsigned item = next_queued(a, qc, per_table, Wt, lane); item < total; item = next_queued(a, qc, per_table, Wt, lane)) {
        const Item it = bulk_item(a, item);
        if (it.P <= 0) continue;
        const char* col = reinterpret_cast<const char*>(a.T + (size_t)it.t * a.sh.V * D + 8 * (lane % Geo<D>::R));
        const float* n2 = a.rownorm2 + (size_t)it.t * a.sh.V;
        const int2* gp = a.pairs + ((long long)it.s * a.n + it.p0) * Kp;
        __syncwarp();
        prefetch_pairs(sp0, gp, Kp, lane);
        int buf = 0;
        long long kvo = kv_elem(a.kv, it.t, H, it.s, it.p0) + c0;
        uint32_t* rec = rq.records + (((long long)it.s * Wt + it.t) * a.n + it.p0) * rq.rec_words;
        for (int p = 0; p < it.P; ++p, rec += rq.rec_words, kvo += a.kv.sp) {
            const int2* sp = sp0 + buf * Kp;
            if (p + 1 < it.P) {
                gp += Kp;
                prefetch_pairs(sp0 + (buf ^ 1) * Kp, gp, Kp, lane);
                pairs_ready<1>();
            } else {
                pairs_ready<0>();
            }
            buf ^= 1;
            float mu[G], sigma2;
            predict<D>(col, n2, sp, Kp, lane, inv_d, mu, sigma2);
            __syncwarp();                                                         // readers of this slot are done
            float y[G];
            if (ENC) {
                load_half_vec<G>(reinterpret_cast<const __half*>(a.kv.base) + kvo, y);
#pragma unroll
                for (int g = 0; g < G; ++g) y[g] = __fsub_rn(y[g], mu[g]) * sgn[g];
                hadamard<D>(y, lane);
                float amax = 0.f;
#pragma unroll
                for (int g = 0; g < G; ++g) amax = fmaxf(amax, fabsf(y[g]));
                const float scale = __uint_as_float(__reduce_max_sync(kFull, __float_as_uint(amax)));   // non-negative floats order like their bits
                const float inv = scale > 0.f ? __fdiv_rn(1.0f, scale) : 0.f;
                uint32_t mine0 = __float_as_uint(scale), mine1 = 0u;               // word 0 of the record is the scale
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    int c = (int)floorf(__fmaf_rn(__fmul_rn(y[g], inv), half_levels, half_levels));
                    c = min(max(c, 0), (1 << B) - 1);
                    for (int b = 0; b < B; ++b) {
                        const uint32_t plane = __ballot_sync(kFull, (c >> b) & 1);
                        const int w = 1 + g * B + b;
                        if ((w & 31) == lane) { if (w < 32) mine0 = plane; else mine1 = plane; }
                    }
                }
                if (lane < rq.rec_words) rec[lane] = mine0;                         // rec_words <= 64
                if (lane + 32 < rq.rec_words) rec[lane + 32] = mine1;
            } else {
                const uint32_t w0 = lane < rq.rec_words ? __ldg(rec + lane) : 0u;
                const uint32_t w1 = lane + 32 < rq.rec_words ? __ldg(rec + lane + 32) : 0u;
                const float scale = __uint_as_float(__shfl_sync(kFull, w0, 0));
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    int c = 0;
                    for (int b = 0; b < B; ++b) {
                        const int w = 1 + g * B + b;
                        const uint32_t plane = __shfl_sync(kFull, w < 32 ? w0 : w1, w & 31);
                        c |= (int)((plane >> lane) & 1u) << b;
                    }
                    y[g] = scale * __fmaf_rn((float)c + 0.5f, cell, -1.0f);
                }
                hadamard<D>(y, lane);
                float out[G];
#pragma unroll
                for (int g = 0; g < G; ++g) out[g] = __fadd_rn(mu[g], y[g] * sgn[g]);
                store_vec<G>(a.kv.base, kvo, out, a.sh.out_dtype);
            }
        }
    }
}

// Decode-time append: one warp per (session, table) predicts the new position and stores its
// symbols and class in slot a.open_slot of the stream's open chunk.  The rows come from HBM at
// random, so what counts is row loads in flight: four blocks per SM (64 registers, the whole
// unrolled batch of row loads issued before the first use) measured best.
#ifndef PLC_APPEND_BLOCKS
#define PLC_APPEND_BLOCKS 4
#endif
template <int D>
__global__ void __launch_bounds__(kThreads, PLC_APPEND_BLOCKS) append_quantise_kernel(const CodecArgs a) {
    constexpr int G = Geo<D>::G;
    const int lane = threadIdx.x & 31;
    const int Wt = 2 * a.sh.L * a.sh.H, H = a.sh.H, Kp = a.sh.Kp;
    int2* sp = g_pair_smem + (threadIdx.x >> 5) * 2 * Kp;
    const long long gw = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const long long nw = (long long)gridDim.x * kWarpsPerBlock;
    const float inv_d = 1.0f / D, inv_delta = a.sh.inv_delta, inv_delta2 = a.sh.inv_delta2,
                floor2 = a.sh.sigma_floor * a.sh.sigma_floor;
    const int c0 = first_comp<D>(lane);
    for (long long item = gw; item < (long long)Wt * a.S; item += nw) {
        const int t = (int)(item / a.S), b = (int)(item % a.S);
        const char* col = reinterpret_cast<const char*>(a.T + (size_t)t * a.sh.V * D + 8 * (lane % Geo<D>::R));
        const int2* gp = a.pairs + (long long)b * Kp;
        __syncwarp();
        prefetch_pairs(sp, gp, Kp, lane);
        pairs_ready<0>();
        float kvv[G];
        load_half_vec<G>(reinterpret_cast<const __half*>(a.kv.base) + kv_elem(a.kv, t, H, b, 0) + c0, kvv);
        float mu[G], sigma2;
        predict<D>(col, a.rownorm2 + (size_t)t * a.sh.V, sp, Kp, lane, inv_d, mu, sigma2);
        const int q = scale_class(sigma2, floor2, inv_delta2);
        const long long o = ((long long)b * Wt + t) * a.sh.chunk_pos + a.open_slot;
        if (lane == 0) a.open_q[o] = q;
#pragma unroll
        for (int g = 0; g < G; ++g) a.open_sym[o * D + c0 + g] = q <= a.sh.zero_q ? 0 : quantise(kvv[g], mu[g], inv_delta);
    }
}

template <class F>
cudaError_t dispatch_d(int d, F&& f) {
    switch (d) {
        case 32: return f(std::integral_constant<int, 32>{});
        case 64: return f(std::integral_constant<int, 64>{});
        case 128: return f(std::integral_constant<int, 128>{});
        case 256: return f(std::integral_constant<int, 256>{});
    }
    return cudaErrorInvalidValue;
}

// Dynamic shared memory of the kernels that stage pairs: one slot of Kp entries per warp.
template <class Kern>
cudaError_t pair_smem_bytes(Kern kern, int Kp, size_t& bytes) {
    bytes = (size_t)kWarpsPerBlock * 2 * Kp * sizeof(int2);
    if (bytes > 24 * 1024) return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    return cudaSuccess;
}

int sm_count() {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms;
}

}  // namespace

int codec_grid_warps(int) { return sm_count() * kBlocksPerSM * kWarpsPerBlock; }

static void set_queues(CodecArgs& a, int n_tables);

// Queue layout of a gather launch.  With one queue for the whole GPU the resident warps span
// about (resident warps / chunks per table) + 1 consecutive tables; if those tables fit in L2 that
// is the layout with the smallest working set and it is kept.  Otherwise L2 cannot hold the tables
// in flight whatever the order, and the only reuse left is between positions that share candidate
// rows: then a queue is served by as few SMs as keep busy with ONE table's chunks (rounded down),
// so that the warps of an SM gather from one or two tables and shared rows stay in that SM's L1.
void codec_schedule(const CodecArgs& a0, int n_tables, int* nq, int* g) {
    CodecArgs a = a0;
    set_queues(a, n_tables);
    *nq = a.sched_nq; *g = a.sched_g;
}

static void set_queues(CodecArgs& a, int n_tables) {
    const int sms = sm_count(), warps_per_sm = kBlocksPerSM * kWarpsPerBlock;
    const long long per_table = std::max(1LL, (long long)a.S * a.st.max_chunks);
    const long long spanned = ((long long)sms * warps_per_sm + per_table - 1) / per_table + 1;
    const double table_bytes = 2.0 * a.sh.V * a.sh.d;
    int dev = 0, l2 = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev);
    long long g = per_table / warps_per_sm;
    if ((double)std::min<long long>(spanned, n_tables) * table_bytes <= (double)l2) g = sms;
    g = std::max(1LL, std::min<long long>(g, sms));
    int nq = (sms + (int)g - 1) / (int)g;
    nq = std::max(1, std::min(nq, std::min(n_tables, kTicketWords)));
    a.sched_g = (int)g; a.sched_nq = nq;
}

cudaError_t launch_rownorm(const __half* T, float* out, long long rows, int d, cudaStream_t st) {
    return dispatch_d(d, [&](auto D) {
        long long blocks = (rows + 7) / 8;
        if (blocks > (long long)sm_count() * 16) blocks = (long long)sm_count() * 16;
        rownorm_kernel<decltype(D)::value><<<(unsigned)blocks, 256, 0, st>>>(T, out, rows);
        count_launch();
        return cudaGetLastError();
    });
}

cudaError_t launch_encode(const CodecArgs& a0, cudaStream_t st) {
    CodecArgs a = a0;
    set_queues(a, 2 * a.sh.L * a.sh.H);
    cudaError_t e = cudaMemsetAsync(a.ticket, 0, sizeof(unsigned int) * kTicketWords, st);
    if (e != cudaSuccess) return e;
    const bool zr = a.sh.zero_q != kZeroOff;
    const bool flex = a.dbg.sym || a.dbg.q || a.dbg.mu || a.dbg.ideal || a.step_exp;
    return dispatch_d(a.sh.d, [&](auto D) {
        constexpr int d = decltype(D)::value;
        if (a.mu_dense) {
            auto kd = zr ? (flex ? encode_kernel<d, kSrcDense, true, true> : encode_kernel<d, kSrcDense, true, false>)
                         : (flex ? encode_kernel<d, kSrcDense, false, true> : encode_kernel<d, kSrcDense, false, false>);
            kd<<<sm_count() * kBlocksPerSM, kThreads, 0, st>>>(a);
            count_launch();
            return cudaGetLastError();
        }
        auto kern = zr ? (flex ? encode_kernel<d, kSrcGather, true, true> : encode_kernel<d, kSrcGather, true, false>)
                       : (flex ? encode_kernel<d, kSrcGather, false, true> : encode_kernel<d, kSrcGather, false, false>);
        size_t sm = 0;
        cudaError_t e2 = pair_smem_bytes(kern, a.sh.Kp, sm);
        if (e2 != cudaSuccess) return e2;
        kern<<<sm_count() * kBlocksPerSM, kThreads, sm, st>>>(a);
        count_launch();
        return cudaGetLastError();
    });
}

cudaError_t launch_append_seal(const CodecArgs& a, cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(a.ticket, 0, sizeof(unsigned int), st);
    if (e != cudaSuccess) return e;
    return dispatch_d(a.sh.d, [&](auto D) {
        long long warps = (long long)a.open_items;
        long long blocks = (warps + kWarpsPerBlock - 1) / kWarpsPerBlock;
        if (blocks > (long long)sm_count() * kBlocksPerSM) blocks = (long long)sm_count() * kBlocksPerSM;
        auto ko = a.sh.zero_q != kZeroOff ? encode_kernel<decltype(D)::value, kSrcOpen, true, false> : encode_kernel<decltype(D)::value, kSrcOpen, false, false>;
        ko<<<(unsigned)blocks, kThreads, 0, st>>>(a);
        count_launch();
        return cudaGetLastError();
    });
}

cudaError_t launch_decode(const CodecArgs& a0, cudaStream_t st) {
    CodecArgs a = a0;
    set_queues(a, 2 * a.sh.L * a.sh.H);
    cudaError_t e = cudaMemsetAsync(a.ticket, 0, sizeof(unsigned int) * kTicketWords, st);
    if (e != cudaSuccess) return e;
    const bool zr = a.sh.zero_q != kZeroOff;
    const bool flex = a.dbg.sym || a.dbg.q || a.dbg.mu || a.step_exp;
    return dispatch_d(a.sh.d, [&](auto D) {
        constexpr int d = decltype(D)::value;
        if (a.mu_dense) {
            auto kd = zr ? (flex ? decode_kernel<d, true, true, true> : decode_kernel<d, true, true, false>)
                         : (flex ? decode_kernel<d, true, false, true> : decode_kernel<d, true, false, false>);
            kd<<<sm_count() * kBlocksPerSM, kThreads, 0, st>>>(a);
            count_launch();
            return cudaGetLastError();
        }
        auto kern = zr ? (flex ? decode_kernel<d, false, true, true> : decode_kernel<d, false, true, false>)
                       : (flex ? decode_kernel<d, false, false, true> : decode_kernel<d, false, false, false>);
        size_t sm = 0;
        cudaError_t e2 = pair_smem_bytes(kern, a.sh.Kp, sm);
        if (e2 != cudaSuccess) return e2;
        kern<<<sm_count() * kBlocksPerSM, kThreads, sm, st>>>(a);
        count_launch();
        return cudaGetLastError();
    });
}

cudaError_t launch_rotq(const CodecArgs& a0, const RotqArgs& r, bool encode, cudaStream_t st) {
    CodecArgs a = a0;
    set_queues(a, 2 * a.sh.L * a.sh.H);
    cudaError_t e = cudaMemsetAsync(a.ticket, 0, sizeof(unsigned int) * kTicketWords, st);
    if (e != cudaSuccess) return e;
    return dispatch_d(a.sh.d, [&](auto D) {
        auto kern = encode ? rotq_kernel<decltype(D)::value, true> : rotq_kernel<decltype(D)::value, false>;
        size_t sm = 0;
        cudaError_t e2 = pair_smem_bytes(kern, a.sh.Kp, sm);
        if (e2 != cudaSuccess) return e2;
        kern<<<sm_count() * kBlocksPerSM, kThreads, sm, st>>>(a, r);
        count_launch();
        return cudaGetLastError();
    });
}

cudaError_t launch_append_quantise(const CodecArgs& a, cudaStream_t st) {
    return dispatch_d(a.sh.d, [&](auto D) {
        long long warps = (long long)a.S * 2 * a.sh.L * a.sh.H;
        long long blocks = (warps + kWarpsPerBlock - 1) / kWarpsPerBlock;
        auto kern = append_quantise_kernel<decltype(D)::value>;
        size_t sm = 0;
        cudaError_t e2 = pair_smem_bytes(kern, a.sh.Kp, sm);
        if (e2 != cudaSuccess) return e2;
        // one wave: as many blocks as are resident together, each walking its share of the items
        int occ = 1;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, kThreads, sm) != cudaSuccess || occ < 1) occ = 1;
        if (blocks > (long long)sm_count() * occ) blocks = (long long)sm_count() * occ;
        kern<<<(unsigned)blocks, kThreads, sm, st>>>(a);
        count_launch();
        return cudaGetLastError();
    });
}

}  // namespace plc

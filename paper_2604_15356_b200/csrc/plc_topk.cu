// Top-K softmax over per-position next-token logits (one thread block per row, rows strided over
// the grid).  Selection is exact (logit descending, index ascending, -0 = +0).
//
// Fast path (K <= 16 per warp of the block: K <= 128 with 256 threads): pass 0 reads the row from HBM and keeps one
// maximum per thread; the ceil(K / warps)-th largest thread maximum of every warp, minimised over the
// warps, is a value with at least K row elements at or above it, i.e. a lower bound of the K-th
// largest logit that needs no histogram.  Pass 1 (served by L2) sums exp(l - l_max) over the row
// and notes the groups of 8 logits that hold an element at or above that bound; after the pass the
// noted groups are taken apart, one per thread, into a candidate list (typically 1.2-2 K entries).
// A list of at most 256 goes to global memory and a second kernel (one warp per row, bitonic sort in
// registers) orders it and writes the K selected, their weights and Z_k; without the scratch for
// that, or for longer lists, the block ranks by counting (long lists: sorted) itself.  Rows whose
// candidates overflow the list (large tie groups, adversarial layouts) and larger K take the radix-select path:
// a 4096-bin histogram of the order-preserving 16-bit key finds the bin that holds the K-th largest,
// a 16-way refinement finds the key itself, and equal keys are taken in index order.
// Reductions use warp shuffles in a fixed order, so results are bit-reproducible from run to run.
// Rows that fit a 64 KB shared-memory buffer (and rows of any length when no selection is asked for)
// first go through topk_staged_kernel further down, which does the same row work on a copy of the
// row in shared memory; this kernel then takes only what that one marks as left over.
#include <type_traits>

#include "plc_common.cuh"

namespace plc {
namespace {

constexpr int kBins = 4096;
constexpr int kCandCap = 1024;
constexpr int kHdrRedo = -2;                        // header mark: the row is left to the general kernel

__device__ __forceinline__ uint32_t key_of(uint32_t u) {
    u &= 0xffffu;
    if ((u & 0x7fffu) == 0) u = 0;                  // -0 and +0 are the same logit
    return (u & 0x8000u) ? (~u & 0xffffu) : (u | 0x8000u);
}
__device__ __forceinline__ uint32_t bits_of_key(uint32_t key) {
    return (key & 0x8000u) ? (key & 0x7fffu) : (~key & 0xffffu);
}
__device__ __forceinline__ float val_of_key(uint32_t key) {
    return __half2float(__ushort_as_half((unsigned short)bits_of_key(key)));
}
constexpr uint32_t kKeyNegInf = 0x03ffu;            // key_of(0xfc00)

template <int THREADS>
struct __align__(16) Smem {
    uint32_t hist[kBins];                           // fast path: candidate list (keys, then indices)
    uint32_t sub[16];
    uint32_t sel_key[kCandCap];
    int32_t sel_idx[kCandCap];
    uint32_t cand_key[kCandCap];
    int32_t cand_idx[kCandCap];
    float ek[kCandCap];
    uint32_t red_k[THREADS / 32];
    uint32_t red_t[THREADS / 32];
    float red_s[THREADS / 32];
    int scan[THREADS / 32];
    int nsel, ncand, bstar, count_above, cstar, thr, need, neq, running, nlist, nhit;
    float row_max, row_sum, sum_k;
    uint32_t theta;
};

// Exclusive scan of one int per thread over the block (thread order); total to all threads.
template <int THREADS>
__device__ __forceinline__ int block_excl_scan(int v, int* scratch, int& total) {
    int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(kFull, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();                                 // scratch free
    if (lane == 31) scratch[wid] = inc;
    __syncthreads();
    int base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < THREADS / 32; ++w) {
        int x = scratch[w];
        if (w < wid) base += x;
        tot += x;
    }
    total = tot;
    return base + inc - v;
}

// Calls f(index, raw binary16 bits) for the elements of the row that this thread owns in tile `t`.
// A tile is THREADS*8 consecutive elements; a thread owns 8 consecutive ones.
template <bool VEC, int THREADS, class F>
__device__ __forceinline__ void for_tile(const __half* row, int V, int t, F&& f) {
    int i0 = t * (THREADS * 8) + threadIdx.x * 8;
    if (VEC) {
        if (i0 < V) {                                // V % 8 == 0: the 8 are all in range
            uint4 r = *reinterpret_cast<const uint4*>(row + i0);
            uint32_t wds[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                f(i0 + 2 * j, wds[j] & 0xffffu);
                f(i0 + 2 * j + 1, wds[j] >> 16);
            }
        }
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (i0 + j < V) f(i0 + j, (uint32_t)__half_as_ushort(row[i0 + j]));
    }
}

// exp(x - l_max) as 2^(x log2(e) - l_max log2(e)): one fused multiply-add and one ex2.approx (relative
// error about 2e-6 at the arguments that matter, inside the tolerance of lse and Z_k; results below
// 2^-126 flush to zero).  nb = -l_max log2(e).
__device__ __forceinline__ float exp_rel(float x, float nb) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(__fmaf_rn(x, 1.44269504088896341f, nb)));
    return r;
}

__device__ __forceinline__ uint32_t hmax2_bits(uint32_t a, uint32_t b) {
    __half2 r = __hmax2(*reinterpret_cast<__half2*>(&a), *reinterpret_cast<__half2*>(&b));
    return *reinterpret_cast<uint32_t*>(&r);
}

// Sorts n_pad (a power of two) order words in shared memory, largest first, with the block.
template <int THREADS, class W>
__device__ __forceinline__ void bitonic_desc(W* v, int n_pad) {
    for (int k = 2; k <= n_pad; k <<= 1)
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int t = threadIdx.x; t < (n_pad >> 1); t += THREADS) {
                const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));       // lower index of the pair
                const W a = v[i], b = v[i | j];
                const bool desc = (i & k) == 0;
                if ((a < b) == desc) { v[i] = b; v[i | j] = a; }
            }
            __syncthreads();
        }
}

// Radix select of the K largest keys of the row into sm.sel_* (unordered); three or more passes
// over the row.
template <bool VEC, int THREADS>
__device__ void select_by_histogram(Smem<THREADS>& sm, const __half* row, int V, int K, int ntiles) {
    const int tid = threadIdx.x;
    for (int i = tid; i < kBins; i += THREADS) sm.hist[i] = 0;
    if (tid < 16) sm.sub[tid] = 0;
    if (tid == 0) { sm.nsel = 0; sm.ncand = 0; sm.running = 0; }
    __syncthreads();
    // Pass A: histogram of the top 12 key bits (keys order like the logits).
    for (int t = 0; t < ntiles; ++t)
        for_tile<VEC, THREADS>(row, V, t, [&](int, uint32_t bits) { atomicAdd(&sm.hist[key_of(bits) >> 4], 1u); });
    __syncthreads();
    // Bin that holds the K-th largest key: thread t owns BPT bins going down from 4095 - BPT*t.
    {
        constexpr int BPT = kBins / THREADS;
        int local = 0;
#pragma unroll
        for (int j = 0; j < BPT; ++j) local += (int)sm.hist[kBins - 1 - (tid * BPT + j)];
        int total;
        int excl = block_excl_scan<THREADS>(local, sm.scan, total);
        if (excl < K && K <= excl + local) {
            int cum = excl;
            for (int j = 0; j < BPT; ++j) {
                int b = kBins - 1 - (tid * BPT + j);
                int c = (int)sm.hist[b];
                if (cum + c >= K) { sm.bstar = b; sm.count_above = cum; sm.cstar = c; break; }
                cum += c;
            }
        }
    }
    __syncthreads();
    const int bstar = sm.bstar, cstar = sm.cstar, count_above = sm.count_above;
    const bool use_cand = cstar <= kCandCap;
    // Pass B: everything above the bin is selected; inside the bin refine on the low 4 key bits.
    for (int t = 0; t < ntiles; ++t)
        for_tile<VEC, THREADS>(row, V, t, [&](int i, uint32_t bits) {
            uint32_t key = key_of(bits);
            int bin = (int)(key >> 4);
            if (bin > bstar) {
                int slot = atomicAdd(&sm.nsel, 1);
                sm.sel_key[slot] = key; sm.sel_idx[slot] = i;
            } else if (bin == bstar) {
                atomicAdd(&sm.sub[key & 15u], 1u);
                if (use_cand) {
                    int slot = atomicAdd(&sm.ncand, 1);
                    sm.cand_key[slot] = key; sm.cand_idx[slot] = i;
                }
            }
        });
    __syncthreads();
    if (tid == 0) {
        int need1 = K - count_above, cum = 0;
        for (int j = 15; j >= 0; --j) {
            int c = (int)sm.sub[j];
            if (cum + c >= need1) { sm.thr = (bstar << 4) | j; sm.need = need1 - cum; sm.neq = c; break; }
            cum += c;
        }
    }
    __syncthreads();
    const uint32_t thr = (uint32_t)sm.thr;
    const int need = sm.need, neq = sm.neq;
    if (use_cand) {
        const int nc = sm.ncand;
        for (int c = tid; c < nc; c += THREADS) {
            uint32_t key = sm.cand_key[c];
            int idx = sm.cand_idx[c];
            bool take = key > thr;
            if (key == thr) {
                if (need == neq) take = true;
                else {
                    int rank = 0;
                    for (int j = 0; j < nc; ++j) rank += (sm.cand_key[j] == thr && sm.cand_idx[j] < idx);
                    take = rank < need;
                }
            }
            if (take) {
                int slot = atomicAdd(&sm.nsel, 1);
                sm.sel_key[slot] = key; sm.sel_idx[slot] = idx;
            }
        }
    } else {
        // Pass C (large tie groups): re-read the row; equal keys are taken in index order.
        for (int t = 0; t < ntiles; ++t) {
            int cnt = 0;
            for_tile<VEC, THREADS>(row, V, t, [&](int i, uint32_t bits) {
                uint32_t key = key_of(bits);
                if ((int)(key >> 4) == bstar && key > thr) {
                    int slot = atomicAdd(&sm.nsel, 1);
                    sm.sel_key[slot] = key; sm.sel_idx[slot] = i;
                }
                cnt += (key == thr);
            });
            int total;
            int rank = block_excl_scan<THREADS>(cnt, sm.scan, total) + sm.running;
            for_tile<VEC, THREADS>(row, V, t, [&](int i, uint32_t bits) {
                uint32_t key = key_of(bits);
                if (key == thr) {
                    if (rank < need) {
                        int slot = atomicAdd(&sm.nsel, 1);
                        sm.sel_key[slot] = key; sm.sel_idx[slot] = i;
                    }
                    ++rank;
                }
            });
            __syncthreads();
            if (tid == 0) sm.running += total;
            __syncthreads();
        }
    }
    __syncthreads();
    // Order the K selected by (key descending, index ascending): a sort of packed order words in the
    // histogram's memory for large K, rank by counting otherwise.
    if (K > 128) {
        unsigned long long* w = reinterpret_cast<unsigned long long*>(sm.hist);
        int n_pad = 256;
        while (n_pad < K) n_pad <<= 1;
        for (int k = tid; k < n_pad; k += THREADS)
            w[k] = k < K ? ((unsigned long long)sm.sel_key[k] << 32) | (0xffffffffu - (uint32_t)sm.sel_idx[k]) : 0ull;
        __syncthreads();
        bitonic_desc<THREADS>(w, n_pad);
        for (int k = tid; k < K; k += THREADS) {
            sm.cand_key[k] = (uint32_t)(w[k] >> 32); sm.cand_idx[k] = (int)(0xffffffffu - (uint32_t)w[k]);
        }
        __syncthreads();
        return;
    }
    for (int k = tid; k < K; k += THREADS) {
        uint32_t key = sm.sel_key[k];
        int idx = sm.sel_idx[k];
        int rank = 0;
        for (int j = 0; j < K; ++j) {
            uint32_t kj = sm.sel_key[j];
            rank += (kj > key) || (kj == key && sm.sel_idx[j] < idx);
        }
        sm.cand_key[rank] = key; sm.cand_idx[rank] = idx;
    }
    __syncthreads();
}

// Candidate list of the fast path: one order word per candidate, larger = earlier in (key
// descending, index ascending); 32-bit words while indices fit 16 bits, 64-bit words otherwise.
__device__ __forceinline__ void list_put(uint32_t* list, bool narrow, int slot, uint32_t key, int idx) {
    if (narrow) list[slot] = (key << 16) | (0xffffu - (uint32_t)idx);
    else reinterpret_cast<unsigned long long*>(list)[slot] = ((unsigned long long)key << 32) | (0xffffffffu - (uint32_t)idx);
}
// Appends those of the two logits in `w` (indices i, i + 1) that reach the bound th2 (the bound in
// both halves).  A warp gets here whenever any of its 256 logits of the moment qualifies, with one
// or two lanes active, so the test is a packed compare and the key is formed for the hits only.
__device__ __forceinline__ void collect2(uint32_t w, uint32_t th2, int i, bool narrow, int* nlist, uint32_t* list) {
    const uint32_t ge = __hge2_mask(*reinterpret_cast<const __half2*>(&w), *reinterpret_cast<const __half2*>(&th2));
    if (ge == 0) return;
    if (ge & 0xffffu) {
        const int slot = atomicAdd(nlist, 1);
        if (slot < kCandCap) list_put(list, narrow, slot, key_of(w & 0xffffu), i);
    }
    if (ge >> 16) {
        const int slot = atomicAdd(nlist, 1);
        if (slot < kCandCap) list_put(list, narrow, slot, key_of(w >> 16), i + 1);
    }
}

template <bool VEC, int THREADS>
__global__ void __launch_bounds__(THREADS) topk_softmax_kernel(TopkArgs a) {
    constexpr int NW = THREADS / 32;
    __shared__ Smem<THREADS> sm;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int V = a.V, K = a.K;
    const int ntiles = (V + THREADS * 8 - 1) / (THREADS * 8);
    const int per_warp = (K + NW - 1) / NW;
    // A warp can offer at most 32 thread maxima, and the bound is only tight while it asks for the
    // upper half of them: beyond 16 per warp the candidates overflow the list on ordinary rows.
    // Calls that want no selected set (only lse / log2 P of the tokens / step exponents) skip the selection.
    const bool select = a.pairs || a.idx || a.w || a.zk;
    const bool fast = select && per_warp <= 16 && K <= kCandCap;
    // The candidate list of the fast path lives in the histogram's memory, which is idle there.
    const bool narrow = V <= 65536;
    uint32_t* list32 = sm.hist;
    unsigned long long* list64 = reinterpret_cast<unsigned long long*>(sm.hist);

    if (a.redo_only && *a.redo == 0) return;                             // nothing was left over
    for (long long rowi = blockIdx.x; rowi < a.N; rowi += gridDim.x) {
        if (a.pos_begin || a.pos_end) {
            int s = (int)(rowi / a.n_per_session), i = (int)(rowi % a.n_per_session);
            int b = a.pos_begin ? a.pos_begin[s] : 0, e = a.pos_end ? a.pos_end[s] : a.n_per_session;
            if (i < b || i >= e) continue;
        }
        if (a.redo_only && __float_as_int(a.cand_hdr[rowi].z) != kHdrRedo) continue;
        const __half* row = a.logits + rowi * (long long)V;
        if (tid == 0) { sm.nlist = 0; sm.nhit = 0; }

        // Pass 0 (HBM): one maximum per thread.
        uint32_t tkey = 0;
        if (VEC) {
            uint32_t m2 = 0xfc00fc00u;                                   // (-inf, -inf)
#pragma unroll 4
            for (int t = 0; t < ntiles; ++t) {
                const int i0 = t * (THREADS * 8) + tid * 8;
                if (i0 < V) {
                    const uint4 r = *reinterpret_cast<const uint4*>(row + i0);
                    m2 = hmax2_bits(m2, hmax2_bits(hmax2_bits(r.x, r.y), hmax2_bits(r.z, r.w)));
                }
            }
            tkey = max(key_of(m2 & 0xffffu), key_of(m2 >> 16));
            if (tid * 8 >= V) tkey = 0;                                   // this thread owns nothing
        } else {
            for (int t = 0; t < ntiles; ++t)
                for_tile<VEC, THREADS>(row, V, t, [&](int, uint32_t bits) { tkey = max(tkey, key_of(bits)); });
        }
        // per warp: the largest and the per_warp-th largest thread maximum
        const uint32_t wmax = __reduce_max_sync(kFull, tkey);
        uint32_t wth = 0;
        if (fast) {
            uint32_t v = tkey;
            for (int r = 0; r < per_warp; ++r) {
                wth = __reduce_max_sync(kFull, v);
                const uint32_t eq = __ballot_sync(kFull, v == wth);
                if (lane == __ffs(eq) - 1) v = 0;
            }
        }
        if (lane == 0) { sm.red_k[wid] = wmax; sm.red_t[wid] = wth; }
        __syncthreads();
        uint32_t km = sm.red_k[0], theta = sm.red_t[0];
#pragma unroll
        for (int w = 1; w < NW; ++w) { km = max(km, sm.red_k[w]); theta = min(theta, sm.red_t[w]); }
        theta = max(theta, kKeyNegInf);
        const float lmax = val_of_key(km);

        // Pass 1 (L2): sum of exp(l - l_max) over the row (fast exponential: its relative error of
        // about 2e-6 at the arguments that matter is inside the tolerance of lse and Z_k) and, on
        // the fast path, the elements at or above the bound.
        const float nb = -lmax * 1.44269504088896341f;
        float s = 0.f;
        if (VEC) {
            const uint32_t tb = bits_of_key(theta);
            const uint32_t th2 = tb | (tb << 16);
#pragma unroll 2
            for (int t = 0; t < ntiles; ++t) {
                const int i0 = t * (THREADS * 8) + tid * 8;
                if (i0 < V) {
                    const uint4 r = *reinterpret_cast<const uint4*>(row + i0);
                    const uint32_t wds[4] = {r.x, r.y, r.z, r.w};
                    const uint32_t top = hmax2_bits(hmax2_bits(r.x, r.y), hmax2_bits(r.z, r.w));
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&wds[j]));
                        s += exp_rel(f.x, nb);
                        s += exp_rel(f.y, nb);
                    }
                    // A group of 8 with a logit at or above the bound is only noted here (few lanes get
                    // here, so anything longer would run once per group with the rest of the warp idle);
                    // the noted groups are taken apart after the pass, one per thread.
                    if (fast && !__hblt2(*reinterpret_cast<const __half2*>(&top), *reinterpret_cast<const __half2*>(&th2))) {
                        const int slot = atomicAdd(&sm.nhit, 1);
                        if (slot < kCandCap) sm.sel_idx[slot] = i0;          // sel_idx is idle on this path
                    }
                }
            }
        } else {
            for (int t = 0; t < ntiles; ++t)
                for_tile<VEC, THREADS>(row, V, t, [&](int i, uint32_t bits) {
                    s += exp_rel(__half2float(__ushort_as_half((unsigned short)bits)), nb);
                    const uint32_t key = key_of(bits);
                    if (fast && key >= theta) {
                        const int slot = atomicAdd(&sm.nlist, 1);
                        if (slot < kCandCap) list_put(sm.hist, narrow, slot, key, i);
                    }
                });
        }
        s = warp_sum(s);
        if (lane == 0) sm.red_s[wid] = s;
        __syncthreads();
        float sum_all = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) sum_all += sm.red_s[w];
        if (VEC && fast) {
            const int nhit = sm.nhit;
            if (nhit > kCandCap) {
                if (tid == 0) sm.nlist = kCandCap + 1;                    // too many: the radix select takes the row
            } else {
                const uint32_t tb = bits_of_key(theta);
                const uint32_t th2 = tb | (tb << 16);
                for (int t = tid; t < nhit; t += THREADS) {
                    const int i0 = sm.sel_idx[t];
                    const uint4 r = *reinterpret_cast<const uint4*>(row + i0);
                    const uint32_t wds[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) collect2(wds[j], th2, i0 + 2 * j, narrow, &sm.nlist, sm.hist);
                }
            }
            __syncthreads();
        }
        const int nlist = sm.nlist;
        // Two-kernel selection: a list that one warp can sort goes to global memory as it is and
        // topk_rank_kernel finishes the row (order, weights, Z_k); everything else stays here.
        const bool handed = fast && a.cand && K <= 128 && nlist >= K && nlist <= kTopkListCap;
        if (a.cand_hdr && tid == 0)
            a.cand_hdr[rowi] = make_float4(lmax, sum_all, __int_as_float(handed ? nlist : -1), 0.f);
        if (handed) {
            if (narrow) {
                uint32_t* dst = static_cast<uint32_t*>(a.cand) + rowi * kTopkListCap;
                for (int c = tid; c < nlist; c += THREADS) dst[c] = list32[c];
            } else {
                unsigned long long* dst = static_cast<unsigned long long*>(a.cand) + rowi * kTopkListCap;
                for (int c = tid; c < nlist; c += THREADS) dst[c] = list64[c];
            }
        } else if (fast && nlist >= K && nlist <= kCandCap) {
            // Order the candidates (at least K of them); the first K are the result.  Short lists are
            // ranked by counting (n^2 / THREADS compares per thread, no barriers), long ones sorted.
            constexpr int kRankMax = 192;
            if (nlist > kRankMax) {
                int n_pad = 256;
                while (n_pad < nlist) n_pad <<= 1;
                if (narrow) {
                    for (int c = nlist + tid; c < n_pad; c += THREADS) list32[c] = 0;    // pad: orders after everything
                    __syncthreads();
                    bitonic_desc<THREADS>(list32, n_pad);
                    for (int k = tid; k < K; k += THREADS) {
                        const uint32_t v = list32[k];
                        sm.cand_key[k] = v >> 16; sm.cand_idx[k] = (int)(0xffffu - (v & 0xffffu));
                    }
                } else {
                    for (int c = nlist + tid; c < n_pad; c += THREADS) list64[c] = 0;
                    __syncthreads();
                    bitonic_desc<THREADS>(list64, n_pad);
                    for (int k = tid; k < K; k += THREADS) {
                        const unsigned long long v = list64[k];
                        sm.cand_key[k] = (uint32_t)(v >> 32); sm.cand_idx[k] = (int)(0xffffffffu - (uint32_t)v);
                    }
                }
            } else if (narrow) {
                const int n4 = (nlist + 3) & ~3;
                for (int c = nlist + tid; c < n4; c += THREADS) list32[c] = 0;           // pad: orders after everything
                __syncthreads();
                for (int c = tid; c < nlist; c += THREADS) {
                    const uint32_t mine = list32[c];
                    int rank = 0;
                    for (int j = 0; j < n4; j += 4) {
                        const uint4 o = *reinterpret_cast<const uint4*>(list32 + j);
                        rank += (o.x > mine) + (o.y > mine) + (o.z > mine) + (o.w > mine);
                    }
                    if (rank < K) { sm.cand_key[rank] = mine >> 16; sm.cand_idx[rank] = (int)(0xffffu - (mine & 0xffffu)); }
                }
            } else {
                for (int c = tid; c < nlist; c += THREADS) {
                    const unsigned long long mine = list64[c];
                    int rank = 0;
                    for (int j = 0; j < nlist; ++j) rank += list64[j] > mine;
                    if (rank < K) { sm.cand_key[rank] = (uint32_t)(mine >> 32); sm.cand_idx[rank] = (int)(0xffffffffu - (uint32_t)mine); }
                }
            }
            __syncthreads();
        } else if (select) {
            __syncthreads();
            select_by_histogram<VEC, THREADS>(sm, row, V, K, ntiles);
        }

        float sum_k = 0.f;
        if (select && !handed) {
            for (int k = tid; k < K; k += THREADS) sm.ek[k] = expf(val_of_key(sm.cand_key[k]) - lmax);
            __syncthreads();
            if (wid == 0) {
                float p = 0.f;
                for (int k = lane; k < K; k += 32) p += sm.ek[k];
                p = warp_sum(p);
                if (lane == 0) sm.sum_k = p;
            }
            __syncthreads();
            sum_k = sm.sum_k;
            for (int k = tid; k < K; k += THREADS) {
                float w = sm.ek[k] / sum_k;
                int idx = sm.cand_idx[k];
                if (a.pairs) a.pairs[rowi * a.Kp + k] = make_int2(idx, __float_as_int(w));
                if (a.idx) a.idx[rowi * K + k] = idx;
                if (a.w) a.w[rowi * K + k] = w;
            }
            if (a.pairs)
                for (int k = K + tid; k < a.Kp; k += THREADS) a.pairs[rowi * a.Kp + k] = make_int2(sm.cand_idx[0], 0);
        }
        if (tid == 0) {
            float lse = lmax + logf(sum_all);
            if (a.lse) a.lse[rowi] = lse;
            if (a.zk && !handed) a.zk[rowi] = sum_k / sum_all;
            if (a.tokens && (a.logp2 || a.step_exp || a.bits_out)) {
                const int tk = a.tokens[rowi];
                const float v = (tk >= 0 && tk < V) ? (__half2float(row[tk]) - lse) * 1.44269504088896341f : __int_as_float(0x7fc00000);
                if (a.logp2) a.logp2[rowi] = v;
                if (a.step_exp || a.bits_out) {
                    // Def. 7: b = max(1, floor(b0 h / hbar)), capped at b0 + extra; decided in binary32
                    const float r = __fmul_rn((float)a.b0, __fdiv_rn(-v, a.hbar));
                    int b = (r >= 1.0f) ? (int)floorf(r) : 1;
                    b = min(b, a.b0 + a.extra);
                    if (a.step_exp) a.step_exp[rowi] = a.b0 - b;
                    if (a.bits_out) a.bits_out[rowi] = b;
                }
            }
        }
        __syncthreads();
    }
}

// ---- rows that fit in shared memory -------------------------------------------------------------
// The same row work as the fast path above, but the row is brought into shared memory ONCE by a
// bulk asynchronous copy (one instruction of one thread, completion on an mbarrier) and both passes
// and the taking apart of the noted groups read it there: the second pass costs no L2 round trips,
// no registers hold loads in flight, and the copy of a block's next row runs under the tail of the
// current one.  Three blocks per SM keep about 190 KB of copies or rows per SM in flight.  Rows
// whose candidates do not fit the hand-over (ties, more than 256 at or above the bound) are marked
// for the general kernel.  A call that wants no selection (lse / log2 P only) may have rows longer
// than the buffer: they pass through it in chunks, one HBM read and no L2 pass at all.  Every wait
// on the barrier is bounded.
constexpr int kStageBytes = 64 * 1024;             // largest row buffer: V <= 32768 binary16 logits
// A row longer than the buffer is staged in equal chunks (a multiple of 8 logits each); only calls
// without a selection take such rows here: maximum and sum are carried from chunk to chunk.
__host__ __device__ constexpr int stage_chunks(int V) { return (V * 2 + kStageBytes - 1) / kStageBytes; }
__host__ __device__ constexpr int stage_chunk_elems(int V) {
    return stage_chunks(V) <= 1 ? V : (((V + stage_chunks(V) - 1) / stage_chunks(V) + 7) & ~7);
}
__host__ __device__ constexpr int stage_buf_bytes(int V) { return (stage_chunk_elems(V) * 2 + 127) & ~127; }
#ifndef PLC_STAGE_THREADS
#define PLC_STAGE_THREADS 256
#endif
constexpr int kStageThreads = PLC_STAGE_THREADS;
constexpr uint32_t kStageSpin = 1u << 24;

struct __align__(16) StageSm {
    unsigned long long bar;
    uint32_t list[kCandCap];
    int32_t hit[kCandCap];
    uint32_t red_k[kStageThreads / 32];
    uint32_t red_t[kStageThreads / 32];
    float red_s[kStageThreads / 32];
    int nlist, nhit;
};

__device__ __forceinline__ bool stage_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kStageSpin; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}

// The row after `rowi` (stride: the grid) that lies inside its session's position range, or N.
__device__ __forceinline__ long long stage_next_row(const TopkArgs& a, long long rowi) {
    for (; rowi < a.N; rowi += gridDim.x) {
        if (!(a.pos_begin || a.pos_end)) return rowi;
        const int s = (int)(rowi / a.n_per_session), i = (int)(rowi % a.n_per_session);
        const int b = a.pos_begin ? a.pos_begin[s] : 0, e = a.pos_end ? a.pos_end[s] : a.n_per_session;
        if (i >= b && i < e) return rowi;
    }
    return a.N;
}

__global__ void __launch_bounds__(kStageThreads) topk_staged_kernel(TopkArgs a) {
    constexpr int THREADS = kStageThreads, NW = THREADS / 32;
    extern __shared__ __align__(128) unsigned char stage_raw[];
    const __half* buf = reinterpret_cast<const __half*>(stage_raw);
    StageSm& sm = *reinterpret_cast<StageSm*>(stage_raw + stage_buf_bytes(a.V));
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int Vrow = a.V, K = a.K;
    const int nchunks = stage_chunks(Vrow), ce = stage_chunk_elems(Vrow);
    const int per_warp = (K + NW - 1) / NW;
    const bool select = a.pairs || a.idx || a.w || a.zk;            // the launcher sends only one-chunk rows of the fast path here with a selection
    const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&sm.bar);
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(stage_raw);

    auto fetch = [&](long long rowi, int c) {                        // one thread: the whole chunk in one copy
        const uint32_t bytes = (uint32_t)min(ce, Vrow - c * ce) * 2u;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the buffer's last readers used ordinary loads
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(dst), "l"(a.logits + rowi * (long long)Vrow + (long long)c * ce), "r"(bytes), "r"(bar) : "memory");
    };

    long long rowi = stage_next_row(a, blockIdx.x);
    int c = 0;
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(1u) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0 && rowi < a.N) fetch(rowi, 0);
    uint32_t parity = 0;
    float run_max = 0.f, run_sum = 0.f;                              // over the chunks of the row so far
    while (rowi < a.N) {
        int next_c = c + 1;
        long long next = rowi;
        if (next_c == nchunks) { next_c = 0; next = stage_next_row(a, rowi + gridDim.x); }
        const int V = min(ce, Vrow - c * ce);                        // logits in the buffer
        const int ntiles = (V + THREADS * 8 - 1) / (THREADS * 8);
        if (tid == 0) { sm.nlist = 0; sm.nhit = 0; }
        bool ok = stage_wait(bar, parity);
        if (!ok) ok = stage_wait(bar, parity);                        // a copy in flight is waited for once more before giving up
        if (__syncthreads_or(!ok)) {
            if (tid == 0 && a.status) atomicOr(a.status, kStTimeout);
            return;
        }
        parity ^= 1u;

        // Pass 0: one maximum per thread.
        uint32_t m2 = 0xfc00fc00u;                                   // (-inf, -inf)
#pragma unroll 4
        for (int t = 0; t < ntiles; ++t) {
            const int i0 = t * (THREADS * 8) + tid * 8;
            if (i0 < V) {
                const uint4 r = *reinterpret_cast<const uint4*>(buf + i0);
                m2 = hmax2_bits(m2, hmax2_bits(hmax2_bits(r.x, r.y), hmax2_bits(r.z, r.w)));
            }
        }
        uint32_t tkey = max(key_of(m2 & 0xffffu), key_of(m2 >> 16));
        if (tid * 8 >= V) tkey = 0;                                   // this thread owns nothing
        const uint32_t wmax = __reduce_max_sync(kFull, tkey);
        uint32_t wth = 0;
        if (select) {
            uint32_t v = tkey;
            for (int r = 0; r < per_warp; ++r) {
                wth = __reduce_max_sync(kFull, v);
                const uint32_t eq = __ballot_sync(kFull, v == wth);
                if (lane == __ffs(eq) - 1) v = 0;
            }
        }
        if (lane == 0) { sm.red_k[wid] = wmax; sm.red_t[wid] = wth; }
        __syncthreads();
        uint32_t km = sm.red_k[0], theta = sm.red_t[0];
#pragma unroll
        for (int w = 1; w < NW; ++w) { km = max(km, sm.red_k[w]); theta = min(theta, sm.red_t[w]); }
        theta = max(theta, kKeyNegInf);
        const float lmax = val_of_key(km);

        // Pass 1: sum of exp(l - l_max); groups of 8 with an element at or above the bound are noted.
        const float nb = -lmax * 1.44269504088896341f;
        const uint32_t tb = bits_of_key(theta);
        const uint32_t th2 = tb | (tb << 16);
        float s = 0.f;
#pragma unroll 2
        for (int t = 0; t < ntiles; ++t) {
            const int i0 = t * (THREADS * 8) + tid * 8;
            if (i0 < V) {
                const uint4 r = *reinterpret_cast<const uint4*>(buf + i0);
                const uint32_t wds[4] = {r.x, r.y, r.z, r.w};
                const uint32_t top = hmax2_bits(hmax2_bits(r.x, r.y), hmax2_bits(r.z, r.w));
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&wds[j]));
                    s += exp_rel(f.x, nb);
                    s += exp_rel(f.y, nb);
                }
                if (select && !__hblt2(*reinterpret_cast<const __half2*>(&top), *reinterpret_cast<const __half2*>(&th2))) {
                    const int slot = atomicAdd(&sm.nhit, 1);
                    if (slot < kCandCap) sm.hit[slot] = i0;
                }
            }
        }
        s = warp_sum(s);
        if (lane == 0) sm.red_s[wid] = s;
        __syncthreads();
        float sum_all = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) sum_all += sm.red_s[w];
        int nlist = 0;
        if (select) {
            const int nhit = sm.nhit;
            if (nhit <= kCandCap) {
                for (int t = tid; t < nhit; t += THREADS) {
                    const int i0 = sm.hit[t];
                    const uint4 r = *reinterpret_cast<const uint4*>(buf + i0);
                    const uint32_t wds[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) collect2(wds[j], th2, i0 + 2 * j, true, &sm.nlist, sm.list);
                }
            }
            __syncthreads();
            nlist = nhit <= kCandCap ? sm.nlist : kCandCap + 1;
        }
        // the buffer is free: the next copy runs under the rest of this row
        if (tid == 0 && next < a.N) fetch(next, next_c);

        // maximum and sum over the chunks so far (the same values in every thread)
        float lmax_row = lmax, sum_row = sum_all;
        if (c > 0) {
            lmax_row = fmaxf(run_max, lmax);
            sum_row = (run_max > -INFINITY ? run_sum * expf(run_max - lmax_row) : 0.f) +
                      (lmax > -INFINITY ? sum_all * expf(lmax - lmax_row) : 0.f);
        }
        run_max = lmax_row; run_sum = sum_row;

        if (next_c == 0) {                                               // last chunk: the row is complete
            const bool handed = select && nlist >= K && nlist <= kTopkListCap;
            if (select) {
                if (tid == 0) {
                    a.cand_hdr[rowi] = make_float4(lmax_row, sum_row, __int_as_float(handed ? nlist : kHdrRedo), 0.f);
                    if (!handed) atomicAdd(a.redo, 1u);
                }
                if (handed) {
                    uint32_t* out = static_cast<uint32_t*>(a.cand) + rowi * kTopkListCap;
                    for (int i = tid; i < nlist; i += THREADS) out[i] = sm.list[i];
                }
            }
            if (tid == 0 && (!select || handed)) {                      // a row that is left over gets these from the general kernel
                const float lse = lmax_row + logf(sum_row);
                if (a.lse) a.lse[rowi] = lse;
                if (a.tokens && (a.logp2 || a.step_exp || a.bits_out)) {
                    const int tk = a.tokens[rowi];
                    const float v = (tk >= 0 && tk < Vrow) ? (__half2float(a.logits[rowi * (long long)Vrow + tk]) - lse) * 1.44269504088896341f
                                                           : __int_as_float(0x7fc00000);
                    if (a.logp2) a.logp2[rowi] = v;
                    if (a.step_exp || a.bits_out) {
                        // Def. 7: b = max(1, floor(b0 h / hbar)), capped at b0 + extra; decided in binary32
                        const float r = __fmul_rn((float)a.b0, __fdiv_rn(-v, a.hbar));
                        int b = (r >= 1.0f) ? (int)floorf(r) : 1;
                        b = min(b, a.b0 + a.extra);
                        if (a.step_exp) a.step_exp[rowi] = a.b0 - b;
                        if (a.bits_out) a.bits_out[rowi] = b;
                    }
                }
            }
        }
        __syncthreads();                                                 // sm.list, sm.nlist are free again
        rowi = next; c = next_c;
    }
}

// One compare-exchange step of a bitonic network on 256 order words held 8 per lane: word e = r * 32 +
// lane sits in v[r].  K2 = the size of the bitonic blocks being merged, J = the distance.  The
// network sorts descending overall.
template <class W, int K2, int J>
__device__ __forceinline__ void bitonic_step(W (&v)[8], int lane) {
    if constexpr (J >= 32) {
        constexpr int RJ = J >> 5;
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            if ((r & RJ) == 0) {
                const bool desc = (((r * 32) & K2) == 0) || K2 == 256;       // K2 >= 64 here: the bit of e lies in r
                const W x = v[r], y = v[r | RJ];
                const bool sw = desc ? (x < y) : (x > y);
                v[r] = sw ? y : x; v[r | RJ] = sw ? x : y;
            }
        }
    } else {
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const W p = __shfl_xor_sync(kFull, v[r], J);
            const int e = r * 32 + lane;
            const bool lower = (lane & J) == 0;
            const bool desc = K2 == 256 || (e & K2) == 0;
            const bool keep_max = lower == desc;
            const W mx = v[r] > p ? v[r] : p, mn = v[r] > p ? p : v[r];
            v[r] = keep_max ? mx : mn;
        }
    }
}
template <class W, int K2, int J>
__device__ __forceinline__ void bitonic_merge(W (&v)[8], int lane) {
    bitonic_step<W, K2, J>(v, lane);
    if constexpr (J > 1) bitonic_merge<W, K2, J / 2>(v, lane);
}
template <class W, int K2>
__device__ __forceinline__ void bitonic_sort256(W (&v)[8], int lane) {
    if constexpr (K2 > 2) bitonic_sort256<W, K2 / 2>(v, lane);
    bitonic_merge<W, K2, K2 / 2>(v, lane);
}

// Second kernel of the two-kernel selection: one warp per row sorts the row's candidate list (at
// most 256 order words, larger = earlier in (logit descending, index ascending)) in registers and
// writes what the streaming kernel would have written for the first K: order, renormalised weights
// (the same sums in the same order), Z_k.  Rows the streaming kernel finished itself carry -1.
template <bool NARROW>
__global__ void __launch_bounds__(256) topk_rank_kernel(TopkArgs a) {
    using W = std::conditional_t<NARROW, uint32_t, unsigned long long>;
    const int lane = threadIdx.x & 31, K = a.K;
    const long long warp = (long long)blockIdx.x * 8 + (threadIdx.x >> 5), nw = (long long)gridDim.x * 8;
    for (long long rowi = warp; rowi < a.N; rowi += nw) {
        if (a.pos_begin || a.pos_end) {
            int s = (int)(rowi / a.n_per_session), i = (int)(rowi % a.n_per_session);
            int b = a.pos_begin ? a.pos_begin[s] : 0, e = a.pos_end ? a.pos_end[s] : a.n_per_session;
            if (i < b || i >= e) continue;
        }
        const float4 hdr = a.cand_hdr[rowi];
        const int nlist = __float_as_int(hdr.z);
        if (nlist < 0) continue;
        const W* src = static_cast<const W*>(a.cand) + rowi * kTopkListCap;
        W v[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) v[r] = r * 32 + lane < nlist ? src[r * 32 + lane] : (W)0;   // 0 orders after everything
        bitonic_sort256<W, 256>(v, lane);
        const float lmax = hdr.x;
        float ek[4];
        int idx[4];
        float p = 0.f;
#pragma unroll
        for (int r = 0; r < 4; ++r) {                   // K <= 128: the first K words sit in v[0..3]
            const uint32_t key = NARROW ? (uint32_t)(v[r] >> 16) : (uint32_t)((unsigned long long)v[r] >> 32);
            idx[r] = NARROW ? (int)(0xffffu - ((uint32_t)v[r] & 0xffffu)) : (int)(0xffffffffu - (uint32_t)v[r]);
            ek[r] = r * 32 + lane < K ? expf(val_of_key(key) - lmax) : 0.f;
            if (r * 32 + lane < K) p += ek[r];
        }
        const float sum_k = warp_sum(p);
        const int idx0 = __shfl_sync(kFull, idx[0], 0);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int k = r * 32 + lane;
            if (k < K) {
                const float w = ek[r] / sum_k;
                if (a.pairs) a.pairs[rowi * a.Kp + k] = make_int2(idx[r], __float_as_int(w));
                if (a.idx) a.idx[rowi * K + k] = idx[r];
                if (a.w) a.w[rowi * K + k] = w;
            }
        }
        if (a.pairs)
            for (int k = K + lane; k < a.Kp; k += 32) a.pairs[rowi * a.Kp + k] = make_int2(idx0, 0);
        if (a.zk && lane == 0) a.zk[rowi] = sum_k / hdr.y;
    }
}

}  // namespace

cudaError_t launch_topk(const TopkArgs& a, cudaStream_t st) {
    if (a.N <= 0) return cudaSuccess;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const bool vec = (a.V % 8 == 0) && ((reinterpret_cast<uintptr_t>(a.logits) & 15) == 0);
    // The second pass over a row should find it in L2: rows of up to 128 KB are read by 256 threads
    // with five blocks per SM, longer rows by 512 threads with two blocks per SM (two, so that one
    // block streams while the other sits at the barrier between its passes).
    const bool wide = (long long)a.V * 2 > 128 * 1024;
    TopkArgs g = a;                                           // what the general kernel is launched with
    auto launch = [&](auto kern, int threads, int cap) {
        int occ = 1;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, threads, 0) != cudaSuccess || occ < 1) occ = 1;
        const long long per_sm = occ < cap ? occ : cap;       // the rows in flight stay within L2
        const long long blocks = a.N < sms * per_sm ? a.N : sms * per_sm;
        kern<<<(unsigned)blocks, threads, 0, st>>>(g);
    };
    const bool select = a.pairs || a.idx || a.w || a.zk;
    // The staged kernel takes what it can finish: calls without a selection (rows of any length, in
    // chunks), and rows that fit in its buffer when the selection can be handed to the ranking
    // kernel (K <= 128 and the scratch for it).
    const bool staged = vec && (select ? (long long)a.V * 2 <= kStageBytes && a.K <= 128 && a.cand && a.cand_hdr && a.redo
                                       : a.V < (1 << 30));
    cudaError_t e = cudaSuccess;
    if (staged) {
        const size_t smem = stage_buf_bytes(a.V) + sizeof(StageSm);
        e = cudaFuncSetAttribute(topk_staged_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (select) {
            e = cudaMemsetAsync(a.redo, 0, sizeof(unsigned int), st);
            if (e != cudaSuccess) return e;
        }
        int occ = 1;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, topk_staged_kernel, kStageThreads, smem) != cudaSuccess || occ < 1) occ = 1;
        const long long blocks = a.N < (long long)sms * occ ? a.N : (long long)sms * occ;
        topk_staged_kernel<<<(unsigned)blocks, kStageThreads, smem, st>>>(a);
        count_launch();
        e = cudaGetLastError();
        if (e != cudaSuccess || !select) return e;
        g.redo_only = 1;                                      // then only what the staged kernel left over
    }
    if (wide) {
        if (vec) launch(topk_softmax_kernel<true, 512>, 512, 2);
        else launch(topk_softmax_kernel<false, 512>, 512, 2);
    } else {
        if (vec) launch(topk_softmax_kernel<true, 256>, 256, 5);
        else launch(topk_softmax_kernel<false, 256>, 256, 5);
    }
    count_launch();
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (a.cand && a.cand_hdr && select && a.K <= 128) {
        const long long want = (a.N + 7) / 8, cap = (long long)sms * 8;
        const unsigned blocks = (unsigned)(want < cap ? want : cap);
        if (a.V <= 65536) topk_rank_kernel<true><<<blocks, 256, 0, st>>>(a);
        else topk_rank_kernel<false><<<blocks, 256, 0, st>>>(a);
        count_launch();
        e = cudaGetLastError();
    }
    return e;
}

}  // namespace plc

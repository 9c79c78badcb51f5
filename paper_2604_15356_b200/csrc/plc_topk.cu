// Top-K softmax over per-position next-token logits (one thread block per row, rows strided over
// the grid).  Selection is exact: a 4096-bin histogram of the order-preserving 16-bit key of each
// binary16 logit finds the bin that holds the K-th largest, a 16-way refinement finds the key
// itself, and equal keys are taken in index order.  Reductions use warp shuffles in a fixed order,
// so results are bit-reproducible from run to run.
#include "plc_common.cuh"

namespace plc {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kBins = 4096;
constexpr int kCandCap = 1024;

__device__ __forceinline__ uint32_t key_of(uint32_t u) {
    u &= 0xffffu;
    if ((u & 0x7fffu) == 0) u = 0;                  // -0 and +0 are the same logit
    return (u & 0x8000u) ? (~u & 0xffffu) : (u | 0x8000u);
}
__device__ __forceinline__ float val_of_key(uint32_t key) {
    uint32_t u = (key & 0x8000u) ? (key & 0x7fffu) : (~key & 0xffffu);
    return __half2float(__ushort_as_half((unsigned short)u));
}

struct Smem {
    uint32_t hist[kBins];
    uint32_t sub[16];
    uint32_t sel_key[kCandCap];
    int32_t sel_idx[kCandCap];
    uint32_t cand_key[kCandCap];
    int32_t cand_idx[kCandCap];
    float ek[kCandCap];
    uint32_t red_k[kWarps];
    float red_s[kWarps];
    int scan[kWarps];
    int nsel, ncand, bstar, count_above, cstar, thr, need, neq, running;
    float row_max, row_sum, sum_k;
};

// Exclusive scan of one int per thread over the block (thread order); total to all threads.
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
    for (int w = 0; w < kWarps; ++w) {
        int x = scratch[w];
        if (w < wid) base += x;
        tot += x;
    }
    total = tot;
    return base + inc - v;
}

// Calls f(index, raw binary16 bits) for the elements of the row that this thread owns in tile `t`.
// A tile is kThreads*8 consecutive elements; a thread owns 8 consecutive ones.
template <bool VEC, class F>
__device__ __forceinline__ void for_tile(const __half* row, int V, int t, F&& f) {
    int i0 = t * (kThreads * 8) + threadIdx.x * 8;
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

template <bool VEC>
__global__ void __launch_bounds__(kThreads) topk_softmax_kernel(TopkArgs a) {
    __shared__ Smem sm;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int V = a.V, K = a.K;
    const int ntiles = (V + kThreads * 8 - 1) / (kThreads * 8);

    for (long long rowi = blockIdx.x; rowi < a.N; rowi += gridDim.x) {
        if (a.pos_begin || a.pos_end) {
            int s = (int)(rowi / a.n_per_session), i = (int)(rowi % a.n_per_session);
            int b = a.pos_begin ? a.pos_begin[s] : 0, e = a.pos_end ? a.pos_end[s] : a.n_per_session;
            if (i < b || i >= e) continue;
        }
        const __half* row = a.logits + rowi * (long long)V;
        for (int i = tid; i < kBins; i += kThreads) sm.hist[i] = 0;
        if (tid < 16) sm.sub[tid] = 0;
        if (tid == 0) { sm.nsel = 0; sm.ncand = 0; sm.running = 0; }
        __syncthreads();

        // Pass A: histogram of the top 12 key bits and the largest key (keys order like the logits).
        uint32_t kmax = 0;
        for (int t = 0; t < ntiles; ++t)
            for_tile<VEC>(row, V, t, [&](int, uint32_t bits) {
                const uint32_t key = key_of(bits);
                atomicAdd(&sm.hist[key >> 4], 1u);
                kmax = max(kmax, key);
            });
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) kmax = max(kmax, __shfl_xor_sync(kFull, kmax, o));
        if (lane == 0) sm.red_k[wid] = kmax;
        __syncthreads();
        if (tid == 0) {
            uint32_t km = sm.red_k[0];
            for (int w = 1; w < kWarps; ++w) km = max(km, sm.red_k[w]);
            sm.row_max = val_of_key(km);
        }

        // Bin that holds the K-th largest key: thread t owns bins 4095-16t ... 4095-16t-15.
        {
            int local = 0;
#pragma unroll
            for (int j = 0; j < 16; ++j) local += (int)sm.hist[kBins - 1 - (tid * 16 + j)];
            int total;
            int excl = block_excl_scan(local, sm.scan, total);
            if (excl < K && K <= excl + local) {
                int cum = excl;
                for (int j = 0; j < 16; ++j) {
                    int b = kBins - 1 - (tid * 16 + j);
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
        // The same pass sums exp(l - l_max) over the row (fast exponential: its relative error of
        // about 2e-6 at the arguments that matter is inside the tolerance of lse and Z_k).
        const float lmax_b = sm.row_max;
        float s = 0.f;
        for (int t = 0; t < ntiles; ++t)
            for_tile<VEC>(row, V, t, [&](int i, uint32_t bits) {
                uint32_t key = key_of(bits);
                s += __expf(__half2float(__ushort_as_half((unsigned short)bits)) - lmax_b);
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
        s = warp_sum(s);
        if (lane == 0) sm.red_s[wid] = s;
        __syncthreads();
        if (tid == 0) {
            float ss = 0.f;
            for (int w = 0; w < kWarps; ++w) ss += sm.red_s[w];
            sm.row_sum = ss;
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
            for (int c = tid; c < nc; c += kThreads) {
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
                for_tile<VEC>(row, V, t, [&](int i, uint32_t bits) {
                    uint32_t key = key_of(bits);
                    if ((int)(key >> 4) == bstar && key > thr) {
                        int slot = atomicAdd(&sm.nsel, 1);
                        sm.sel_key[slot] = key; sm.sel_idx[slot] = i;
                    }
                    cnt += (key == thr);
                });
                int total;
                int rank = block_excl_scan(cnt, sm.scan, total) + sm.running;
                for_tile<VEC>(row, V, t, [&](int i, uint32_t bits) {
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

        // Order the K selected by (key descending, index ascending): rank by counting.
        for (int k = tid; k < K; k += kThreads) {
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
        const float lmax = sm.row_max;
        for (int k = tid; k < K; k += kThreads) sm.ek[k] = expf(val_of_key(sm.cand_key[k]) - lmax);
        __syncthreads();
        if (wid == 0) {
            float p = 0.f;
            for (int k = lane; k < K; k += 32) p += sm.ek[k];
            p = warp_sum(p);
            if (lane == 0) sm.sum_k = p;
        }
        __syncthreads();
        const float sum_k = sm.sum_k, sum_all = sm.row_sum;
        for (int k = tid; k < K; k += kThreads) {
            float w = sm.ek[k] / sum_k;
            int idx = sm.cand_idx[k];
            if (a.pairs) a.pairs[rowi * a.Kp + k] = make_int2(idx, __float_as_int(w));
            if (a.idx) a.idx[rowi * K + k] = idx;
            if (a.w) a.w[rowi * K + k] = w;
        }
        if (a.pairs)
            for (int k = K + tid; k < a.Kp; k += kThreads) a.pairs[rowi * a.Kp + k] = make_int2(sm.cand_idx[0], 0);
        if (tid == 0) {
            float lse = lmax + logf(sum_all);
            if (a.lse) a.lse[rowi] = lse;
            if (a.zk) a.zk[rowi] = sum_k / sum_all;
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

}  // namespace

cudaError_t launch_topk(const TopkArgs& a, cudaStream_t st) {
    if (a.N <= 0) return cudaSuccess;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    long long blocks = a.N < (long long)sms * 4 ? a.N : (long long)sms * 4;
    bool vec = (a.V % 8 == 0) && ((reinterpret_cast<uintptr_t>(a.logits) & 15) == 0);
    if (vec) topk_softmax_kernel<true><<<(unsigned)blocks, kThreads, 0, st>>>(a);
    else topk_softmax_kernel<false><<<(unsigned)blocks, kThreads, 0, st>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace plc

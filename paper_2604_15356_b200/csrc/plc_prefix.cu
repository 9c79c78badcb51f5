// Batched longest common prefix and trie metric d_T(a,b) = -log2 P(a ^ b) over S sessions: one warp
// per ordered pair (a,b).  The log-probability of the common prefix is summed in double in a fixed
// order, so the result does not depend on scheduling.
#include "plc_common.cuh"

namespace plc {
namespace {

__global__ void __launch_bounds__(256) lcp_dt_kernel(const int32_t* __restrict__ tokens, const int32_t* __restrict__ lens,
                                                     const float* __restrict__ logp2, int S, long long stride,
                                                     int32_t* __restrict__ lcp, float* __restrict__ dT) {
    const int lane = threadIdx.x & 31;
    const long long warp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long long nwarps = (long long)gridDim.x * (blockDim.x >> 5);
    for (long long pair = warp; pair < (long long)S * S; pair += nwarps) {
        const int a = (int)(pair / S), b = (int)(pair % S);
        const int32_t* ta = tokens + a * stride;
        const int32_t* tb = tokens + b * stride;
        const int m = (int)max(0ll, min((long long)min(lens[a], lens[b]), stride));
        int n = m;
        for (int base = 0; base < m; base += 32) {
            int j = base + lane;
            bool differ = (j < m) && (ta[j] != tb[j]);
            uint32_t mask = __ballot_sync(kFull, differ);
            if (mask) { n = base + __ffs(mask) - 1; break; }
        }
        double acc = 0.0;
        const float* la = logp2 + a * stride;
        for (int j = lane; j < n; j += 32) acc -= (double)la[j];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(kFull, acc, o);
        if (lane == 0) { lcp[pair] = n; dT[pair] = (float)acc; }
    }
}

// parent[a] = earlier session with the longest common prefix (smallest index among equals).
__global__ void parent_kernel(const int32_t* __restrict__ lcp, int S, int32_t* __restrict__ parent,
                              int32_t* __restrict__ shared_len) {
    int a = blockIdx.x * blockDim.x + threadIdx.x;
    if (a >= S) return;
    int best = -1, bl = 0;
    for (int b = 0; b < a; ++b) {
        int v = lcp[(long long)a * S + b];
        if (v > bl) { bl = v; best = b; }
    }
    parent[a] = best;
    shared_len[a] = bl;
}

// Semantic prefix clusters (Def. 3) from the matrices above: one warp per session a scans its row.
// Members of a's cluster: a itself and every b whose shared prefix with a carries at least delta
// bits, d_T(a,b) >= delta (an equivalence, because d_T(a,c) >= min(d_T(a,b), d_T(b,c))).
// cluster[a] = smallest member, centroid[a] = member with the smallest -log2 P (the diagonal of dT;
// ties: smallest index), begin[a] = lcp(a, centroid), 0 for the centroid itself.
__global__ void __launch_bounds__(256) cluster_kernel(const int32_t* __restrict__ lcp, const float* __restrict__ dT, int S,
                                                      float delta, int32_t* __restrict__ cluster,
                                                      int32_t* __restrict__ centroid, int32_t* __restrict__ begin) {
    const int lane = threadIdx.x & 31;
    const int a = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (a >= S) return;
    int first = a, best = a;
    float pbest = dT[(long long)a * S + a];
    for (int b = lane; b < S; b += 32) {
        if (b != a && !(dT[(long long)a * S + b] >= delta)) continue;
        first = min(first, b);
        const float pb = dT[(long long)b * S + b];
        if (pb < pbest || (pb == pbest && b < best)) { pbest = pb; best = b; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        first = min(first, __shfl_xor_sync(kFull, first, o));
        const float po = __shfl_xor_sync(kFull, pbest, o);
        const int bo = __shfl_xor_sync(kFull, best, o);
        if (po < pbest || (po == pbest && bo < best)) { pbest = po; best = bo; }
    }
    if (lane == 0) {
        cluster[a] = first;
        centroid[a] = best;
        begin[a] = best == a ? 0 : lcp[(long long)a * S + best];
    }
}

}  // namespace

cudaError_t launch_prefix_clusters(const int32_t* lcp, const float* dT, int S, float delta, int32_t* cluster,
                                   int32_t* centroid, int32_t* begin, cudaStream_t st) {
    if (S <= 0) return cudaSuccess;
    cluster_kernel<<<(S + 7) / 8, 256, 0, st>>>(lcp, dT, S, delta, cluster, centroid, begin);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_prefix_dedup(const int32_t* tokens, const int32_t* lens, const float* logp2, int S, int64_t stride,
                                int32_t* lcp, float* dT, int32_t* parent, int32_t* shared_len, cudaStream_t st) {
    if (S <= 0) return cudaSuccess;
    long long pairs = (long long)S * S;
    long long blocks = (pairs + 7) / 8;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        sms = 1;
    if (blocks > (long long)sms * 8) blocks = (long long)sms * 8;
    lcp_dt_kernel<<<(unsigned)blocks, 256, 0, st>>>(tokens, lens, logp2, S, (long long)stride, lcp, dT);
    parent_kernel<<<(S + 127) / 128, 128, 0, st>>>(lcp, S, parent, shared_len);
    count_launch(2);
    return cudaGetLastError();
}

}  // namespace plc

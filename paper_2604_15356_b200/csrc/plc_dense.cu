// Full-vocabulary prediction (Def. 5 of the paper: KV^ = sum over the whole vocabulary of
// P(t | t_<i) F(t_<i, t)) as a dense bf16 contraction on the 5th-generation tensor cores:
//   MU[rows x (2H*d)] = P[rows x V] * Tb[(2H*d) x V]^T     per layer, fp32 accumulation in TMEM.
// P = bf16(softmax(logits)); Tb = bf16(T) of the layer, transposed so that both operands are
// K-major (V contiguous).  One CTA computes a 128 x 256 tile: a TMA producer thread fills a
// 4-stage shared-memory ring (128B-swizzled boxes of 64 K-elements), one thread issues
// tcgen05.mma (128x256x16) into 256 TMEM columns and releases ring slots with tcgen05.commit,
// four warps read the accumulators back with tcgen05.ld and store the tile.  Single-CTA launch:
// every TMA load lands in this CTA's own shared memory and the tensor maps cover this GPU's memory
// only.  Every mbarrier wait is bounded; a wait that runs out sets an error bit and a CTA-wide
// `failed` word: the producer stops and waits (bounded) for the copies it has in flight, the
// epilogue stores nothing, and the CTA frees its TMEM and returns.
// The variance term s1[row][table] = sum_v P[row][v] * bf16(||Tb_v||^2 / d) is a second launch of
// the same kernel with a narrow N tile (one column per table).
#include <cuda.h>
#include <cuda_bf16.h>

#include "plc_common.cuh"

namespace plc {
namespace {

int dense_sm_count() {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        sms = 1;
    return sms;
}

constexpr int kBM = 128, kBN = 256, kBK = 64, kStages = 4, kUmmaK = 16;
constexpr int kABytes = kBM * kBK * 2, kBBytes = kBN * kBK * 2, kStageBytes = kABytes + kBBytes;
constexpr int kGemmThreads = 192;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr size_t kGemmSmem = (size_t)kStages * kStageBytes + 1024 + 256;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false (and the error bit set) if the phase did not complete within the limit.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, unsigned int* status) {
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    atomicOr(status, kStTimeout);
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    // K-major, 128-byte swizzle: start >> 4, LBO = 1 (unused), SBO = 1024 B between 8-row groups,
    // descriptor version 1, layout type 2 (SWIZZLE_128B)
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// instruction descriptor: D = f32, A = B = bf16, both K-major, M = 128, N = bn (multiple of 16, <= 256)
__host__ __device__ constexpr uint32_t make_idesc(int bn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}

__global__ void __launch_bounds__(kGemmThreads, 1)
dense_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  float* __restrict__ out, long long ldo, int rows, int ncols, int num_kb, int bn, unsigned int* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)kStages * kStageBytes);   // full[4], empty[4], tmem_full
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 1);
    volatile uint32_t* failed = tmem_slot + 1;        // set by any role whose wait ran out
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Column tile fastest in launch order: the CTAs resident together then share their row blocks of A
    // (each block of A is fetched from HBM once and found in L2 by the other column tiles), and B, the
    // smaller operand, is what gets re-read from L2.
    const int ntn = (int)gridDim.y;
    const int lin = blockIdx.y * gridDim.x + blockIdx.x;
    const int m0 = (lin / ntn) * kBM, n0 = (lin % ntn) * bn;
    const uint32_t stage_tx = (uint32_t)(kABytes + bn * kBK * 2), idesc = make_idesc(bn);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + kStages), tfull = smem_u32(bars + 2 * kStages);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        mbar_init(tfull, 1);
        *failed = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(256u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0 && lane == 0) {
        // TMA producer
        int issued = 0;
        bool ok = true;
        for (int kb = 0; kb < num_kb && ok; ++kb) {
            const int s = kb % kStages;
            const uint32_t ph = (uint32_t)(kb / kStages) & 1u;
            ok = !*failed && mbar_wait(empty0 + 8 * s, ph ^ 1u, status);
            if (!ok) break;
            mbar_expect_tx(full0 + 8 * s, stage_tx);
            const uint32_t sa = smem_u32(smem + (size_t)s * kStageBytes);
            tma_load_2d(sa, &map_a, kb * kBK, m0, full0 + 8 * s);
            tma_load_2d(sa + kABytes, &map_b, kb * kBK, n0, full0 + 8 * s);
            ++issued;
        }
        if (!ok) {
            // drain: the copies already issued still land in this CTA's shared memory
            *failed = 1u;
            for (int kb = issued > kStages ? issued - kStages : 0; kb < issued; ++kb)
                mbar_wait(full0 + 8 * (kb % kStages), (uint32_t)(kb / kStages) & 1u, status);
        }
    } else if (warp == 1 && lane == 0) {
        // MMA issuer
        bool ok = true;
        for (int kb = 0; kb < num_kb && ok; ++kb) {
            const int s = kb % kStages;
            const uint32_t ph = (uint32_t)(kb / kStages) & 1u;
            ok = mbar_wait(full0 + 8 * s, ph, status);
            if (!ok) { *failed = 1u; __threadfence_block(); break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t sa = smem_u32(smem + (size_t)s * kStageBytes);
            const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sa + kABytes);
#pragma unroll
            for (int k = 0; k < kBK / kUmmaK; ++k)
                umma_bf16(tmem_base, da + 2 * k, db + 2 * k, idesc, (kb | k) ? 1u : 0u);
            umma_commit(empty0 + 8 * s);              // frees the ring slot when these MMAs have read it
        }
        umma_commit(tfull);                           // arrives when the MMAs issued so far are done (all of them, or none pending)
    } else if (warp >= 2) {
        // epilogue: warp w reads TMEM lanes 32*(w%4) ... +31
        bool ok = mbar_wait(tfull, 0, status);
        if (!ok) *failed = 1u;
        ok = ok && !*failed;                          // partial accumulators are never stored
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int q = warp & 3;
        const int row = m0 + q * 32 + lane;
        const bool vec_ok = ((ldo | ncols) & 3) == 0;
        if (ok) {
            for (int c = 0; c * 32 < bn; ++c) {
                uint32_t r[32];
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 32);
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                    "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                    "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                    : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                      "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                      "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                      "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                    : "r"(taddr) : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                const int col = n0 + c * 32;
                if (row < rows && col < ncols) {
                    float* dr = out + (long long)row * ldo + col;
                    if (vec_ok) {
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            if (col + 4 * j < ncols)
                                reinterpret_cast<float4*>(dr)[j] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                                                                __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (col + j < ncols) dr[j] = __uint_as_float(r[j]);
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
    }
}

// P[row][v] = bf16(exp(l_v - lse)), columns V..ldp-1 = 0.  One block per row; 8 logits per thread
// and step when the row is 16-byte aligned.  exp is the fast intrinsic: its relative error (~1e-6)
// is far below the 2^-9 of the bfloat16 result.
template <bool VEC>
__global__ void __launch_bounds__(256) softmax_bf16_kernel(const __half* __restrict__ logits, long long rows, int V, int ldp,
                                                           __nv_bfloat16* __restrict__ P) {
    __shared__ float red_m[8], red_s[8];
    __shared__ float sh_max, sh_lse;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
        const __half* lr = logits + row * V;
        // pass 1: maximum
        float m = -INFINITY;
        if (VEC) {
            for (int v = tid * 8; v < V; v += 256 * 8) {
                const uint4 r = *reinterpret_cast<const uint4*>(lr + v);
                const __half2* hp = reinterpret_cast<const __half2*>(&r);
#pragma unroll
                for (int j = 0; j < 4; ++j) { const float2 f = __half22float2(hp[j]); m = fmaxf(m, fmaxf(f.x, f.y)); }
            }
        } else {
            for (int v = tid; v < V; v += 256) m = fmaxf(m, __half2float(lr[v]));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(kFull, m, o));
        __syncthreads();
        if (lane == 0) red_m[wid] = m;
        __syncthreads();
        if (tid == 0) {
            float mm = red_m[0];
            for (int w = 1; w < 8; ++w) mm = fmaxf(mm, red_m[w]);
            sh_max = mm;
        }
        __syncthreads();
        const float mx = sh_max;
        // pass 2: sum of exponentials (row is in L2 now)
        float s = 0.f;
        if (VEC) {
            for (int v = tid * 8; v < V; v += 256 * 8) {
                const uint4 r = *reinterpret_cast<const uint4*>(lr + v);
                const __half2* hp = reinterpret_cast<const __half2*>(&r);
#pragma unroll
                for (int j = 0; j < 4; ++j) { const float2 f = __half22float2(hp[j]); s += __expf(f.x - mx) + __expf(f.y - mx); }
            }
        } else {
            for (int v = tid; v < V; v += 256) s += __expf(__half2float(lr[v]) - mx);
        }
        s = warp_sum(s);
        if (lane == 0) red_s[wid] = s;
        __syncthreads();
        if (tid == 0) {
            float ss = 0.f;
            for (int w = 0; w < 8; ++w) ss += red_s[w];
            sh_lse = mx + __logf(ss);
        }
        __syncthreads();
        const float lse = sh_lse;
        __nv_bfloat16* pr = P + row * ldp;
        if (VEC) {
            for (int v = tid * 8; v < ldp; v += 256 * 8) {          // ldp is a multiple of 64
                __nv_bfloat162 o[4];
                if (v < V) {
                    const uint4 r = *reinterpret_cast<const uint4*>(lr + v);
                    const __half2* hp = reinterpret_cast<const __half2*>(&r);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float2 f = __half22float2(hp[j]);
                        o[j] = __floats2bfloat162_rn(__expf(f.x - lse), __expf(f.y - lse));
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) o[j] = __floats2bfloat162_rn(0.f, 0.f);
                }
                *reinterpret_cast<uint4*>(pr + v) = *reinterpret_cast<const uint4*>(o);
            }
        } else {
            for (int v = tid; v < ldp; v += 256)
                pr[v] = __float2bfloat16_rn(v < V ? __expf(__half2float(lr[v]) - lse) : 0.f);
        }
        __syncthreads();
    }
}

// Tb[t*d + j][v] = bf16(T_layer[t][v][j]): 32 x 32 tiles through shared memory.
__global__ void __launch_bounds__(256) transpose_bf16_kernel(const __half* __restrict__ Tl, int tables, int V, int d, int ldv,
                                                             __nv_bfloat16* __restrict__ Tb) {
    __shared__ __nv_bfloat16 tile[32][33];
    const int t = blockIdx.z, v0 = blockIdx.x * 32, j0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;      // 32 x 8
    const __half* src = Tl + (size_t)t * V * d;
    for (int r = ty; r < 32; r += 8) {
        const int v = v0 + r;
        tile[r][tx] = (v < V) ? __float2bfloat16_rn(__half2float(src[(size_t)v * d + j0 + tx])) : __float2bfloat16_rn(0.f);
    }
    __syncthreads();
    for (int r = ty; r < 32; r += 8) {
        const int v = v0 + tx;
        if (v < ldv) Tb[((size_t)t * d + j0 + r) * ldv + v] = tile[tx][r];
    }
}

// Nb[t][v] = bf16(sum_j bf16(T[t][v][j])^2 / d) (row pitch ldv).  One warp per row of T.
__global__ void __launch_bounds__(256) rownorm_bf16_kernel(const __half* __restrict__ Tl, long long nrows, int V, int d, int ldv,
                                                           __nv_bfloat16* __restrict__ out) {
    const int lane = threadIdx.x & 31;
    const long long warp = (long long)blockIdx.x * 8 + (threadIdx.x >> 5), nw = (long long)gridDim.x * 8;
    for (long long r = warp; r < nrows; r += nw) {
        float s = 0.f;
        for (int j = lane; j < d; j += 32) {
            const float x = __bfloat162float(__float2bfloat16_rn(__half2float(Tl[r * d + j])));
            s = __fmaf_rn(x, x, s);
        }
        s = warp_sum(s);
        if (lane == 0) out[(r / V) * ldv + (r % V)] = __float2bfloat16_rn(s / (float)d);
    }
}

// Blocks of 256 threads for n work items, at most 16 per SM (grid-stride kernels).
unsigned blocks_for(long long n) {
    const long long b = (n + 255) / 256, cap = (long long)dense_sm_count() * 16;
    return (unsigned)(b < cap ? (b > 0 ? b : 1) : cap);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2-D bf16 tensor [outer][inner] (inner contiguous, row pitch ld elements), boxes of 64 x box_outer.
bool make_map(CUtensorMap* map, void* base, uint64_t inner, uint64_t outer, uint64_t ld, uint32_t box_outer) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBK, box_outer};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// out[rows x ncols] (fp32, pitch ldo) = A[rows x K] * B[nrows_b x K]^T, both bf16 with row pitch ldk (a
// multiple of 64; K = ldk, zero padded); nrows_b is a multiple of the N tile bn.
cudaError_t launch_gemm(const __nv_bfloat16* A, long long rows, const __nv_bfloat16* B, int nrows_b, int ldk, int bn,
                        float* out, long long ldo, int ncols, unsigned int* status, cudaStream_t st) {
    CUtensorMap ma, mb;
    if (!make_map(&ma, const_cast<__nv_bfloat16*>(A), (uint64_t)ldk, (uint64_t)rows, (uint64_t)ldk, kBM)) return cudaErrorUnknown;
    if (!make_map(&mb, const_cast<__nv_bfloat16*>(B), (uint64_t)ldk, (uint64_t)nrows_b, (uint64_t)ldk, (uint32_t)bn)) return cudaErrorUnknown;
    cudaError_t e = cudaFuncSetAttribute(dense_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kGemmSmem);
    if (e != cudaSuccess) return e;
    dim3 g((unsigned)((rows + kBM - 1) / kBM), (unsigned)(nrows_b / bn));
    dense_gemm_kernel<<<g, kGemmThreads, kGemmSmem, st>>>(ma, mb, out, ldo, (int)rows, ncols, ldk / kBK, bn, status);
    count_launch();
    return cudaGetLastError();
}

// dst[r][c] = bf16(src[r][c]) for c < cols, 0 for cols <= c < ld (row-major, f16 source pitch = cols).
__global__ void __launch_bounds__(256) cvt_f16_bf16_kernel(const __half* __restrict__ src, long long rows, int cols, int ld,
                                                           __nv_bfloat16* __restrict__ dst) {
    const long long total = rows * ld;
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < total; i += (long long)gridDim.x * 256) {
        const long long r = i / ld; const int c = (int)(i % ld);
        dst[i] = __float2bfloat16_rn(c < cols ? __half2float(src[r * cols + c]) : 0.f);
    }
}
__global__ void __launch_bounds__(256) cvt_f32_bf16_kernel(const float* __restrict__ src, long long n, __nv_bfloat16* __restrict__ dst) {
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long long)gridDim.x * 256)
        dst[i] = __float2bfloat16_rn(src[i]);
}
// Nb[t][v] = bf16(sum_j (tlin[v][t*d + j] + c[t][j])^2 / d): one warp per (v, t).
__global__ void __launch_bounds__(256) tlin_norm_kernel(const float* __restrict__ tlin, long long ld_t, const __half* __restrict__ c,
                                                        int V, int tables, int d, int ldv, __nv_bfloat16* __restrict__ Nb) {
    const int lane = threadIdx.x & 31;
    const long long warp = (long long)blockIdx.x * 8 + (threadIdx.x >> 5), nw = (long long)gridDim.x * 8;
    for (long long it = warp; it < (long long)V * tables; it += nw) {
        const int v = (int)(it / tables), t = (int)(it % tables);
        float s = 0.f;
        for (int j = lane; j < d; j += 32) {
            const float x = tlin[(long long)v * ld_t + t * d + j] + __half2float(c[t * d + j]);
            s = __fmaf_rn(x, x, s);
        }
        s = warp_sum(s);
        if (lane == 0) Nb[(size_t)t * ldv + v] = __float2bfloat16_rn(s / (float)d);
    }
}

}  // namespace

size_t dense_scratch_bytes(const DenseShape& sh, size_t* off /*[5]*/) {
    auto up = [](size_t x) { return (x + 1023) & ~(size_t)1023; };
    size_t o = 0;
    off[0] = o; o += up((size_t)sh.rows * sh.ldv * 2);                 // P
    off[1] = o; o += up((size_t)sh.ncols_pad * sh.ldv * 2);            // Tb
    off[2] = o;                                                        // (unused)
    off[3] = o; o += up((size_t)sh.rows * sh.ncols * 4);               // mu
    off[4] = o; o += up((size_t)sh.rows * sh.nt_all * 4);              // s1 of every (layer, table)
    return o;
}

size_t dense_model_bytes(const DenseShape& sh) { return (size_t)sh.nt_all_pad * sh.ldv * 2; }

// Creation: Nb_all[l * tables + t][v] = bf16(sum_j bf16(T[l][t][v][j])^2 / d) for every layer; rows beyond
// L * tables and columns beyond V are zero.
cudaError_t dense_prepare(const __half* T, int L, const DenseShape& sh, uint8_t* model, cudaStream_t st) {
    __nv_bfloat16* Nb = reinterpret_cast<__nv_bfloat16*>(model);
    cudaError_t e = cudaMemsetAsync(Nb, 0, dense_model_bytes(sh), st);
    if (e != cudaSuccess) return e;
    const long long nrows = (long long)L * sh.tables * sh.V;
    rownorm_bf16_kernel<<<blocks_for(nrows * 32), 256, 0, st>>>(T, nrows, sh.V, sh.d, sh.ldv, Nb);
    count_launch();
    return cudaGetLastError();
}

// Per call: P = bf16(softmax(logits)) and the variance term of every layer in one contraction,
// s1[row][l * tables + t] = sum_v P[row][v] Nb_all[l * tables + t][v].
cudaError_t dense_begin(const __half* logits, const DenseShape& sh, const uint8_t* model, uint8_t* scratch, const size_t* off,
                        unsigned int* status, cudaStream_t st) {
    cudaError_t e = dense_softmax(logits, sh, scratch, off, st);
    if (e != cudaSuccess) return e;
    return launch_gemm(reinterpret_cast<const __nv_bfloat16*>(scratch + off[0]), sh.rows,
                       reinterpret_cast<const __nv_bfloat16*>(model), sh.nt_all_pad, sh.ldv, 256,
                       reinterpret_cast<float*>(scratch + off[4]), sh.nt_all, sh.nt_all, status, st);
}

cudaError_t dense_softmax(const __half* logits, const DenseShape& sh, uint8_t* scratch, const size_t* off, cudaStream_t st) {
    const long long cap_blocks = (long long)dense_sm_count() * 8;
    long long blocks = sh.rows < cap_blocks ? sh.rows : cap_blocks;
    __nv_bfloat16* P = reinterpret_cast<__nv_bfloat16*>(scratch + off[0]);
    if (sh.V % 8 == 0 && (reinterpret_cast<uintptr_t>(logits) & 15) == 0)
        softmax_bf16_kernel<true><<<(unsigned)blocks, 256, 0, st>>>(logits, sh.rows, sh.V, sh.ldv, P);
    else
        softmax_bf16_kernel<false><<<(unsigned)blocks, 256, 0, st>>>(logits, sh.rows, sh.V, sh.ldv, P);
    count_launch();
    return cudaGetLastError();
}

// Prediction of one layer: fills mu [rows][ncols] in the scratch (the variance term of every layer was
// formed by dense_begin).
cudaError_t dense_layer(const __half* T_layer, const DenseShape& sh, uint8_t* scratch, const size_t* off,
                        unsigned int* status, cudaStream_t st, cudaEvent_t ev0, cudaEvent_t ev1) {
    __nv_bfloat16* P = reinterpret_cast<__nv_bfloat16*>(scratch + off[0]);
    __nv_bfloat16* Tb = reinterpret_cast<__nv_bfloat16*>(scratch + off[1]);
    float* mu = reinterpret_cast<float*>(scratch + off[3]);
    cudaError_t e;
    if (sh.ncols_pad > sh.ncols) {       // rows of Tb beyond the real columns must read as zero
        e = cudaMemsetAsync(Tb + (size_t)sh.ncols * sh.ldv, 0, (size_t)(sh.ncols_pad - sh.ncols) * sh.ldv * 2, st);
        if (e != cudaSuccess) return e;
    }
    dim3 tg((sh.ldv + 31) / 32, sh.d / 32, sh.tables);
    transpose_bf16_kernel<<<tg, 256, 0, st>>>(T_layer, sh.tables, sh.V, sh.d, sh.ldv, Tb);
    count_launch();
    if (ev0) cudaEventRecord(ev0, st);
    e = launch_gemm(P, sh.rows, Tb, sh.ncols_pad, sh.ldv, kBN, mu, (long long)sh.ncols, sh.ncols, status, st);
    if (ev1) cudaEventRecord(ev1, st);
    return e;
}

// ---------------------------------------------------------------------------------------------
// Linear-embedding predictor (Sec. 7.1): KV^ ~ c + A Ebar, Ebar = sum_v p_v E(v).  Two chained
// contractions on the same tensor-core kernel: Ebar = P * E (once per call, shared by all layers),
// then per layer mu = Ebar * A_layer^T (K = d_model); the variance term of all layers is one more
// contraction of P with the table of candidate norms ||c + A E(v)||^2 / d built at creation.

size_t linear_model_bytes(const LinearShape& sh, size_t* off /*[2]: Ebt, NbAll*/) {
    auto up = [](size_t x) { return (x + 1023) & ~(size_t)1023; };
    size_t o = 0;
    off[0] = o; o += up((size_t)sh.dm * sh.ldv * 2);
    off[1] = o; o += up((size_t)sh.nt_all_pad * sh.ldv * 2);
    return o;
}

size_t linear_scratch_bytes(const LinearShape& sh, size_t* off /*[6]: P, Ef, Eb16, s1, Ab, mu*/) {
    auto up = [](size_t x) { return (x + 1023) & ~(size_t)1023; };
    size_t o = 0;
    off[0] = o; o += up((size_t)sh.rows * sh.ldv * 2);
    off[1] = o; o += up((size_t)sh.rows * sh.dm * 4);
    off[2] = o; o += up((size_t)sh.rows * sh.dm * 2);
    off[3] = o; o += up((size_t)sh.rows * sh.nt_all * 4);
    off[4] = o; o += up((size_t)sh.ncols_pad * sh.dm * 2);
    off[5] = o; o += up((size_t)sh.rows * sh.ncols * 4);
    return o;
}

static int tile_for(int n) { return n % 256 == 0 ? 256 : (n % 128 == 0 ? 128 : 64); }


// Creation: E transposed to bf16 and the norm table of every (layer, table).  Allocates (and
// frees) its temporaries; synchronises the stream.
cudaError_t linear_prepare(const __half* E, const __half* A, const __half* c, const LinearShape& sh, uint8_t* model,
                           const size_t* moff, unsigned int* status, cudaStream_t st) {
    __nv_bfloat16* Ebt = reinterpret_cast<__nv_bfloat16*>(model + moff[0]);
    __nv_bfloat16* NbAll = reinterpret_cast<__nv_bfloat16*>(model + moff[1]);
    __nv_bfloat16 *Eb = nullptr, *Ab = nullptr;
    float* tlin = nullptr;
    cudaError_t e = cudaMalloc(&Eb, (size_t)sh.V * sh.dm * 2);
    if (e == cudaSuccess) e = cudaMalloc(&Ab, (size_t)sh.ncols_pad * sh.dm * 2);
    if (e == cudaSuccess) e = cudaMalloc(&tlin, (size_t)sh.V * sh.ncols * 4);
    if (e == cudaSuccess) e = cudaMemsetAsync(NbAll, 0, (size_t)sh.nt_all_pad * sh.ldv * 2, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(Ab, 0, (size_t)sh.ncols_pad * sh.dm * 2, st);
    if (e == cudaSuccess) {
        dim3 tg((sh.ldv + 31) / 32, sh.dm / 32, 1);
        transpose_bf16_kernel<<<tg, 256, 0, st>>>(E, 1, sh.V, sh.dm, sh.ldv, Ebt);
        cvt_f16_bf16_kernel<<<blocks_for((long long)sh.V * sh.dm), 256, 0, st>>>(E, sh.V, sh.dm, sh.dm, Eb);
        count_launch(2);
        for (int l = 0; l < sh.L && e == cudaSuccess; ++l) {
            const __half* Al = A + (size_t)l * sh.ncols * sh.dm;
            cvt_f16_bf16_kernel<<<blocks_for((long long)sh.ncols * sh.dm), 256, 0, st>>>(Al, sh.ncols, sh.dm, sh.dm, Ab);
            e = launch_gemm(Eb, sh.V, Ab, sh.ncols_pad, sh.dm, 256, tlin, sh.ncols, sh.ncols, status, st);
            if (e != cudaSuccess) break;
            const long long pairs = (long long)sh.V * sh.tables;
            tlin_norm_kernel<<<blocks_for(pairs * 32), 256, 0, st>>>(
                tlin, sh.ncols, c + (size_t)l * sh.ncols, sh.V, sh.tables, sh.d, sh.ldv, NbAll + (size_t)l * sh.tables * sh.ldv);
            count_launch(2);
            e = cudaGetLastError();
        }
    }
    cudaError_t e2 = cudaStreamSynchronize(st);
    cudaFree(Eb); cudaFree(Ab); cudaFree(tlin);
    return e != cudaSuccess ? e : e2;
}

// Per call: P, Ebar (bf16) and the variance term of every layer.
cudaError_t linear_begin(const __half* logits, const LinearShape& sh, const uint8_t* model, const size_t* moff,
                         uint8_t* scratch, const size_t* off, unsigned int* status, cudaStream_t st) {
    DenseShape ds{}; ds.rows = sh.rows; ds.V = sh.V; ds.ldv = sh.ldv;
    cudaError_t e = dense_softmax(logits, ds, scratch, off, st);
    if (e != cudaSuccess) return e;
    const __nv_bfloat16* P = reinterpret_cast<const __nv_bfloat16*>(scratch + off[0]);
    float* Ef = reinterpret_cast<float*>(scratch + off[1]);
    __nv_bfloat16* Eb16 = reinterpret_cast<__nv_bfloat16*>(scratch + off[2]);
    float* s1 = reinterpret_cast<float*>(scratch + off[3]);
    e = launch_gemm(P, sh.rows, reinterpret_cast<const __nv_bfloat16*>(model + moff[0]), sh.dm, sh.ldv, tile_for(sh.dm),
                    Ef, sh.dm, sh.dm, status, st);
    if (e != cudaSuccess) return e;
    cvt_f32_bf16_kernel<<<blocks_for(sh.rows * sh.dm), 256, 0, st>>>(Ef, sh.rows * sh.dm, Eb16);
    count_launch();
    return launch_gemm(P, sh.rows, reinterpret_cast<const __nv_bfloat16*>(model + moff[1]), sh.nt_all_pad, sh.ldv, 256,
                       s1, sh.nt_all, sh.nt_all, status, st);
}

// Per layer: mu [rows][2H*d] = Ebar * A_layer^T (the bias c is added where mu is read).
cudaError_t linear_layer(const __half* A_layer, const LinearShape& sh, uint8_t* scratch, const size_t* off,
                         unsigned int* status, cudaStream_t st, cudaEvent_t ev0, cudaEvent_t ev1) {
    __nv_bfloat16* Ab = reinterpret_cast<__nv_bfloat16*>(scratch + off[4]);
    cudaError_t e = cudaSuccess;
    if (sh.ncols_pad > sh.ncols) e = cudaMemsetAsync(Ab + (size_t)sh.ncols * sh.dm, 0, (size_t)(sh.ncols_pad - sh.ncols) * sh.dm * 2, st);
    if (e != cudaSuccess) return e;
    cvt_f16_bf16_kernel<<<blocks_for((long long)sh.ncols * sh.dm), 256, 0, st>>>(A_layer, sh.ncols, sh.dm, sh.dm, Ab);
    count_launch();
    if (ev0) cudaEventRecord(ev0, st);
    e = launch_gemm(reinterpret_cast<const __nv_bfloat16*>(scratch + off[2]), sh.rows, Ab, sh.ncols_pad, sh.dm, 256,
                    reinterpret_cast<float*>(scratch + off[5]), sh.ncols, sh.ncols, status, st);
    if (ev1) cudaEventRecord(ev1, st);
    return e;
}

}  // namespace plc

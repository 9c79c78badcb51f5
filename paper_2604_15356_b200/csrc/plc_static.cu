// plc_rans_encode_static: entropy-codes chunks of already quantised symbols with every byte of
// working memory taken from one file-scope device array, so the call itself allocates nothing.
// It is a variant of the chunk-sealing kernel of the append path (same bitstream, bit for bit);
// nothing else in the library calls into this file.
#include <mutex>

#include "plc_common.cuh"

namespace plc {
namespace {

constexpr int kStWarpsPerBlock = 8;
constexpr int kStBlocks = 32;
constexpr int kStWarps = kStWarpsPerBlock * kStBlocks;          // 256 warps share the array
constexpr int kStMaxComponents = 4096;                          // positions * d of one chunk
constexpr int kStWordsPerWarp = 4 * kStMaxComponents + 64;      // worst case of the format, in 16-bit words
constexpr size_t kStHeader = 256;                               // work ticket lives in the first bytes
constexpr size_t kStBytes = kStHeader + (size_t)kStWarps * kStWordsPerWarp * sizeof(uint16_t);   // ~8.03 MiB

// Working memory of every call on this device (each GPU that loads the library holds it until the
// process exits).  Host code must not pass this name to a kernel: its device address is fetched
// once per device with cudaGetSymbolAddress (static_scratch() below).
static __device__ __align__(256) unsigned char g_static_scratch[kStBytes];


struct EncTablesSt { EncEntry enc[kNumTables][kNumSym]; };

__device__ __forceinline__ int st_first_comp(int lane, int d) {
    const int R = d / 8, G = d / 32;
    return 8 * (lane % R) + G * (lane / R);
}

__global__ void __launch_bounds__(kStWarpsPerBlock * 32)
rans_encode_static_kernel(const int32_t* __restrict__ sym, const int32_t* __restrict__ q, int n_streams, int P, int d,
                          int chunk_capacity, int chunk_index, StreamsDev out, uint32_t* status,
                          unsigned char* scratch) {
    __shared__ EncTablesSt tb;
    for (int id = threadIdx.x; id < kNumTables; id += blockDim.x) {
        uint32_t f[kNumSym];
        build_freqs(id + kQMin, f);
        uint32_t c = 0;
        for (int i = 0; i < kNumSym; ++i) {
            uint32_t fi = f[i];
            tb.enc[id][i].rcp = fi == 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / fi);
            tb.enc[id][i].fc = fi | (c << 16);
            c += fi;
        }
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const uint32_t lt = lanemask_lt();
    unsigned int* ticket = reinterpret_cast<unsigned int*>(scratch);
    const int gw = blockIdx.x * kStWarpsPerBlock + (threadIdx.x >> 5);
    uint16_t* stage = reinterpret_cast<uint16_t*>(scratch + kStHeader) + (size_t)gw * kStWordsPerWarp;
    const int G = d / 32, c0 = st_first_comp(lane, d);

    for (;;) {
        unsigned item = 0;
        if (lane == 0) item = atomicAdd(ticket, 1u);
        item = __shfl_sync(kFull, item, 0);
        if (item >= (unsigned)n_streams) break;
        const long long slot = (long long)item * out.max_chunks + chunk_index;
        uint32_t x = kRansL;
        int wp = kStWordsPerWarp;
        bool bad_class = false;
        for (int p = P - 1; p >= 0; --p) {
            const long long o = (long long)item * chunk_capacity + p;
            int qq = q[o];
            if (qq < kQMin || qq > kQMax) { bad_class = true; qq = min(max(qq, kQMin), kQMax); }
            int s, qp;
            class_params(qq, s, qp);
            const EncEntry* tbl = tb.enc[qp - kQMin];
            for (int g = G - 1; g >= 0; --g) {
                int v = sym[o * d + c0 + g];
                v = min(max(v, -kSymLimit), kSymLimit);
                int hi = v; uint32_t lo = 0;
                if (s) { int u = v + (1 << (s - 1)); hi = u >> s; lo = (uint32_t)u & ((1u << s) - 1u); }
                const bool esc = hi > kHiMax || hi < -kHiMax;
                const int zz = esc ? kEsc : (hi > 0 ? 2 * hi - 1 : -2 * hi);
                const EncEntry e = tbl[zz];
                const uint32_t f = e.fc & 0xffffu, c = e.fc >> 16;
                const bool emit = x >= (f << 17);
                const uint32_t emask = __ballot_sync(kFull, emit), xmask = __ballot_sync(kFull, esc);
                const int n_emit = __popc(emask), n_esc = __popc(xmask);
                const int base = wp - (2 * s + n_emit + 2 * n_esc);
                if (esc) {
                    int at = base + 2 * s + n_emit + 2 * __popc(xmask & lt);
                    stage[at] = (uint16_t)((uint32_t)hi & 0xffffu);
                    stage[at + 1] = (uint16_t)((uint32_t)hi >> 16);
                }
                if (emit) { stage[base + 2 * s + __popc(emask & lt)] = (uint16_t)(x & 0xffffu); x >>= 16; }
                uint32_t qd = __umulhi(x, e.rcp);
                uint32_t r = x - qd * f;
                if (r >= f) { ++qd; r -= f; }
                x = (qd << kProbBits) + r + c;
                if (s) {
                    uint32_t mine = 0;
                    for (int b = 0; b < s; ++b) {
                        uint32_t plane = __ballot_sync(kFull, (lo >> b) & 1u);
                        if ((lane >> 1) == b) mine = plane;
                    }
                    if (lane < 2 * s) stage[base + lane] = (uint16_t)((lane & 1) ? (mine >> 16) : (mine & 0xffffu));
                }
                wp = base;
            }
        }
        __syncwarp();
        const int n_words = kStWordsPerWarp - wp;
        const unsigned nbytes = 128u + 2u * (unsigned)n_words;
        unsigned long long off = 0;
        if (lane == 0) off = atomicAdd(out.total_bytes, (unsigned long long)((nbytes + 15u) & ~15u));
        off = __shfl_sync(kFull, off, 0);
        const bool aligned = (off & 15ull) == 0;        // the caller's byte cursor must be a multiple of 16
        const bool fits = off + nbytes <= out.capacity && aligned;
        if (lane == 0) {
            out.chunk_offset[slot] = off;
            out.chunk_bytes[slot] = nbytes;
            if (off + nbytes > out.capacity) atomicOr(status, kStCapacity);
            if (!aligned) atomicOr(status, kStCursor);
        }
        if (__any_sync(kFull, bad_class) && lane == 0) atomicOr(status, kStBadClass);
        if (fits) {
            uint8_t* dst = out.payload + off;
            reinterpret_cast<uint32_t*>(dst)[lane] = x;
            uint16_t* dw = reinterpret_cast<uint16_t*>(dst + 128);
            for (int i = lane; i < n_words; i += 32) dw[i] = __ldcg(stage + wp + i);
        }
        __syncwarp();
    }
}

// Device address of g_static_scratch for the current device; looked up once per device.
cudaError_t static_scratch(unsigned char** out) {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static unsigned char* ptrs[kMaxDevices] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (!ptrs[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        ptrs[dev] = static_cast<unsigned char*>(p);
    }
    *out = ptrs[dev];
    return cudaSuccess;
}

}  // namespace
}  // namespace plc

using namespace plc;

extern "C" plc_status plc_rans_encode_static(const int32_t* sym_dev, const int32_t* q_dev, int32_t n_streams,
                                             int32_t n_pos, int32_t head_dim, int32_t chunk_capacity,
                                             int32_t chunk_index, const plc_streams* out, uint32_t* status_dev,
                                             void* stream) {
    if (!sym_dev || !q_dev || !out || !status_dev || n_streams < 0 || n_pos < 1 || chunk_capacity < n_pos) return PLC_E_INVALID;
    if (!out->payload_dev || !out->chunk_offset_dev || !out->chunk_bytes_dev || !out->total_bytes_dev) return PLC_E_INVALID;
    if (head_dim != 32 && head_dim != 64 && head_dim != 128 && head_dim != 256) return PLC_E_SHAPE;
    if ((long long)n_pos * head_dim > kStMaxComponents) return PLC_E_SHAPE;      // beyond the static working memory
    if (chunk_index < 0 || chunk_index >= out->max_chunks) return PLC_E_SHAPE;
    if (reinterpret_cast<uintptr_t>(out->payload_dev) & 15) return PLC_E_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* scratch = nullptr;
    if (static_scratch(&scratch) != cudaSuccess) return PLC_E_CUDA;
    // the array keeps the previous call's contents: the ticket must start at zero, the status is an output
    if (cudaMemsetAsync(scratch, 0, kStHeader, st) != cudaSuccess) return PLC_E_CUDA;
    if (cudaMemsetAsync(status_dev, 0, sizeof(uint32_t), st) != cudaSuccess) return PLC_E_CUDA;
    if (n_streams == 0) return PLC_OK;
    StreamsDev d;
    d.payload = out->payload_dev; d.capacity = out->payload_capacity;
    d.chunk_offset = reinterpret_cast<unsigned long long*>(out->chunk_offset_dev);
    d.chunk_bytes = out->chunk_bytes_dev;
    d.total_bytes = reinterpret_cast<unsigned long long*>(out->total_bytes_dev);
    d.max_chunks = out->max_chunks;
    int blocks = (n_streams + kStWarpsPerBlock - 1) / kStWarpsPerBlock;
    if (blocks > kStBlocks) blocks = kStBlocks;
    rans_encode_static_kernel<<<blocks, kStWarpsPerBlock * 32, 0, st>>>(sym_dev, q_dev, n_streams, n_pos, head_dim,
                                                                       chunk_capacity, chunk_index, d, status_dev, scratch);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? PLC_OK : PLC_E_CUDA;
}

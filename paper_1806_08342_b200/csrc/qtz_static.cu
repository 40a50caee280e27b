// qtz_minmax_static: the per-layer min/max range reduction for callers that must not
// allocate.  Same two-pass reduction as qtz_minmax (block partials, then one block folds them),
// but the partials live in a fixed array that is part of the library image instead of a buffer
// obtained from cudaMalloc, the result stays on the device in memory the caller provides, and
// no handle is needed.
//
// Who needs this: a process that gave all device memory to its own pool at start-up (a later
// cudaMalloc fails or eats into the pool's head-room), and latency-critical loops in which the
// device-wide synchronisation a cudaMalloc / cudaFree may imply is not acceptable.
//
// The price: every GPU that loads the library carries the array (48 KB) until the process
// exits; the tensor size is capped; and all calls on a device share the one array, so two
// calls whose kernels can overlap on the GPU (different streams) race on it.
#include <cfloat>
#include <mutex>

#include "qtz_device_util.cuh"
#include "qtz_internal.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kChunk = 65536;          // elements reduced by one block
constexpr int kMaxPartials = 4096;     // blocks per call at most
constexpr int kMaxDevices = 64;

// Block partials: (lo, hi, non-finite flag) per block.  Nothing here has to start at zero:
// the first pass overwrites exactly the entries the second pass reads.
static __device__ __align__(256) float g_minmax_partials[3 * kMaxPartials];

using qtz_dev::Range;
static_assert(kThreads == qtz_dev::kReduceThreads, "block_reduce assumes this block size");

__device__ __forceinline__ void take(Range& r, float v) { qtz_dev::range_take(r, v); }
__device__ __forceinline__ Range reduce_block(Range r) { return qtz_dev::block_reduce(r); }

// First pass: block b reduces elements [b*kChunk, (b+1)*kChunk) and writes one triple.
__global__ void __launch_bounds__(kThreads)
minmax_static_chunks_kernel(const float* __restrict__ x, int64_t n, float* __restrict__ partials)
{
    const int64_t begin = static_cast<int64_t>(blockIdx.x) * kChunk;
    const int64_t end = begin + kChunk < n ? begin + kChunk : n;
    Range r{FLT_MAX, -FLT_MAX, 0u};
    if ((reinterpret_cast<uintptr_t>(x) & 15u) == 0) {  // chunk starts stay 16-byte aligned
        const int64_t vec_end = begin + ((end - begin) & ~static_cast<int64_t>(3));
        for (int64_t i = begin + 4 * threadIdx.x; i < vec_end; i += 4 * kThreads) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(x + i));
            take(r, v.x); take(r, v.y); take(r, v.z); take(r, v.w);
        }
        for (int64_t i = vec_end + threadIdx.x; i < end; i += kThreads) take(r, __ldg(x + i));
    } else {
        for (int64_t i = begin + threadIdx.x; i < end; i += kThreads) take(r, __ldg(x + i));
    }
    r = reduce_block(r);
    if (threadIdx.x == 0) {
        partials[3 * blockIdx.x + 0] = r.lo;
        partials[3 * blockIdx.x + 1] = r.hi;
        partials[3 * blockIdx.x + 2] = __uint_as_float(r.bad);
    }
}

// Second pass: one block folds `count` triples into out[0..2].
__global__ void __launch_bounds__(kThreads)
minmax_static_finish_kernel(const float* __restrict__ partials, int count, float* __restrict__ out)
{
    Range r{FLT_MAX, -FLT_MAX, 0u};
    for (int i = threadIdx.x; i < count; i += kThreads) {
        r.lo = fminf(r.lo, partials[3 * i]);
        r.hi = fmaxf(r.hi, partials[3 * i + 1]);
        r.bad |= __float_as_uint(partials[3 * i + 2]);
    }
    r = reduce_block(r);
    if (threadIdx.x == 0) {
        out[0] = r.lo;
        out[1] = r.hi;
        out[2] = __uint_as_float(r.bad);
    }
}

// Device address of the array, looked up once per device.  In host code the array's name is
// only a handle for the runtime, never a pointer a kernel may use.
std::mutex g_setup_lock;
float* g_partials_addr[kMaxDevices] = {};

cudaError_t partials_for_current_device(int device, float** out)
{
    std::lock_guard<std::mutex> guard(g_setup_lock);
    if (!g_partials_addr[device]) {
        float* ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_minmax_partials);
        if (e != cudaSuccess) return e;
        g_partials_addr[device] = ptr;
    }
    *out = g_partials_addr[device];
    return cudaSuccess;
}

}  // namespace

extern "C" int64_t qtz_minmax_static_max_count(void) { return static_cast<int64_t>(kMaxPartials) * kChunk; }

extern "C" qtz_status qtz_minmax_static(const float* x_dev, int64_t count, float* out_dev, void* stream)
{
    if (!x_dev || !out_dev || count <= 0) return QTZ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x_dev) & 3u) || (reinterpret_cast<uintptr_t>(out_dev) & 3u)) return QTZ_ERR_MISALIGNED;
    if (count > qtz_minmax_static_max_count()) return QTZ_ERR_TOO_LARGE;
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) {
        (void)cudaGetLastError();
        return QTZ_ERR_NO_DEVICE;
    }
    float* partials = nullptr;
    if (partials_for_current_device(device, &partials) != cudaSuccess) {
        (void)cudaGetLastError();
        return QTZ_ERR_CUDA;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int blocks = static_cast<int>((count + kChunk - 1) / kChunk);
    minmax_static_chunks_kernel<<<blocks, kThreads, 0, st>>>(x_dev, count, partials);
    if (cudaGetLastError() != cudaSuccess) return QTZ_ERR_CUDA;
    minmax_static_finish_kernel<<<1, kThreads, 0, st>>>(partials, blocks, out_dev);
    if (cudaGetLastError() != cudaSuccess) return QTZ_ERR_CUDA;
    return QTZ_OK;
}

// Measurement and self-test kernels of libqtz.
//
//  * qtz_probe_int8_peak: the rate of the tensor cores alone.  One CTA per SM keeps one A tile
//    (128 x 128 bytes) and one B tile (256 x 128 bytes) resident in shared memory and issues
//    tcgen05.mma kind::i8 (M = 128, N = 256, K = 32) back to back into two TMEM accumulators;
//    nothing is loaded inside the loop, so the figure is the ceiling a u8 x s8 -> s32
//    contraction (Eq. 5, first term) can reach on this part at the clocks it holds.
//  * qtz_probe_requant_rate: the rate at which the CUDA cores produce requantised outputs (three dp4a and
//    one 32x32->64 multiply-shift-clamp each), which is the ceiling of the depthwise kernel and of every
//    requantising epilogue.
//  * qtz_selftest_wait_timeout: one CTA waits, with a small cycle budget, on an mbarrier that
//    nobody ever signals.  The wait gives up by itself, records (QTZ_ERR_DEVICE_TIMEOUT, site)
//    in the handle's status word and the kernel returns: the path every bounded wait of the
//    convolution kernels takes when something upstream stalls, exercised without any fault.
#include "qtz_internal.cuh"
#include "qtz_ptx.cuh"

using namespace qtz_ptx;

namespace {

constexpr int kProbeM = 128, kProbeN = 256, kProbeRowBytes = 128;
constexpr int kProbeBatch = 32;          // MMAs between two commits
constexpr int kProbeThreads = 128;

__global__ void __launch_bounds__(kProbeThreads, 1)
probe_i8_mma_kernel(int batches, long long wait_budget, int32_t* status)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* const smem = smem_raw + (base - smem_u32(smem_raw));
    __shared__ __align__(8) uint64_t bars[2];
    __shared__ uint32_t tmem_slot;
    const uint32_t a_addr = base, b_addr = base + kProbeM * kProbeRowBytes;
    const int warp = threadIdx.x >> 5;

    // operands: pseudo-random bytes (all-zero operands would draw less power than real data)
    for (uint32_t i = threadIdx.x; i < (kProbeM + kProbeN) * kProbeRowBytes / 4; i += kProbeThreads) {
        uint32_t v = (i + 1u) * 2654435761u + blockIdx.x * 40503u;
        v ^= v >> 15; v *= 2246822519u; v ^= v >> 13;
        reinterpret_cast<uint32_t*>(smem)[i] = v;
    }
    fence_proxy_async_smem();
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars[0]), 1);
        mbar_init(smem_u32(&bars[1]), 1);
        fence_barrier_init();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;

    if (warp == 0) {
        const uint64_t da = make_kmajor_desc(a_addr, kProbeRowBytes), db = make_kmajor_desc(b_addr, kProbeRowBytes);
        // s32 accumulate, A = u8, B = s8, both K-major
        const uint32_t idesc = (2u << 4) | (0u << 7) | (1u << 10) | (static_cast<uint32_t>(kProbeN >> 3) << 17) |
                               (static_cast<uint32_t>(kProbeM >> 4) << 24);
        bool ok = true;
        for (int b = 0; b < batches && ok; ++b) {
            // batch b reuses the barrier of batch b - 2: wait until that one has retired
            if (b >= 2) ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars[b & 1]), ((b >> 1) - 1) & 1, wait_budget, 64u));
            if (!ok) break;
            const uint32_t d = tmem_base + (b & 1) * kProbeN;
            if (elect_one()) {
                // straight-line issue: the four K slices of the resident tiles, eight times over
#pragma unroll
                for (int i = 0; i < kProbeBatch; ++i) mma_i8(d, da + 2 * (i & 3), db + 2 * (i & 3), idesc, i > 0 ? 1u : 0u);
                mma_commit(smem_u32(&bars[b & 1]));
            }
            __syncwarp();
        }
        // drain: the last two batches
        for (int b = max(0, batches - 2); b < batches && ok; ++b)
            ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars[b & 1]), (b >> 1) & 1, wait_budget, 64u));
        if (!ok && (threadIdx.x & 31) == 0 && atomicCAS(status, 0, QTZ_ERR_DEVICE_TIMEOUT) == 0) status[1] = QTZ_SITE_PROBE;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

__global__ void __launch_bounds__(32, 1)
selftest_wait_kernel(long long budget, int32_t* status)
{
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        fence_barrier_init();
    }
    __syncwarp();
    // nobody arrives on this barrier: the wait must run out of budget and come back
    const bool done = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar), 0, budget, 64u));
    if (!done && threadIdx.x == 0 && atomicCAS(status, 0, QTZ_ERR_DEVICE_TIMEOUT) == 0) status[1] = QTZ_SITE_SELFTEST;
}

// Integer-issue rate of the requantising arithmetic: every thread runs independent chains of
//   kind 0: three dp4a per output (a depthwise output's nine taps)
//   kind 1: the 32x32->64 multiply-add, the shift of its high word and the clamp (one requantisation)
//   kind 2: both (a depthwise output from taps to code)
// on register operands, eight outputs per loop pass.  Nothing touches memory inside the loop.
template <int kKind>
__global__ void __launch_bounds__(256)
probe_requant_kernel(const uint32_t* __restrict__ seed, int32_t* __restrict__ sink_out, int iters, int32_t m, int sh, long long add64)
{
    const int tid = blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t x0 = seed[tid & 255], x1 = seed[(tid + 1) & 255], x2 = seed[(tid + 2) & 255];
    const uint32_t w0 = seed[(tid + 3) & 255], w1 = seed[(tid + 4) & 255], w2 = seed[(tid + 5) & 255];
    int32_t sink = 0;
    for (int it = 0; it < iters; ++it) {
        int32_t acc[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (kKind != 1) {
                int32_t d0, d1, d2;
                asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d0) : "r"(x0 + u), "r"(w0), "r"(0));
                asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d1) : "r"(x1 + u), "r"(w1), "r"(d0));
                asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d2) : "r"(x2 + u), "r"(w2), "r"(d1));
                acc[u] = d2;
            } else {
                acc[u] = static_cast<int32_t>(x0 + 77u * u);
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            int32_t y = acc[u];
            if (kKind != 0) {
                const long long p = static_cast<long long>(acc[u]) * m + add64;
                y = __vimin_s32_relu(static_cast<int32_t>(p >> 32) >> sh, 255);
            }
            sink ^= y;
        }
        x0 += sink & 1; x1 += 3; x2 += 5;
    }
    sink_out[tid] = sink;
}

}  // namespace

extern "C" qtz_status qtz_probe_requant_rate(qtz_handle h, int32_t kind, double* outputs_per_clock_sm, double* outputs_per_second,
                                             void* stream)
{
    if (!h || !outputs_per_clock_sm || kind < 0 || kind > 2) return QTZ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    qtz_device_guard guard(h->device);
    const int blocks = h->num_sms * 8, threads = 256, iters = 4000;
    qtz_status s = qtz_ensure_reduce(h, sizeof(int32_t) * (static_cast<size_t>(blocks) * threads + 256));
    if (s != QTZ_OK) return s;
    uint32_t* seed = reinterpret_cast<uint32_t*>(h->reduce_dev);
    int32_t* sink = reinterpret_cast<int32_t*>(h->reduce_dev) + 256;
    uint32_t host_seed[256];
    for (int i = 0; i < 256; ++i) host_seed[i] = static_cast<uint32_t>(i + 1) * 2654435761u;
    QTZ_CUDA(h, cudaMemcpyAsync(seed, host_seed, sizeof(host_seed), cudaMemcpyHostToDevice, st));
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    QTZ_CUDA(h, cudaEventCreate(&e0));
    QTZ_CUDA(h, cudaEventCreate(&e1));
    const int32_t m = 1518500250;
    const long long add64 = 1ll << 39;
    auto launch = [&](int n) {
        if (kind == 0) probe_requant_kernel<0><<<blocks, threads, 0, st>>>(seed, sink, n, m, 8, add64);
        else if (kind == 1) probe_requant_kernel<1><<<blocks, threads, 0, st>>>(seed, sink, n, m, 8, add64);
        else probe_requant_kernel<2><<<blocks, threads, 0, st>>>(seed, sink, n, m, 8, add64);
    };
    launch(10);
    cudaError_t e = cudaEventRecord(e0, st);
    launch(iters);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaEventRecord(e1, st);
    if (e == cudaSuccess) e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    int khz = 0;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, h->device);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (e != cudaSuccess) return qtz_cuda_fail(h, e, "probe_requant_kernel");
    const double outputs = static_cast<double>(blocks) * threads * iters * 8.0;
    const double per_second = outputs / (static_cast<double>(ms) * 1e-3);
    if (outputs_per_second) *outputs_per_second = per_second;
    *outputs_per_clock_sm = per_second / h->num_sms / (static_cast<double>(khz) * 1e3);   // at the maximum SM clock
    return QTZ_OK;
}

extern "C" qtz_status qtz_probe_int8_peak(qtz_handle h, int32_t mmas_per_cta, int32_t launches, double* tops_out,
                                          float* ms_out, void* stream)
{
    if (!h || !tops_out || mmas_per_cta < kProbeBatch || launches < 1 || launches > 100000) return QTZ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int prev = 0;
    QTZ_CUDA(h, cudaGetDevice(&prev));
    QTZ_CUDA(h, cudaSetDevice(h->device));
    const int batches = mmas_per_cta / kProbeBatch;
    const size_t smem = static_cast<size_t>(kProbeM + kProbeN) * kProbeRowBytes + 1024;
    QTZ_CUDA(h, cudaFuncSetAttribute(probe_i8_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    QTZ_CUDA(h, cudaEventCreate(&e0));
    QTZ_CUDA(h, cudaEventCreate(&e1));
    probe_i8_mma_kernel<<<h->num_sms, kProbeThreads, smem, st>>>(batches, h->wait_budget, h->status_dev);   // warm-up
    cudaError_t e = cudaEventRecord(e0, st);
    for (int i = 0; i < launches && e == cudaSuccess; ++i) {
        probe_i8_mma_kernel<<<h->num_sms, kProbeThreads, smem, st>>>(batches, h->wait_budget, h->status_dev);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaEventRecord(e1, st);
    if (e == cudaSuccess) e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaSetDevice(prev);
    if (e != cudaSuccess) return qtz_cuda_fail(h, e, "probe_i8_mma_kernel");
    const double ops = 2.0 * kProbeM * kProbeN * 32.0 * batches * kProbeBatch * h->num_sms * launches;
    *tops_out = ops / (static_cast<double>(ms) * 1e-3) / 1e12;
    if (ms_out) *ms_out = ms;
    return QTZ_OK;
}

extern "C" qtz_status qtz_selftest_wait_timeout(qtz_handle h, int64_t budget_cycles, void* stream)
{
    if (!h || budget_cycles < 1 || budget_cycles > 100000000LL) return QTZ_ERR_INVALID_ARG;
    int prev = 0;
    QTZ_CUDA(h, cudaGetDevice(&prev));
    QTZ_CUDA(h, cudaSetDevice(h->device));
    selftest_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(budget_cycles, h->status_dev);
    const cudaError_t e = cudaGetLastError();
    cudaSetDevice(prev);
    if (e != cudaSuccess) return qtz_cuda_fail(h, e, "selftest_wait_kernel");
    return QTZ_OK;
}

extern "C" qtz_status qtz_set_wait_budget(qtz_handle h, int64_t cycles)
{
    if (!h || cycles < 1000) return QTZ_ERR_INVALID_ARG;
    h->wait_budget = cycles;
    return QTZ_OK;
}

// Measured ceilings of the on-chip resources the reconstruction (Algorithm 2) runs on: the fp32
// min/max rate of the ALU pipe, which carries the element-wise medians, and the shared-memory read
// rate, which carries the cell reads.  The decode kernels are compared with these numbers, not with
// table values.  Each probe is a register-only (or shared-memory-only) loop with enough independent
// chains per thread and enough warps per SM to keep its pipe full; nothing here touches the method.
#include "kvr_internal.h"

namespace {

constexpr int PROBE_THREADS = 1024;
constexpr int CHAINS = 8;

// 2 * CHAINS min/max per iteration and thread (inline PTX so that no other arithmetic is added).
__global__ void __launch_bounds__(PROBE_THREADS, 1)
probe_minmax_kernel(const float* __restrict__ seed, float* __restrict__ sink, int iters) {
    float x[CHAINS];
    const float lo = seed[threadIdx.x & 31], hi = seed[32 + (threadIdx.x & 31)];
#pragma unroll
    for (int c = 0; c < CHAINS; ++c) x[c] = seed[64 + ((threadIdx.x + c) & 31)];
#pragma unroll 1
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int c = 0; c < CHAINS; ++c) {
            asm volatile("min.f32 %0, %0, %1;\n" : "+f"(x[c]) : "f"(hi));
            asm volatile("max.f32 %0, %0, %1;\n" : "+f"(x[c]) : "f"(lo));
        }
    }
    float s = 0.f;
#pragma unroll
    for (int c = 0; c < CHAINS; ++c) s += x[c];
    if (s == 12345.678f) sink[0] = s;
}

// 16-byte shared-memory loads, conflict-free (a warp reads 512 contiguous bytes per instruction).
__global__ void __launch_bounds__(PROBE_THREADS, 1)
probe_lds_kernel(float* __restrict__ sink, int iters) {
    extern __shared__ __align__(16) unsigned char smem[];
    float4* s4 = reinterpret_cast<float4*>(smem);
    for (int i = threadIdx.x; i < 8 * PROBE_THREADS; i += PROBE_THREADS) s4[i] = make_float4(1.f, 2.f, 3.f, 4.f);
    __syncthreads();
    const uint32_t base = (uint32_t)__cvta_generic_to_shared(smem) + threadIdx.x * 16u;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            float4 v;
            asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];\n"
                         : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(base + (uint32_t)k * (PROBE_THREADS * 16u)));
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
    }
    if (acc.x + acc.y + acc.z + acc.w == 12345.678f) sink[0] = acc.x;
}

}  // namespace

extern "C" kvr_status_t kvr_measure_pipe_peaks(double* peaks, void* cuda_stream) {
    if (!peaks) return KVR_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return KVR_ERR_CUDA;
    if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return KVR_ERR_CUDA;
    float* buf = nullptr;
    if (cudaMalloc(&buf, 128 * sizeof(float)) != cudaSuccess) { cudaGetLastError(); return KVR_ERR_ALLOC; }
    float h[128];
    for (int i = 0; i < 128; ++i) h[i] = (i < 32) ? -1.0f - i : (i < 64) ? 1.0f + i : 0.01f * i;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaError_t e = cudaMemcpyAsync(buf, h, sizeof(h), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    const size_t lds_smem = 8 * PROBE_THREADS * 16;
    if (e == cudaSuccess) e = cudaFuncSetAttribute(probe_lds_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lds_smem);
    const int iters = 4096, grid = 2 * n_sm;
    auto timed = [&](int which, float* ms) -> cudaError_t {
        for (int rep = 0; rep < 2; ++rep) {                 // first round warms up
            cudaError_t r = cudaEventRecord(e0, st);
            if (r != cudaSuccess) return r;
            if (which == 0) probe_minmax_kernel<<<grid, PROBE_THREADS, 0, st>>>(buf, buf + 96, iters);
            else probe_lds_kernel<<<grid, PROBE_THREADS, lds_smem, st>>>(buf + 96, iters);
            r = cudaGetLastError();
            if (r != cudaSuccess) return r;
            r = cudaEventRecord(e1, st);
            if (r != cudaSuccess) return r;
            r = cudaEventSynchronize(e1);
            if (r != cudaSuccess) return r;
            r = cudaEventElapsedTime(ms, e0, e1);
            if (r != cudaSuccess) return r;
        }
        return cudaSuccess;
    };
    float ms0 = 0.f, ms1 = 0.f;
    if (e == cudaSuccess) e = timed(0, &ms0);
    if (e == cudaSuccess) e = timed(1, &ms1);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(buf);
    if (e != cudaSuccess) { cudaGetLastError(); return KVR_ERR_CUDA; }
    const double threads = (double)grid * PROBE_THREADS;
    peaks[0] = threads * iters * (2.0 * CHAINS) / (ms0 * 1e-3);          // fp32 min/max lane-ops per second
    peaks[1] = threads * iters * 8.0 * 16.0 / (ms1 * 1e-3);              // shared-memory bytes read per second
    return KVR_OK;
}

// Device micro-probes used to put the forward kernels' numbers in context: fp32 FMA rate, shared-memory
// load bandwidth, L2 read bandwidth and the cost of an empty launch.  They touch only buffers they
// allocate themselves and are not part of the forward path.
#include "cfi.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>

namespace {

__global__ void probe_fma_kernel(float* out, int iters, float seed) {
    float a[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] = seed + i + threadIdx.x;
    const float m = 0.999f, c = 0.001f;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 8; ++i) a[i] = fmaf(a[i], m, c);
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) s += a[i];
    if (s == 123.456f) out[0] = s;  // never true; keeps the chains alive
}

__global__ void probe_lds_kernel(float* out, int iters) {
    extern __shared__ __align__(16) float sm[];
    for (int i = threadIdx.x; i < 8192; i += blockDim.x) sm[i] = (float)i;
    __syncthreads();
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    int idx = threadIdx.x * 4;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float4 v = *reinterpret_cast<const float4*>(sm + ((idx + u * 1024) & 8188));
            acc.x += v.x, acc.y += v.y, acc.z += v.z, acc.w += v.w;
        }
        idx = (idx + 4096) & 8188;
    }
    if (acc.x + acc.y + acc.z + acc.w == 123.456f) out[0] = acc.x;
}

// Every CTA reads the whole buffer (`n4` float4) `passes` times; CTA i starts at a different offset.
__global__ void probe_l2_kernel(const float4* __restrict__ buf, size_t n4, int passes, float* out, int same_start) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const size_t start = same_start ? 0 : ((size_t)blockIdx.x * 8191u * 64u) % n4;
    for (int p = 0; p < passes; ++p) {
        for (size_t i = threadIdx.x; i < n4; i += (size_t)blockDim.x * 4) {
            float4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                size_t j = start + i + (size_t)u * blockDim.x;
                if (j >= n4) j -= n4;
                if (j >= n4) j = 0;
                v[u] = __ldcg(buf + j);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) acc.x += v[u].x, acc.y += v[u].y, acc.z += v[u].z, acc.w += v[u].w;
        }
    }
    if (acc.x + acc.y + acc.z + acc.w == 123.456f) out[0] = acc.x;
}

__global__ void probe_empty_kernel() {}

// The two kernels of cfi_probe_floor_launch.  Both start and finish the way the forward kernels do (they let the next
// kernel in the stream start early and wait for the one before them), so a chain of them in a stream or graph costs
// what a chain of forward launches would cost with all of their work taken out.
__global__ void probe_floor_empty_kernel(float* out) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (out == nullptr) return;  // never: keeps the argument alive
}
// One dependent trip to DRAM per CTA and one store: thread 0 reads the launch counter (on chip), then a line of
// `buf` that no recent launch has touched, and writes what it read to out[cta]; CTA 0 then advances the counter.
__global__ void probe_floor_roundtrip_kernel(const float* __restrict__ buf, unsigned long long lines, unsigned long long* counter,
                                             float* out) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (threadIdx.x == 0) {
        const unsigned long long c = *reinterpret_cast<volatile unsigned long long*>(counter);
        const unsigned long long line = ((c * gridDim.x + blockIdx.x) * 4099ull) % lines;
        out[blockIdx.x] = __ldcg(buf + line * 32ull);
        if (blockIdx.x == 0) atomicAdd(counter, 1ull);
    }
}

float elapsed_ms(cudaEvent_t a, cudaEvent_t b) {
    float ms = 0.f;
    cudaEventElapsedTime(&ms, a, b);
    return ms;
}

}  // namespace

extern "C" cfi_status_t cfi_probe_device(cfi_device_probe_t* p) {
    if (!p) return CFI_ERR_NULL;
    int dev = 0;
    cudaDeviceProp prop{};
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
        cudaGetLastError();
        return CFI_ERR_CUDA;
    }
    *p = cfi_device_probe_t{};
    p->sm_count = prop.multiProcessorCount;
    p->l2_bytes = prop.l2CacheSize;
    p->smem_per_block_optin = (int64_t)prop.sharedMemPerBlockOptin;
    int clk_khz = 0;
    cudaDeviceGetAttribute(&clk_khz, cudaDevAttrClockRate, dev);
    p->sm_clock_mhz_nominal = clk_khz / 1000.0;

    float* out = nullptr;
    float4* buf = nullptr;
    const size_t l2_probe_bytes = 16u << 20, hot_bytes = 768u << 10;
    if (cudaMalloc(&out, 256) != cudaSuccess || cudaMalloc(&buf, l2_probe_bytes) != cudaSuccess) {
        cudaGetLastError();
        if (out) cudaFree(out);
        return CFI_ERR_ALLOC;
    }
    cudaMemset(buf, 0, l2_probe_bytes);
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    const int sms = prop.multiProcessorCount;

    // fp32 FMA: 8 chains x iters per thread
    {
        const int iters = 1 << 15, threads = 1024, blocks = sms * 2;
        probe_fma_kernel<<<blocks, threads>>>(out, 1024, 1.0f);
        cudaEventRecord(e0);
        probe_fma_kernel<<<blocks, threads>>>(out, iters, 1.0f);
        cudaEventRecord(e1);
        cudaEventSynchronize(e1);
        p->fma_tflops = 2.0 * 8.0 * iters * (double)threads * blocks / (elapsed_ms(e0, e1) * 1e-3) / 1e12;
    }
    // shared memory: 16-byte loads, conflict free
    {
        const int iters = 1 << 12, threads = 1024, blocks = sms;
        probe_lds_kernel<<<blocks, threads, 32768>>>(out, 64);
        cudaEventRecord(e0);
        probe_lds_kernel<<<blocks, threads, 32768>>>(out, iters);
        cudaEventRecord(e1);
        cudaEventSynchronize(e1);
        p->smem_load_gbs = 16.0 * 8.0 * iters * (double)threads * blocks / (elapsed_ms(e0, e1) * 1e-3) / 1e9;
    }
    // L2: every CTA streams a 16 MB resident buffer; then every CTA streams the same 768 KB
    for (int hot = 0; hot < 2; ++hot) {
        const size_t bytes = hot ? hot_bytes : l2_probe_bytes;
        const size_t n4 = bytes / 16;
        const int passes = hot ? 16 : 1, threads = 512, blocks = sms;
        probe_l2_kernel<<<blocks, threads>>>(buf, n4, 1, out, hot);
        cudaEventRecord(e0);
        probe_l2_kernel<<<blocks, threads>>>(buf, n4, passes, out, hot);
        cudaEventRecord(e1);
        cudaEventSynchronize(e1);
        const double gbs = (double)bytes * passes * blocks / (elapsed_ms(e0, e1) * 1e-3) / 1e9;
        if (hot) p->l2_read_same_lines_gbs = gbs;
        else p->l2_read_gbs = gbs;
    }
    // empty launches back to back on one stream
    {
        const int n = 2000;
        for (int i = 0; i < 10; ++i) probe_empty_kernel<<<1, 32>>>();
        cudaEventRecord(e0);
        for (int i = 0; i < n; ++i) probe_empty_kernel<<<1, 32>>>();
        cudaEventRecord(e1);
        cudaEventSynchronize(e1);
        p->empty_launch_us = elapsed_ms(e0, e1) * 1e3 / n;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(buf);
    cudaFree(out);
    const cudaError_t err = cudaDeviceSynchronize();
    if (err != cudaSuccess) {
        cudaGetLastError();
        return CFI_ERR_CUDA;
    }
    return CFI_OK;
}

extern "C" cfi_status_t cfi_probe_floor_launch(int32_t kind, const void* buf, size_t buf_bytes, void* scratch, cfi_stream_t stream) {
    if (kind != 0 && kind != 1) return CFI_ERR_DTYPE;
    if (!scratch || (kind == 1 && !buf)) return CFI_ERR_NULL;
    if (((uintptr_t)buf | (uintptr_t)scratch) & 255u) return CFI_ERR_ALIGNMENT;
    if (kind == 1 && buf_bytes < (1u << 20)) return CFI_ERR_BUFFER_TOO_SMALL;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        return CFI_ERR_CUDA;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)sms);
    cfg.blockDim = dim3(128);
    cfg.stream = reinterpret_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    unsigned long long* counter = static_cast<unsigned long long*>(scratch);
    float* out = reinterpret_cast<float*>(counter + 32);
    cudaError_t e;
    if (kind == 0) e = cudaLaunchKernelEx(&cfg, probe_floor_empty_kernel, out);
    else e = cudaLaunchKernelEx(&cfg, probe_floor_roundtrip_kernel, static_cast<const float*>(buf), (unsigned long long)(buf_bytes / 128),
                                counter, out);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return CFI_ERR_CUDA;
    }
    return CFI_OK;
}

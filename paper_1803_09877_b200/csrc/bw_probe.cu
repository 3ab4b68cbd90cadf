// Stand-alone bandwidth probe (not part of libdraco): what this GPU streams for the traffic mixes of the
// cyclic encoder, without any arithmetic.  n rows of d fp32 in (4 n d bytes), n rows of d complex64 out
// (8 n d bytes), the shapes of Z = G W (Section 3, "Cyclic Code").
//
//   copy / fill / expand   contiguous streams: 1 : 1, 0 : 1 and 1 : 2 read : write
//   ring                   the encoder's data path: every warp walks 128-coordinate strips over the n rows, each
//                          lane copying its 16 bytes of a row into a private shared-memory ring with cp.async
//                          (coordinates 2l, 2l+1, 64+2l, 64+2l+1) and writing two 16-byte stores 512 bytes apart
//
// Build and run:  python -m paper_1803_09877_b200.build --probe   (writes paper_1803_09877_b200/bw_probe), then
//                 ./paper_1803_09877_b200/bw_probe [d]        (d = 60200000 by default; 33 GB of device memory)
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <vector>

#define CK(x)                                                                              \
    do {                                                                                   \
        cudaError_t e__ = (x);                                                             \
        if (e__ != cudaSuccess) {                                                          \
            printf("CUDA error %s at line %d\n", cudaGetErrorString(e__), __LINE__);       \
            exit(1);                                                                       \
        }                                                                                  \
    } while (0)

// U float4 per lane in flight; every warp instruction covers 512 contiguous bytes
template <int U>
__global__ void copy_kernel(const float4* __restrict__ in, float4* __restrict__ out, int64_t nvec) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t base = warp * (U * 32); base < nvec; base += nwarps * (U * 32)) {
        float4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t i = base + u * 32 + lane;
            if (i < nvec) v[u] = __ldcs(in + i);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t i = base + u * 32 + lane;
            if (i < nvec) __stcs(out + i, v[u]);
        }
    }
}

template <int U>
__global__ void fill_kernel(float4* __restrict__ out, int64_t nvec) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const float4 v = make_float4(1.f, 2.f, 3.f, (float)lane);
    for (int64_t base = warp * (U * 32); base < nvec; base += nwarps * (U * 32)) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t i = base + u * 32 + lane;
            if (i < nvec) __stcs(out + i, v);
        }
    }
}

// 32 input float4 of a warp (512 B) become 64 output float4 (1 KB): lane l writes out[2 c + l] and out[2 c + 32 + l]
template <int U>
__global__ void expand_kernel(const float4* __restrict__ in, float4* __restrict__ out, int64_t nvec) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t base = warp * (U * 32); base < nvec; base += nwarps * (U * 32)) {
        float4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t i = base + u * 32 + lane;
            if (i < nvec) v[u] = __ldcs(in + i);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t c = base + u * 32;              // nvec is a multiple of 32: a chunk is whole or absent
            if (c + lane < nvec) {
                __stcs(out + 2 * c + lane, v[u]);
                __stcs(out + 2 * c + 32 + lane, make_float4(v[u].y, v[u].x, v[u].w, v[u].z));
            }
        }
    }
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// The encoder's data path.  RING rows in flight per lane, running on across strips; d must be a multiple of 128.
template <int RING>
__global__ void ring_kernel(const float* __restrict__ G, float* __restrict__ Z, int64_t d, int n) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t nstrips = d / 128;
    const uint32_t ring0 = smem_u32(smem) + threadIdx.x * 16;
    const uint32_t rowb = blockDim.x * 16;
    int64_t fs = warp;                                    // fetch cursor: strip and row of the next copy
    int fr = 0;
    auto fetch = [&](uint32_t dst) {
        if (fs < nstrips) {
            const float* ga = G + fs * 128 + 2 * lane + (int64_t)fr * d;
            asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst), "l"(ga) : "memory");
            asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst + 8), "l"(ga + 64) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");   // an empty group keeps every thread's count equal
        if (++fr == n) { fr = 0; fs += nwarps; }
    };
    for (int q = 0; q < RING; ++q) fetch(ring0 + q * rowb);
    uint32_t rd = 0;
    for (int64_t s = warp; s < nstrips; s += nwarps) {
        float* z = Z + s * 256;
        for (int r = 0; r < n; ++r) {
            asm volatile("cp.async.wait_group %0;" ::"n"(RING - 1) : "memory");
            float4 x;
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(x.x), "=f"(x.y), "=f"(x.z), "=f"(x.w) : "r"(ring0 + rd) : "memory");
            float* zr = z + (int64_t)r * (2 * d);
            __stcs(reinterpret_cast<float4*>(zr) + lane, make_float4(x.x, x.y, x.y, x.x));
            __stcs(reinterpret_cast<float4*>(zr) + 32 + lane, make_float4(x.z, x.w, x.w, x.z));
            fetch(ring0 + rd);                            // refill the slot just read (the stores above needed its value)
            rd += rowb;
            if (rd == RING * rowb) rd = 0;
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

template <typename F>
float median_ms(F launch, int reps = 8) {
    cudaEvent_t a, b;
    CK(cudaEventCreate(&a));
    CK(cudaEventCreate(&b));
    launch();
    launch();
    CK(cudaDeviceSynchronize());
    std::vector<float> ts;
    for (int i = 0; i < reps; ++i) {
        CK(cudaEventRecord(a));
        launch();
        CK(cudaEventRecord(b));
        CK(cudaEventSynchronize(b));
        float ms;
        CK(cudaEventElapsedTime(&ms, a, b));
        ts.push_back(ms);
    }
    CK(cudaGetLastError());
    std::sort(ts.begin(), ts.end());
    return ts[ts.size() / 2];
}

int main(int argc, char** argv) {
    const int n = 45;
    const int64_t d = argc > 1 ? atoll(argv[1]) : 60200000;       // the ring kernel leaves a ragged tail (d mod 128) alone
    if (d < 128 || d > 200000000 || d % 4 != 0) { printf("d must be a multiple of 4 in [128, 2e8]\n"); return 2; }   // 16-byte rows
    const int64_t nin = (int64_t)n * d;                           // floats in; 2 nin floats out
    float *in, *out;
    CK(cudaMalloc(&in, nin * 4));
    CK(cudaMalloc(&out, nin * 8));
    CK(cudaMemset(in, 0, nin * 4));
    CK(cudaMemset(out, 0, nin * 8));
    const int64_t nvec = (nin / 4) / 32 * 32;                     // whole 512-byte warp chunks
    int sms;
    CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0));
    printf("%d SMs; n = %d rows, d = %lld (row pitch %lld B): %.2f GB in, %.2f GB out\n", sms, n, (long long)d,
           (long long)d * 4, nin * 4 / 1e9, nin * 8 / 1e9);
    auto report = [&](const char* name, double bytes, float ms) {
        printf("%-58s %8.3f ms  %7.1f GB/s\n", name, ms, bytes / ms / 1e6);
        fflush(stdout);
    };
    char nm[128];
    const double b_copy = nvec * 32.0, b_fill = nvec * 32.0, b_expand = nvec * 48.0;
#define COPY(U, BPS, T)                                                                                        \
    {                                                                                                          \
        const float ms = median_ms([&] { copy_kernel<U><<<sms * BPS, T>>>((const float4*)in, (float4*)out, nvec); }); \
        snprintf(nm, sizeof nm, "copy    %d x 16 B in flight/lane, %d blocks/SM x %d thr", U, BPS, T);          \
        report(nm, b_copy, ms);                                                                                \
    }
#define FILL(U, BPS, T)                                                                                        \
    {                                                                                                          \
        const float ms = median_ms([&] { fill_kernel<U><<<sms * BPS, T>>>((float4*)out, 2 * nvec); });          \
        snprintf(nm, sizeof nm, "fill    %d x 16 B/lane, %d blocks/SM x %d thr", U, BPS, T);                    \
        report(nm, b_fill, ms);                                                                                \
    }
#define EXPAND(U, BPS, T)                                                                                      \
    {                                                                                                          \
        const float ms = median_ms([&] { expand_kernel<U><<<sms * BPS, T>>>((const float4*)in, (float4*)out, nvec); }); \
        snprintf(nm, sizeof nm, "expand  %d x 16 B in flight/lane, %d blocks/SM x %d thr", U, BPS, T);          \
        report(nm, b_expand, ms);                                                                              \
    }
#define RINGK(RING, T)                                                                                         \
    {                                                                                                          \
        const size_t sm = (size_t)T * 16 * RING;                                                               \
        CK(cudaFuncSetAttribute(ring_kernel<RING>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm));     \
        const float ms = median_ms([&] { ring_kernel<RING><<<sms, T, sm>>>(in, out, d, n); });                  \
        snprintf(nm, sizeof nm, "ring    %d rows in flight/lane, 1 block/SM x %d thr (%zu KB)", RING, T, sm >> 10); \
        report(nm, (double)(d / 128 * 128) * n * 12.0, ms);                                                    \
    }
    COPY(8, 4, 256) COPY(2, 8, 256) COPY(8, 1, 384)
    FILL(8, 4, 256) FILL(2, 1, 384)
    EXPAND(2, 8, 256) EXPAND(4, 8, 256) EXPAND(8, 4, 256) EXPAND(16, 2, 256) EXPAND(8, 1, 384)
    RINGK(12, 384) RINGK(12, 352) RINGK(12, 256) RINGK(12, 512) RINGK(10, 384) RINGK(14, 384) RINGK(16, 384) RINGK(8, 384)
    CK(cudaFree(in));
    CK(cudaFree(out));
    return 0;
}

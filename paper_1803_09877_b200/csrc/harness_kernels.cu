// Seeded synthetic inputs and the adversary (R = Z + N): the generator side of the library.
// Counter-based and built from integer arithmetic plus single correctly rounded fp32
// operations, so every value has the same bits as any other implementation of the same
// definition (see draco_generate in draco.h).
#include <math.h>

#include "draco_internal.cuh"

namespace draco {

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ uint64_t splitmix64_at(uint64_t seed, uint64_t ctr) {
    uint64_t z = seed + (ctr + 1ull) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__device__ __forceinline__ uint32_t sum16(uint64_t h) {
    const uint32_t lo = (uint32_t)h, hi = (uint32_t)(h >> 32);
    return (lo & 0xFFFFu) + (lo >> 16) + (hi & 0xFFFFu) + (hi >> 16);
}

// Irwin-Hall(8) approximation of a standard normal, element i of the row with key `key`.
__device__ __forceinline__ float approx_normal(uint64_t key, uint64_t i, float inv_sigma) {
    const uint32_t s = sum16(splitmix64_at(key, 2ull * i)) + sum16(splitmix64_at(key, 2ull * i + 1ull));
    return __fmul_rn((float)((int)s - 262140), inv_sigma);
}

__global__ void __launch_bounds__(kThreads)
generate_kernel(float* __restrict__ out, int rows, int64_t len, int64_t ld, int64_t i0, int row0, float mean, float sd,
                uint64_t seed, float inv_sigma) {
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    for (int r = 0; r < rows; ++r) {
        const uint64_t key = splitmix64_at(seed, (uint64_t)(row0 + r));
        float* dst = out + (int64_t)r * ld;
        for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < len; i += stride) {
            const float x = approx_normal(key, (uint64_t)(i0 + i), inv_sigma);
            dst[i] = __fadd_rn(__fmul_rn(x, sd), mean);
        }
    }
}

__device__ __forceinline__ float corrupt_value(float v, int64_t idx, int model, float param, uint64_t key, int is_complex,
                                               float inv_sigma) {
    if (model == DRACO_ADV_REVGRAD) return __fmul_rn(v, -param);
    if (model == DRACO_ADV_CONST) return (is_complex && (idx & 1)) ? 0.0f : param;
    return __fadd_rn(v, __fmul_rn(approx_normal(key, (uint64_t)idx, inv_sigma), param));
}

// One adversarial row, in place; VEC = 4 when the row slice is 16-byte aligned and a multiple of 4 values.
template <int VEC>
__global__ void __launch_bounds__(kThreads)
corrupt_kernel(float* __restrict__ row, int64_t nvals, int64_t v0, int model, float param, uint64_t key, int is_complex,
               float inv_sigma) {
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    if (VEC == 4) {
        float4* row4 = reinterpret_cast<float4*>(row);
        for (int64_t q = (int64_t)blockIdx.x * kThreads + threadIdx.x; q < nvals / 4; q += stride) {
            float4 v = model == DRACO_ADV_CONST ? make_float4(0.f, 0.f, 0.f, 0.f) : __ldcs(row4 + q);
            const int64_t i = v0 + q * 4;
            v.x = corrupt_value(v.x, i, model, param, key, is_complex, inv_sigma);
            v.y = corrupt_value(v.y, i + 1, model, param, key, is_complex, inv_sigma);
            v.z = corrupt_value(v.z, i + 2, model, param, key, is_complex, inv_sigma);
            v.w = corrupt_value(v.w, i + 3, model, param, key, is_complex, inv_sigma);
            __stcs(row4 + q, v);
        }
    } else {
        for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < nvals; i += stride)
            row[i] = corrupt_value(row[i], v0 + i, model, param, key, is_complex, inv_sigma);
    }
}

float inv_sigma_f32() { return (float)(1.0 / sqrt(8.0 * (4294967296.0 - 1.0) / 12.0)); }

uint64_t host_splitmix64_at(uint64_t seed, uint64_t ctr) {
    uint64_t z = seed + (ctr + 1ull) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

int grid_for(int64_t work) {
    int64_t want = (work + kThreads - 1) / kThreads;
    if (want > 148 * 16) want = 148 * 16;
    if (want < 1) want = 1;
    return (int)want;
}

}  // namespace

int launch_generate(float* out, int rows, int64_t len, int64_t ld, int64_t i0, int row0, float mean, float sd,
                    uint64_t seed, cudaStream_t st) {
    generate_kernel<<<grid_for(len), kThreads, 0, st>>>(out, rows, len, ld, i0, row0, mean, sd, seed, inv_sigma_f32());
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

int launch_corrupt_row(float* row, int64_t nvals, int64_t v0, int model, float param, uint64_t seed, int node,
                       bool is_complex, cudaStream_t st) {
    const uint64_t key = host_splitmix64_at(seed, (uint64_t)node);
    const bool vec4 = (nvals % 4 == 0) && ((reinterpret_cast<uintptr_t>(row) & 15u) == 0);
    if (vec4)
        corrupt_kernel<4><<<grid_for(nvals / 4), kThreads, 0, st>>>(row, nvals, v0, model, param, key, is_complex ? 1 : 0,
                                                                    inv_sigma_f32());
    else
        corrupt_kernel<1><<<grid_for(nvals), kThreads, 0, st>>>(row, nvals, v0, model, param, key, is_complex ? 1 : 0,
                                                                inv_sigma_f32());
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

}  // namespace draco

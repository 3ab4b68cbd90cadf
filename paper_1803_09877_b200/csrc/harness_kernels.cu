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

// All adversarial rows in one launch, in place: blockIdx.y picks the adversary, blockIdx.x strides over its row
// slice.  VEC = 4 when every row slice is 16-byte aligned and a multiple of 4 values long.
struct CorruptTable {
    int32_t node[kMaxN];
    int32_t model[kMaxN];
    float param[kMaxN];
    unsigned long long key[kMaxN];        // generator key of the node's noise row
};

template <int VEC>
__global__ void __launch_bounds__(kThreads)
corrupt_kernel(float* __restrict__ R, int64_t row_pitch, int64_t nvals, int64_t v0, int is_complex, float inv_sigma,
               const __grid_constant__ CorruptTable tab) {
    const int a = blockIdx.y;
    const int model = tab.model[a];
    const float param = tab.param[a];
    const uint64_t key = tab.key[a];
    float* row = R + (int64_t)tab.node[a] * row_pitch + v0;
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

int grid_for(int64_t work, int sm_count, int per_sm) {
    int64_t want = (work + kThreads - 1) / kThreads;
    const int64_t cap = (int64_t)(sm_count > 0 ? sm_count : 1) * per_sm;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    return (int)want;
}

int device_sm_count() {                     // of the current device; looked up once per device
    static int cached[64] = {};
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 1;
    if (dev >= 0 && dev < 64 && cached[dev] > 0) return cached[dev];
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return 1;
    if (dev >= 0 && dev < 64) cached[dev] = sms;
    return sms;
}

}  // namespace

int launch_generate(float* out, int rows, int64_t len, int64_t ld, int64_t i0, int row0, float mean, float sd,
                    uint64_t seed, cudaStream_t st) {
    generate_kernel<<<grid_for(len, device_sm_count(), 16), kThreads, 0, st>>>(out, rows, len, ld, i0, row0, mean, sd, seed,
                                                                              inv_sigma_f32());
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

// R = Z + N on the rows node[0 .. n_adv-1]: values [v0, v0 + nvals) of each (fp32 values; a complex entry is two).
int launch_corrupt(float* R, int64_t row_pitch, int64_t nvals, int64_t v0, const int* node, const int* model,
                   const float* param, int n_adv, uint64_t seed, bool is_complex, int sm_count, cudaStream_t st) {
    if (n_adv == 0) return DRACO_OK;
    CorruptTable tab;
    for (int a = 0; a < n_adv; ++a) {
        tab.node[a] = node[a];
        tab.model[a] = model[a];
        tab.param[a] = param[a];
        tab.key[a] = host_splitmix64_at(seed, (uint64_t)node[a]);
    }
    const bool vec4 = (nvals % 4 == 0) && (row_pitch % 4 == 0) && (v0 % 4 == 0) && ((reinterpret_cast<uintptr_t>(R) & 15u) == 0);
    // enough blocks per adversary that all of them together fill the device about sixteen times over
    int per_sm = 16 / n_adv;
    if (per_sm < 2) per_sm = 2;
    const dim3 grid(grid_for(vec4 ? nvals / 4 : nvals, sm_count, per_sm), n_adv);
    if (vec4) corrupt_kernel<4><<<grid, kThreads, 0, st>>>(R, row_pitch, nvals, v0, is_complex ? 1 : 0, inv_sigma_f32(), tab);
    else corrupt_kernel<1><<<grid, kThreads, 0, st>>>(R, row_pitch, nvals, v0, is_complex ? 1 : 0, inv_sigma_f32(), tab);
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

}  // namespace draco

// Cyclic-code recovery, Algorithm 1 step 4: u = Re(R_{.,U} b) for the decode vector b left
// in the plan's device state by the decode-vector kernel.
//
// One pass over the rows with b_j != 0.  The code cancels entries of W as large as 1e5 back
// to 1, so the running sums are kept in fp64 (fp32 would lose about kappa * 2^-24 of the
// result); R stays fp32 in memory.  HBM traffic: 8 |U| len bytes read + 4 len written.
#include "draco_internal.cuh"

namespace draco {

namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 8;

template <bool VEC2>
__global__ void __launch_bounds__(kThreads)
cyc_recover_kernel(const float2* __restrict__ R, int64_t len, int64_t ld, const CycDevice* __restrict__ cd,
                   const DeviceInfo* __restrict__ info, float* __restrict__ u) {
    __shared__ double2 bs[kMaxN];
    __shared__ int rows[kMaxN];
    const int count = info->n_active;
    for (int k = threadIdx.x; k < count; k += kThreads) {
        bs[k] = cd->b_active[k];
        rows[k] = cd->active[k];
    }
    __syncthreads();
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    if (VEC2) {
        const int64_t nvec = len / 2;
        for (int64_t v = (int64_t)blockIdx.x * kThreads + threadIdx.x; v < nvec; v += stride) {
            const float2* col = R + v * 2;
            double a0 = 0.0, a1 = 0.0;
            for (int k0 = 0; k0 < count; k0 += kUnroll) {
                float4 x[kUnroll];
#pragma unroll
                for (int q = 0; q < kUnroll; ++q)
                    if (k0 + q < count) x[q] = __ldcs(reinterpret_cast<const float4*>(col + (int64_t)rows[k0 + q] * ld));
#pragma unroll
                for (int q = 0; q < kUnroll; ++q)
                    if (k0 + q < count) {
                        const double2 b = bs[k0 + q];
                        a0 = fma(b.x, (double)x[q].x, a0);
                        a0 = fma(-b.y, (double)x[q].y, a0);
                        a1 = fma(b.x, (double)x[q].z, a1);
                        a1 = fma(-b.y, (double)x[q].w, a1);
                    }
            }
            __stcs(reinterpret_cast<float2*>(u + v * 2), make_float2((float)a0, (float)a1));
        }
    } else {
        for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < len; i += stride) {
            double a0 = 0.0;
            for (int k = 0; k < count; ++k) {
                const float2 x = __ldcs(R + (int64_t)rows[k] * ld + i);
                const double2 b = bs[k];
                a0 = fma(b.x, (double)x.x, a0);
                a0 = fma(-b.y, (double)x.y, a0);
            }
            u[i] = (float)a0;
        }
    }
}

}  // namespace

int launch_cyc_recover(draco_plan* p, const float2* R, int64_t len, int64_t ld, float* u, cudaStream_t st) {
    const bool vec2 = (len % 2 == 0) && (ld % 2 == 0);
    const int64_t nvec = vec2 ? len / 2 : len;
    int64_t want = (nvec + kThreads - 1) / kThreads;
    const int64_t cap = (int64_t)p->sm_count * 16;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    if (vec2)
        cyc_recover_kernel<true><<<(int)want, kThreads, 0, st>>>(R, len, ld, p->cyc_dev, p->info_dev, u);
    else
        cyc_recover_kernel<false><<<(int)want, kThreads, 0, st>>>(R, len, ld, p->cyc_dev, p->info_dev, u);
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

}  // namespace draco

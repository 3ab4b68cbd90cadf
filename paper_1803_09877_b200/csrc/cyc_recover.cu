// Cyclic-code recovery, Algorithm 1 step 4: u = Re(R_{.,U} b) for the decode vector b left
// in the plan's device state by the decode-vector kernel.
//
// One pass over the rows with b_j != 0.  The code cancels entries of W as large as 1e5 back
// to 1, so the running sums are kept in fp64 (fp32 would lose about kappa * 2^-24 of the
// result); R stays fp32 in memory.  HBM traffic: 8 |U| len bytes read + 4 len written.
//
// Self-check (unpacked plans).  u-hat = G 1_P is real, so Im(u-hat) is rounding residue as long as every
// row of U is honest, and of the size of the result when an adversary is left in U.  The kernel forms
// Im(u-hat_i) on one coordinate run in eight (floor(i / 64) mod 8 = 0, uniform in a warp) and leaves max |Im| and
// max |Re| over those coordinates in the plan's info block.  (The compiler predicates the extra multiply-adds
// instead of branching, so the fp64 pipe is 19 % busy instead of 10 %; the kernel stays memory-bound, and two
// specialised copies of the loop behind a real branch cost 118 registers instead of 80.)
#include "draco_internal.cuh"

namespace draco {

namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 8;

// PACKED: the vectors carry two gradient coordinates per complex entry (Section 3, last
// paragraph): u[i] = Re(u-hat_i), u[len + i] = Im(u-hat_i) for len + i < d_packed.
template <bool VEC2, bool PACKED>
__global__ void __launch_bounds__(kThreads)
cyc_recover_kernel(const float2* __restrict__ R, int64_t len, int64_t ld, const CycDevice* __restrict__ cd,
                   DeviceInfo* info, float* __restrict__ u, int64_t d_packed, float* __restrict__ w, float scale) {
    __shared__ double2 bs[kMaxN];
    __shared__ int rows[kMaxN];
    const int count = info->n_active;
    double im_max = 0.0, re_max = 0.0;                    // over this thread's sampled coordinates
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
            const bool sampled = !PACKED && ((v >> 5) & 7) == 0;       // coordinates 2 v, 2 v + 1: floor(i / 64) mod 8 == 0
            double a0 = 0.0, a1 = 0.0, i0 = 0.0, i1 = 0.0;
            for (int k0 = 0; k0 < count; k0 += kUnroll) {
                float4 x[kUnroll];
#pragma unroll
                for (int q = 0; q < kUnroll; ++q)
                    if (k0 + q < count) x[q] = __ldcs(reinterpret_cast<const float4*>(col + (int64_t)rows[k0 + q] * ld));
#pragma unroll
                for (int q = 0; q < kUnroll; ++q)
                    if (k0 + q < count) {
                        const double2 b = bs[k0 + q];
                        const double xr0 = (double)x[q].x, xi0 = (double)x[q].y, xr1 = (double)x[q].z, xi1 = (double)x[q].w;
                        a0 = fma(b.x, xr0, a0);
                        a0 = fma(-b.y, xi0, a0);
                        a1 = fma(b.x, xr1, a1);
                        a1 = fma(-b.y, xi1, a1);
                        if (PACKED || sampled) {
                            i0 = fma(b.x, xi0, i0);
                            i0 = fma(b.y, xr0, i0);
                            i1 = fma(b.x, xi1, i1);
                            i1 = fma(b.y, xr1, i1);
                        }
                    }
            }
            if (sampled) {
                im_max = fmax(im_max, fmax(fabs(i0), fabs(i1)));
                re_max = fmax(re_max, fmax(fabs(a0), fabs(a1)));
            }
            if (u != nullptr) {
                __stcs(reinterpret_cast<float2*>(u + v * 2), make_float2((float)a0, (float)a1));
                if (PACKED) __stcs(reinterpret_cast<float2*>(u + len + v * 2), make_float2((float)i0, (float)i1));
            }
            if (w != nullptr) {                          // w <- w - scale * u, u rounded to fp32 first as when stored
                float2* wp = reinterpret_cast<float2*>(w + v * 2);
                float2 wv = *wp;
                wv.x = fmaf(-scale, (float)a0, wv.x);
                wv.y = fmaf(-scale, (float)a1, wv.y);
                *wp = wv;
                if (PACKED) {
                    wp = reinterpret_cast<float2*>(w + len + v * 2);
                    wv = *wp;
                    wv.x = fmaf(-scale, (float)i0, wv.x);
                    wv.y = fmaf(-scale, (float)i1, wv.y);
                    *wp = wv;
                }
            }
        }
    } else {
        for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < len; i += stride) {
            const bool sampled = !PACKED && ((i >> 6) & 7) == 0;
            double a0 = 0.0, i0 = 0.0;
            for (int k = 0; k < count; ++k) {
                const float2 x = __ldcs(R + (int64_t)rows[k] * ld + i);
                const double2 b = bs[k];
                a0 = fma(b.x, (double)x.x, a0);
                a0 = fma(-b.y, (double)x.y, a0);
                if (PACKED || sampled) {
                    i0 = fma(b.x, (double)x.y, i0);
                    i0 = fma(b.y, (double)x.x, i0);
                }
            }
            if (sampled) {
                im_max = fmax(im_max, fabs(i0));
                re_max = fmax(re_max, fabs(a0));
            }
            if (u != nullptr) {
                u[i] = (float)a0;
                if (PACKED && len + i < d_packed) u[len + i] = (float)i0;
            }
            if (w != nullptr) {
                w[i] = fmaf(-scale, (float)a0, w[i]);
                if (PACKED && len + i < d_packed) w[len + i] = fmaf(-scale, (float)i0, w[len + i]);
            }
        }
    }
    if (!PACKED) {
        // non-negative doubles order like their bit patterns; NaN (an adversary may send it) counts as the largest
        if (!(im_max == im_max)) im_max = __longlong_as_double(0x7ff0000000000000ll);
        if (!(re_max == re_max)) re_max = __longlong_as_double(0x7ff0000000000000ll);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            im_max = fmax(im_max, __shfl_xor_sync(0xffffffffu, im_max, off));
            re_max = fmax(re_max, __shfl_xor_sync(0xffffffffu, re_max, off));
        }
        if ((threadIdx.x & 31) == 0) {
            if (im_max > 0.0) atomicMax(&info->im_residual_bits, (unsigned long long)__double_as_longlong(im_max));
            if (re_max > 0.0) atomicMax(&info->re_max_bits, (unsigned long long)__double_as_longlong(re_max));
        }
    }
}

}  // namespace

int launch_cyc_recover(draco_plan* p, const float2* R, int64_t len, int64_t ld, float* u, int64_t d_packed,
                       cudaStream_t st, float* w, float scale) {
    const bool packed = d_packed > 0;
    // 64-bit stores of u need len even; in packed mode the second half starts at u + len and must cover it fully
    const bool vec2 = (len % 2 == 0) && (ld % 2 == 0) && (!packed || d_packed == 2 * len);
    const int64_t nvec = vec2 ? len / 2 : len;
    int64_t want = (nvec + kThreads - 1) / kThreads;
    const int64_t cap = (int64_t)p->sm_count * 16;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
#define DRACO_REC(V2, PK) \
    cyc_recover_kernel<V2, PK><<<(int)want, kThreads, 0, st>>>(R, len, ld, p->cyc_dev, p->info_dev, u, d_packed, w, scale)
    if (vec2) {
        if (packed) DRACO_REC(true, true); else DRACO_REC(true, false);
    } else {
        if (packed) DRACO_REC(false, true); else DRACO_REC(false, false);
    }
#undef DRACO_REC
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

}  // namespace draco

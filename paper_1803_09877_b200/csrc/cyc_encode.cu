// Cyclic-code encoder (Section 3, "Cyclic Code"): Z = G W, z_j = G W_{.,j}.
//
// W = [Q 1_P] C_L has the closed form W[j][k] = n^(-1/2) prod_{m in alpha_j} (w^k - w^m),
// w = exp(2 pi i / n), alpha_j = {j+2s+1 .. j+n-1} mod n, so its rows are shifted copies of
// row 0 up to a unit phase: W[j][k] = w^(j M) W[0][(k - j) mod n], M = n - 2 s - 1.  Hence
//
//     z_j = phase[j] * sum_{t=0..2s} tap[t] * g_{(j - t) mod n},
//     tap[t] = w^(-t M) W[0][t],   phase[j] = w^(j M):
//
// one fixed (2 s + 1)-tap complex filter run around the circle of gradients, then one unit
// rotation per output.  The taps do not depend on j, so they sit in the kernel's constant
// parameter bank and every multiply-add takes its coefficient from there.
//
// A thread owns 4 consecutive coordinates and walks the n rows once, keeping a sliding
// window of 2 s + 1 rows (plus PF rows of prefetch) in registers; the first 2 s rows of the
// circle are fetched a second time at the end of the walk (they come from L2).
// HBM traffic: 4 n len bytes read + 8 n len bytes written; 2 n (2 s + 1) FMA per coordinate.
#include "draco_internal.cuh"

namespace draco {

namespace {

constexpr int kThreads = 256;

template <int S, int PF>
__global__ void __launch_bounds__(kThreads, 2)
cyc_encode_kernel(const float* __restrict__ G, float2* __restrict__ Z, int64_t len, int64_t ldg, int64_t ldz, int n,
                  const __grid_constant__ EncodeTaps taps, const __grid_constant__ EncodePhase ph) {
    constexpr int R = 2 * S + 1;
    constexpr int SLOTS = R + PF;
    const int total = n + 2 * S;          // virtual rows: the last 2 s rows of the circle, then rows 0 .. n-1
    const int64_t nvec = len / 4;
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    for (int64_t v = (int64_t)blockIdx.x * kThreads + threadIdx.x; v < nvec; v += stride) {
        const float* gcol = G + v * 4;
        float2* zcol = Z + v * 4;
        float4 win[SLOTS];
#pragma unroll
        for (int p = 0; p < PF; ++p) {
            if (p < total) {
                int r = p - 2 * S;
                if (r < 0) r += n;
                win[p] = __ldcs(reinterpret_cast<const float4*>(gcol + (int64_t)r * ldg));
            }
        }
        for (int v0 = 0; v0 < total; v0 += SLOTS) {
#pragma unroll
            for (int p = 0; p < SLOTS; ++p) {
                const int vv = v0 + p;
                if (vv < total) {
                    if (vv + PF < total) {
                        int r = vv + PF - 2 * S;
                        if (r < 0) r += n;
                        win[(p + PF) % SLOTS] = __ldcs(reinterpret_cast<const float4*>(gcol + (int64_t)r * ldg));
                    }
                    if (vv >= 2 * S) {
                        const int j = vv - 2 * S;
                        float ar0 = 0.f, ar1 = 0.f, ar2 = 0.f, ar3 = 0.f;
                        float ai0 = 0.f, ai1 = 0.f, ai2 = 0.f, ai3 = 0.f;
#pragma unroll
                        for (int t = 0; t < R; ++t) {
                            const float4 g = win[(p - t + 2 * SLOTS) % SLOTS];
                            const float cr = taps.tap[t].x, ci = taps.tap[t].y;
                            ar0 = fmaf(cr, g.x, ar0); ai0 = fmaf(ci, g.x, ai0);
                            ar1 = fmaf(cr, g.y, ar1); ai1 = fmaf(ci, g.y, ai1);
                            ar2 = fmaf(cr, g.z, ar2); ai2 = fmaf(ci, g.z, ai2);
                            ar3 = fmaf(cr, g.w, ar3); ai3 = fmaf(ci, g.w, ai3);
                        }
                        const float2 w = ph.phase[j];
                        float4 lo, hi;
                        lo.x = fmaf(ar0, w.x, -ai0 * w.y); lo.y = fmaf(ar0, w.y, ai0 * w.x);
                        lo.z = fmaf(ar1, w.x, -ai1 * w.y); lo.w = fmaf(ar1, w.y, ai1 * w.x);
                        hi.x = fmaf(ar2, w.x, -ai2 * w.y); hi.y = fmaf(ar2, w.y, ai2 * w.x);
                        hi.z = fmaf(ar3, w.x, -ai3 * w.y); hi.w = fmaf(ar3, w.y, ai3 * w.x);
                        float4* dst = reinterpret_cast<float4*>(zcol + (int64_t)j * ldz);
                        __stcs(dst, lo);
                        __stcs(dst + 1, hi);
                    }
                }
            }
        }
    }
}

// Any s, any length / alignment: one coordinate per thread, rows re-read through the caches.
__global__ void __launch_bounds__(kThreads)
cyc_encode_generic_kernel(const float* __restrict__ G, float2* __restrict__ Z, int64_t len, int64_t ldg, int64_t ldz,
                          int n, int s,
                          const float2* __restrict__ taps, const __grid_constant__ EncodePhase ph) {
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < len; i += stride) {
        for (int j = 0; j < n; ++j) {
            float ar = 0.f, ai = 0.f;
            for (int t = 0; t <= 2 * s; ++t) {
                int r = j - t;
                if (r < 0) r += n;
                const float g = G[(int64_t)r * ldg + i];
                const float2 c = taps[t];
                ar = fmaf(c.x, g, ar);
                ai = fmaf(c.y, g, ai);
            }
            const float2 w = ph.phase[j];
            Z[(int64_t)j * ldz + i] = make_float2(fmaf(ar, w.x, -ai * w.y), fmaf(ar, w.y, ai * w.x));
        }
    }
}

template <int S>
void launch_fast(const draco_plan* p, const float* G, float2* Z, int64_t len, int64_t ldg, int64_t ldz, cudaStream_t st) {
    constexpr int PF = 6;
    const int64_t nvec = len / 4;
    int64_t want = (nvec + kThreads - 1) / kThreads;
    const int64_t cap = (int64_t)p->sm_count * 2 * 8;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    cyc_encode_kernel<S, PF><<<(int)want, kThreads, 0, st>>>(G, Z, len, ldg, ldz, p->n, p->taps, p->phase);
}

}  // namespace

int launch_cyc_encode(const draco_plan* p, const float* G, float2* Z, int64_t len, int64_t ldg, int64_t ldz,
                      cudaStream_t st) {
    const bool fast = (len % 4 == 0) && (ldg % 4 == 0) && (ldz % 2 == 0) && p->s <= 7;
    if (fast) {
        switch (p->s) {
            case 0: launch_fast<0>(p, G, Z, len, ldg, ldz, st); break;
            case 1: launch_fast<1>(p, G, Z, len, ldg, ldz, st); break;
            case 2: launch_fast<2>(p, G, Z, len, ldg, ldz, st); break;
            case 3: launch_fast<3>(p, G, Z, len, ldg, ldz, st); break;
            case 4: launch_fast<4>(p, G, Z, len, ldg, ldz, st); break;
            case 5: launch_fast<5>(p, G, Z, len, ldg, ldz, st); break;
            case 6: launch_fast<6>(p, G, Z, len, ldg, ldz, st); break;
            default: launch_fast<7>(p, G, Z, len, ldg, ldz, st); break;
        }
    } else {
        int64_t want = (len + kThreads - 1) / kThreads;
        const int64_t cap = (int64_t)p->sm_count * 16;
        if (want > cap) want = cap;
        if (want < 1) want = 1;
        cyc_encode_generic_kernel<<<(int)want, kThreads, 0, st>>>(G, Z, len, ldg, ldz, p->n, p->s, p->taps_full_dev, p->phase);
    }
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

}  // namespace draco

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
// Data movement.  A thread block owns a tile of 1536 coordinates (1408 for s >= 6) and walks the n rows
// once.  One producer lane streams the row tiles (6 KB each) from global memory into a ring of
// shared-memory stages with bulk asynchronous copies (cp.async.bulk + mbarrier, no
// multicast); 12 (11) consumer warps take each row from the ring into a register window of the
// last 2 s + 1 rows, 4 coordinates per thread.  The first 2 s rows are also kept in shared
// memory, because the circle closes on them at the end of the walk; nothing is read twice.
// HBM traffic is the algorithmic minimum: 4 n len bytes read + 8 n len bytes written.
//
// Arithmetic.  |tap| peaks in the middle of the filter (1.8e5 at n = 45, s = 5) and decoding
// cancels the sum back to O(1), so rounding in the encoder is amplified by that factor.  The
// outer taps are accumulated in fp32, smallest first; the three centre taps, the rotation
// and the final sum run in fp64, and each output is rounded to fp32 once.  That keeps the
// encoder at the accuracy floor of complex64 transport (2 n (2 s + 1) FMA per coordinate,
// of which 6 n + 4 n in fp64).
#include "draco_internal.cuh"

namespace draco {

namespace {

constexpr int kVec = 4;                         // coordinates per consumer thread
// Block shape per s.  A scheduler's 16 K registers cap a thread at 128 registers once it hosts 4 warps,
// and the s >= 6 window needs about 155: those kernels run 11 consumer warps + the producer (3 warps per
// scheduler) instead of 12 + 1 (measured at n = 45: 7.1 ms against 8.0 ms with spills; for s = 5 the
// 12-warp shape is the faster one, 6.0 ms against 6.4 ms).
template <int S>
struct RingCfg {
    static constexpr int kConsumers = S >= 6 ? 352 : 384;    // consumer threads; the next warp is the producer
    static constexpr int kThreads = kConsumers + 32;
    static constexpr int kTile = kConsumers * kVec;           // coordinates per tile = floats per stage
};
constexpr int kStages = 16;                     // ring depth (up to 96 KB in flight per block)
static_assert((kStages & (kStages - 1)) == 0, "stage indices and parities are derived with masks: kStages must be a power of two");
constexpr int kGenericThreads = 256;

// ---------------------------------------------------------------- mbarrier / bulk-copy wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t a, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(a), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t a, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(a), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t a, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(a), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: every wait in this file gives up after about 4 M polls (seconds), so a
// protocol error ends the kernel with an error flag instead of hanging the device.
__device__ __noinline__ bool mbar_wait_slow(uint32_t a, uint32_t parity) {
    for (int i = 0; i < (1 << 22); ++i)
        if (mbar_try_wait(a, parity)) return true;
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t a, uint32_t parity) {
    if (mbar_try_wait(a, parity)) return true;
    return mbar_wait_slow(a, parity);
}
// Hand a ring stage back to the producer after its contents were read into registers with
// value bits `bits`.  The arrival count is 1 + ((bits * bits + bits) & 1) = 1 (x (x + 1) is
// even), written so that the instruction carries a true register dependency on the loaded
// data: the stage cannot be returned to the copy engine (which overwrites it through the
// asynchronous proxy) before the shared-memory read that produced `bits` has completed.
// Releasing straight after issuing the read lost that race under load.
__device__ __forceinline__ void mbar_release_after_read(uint32_t a, uint32_t bits) {
    const uint32_t count = 1u + ((bits * bits + bits) & 1u);
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(a), "r"(count) : "memory");
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t mbar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(mbar)
                 : "memory");
}

// ---------------------------------------------------------------- consumer state
template <int S>
struct Window {
    static constexpr int R = 2 * S + 1;
    static constexpr int NBIG = R < 3 ? R : 3;                     // centre taps in fp64
    static constexpr int H = (NBIG - 1) / 2;
    static constexpr int SL = ((R + NBIG - 1) / NBIG) * NBIG;      // register slots: a multiple of NBIG
    float4 win[SL];                                                // rows (vv - t), slot = vv mod SL
    double cw[NBIG][4];                                            // fp64 copies of the rows under the centre taps
};

struct RingState {
    uint32_t full0, empty0;      // shared addresses of the barrier arrays
    uint32_t st, par;            // next stage to consume and its phase parity
    uint32_t pend_bar, pend_bits;
    bool pending;                // a stage was read in the previous step and is not released yet
};

// One step of the walk: bring row vv of the tile into window slot P (from the ring, or from
// the stash once the circle has closed), and emit z_{vv mod n} when the window is full.
// MODE 0: first SL steps of a tile (all rows from the ring; outputs from step 2 S on; nothing
//         pending at step 0);  MODE 1: steady state (ring row + output, previous stage pending);
// MODE 2: anything (run-time guards).  Returns false when a wait gave up.
template <int S, int P, int MODE, bool PACKED>
__device__ __forceinline__ bool encode_step(Window<S>& w, RingState& rs, int vv, int n, const float* ring_t,
                                            float* stash_t, float2* zcol, int64_t ldz, int active, int lane,
                                            const EncodeTaps& taps, const EncodeTaps64& taps64,
                                            const EncodePhase64& ph64) {
    constexpr int R = Window<S>::R, NBIG = Window<S>::NBIG, H = Window<S>::H, SL = Window<S>::SL;
    constexpr int kTile = RingCfg<S>::kTile;
    const int total = n + 2 * S;
    if (MODE == 2 && vv >= total) return true;
    const bool from_ring = (MODE != 2) || (vv < n);
    const bool release_first = (MODE == 1) || (MODE == 0 && P > 0) || (MODE == 2 && rs.pending);
    if (release_first) {
        __syncwarp();
        if (lane == 0) mbar_release_after_read(rs.pend_bar, rs.pend_bits);
        rs.pending = false;
    }
    float4 x;
    if (from_ring) {
        const uint32_t bar = rs.full0 + 8 * rs.st;
        if (!mbar_wait(bar, rs.par)) return false;
        if (PACKED) {      // first half of the gradient -> real parts, second half -> imaginary parts
            const float2 a = *reinterpret_cast<const float2*>(ring_t + rs.st * kTile);
            const float2 b = *reinterpret_cast<const float2*>(ring_t + rs.st * kTile + kTile / 2);
            x = make_float4(a.x, a.y, b.x, b.y);
        } else {           // coordinates 2l, 2l+1 and 64+2l, 64+2l+1 of the warp's 128: see the stores below
            const float2 a = *reinterpret_cast<const float2*>(ring_t + rs.st * kTile);
            const float2 b = *reinterpret_cast<const float2*>(ring_t + rs.st * kTile + 64);
            x = make_float4(a.x, a.y, b.x, b.y);
        }
        rs.pend_bar = rs.empty0 + 8 * rs.st;
        rs.pend_bits = __float_as_uint(x.x);
        rs.pending = true;
        rs.st = (rs.st + 1) & (kStages - 1);
        rs.par ^= (rs.st == 0);
        if ((MODE == 0 && P < 2 * S) || (MODE == 2 && vv < 2 * S))
            *reinterpret_cast<float4*>(stash_t + vv * kTile) = x;
    } else {
        x = *reinterpret_cast<const float4*>(stash_t + (vv - n) * kTile);
    }
    w.win[P] = x;
    if (MODE != 2 || vv >= S - H) {          // the row now under tap S-H enters the fp64 window
        constexpr int Q = (P - (S - H) + 2 * SL) % SL;
        w.cw[Q % NBIG][0] = (double)w.win[Q].x;
        w.cw[Q % NBIG][1] = (double)w.win[Q].y;
        w.cw[Q % NBIG][2] = (double)w.win[Q].z;
        w.cw[Q % NBIG][3] = (double)w.win[Q].w;
    }
    const bool emit = (MODE == 1) || (MODE == 0 && P >= 2 * S) || (MODE == 2 && vv >= 2 * S);
    if (emit) {
        // win[(P - t) mod SL] = row (vv - t) mod n: this output is z_j, j = vv mod n
        const int j = (MODE == 2 && vv >= n) ? vv - n : vv;
        float ar[4] = {0.f, 0.f, 0.f, 0.f}, ai[4] = {0.f, 0.f, 0.f, 0.f};
        // taps grow towards the middle of the filter: add the outer (small) terms first so the
        // running sums stay small while most of the fp32 roundings happen
#pragma unroll
        for (int k = 0; k < R; ++k) {
            const int t = (k & 1) ? 2 * S - (k >> 1) : (k >> 1);
            if (t >= S - H && t <= S + H) continue;
            const float4 g = w.win[(P - t + 2 * SL) % SL];
            const float cr = taps.tap[t].x, ci = taps.tap[t].y;
            ar[0] = fmaf(cr, g.x, ar[0]); ai[0] = fmaf(ci, g.x, ai[0]);
            ar[1] = fmaf(cr, g.y, ar[1]); ai[1] = fmaf(ci, g.y, ai[1]);
            ar[2] = fmaf(cr, g.z, ar[2]); ai[2] = fmaf(ci, g.z, ai[2]);
            ar[3] = fmaf(cr, g.w, ar[3]); ai[3] = fmaf(ci, g.w, ai[3]);
        }
        double dr[4], di[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) { dr[c] = (double)ar[c]; di[c] = (double)ai[c]; }
#pragma unroll
        for (int t = S - H; t <= S + H; ++t) {
            constexpr int dummy = 0;
            (void)dummy;
            const int q = ((P - t + 2 * SL) % SL) % NBIG;
            const double cr = taps64.tap[t].x, ci = taps64.tap[t].y;
#pragma unroll
            for (int c = 0; c < 4; ++c) { dr[c] = fma(cr, w.cw[q][c], dr[c]); di[c] = fma(ci, w.cw[q][c], di[c]); }
        }
        const double2 rot = ph64.phase[j];
        double xr[4], xi[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            xr[c] = fma(dr[c], rot.x, -di[c] * rot.y);
            xi[c] = fma(dr[c], rot.y, di[c] * rot.x);
        }
        if (PACKED) {
            // components 0,1 filtered the real parts (X), 2,3 the imaginary parts (Y): z = X + i Y
            if (active & 1) {
                float4* dst = reinterpret_cast<float4*>(zcol + (int64_t)j * ldz);
                __stcs(dst, make_float4((float)(xr[0] - xi[2]), (float)(xi[0] + xr[2]), (float)(xr[1] - xi[3]),
                                        (float)(xi[1] + xr[3])));
            }
        } else {
            // A lane's two 16-byte stores are 512 bytes apart, so that each store instruction of the warp
            // covers 512 contiguous bytes (whole 32-byte sectors).  With the 4 coordinates of a lane adjacent,
            // every instruction wrote half of 32 sectors and the kernel stopped at 4.9 TB/s.
            float2* dst = zcol + (int64_t)j * ldz;
            if (active & 1) __stcs(reinterpret_cast<float4*>(dst), make_float4((float)xr[0], (float)xi[0], (float)xr[1], (float)xi[1]));
            if (active & 2) __stcs(reinterpret_cast<float4*>(dst + 64), make_float4((float)xr[2], (float)xi[2], (float)xr[3], (float)xi[3]));
        }
    }
    return true;
}

template <int S, int MODE, bool PACKED, int P = 0>
__device__ __forceinline__ bool encode_chunk(Window<S>& w, RingState& rs, int v0, int n, const float* ring_t,
                                             float* stash_t, float2* zcol, int64_t ldz, int active, int lane,
                                             const EncodeTaps& taps, const EncodeTaps64& taps64,
                                             const EncodePhase64& ph64) {
    if constexpr (P < Window<S>::SL) {
        if (!encode_step<S, P, MODE, PACKED>(w, rs, v0 + P, n, ring_t, stash_t, zcol, ldz, active, lane, taps, taps64, ph64))
            return false;
        return encode_chunk<S, MODE, PACKED, P + 1>(w, rs, v0, n, ring_t, stash_t, zcol, ldz, active, lane, taps, taps64, ph64);
    } else {
        return true;
    }
}

// PACKED: the real -> complex packing of Section 3's last paragraph.  `len` then counts complex
// coordinates, a tile holds kTile / 2 of them, and a stage receives two slices of each row:
// G[r][c0 ..] (real parts) and G[r][half + c0 ..] (imaginary parts).
template <int S, bool PACKED>
__global__ void __launch_bounds__(RingCfg<S>::kThreads, 1)
cyc_encode_ring_kernel(const float* __restrict__ G, float2* __restrict__ Z, int64_t len, int64_t ldg, int64_t ldz,
                       int64_t half, int n,
                       const __grid_constant__ EncodeTaps taps, const __grid_constant__ EncodeTaps64 taps64,
                       const __grid_constant__ EncodePhase64 ph64, int* err) {
    constexpr int SL = Window<S>::SL;
    constexpr int NSTASH = S > 0 ? 2 * S : 1;
    constexpr int kConsumers = RingCfg<S>::kConsumers, kTile = RingCfg<S>::kTile;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float* ring = reinterpret_cast<float*>(smem_raw);                        // [kStages][kTile]
    float* stash = ring + kStages * kTile;                                   // [2 S][kTile]
    uint64_t* bars = reinterpret_cast<uint64_t*>(stash + NSTASH * kTile);    // full[kStages], empty[kStages]
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + kStages);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(full0 + 8 * i, 1);
            mbar_init(empty0 + 8 * i, kConsumers / 32);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    constexpr int kTileCoords = PACKED ? kTile / 2 : kTile;      // coordinates of Z per tile
    constexpr int kPerThread = PACKED ? 2 : kVec;
    const int64_t ntiles = (len + kTileCoords - 1) / kTileCoords;

    if (warp == kConsumers / 32) {
        // ---------------- producer: one lane streams row tiles into the ring
        if (lane == 0) {
            uint32_t cnt = 0;
            bool ok = true;
            for (int64_t tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                const int64_t c0 = tile * kTileCoords;
                const uint32_t bytes = (uint32_t)(((len - c0) < kTileCoords ? (len - c0) : kTileCoords) * 4);
                const float* src = G + c0;
                for (int r = 0; r < n; ++r, ++cnt, src += ldg) {
                    const uint32_t st = cnt & (kStages - 1), par = (cnt / kStages) & 1;
                    if (!mbar_wait(empty0 + 8 * st, par ^ 1)) { ok = false; break; }
                    mbar_expect_tx(full0 + 8 * st, PACKED ? 2 * bytes : bytes);
                    bulk_g2s(smem_u32(ring + st * kTile), src, bytes, full0 + 8 * st);
                    if (PACKED) bulk_g2s(smem_u32(ring + st * kTile + kTile / 2), src + half, bytes, full0 + 8 * st);
                }
            }
            if (!ok) {
                atomicExch(err, 1);
                // let the copies already in flight land before the block's shared memory is released
                for (uint32_t back = 1; back <= kStages && back <= cnt; ++back) {
                    const uint32_t c = cnt - back;
                    mbar_wait(full0 + 8 * (c & (kStages - 1)), (c / kStages) & 1);
                }
            }
        }
        return;
    }

    // ---------------- consumers
    Window<S> w;
    RingState rs;
    rs.full0 = full0; rs.empty0 = empty0; rs.st = 0; rs.par = 0;
    rs.pend_bar = 0; rs.pend_bits = 0; rs.pending = false;
    // unpacked: a lane owns coordinates 2l, 2l+1, 64+2l, 64+2l+1 of its warp's 128; packed: entries 2 tid, 2 tid + 1
    const int first = PACKED ? tid * 2 : warp * 128 + lane * 2;
    const float* ring_t = ring + first;
    float* stash_t = stash + tid * kVec;
    const int total = n + 2 * S;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const int64_t c0 = tile * kTileCoords;
        const int active = (c0 + first < len ? 1 : 0) | ((PACKED || c0 + first + 64 < len) ? 2 : 0);
        float2* zcol = Z + c0 + first;
        bool ok = true;
        int v0 = 0;
        if (n >= SL && S > 0) {
            ok = encode_chunk<S, 0, PACKED>(w, rs, 0, n, ring_t, stash_t, zcol, ldz, active, lane, taps, taps64, ph64);
            for (v0 = SL; ok && v0 + SL <= n; v0 += SL)
                ok = encode_chunk<S, 1, PACKED>(w, rs, v0, n, ring_t, stash_t, zcol, ldz, active, lane, taps, taps64, ph64);
        }
        for (; ok && v0 < total; v0 += SL)
            ok = encode_chunk<S, 2, PACKED>(w, rs, v0, n, ring_t, stash_t, zcol, ldz, active, lane, taps, taps64, ph64);
        if (!ok) {
            atomicExch(err, 2);
            return;
        }
        if (rs.pending) {                      // only when the tile ended on a ring row (s = 0)
            __syncwarp();
            if (lane == 0) mbar_release_after_read(rs.pend_bar, rs.pend_bits);
            rs.pending = false;
        }
    }
}

// Any s, any length / alignment: one coordinate per thread, rows re-read through the caches,
// fp64 accumulation throughout.  half > 0: packed mode (len complex coordinates; the imaginary
// parts come from G[r][half + i], zero beyond d_real).
__global__ void __launch_bounds__(kGenericThreads)
cyc_encode_generic_kernel(const float* __restrict__ G, float2* __restrict__ Z, int64_t len, int64_t ldg, int64_t ldz,
                          int64_t half, int64_t d_real, int n, int s, const float2* __restrict__ taps,
                          const __grid_constant__ EncodePhase64 ph) {
    const int64_t stride = (int64_t)gridDim.x * kGenericThreads;
    for (int64_t i = (int64_t)blockIdx.x * kGenericThreads + threadIdx.x; i < len; i += stride) {
        const bool has_b = half > 0 && half + i < d_real;
        for (int j = 0; j < n; ++j) {
            double ar = 0.0, ai = 0.0, br = 0.0, bi = 0.0;
            for (int t = 0; t <= 2 * s; ++t) {
                int r = j - t;
                if (r < 0) r += n;
                const float2 c = taps[t];
                const double g = (double)G[(int64_t)r * ldg + i];
                ar = fma((double)c.x, g, ar);
                ai = fma((double)c.y, g, ai);
                if (has_b) {
                    const double gb = (double)G[(int64_t)r * ldg + half + i];
                    br = fma((double)c.x, gb, br);
                    bi = fma((double)c.y, gb, bi);
                }
            }
            const double2 rot = ph.phase[j];
            const double xr = fma(ar, rot.x, -ai * rot.y), xi = fma(ar, rot.y, ai * rot.x);
            const double yr = fma(br, rot.x, -bi * rot.y), yi = fma(br, rot.y, bi * rot.x);
            Z[(int64_t)j * ldz + i] = make_float2((float)(xr - yi), (float)(xi + yr));
        }
    }
}

template <int S, bool PACKED>
int launch_ring(const draco_plan* p, const float* G, float2* Z, int64_t len, int64_t ldg, int64_t ldz, int64_t half,
                cudaStream_t st) {
    constexpr int NSTASH = S > 0 ? 2 * S : 1;
    constexpr int kTile = RingCfg<S>::kTile, kRingThreads = RingCfg<S>::kThreads;
    const size_t smem = sizeof(float) * kTile * (kStages + NSTASH) + 16 * kStages;
    auto kern = cyc_encode_ring_kernel<S, PACKED>;
    static bool configured[64] = {};
    int dev = p->device;
    if (dev < 0 || dev >= 64) dev = 0;
    if (!configured[dev]) {
        DRACO_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        configured[dev] = true;
    }
    int per_sm = 1;
    DRACO_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kRingThreads, smem));
    if (per_sm < 1) per_sm = 1;
    constexpr int kTileCoords = PACKED ? kTile / 2 : kTile;
    const int64_t ntiles = (len + kTileCoords - 1) / kTileCoords;
    int64_t grid = (int64_t)p->sm_count * per_sm;
    if (grid > ntiles) grid = ntiles;
    if (grid < 1) grid = 1;
    kern<<<(int)grid, kRingThreads, smem, st>>>(G, Z, len, ldg, ldz, half, p->n, p->taps, p->taps64, p->phase64,
                                               &p->info_dev->internal_error);
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

template <bool PACKED>
int launch_ring_any(const draco_plan* p, const float* G, float2* Z, int64_t len, int64_t ldg, int64_t ldz, int64_t half,
                    cudaStream_t st) {
    switch (p->s) {
        case 0: return launch_ring<0, PACKED>(p, G, Z, len, ldg, ldz, half, st);
        case 1: return launch_ring<1, PACKED>(p, G, Z, len, ldg, ldz, half, st);
        case 2: return launch_ring<2, PACKED>(p, G, Z, len, ldg, ldz, half, st);
        case 3: return launch_ring<3, PACKED>(p, G, Z, len, ldg, ldz, half, st);
        case 4: return launch_ring<4, PACKED>(p, G, Z, len, ldg, ldz, half, st);
        case 5: return launch_ring<5, PACKED>(p, G, Z, len, ldg, ldz, half, st);
        case 6: return launch_ring<6, PACKED>(p, G, Z, len, ldg, ldz, half, st);
        default: return launch_ring<7, PACKED>(p, G, Z, len, ldg, ldz, half, st);
    }
}

}  // namespace

// half == 0: Z[j][i], i < len, from G[.][i].  half > 0 (packed): Z[j][i], i < len complex coordinates,
// from G[.][i] (real parts) and G[.][half + i] (imaginary parts, zero for half + i >= d_real).
int launch_cyc_encode(const draco_plan* p, const float* G, float2* Z, int64_t len, int64_t ldg, int64_t ldz,
                      int64_t half, int64_t d_real, cudaStream_t st) {
    // the ring kernel needs 16-byte aligned row slices: row starts, tile starts and the half offset multiples of 4 floats
    const bool packed = half > 0;
    bool fast = (ldg % 4 == 0) && (ldz % 2 == 0) && p->s <= 7;
    if (packed) fast = fast && (len % 4 == 0) && (half % 4 == 0) && (half + len <= d_real);
    else fast = fast && (len % 4 == 0);
    if (fast) return packed ? launch_ring_any<true>(p, G, Z, len, ldg, ldz, half, st)
                            : launch_ring_any<false>(p, G, Z, len, ldg, ldz, 0, st);
    int64_t want = (len + kGenericThreads - 1) / kGenericThreads;
    const int64_t cap = (int64_t)p->sm_count * 16;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    cyc_encode_generic_kernel<<<(int)want, kGenericThreads, 0, st>>>(G, Z, len, ldg, ldz, half, d_real, p->n, p->s,
                                                                     p->taps_full_dev, p->phase64);
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

}  // namespace draco

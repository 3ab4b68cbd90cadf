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
// Data movement.  Every warp walks strips of 128 coordinates (64 complex coordinates in packed mode)
// on its own, a lane owning 4 of them, and visits the n rows of a strip once.  Each lane streams its
// 16 bytes of every row from global memory into a private column of a shared-memory ring with
// asynchronous copies (cp.async, one group per row, 12 rows in flight, running on into the next strip),
// and takes them from there into a register window of the last 2 s + 1 rows.  No thread reads what
// another thread copied, so the kernel has no barrier, no flag and no wait other than
// cp.async.wait_group.  The first 2 s rows of a strip are also kept in shared memory, because the
// circle closes on them at the end of the walk; nothing is read twice.
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

constexpr int kVec = 4;                         // coordinates per thread
constexpr int kRing = 12;                       // rows in flight per thread
constexpr int kGenericThreads = 256;

// Shapes per s.  The window of the s >= 3 kernels needs 140-168 registers, which a scheduler's 16 K
// registers allow for 3 warps: 12 warps per block, one block per SM.  The s <= 2 kernels fit in 128
// registers and run 16 warps.
template <int S>
struct StreamCfg {
    static constexpr int R = 2 * S + 1;                            // taps
    static constexpr int NBIG = R < 3 ? R : 3;                     // centre taps in fp64
    static constexpr int H = (NBIG - 1) / 2;
    static constexpr int SL = ((R + NBIG - 1) / NBIG) * NBIG;      // register slots: a multiple of NBIG
    static constexpr int kThreads = S <= 2 ? 512 : 384;
    static constexpr int NSTASH = S > 0 ? 2 * S : 1;
    static constexpr uint32_t kRowBytes = kThreads * 16;           // one ring / stash row: 16 bytes per thread
    static constexpr size_t kSmem = (size_t)kRowBytes * (kRing + NSTASH);
};

// ---------------------------------------------------------------- asynchronous-copy and shared-memory wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// The same copy with its source switched off by a predicate (ignore-src: zeros are written, src is not read), so that
// a lane outside the vector needs no branch around its copies.
__device__ __forceinline__ void cp_async8_if(uint32_t dst, const void* src, bool on) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, %2, 0;\n\tcp.async.ca.shared.global [%0], [%1], 8, p;\n\t}" ::"r"(dst), "l"(src), "r"((uint32_t)on) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {          // at most N of this thread's groups still pending
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ float4 lds128(uint32_t a) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ void sts128(uint32_t a, float4 v) {
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(a), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}

// ---------------------------------------------------------------- per-thread state
template <int S>
struct Window {
    float4 win[StreamCfg<S>::SL];                  // rows (vv - t), slot = vv mod SL
    double cw[StreamCfg<S>::NBIG][4];              // fp64 copies of the rows under the centre taps
};

// The fetch side: the rows of this warp's strips, one after the other, kRing rows ahead of the row being
// consumed.  A lane copies coordinates 2l, 2l+1 and 64+2l, 64+2l+1 of the strip (packed: complex
// coordinates 2l, 2l+1, real parts from G[r][c], imaginary parts from G[r][half + c]).
template <bool PACKED>
struct Fetcher {
    const float* G;
    const float* ga;            // this lane's first pair in the next row to fetch
    int64_t boff;               // from there to its second pair: 64, or `half` when PACKED
    int64_t boff_now;           // the same, 0 while the second pair is switched off
    int64_t strip, nstrips, strip_step, len, ldg;
    int row, n, lane;
    bool act0, act1;            // the pairs lie inside the vector (and the strip exists)
    __device__ __forceinline__ void open_strip() {
        constexpr int kStrip = PACKED ? 64 : 128;
        const int64_t c = strip * kStrip + 2 * lane;
        act0 = strip < nstrips && c < len;
        act1 = PACKED ? act0 : (strip < nstrips && c + 64 < len);
        // switched-off copies still carry an address: keep it inside the matrix (this lane's first pair of strip 0, and
        // the first pair again for a second pair beyond the row's end)
        ga = G + (act0 ? c : (int64_t)(2 * lane < len ? 2 * lane : 0));
        boff_now = act1 ? boff : 0;
        row = 0;
    }
    // copy this lane's 16 bytes of the next row to shared address dst and close the group (copies of a lane
    // outside the vector are switched off; every thread counts the same groups)
    __device__ __forceinline__ void fetch(uint32_t dst) {
        cp_async8_if(dst, ga, act0);
        cp_async8_if(dst + 8, ga + boff_now, act1);
        cp_async_commit();
        ga += ldg;
        if (++row == n) {
            strip += strip_step;
            open_strip();
        }
    }
};

struct Cursor {
    uint32_t ring0, rd;         // this thread's column of the ring, and the byte offset of the next row to consume
    float2* zout;               // next output row (modes 0 and 1)
};

// One step of the walk: bring row vv of the strip into window slot P (from the ring, or from the stash once
// the circle has closed), emit z_{vv mod n} when the window is full, and refill the ring slot.
// MODE 0: first SL steps of a strip (all rows from the ring; outputs from step 2 S on);
// MODE 1: steady state (ring row + output);  MODE 2: anything (run-time guards).
template <int S, int P, int MODE, bool PACKED>
__device__ __forceinline__ void encode_step(Window<S>& w, Cursor& cur, Fetcher<PACKED>& f, int vv, int n, int64_t ldz,
                                            uint32_t stash0, float2* zcol, bool act0, bool act1,
                                            const EncodeTaps& taps, const EncodeTaps64& taps64,
                                            const EncodePhase64& ph64) {
    using Cfg = StreamCfg<S>;
    constexpr int R = Cfg::R, NBIG = Cfg::NBIG, H = Cfg::H, SL = Cfg::SL;
    constexpr uint32_t kRowBytes = Cfg::kRowBytes;
    const int total = n + 2 * S;
    if (MODE == 2 && vv >= total) return;
    const bool from_ring = (MODE != 2) || (vv < n);
    float4 x;
    if (from_ring) {
        cp_async_wait<kRing - 1>();          // kRing groups were committed after the one that carries this row
        x = lds128(cur.ring0 + cur.rd);
        if ((MODE == 0 && P < 2 * S) || (MODE == 2 && vv < 2 * S)) sts128(stash0 + (uint32_t)vv * kRowBytes, x);
    } else {
        x = lds128(stash0 + (uint32_t)(vv - n) * kRowBytes);
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
        float2* dst;
        if (MODE == 2) {
            dst = zcol + (int64_t)j * ldz;
        } else {
            dst = cur.zout;
            cur.zout += ldz;
        }
        if (PACKED) {
            // components 0,1 filtered the real parts (X), 2,3 the imaginary parts (Y): z = X + i Y
            if (act0)
                __stcs(reinterpret_cast<float4*>(dst), make_float4((float)(xr[0] - xi[2]), (float)(xi[0] + xr[2]),
                                                                   (float)(xr[1] - xi[3]), (float)(xi[1] + xr[3])));
        } else {
            // A lane's two 16-byte stores are 512 bytes apart, so that each store instruction of the warp
            // covers 512 contiguous bytes (whole 32-byte sectors).  With the 4 coordinates of a lane adjacent,
            // every instruction wrote half of 32 sectors and the kernel stopped at 4.9 TB/s.
            if (act0) __stcs(reinterpret_cast<float4*>(dst), make_float4((float)xr[0], (float)xi[0], (float)xr[1], (float)xi[1]));
            if (act1) __stcs(reinterpret_cast<float4*>(dst + 64), make_float4((float)xr[2], (float)xi[2], (float)xr[3], (float)xi[3]));
        }
    }
    if (from_ring) {
        // The slot just consumed is refilled with the row kRing ahead.  Its read has completed by then: the stash
        // store or the global stores above need the value read and come before the copy in program order (a lane
        // without stores issues no copy either).
        f.fetch(cur.ring0 + cur.rd);
        cur.rd += kRowBytes;
        if (cur.rd == kRing * kRowBytes) cur.rd = 0;
    }
}

template <int S, int MODE, bool PACKED, int P = 0>
__device__ __forceinline__ void encode_chunk(Window<S>& w, Cursor& cur, Fetcher<PACKED>& f, int v0, int n, int64_t ldz,
                                             uint32_t stash0, float2* zcol, bool act0, bool act1,
                                             const EncodeTaps& taps, const EncodeTaps64& taps64,
                                             const EncodePhase64& ph64) {
    if constexpr (P < StreamCfg<S>::SL) {
        encode_step<S, P, MODE, PACKED>(w, cur, f, v0 + P, n, ldz, stash0, zcol, act0, act1, taps, taps64, ph64);
        encode_chunk<S, MODE, PACKED, P + 1>(w, cur, f, v0, n, ldz, stash0, zcol, act0, act1, taps, taps64, ph64);
    }
}

// PACKED: the real -> complex packing of Section 3's last paragraph.  `len` then counts complex
// coordinates, a strip holds 64 of them, and a lane receives two pairs of each row:
// G[r][c], G[r][c + 1] (real parts) and G[r][half + c], G[r][half + c + 1] (imaginary parts).
template <int S, bool PACKED>
__global__ void __launch_bounds__(StreamCfg<S>::kThreads, 1)
cyc_encode_stream_kernel(const float* __restrict__ G, float2* __restrict__ Z, int64_t len, int64_t ldg, int64_t ldz,
                         int64_t half, int n,
                         const __grid_constant__ EncodeTaps taps, const __grid_constant__ EncodeTaps64 taps64,
                         const __grid_constant__ EncodePhase64 ph64) {
    using Cfg = StreamCfg<S>;
    constexpr int SL = Cfg::SL, kWarps = Cfg::kThreads / 32;
    constexpr int kStrip = PACKED ? 64 : 128;
    extern __shared__ __align__(16) unsigned char smem_raw[];        // ring[kRing][kThreads], stash[2 S][kThreads], 16 bytes each
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t nstrips = (len + kStrip - 1) / kStrip;
    const int64_t strip0 = (int64_t)blockIdx.x * kWarps + warp, strip_step = (int64_t)gridDim.x * kWarps;
    Cursor cur;
    cur.ring0 = smem_u32(smem_raw) + threadIdx.x * 16;
    cur.rd = 0;
    const uint32_t stash0 = cur.ring0 + kRing * Cfg::kRowBytes;
    Fetcher<PACKED> f;
    f.G = G; f.boff = PACKED ? half : 64; f.nstrips = nstrips; f.len = len; f.ldg = ldg; f.n = n; f.lane = lane;
    f.strip = strip0; f.strip_step = strip_step;
    f.open_strip();
#pragma unroll 1
    for (int q = 0; q < kRing; ++q) f.fetch(cur.ring0 + q * Cfg::kRowBytes);
    Window<S> w;
#pragma unroll
    for (int q = 0; q < SL; ++q) w.win[q] = make_float4(0.f, 0.f, 0.f, 0.f);
    const int total = n + 2 * S;
    for (int64_t strip = strip0; strip < nstrips; strip += strip_step) {
        const int64_t c = strip * kStrip + 2 * lane;
        const bool act0 = c < len;
        const bool act1 = PACKED ? act0 : (c + 64 < len);
        float2* zcol = Z + c;
        cur.zout = zcol + (int64_t)(2 * S) * ldz;
        int v0 = 0;
        if (n >= SL && S > 0) {
            encode_chunk<S, 0, PACKED>(w, cur, f, 0, n, ldz, stash0, zcol, act0, act1, taps, taps64, ph64);
            for (v0 = SL; v0 + SL <= n; v0 += SL)
                encode_chunk<S, 1, PACKED>(w, cur, f, v0, n, ldz, stash0, zcol, act0, act1, taps, taps64, ph64);
        }
        for (; v0 < total; v0 += SL)
            encode_chunk<S, 2, PACKED>(w, cur, f, v0, n, ldz, stash0, zcol, act0, act1, taps, taps64, ph64);
    }
    cp_async_wait<0>();
}

// Any s, any length / alignment: one coordinate per thread, rows re-read through the caches,
// fp64 taps and fp64 accumulation throughout (a tap rounded to fp32 is a fixed error of 2^-24 |tap| that
// the decoder's cancellation amplifies like any other).  half > 0: packed mode (len complex coordinates; the imaginary
// parts come from G[r][half + i], zero beyond d_real).
__global__ void __launch_bounds__(kGenericThreads)
cyc_encode_generic_kernel(const float* __restrict__ G, float2* __restrict__ Z, int64_t len, int64_t ldg, int64_t ldz,
                          int64_t half, int64_t d_real, int n, int s, const double2* __restrict__ taps,
                          const __grid_constant__ EncodePhase64 ph) {
    const int64_t stride = (int64_t)gridDim.x * kGenericThreads;
    for (int64_t i = (int64_t)blockIdx.x * kGenericThreads + threadIdx.x; i < len; i += stride) {
        const bool has_b = half > 0 && half + i < d_real;
        for (int j = 0; j < n; ++j) {
            double ar = 0.0, ai = 0.0, br = 0.0, bi = 0.0;
            for (int t = 0; t <= 2 * s; ++t) {
                int r = j - t;
                if (r < 0) r += n;
                const double2 c = taps[t];
                const double g = (double)G[(int64_t)r * ldg + i];
                ar = fma(c.x, g, ar);
                ai = fma(c.y, g, ai);
                if (has_b) {
                    const double gb = (double)G[(int64_t)r * ldg + half + i];
                    br = fma(c.x, gb, br);
                    bi = fma(c.y, gb, bi);
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
int launch_stream(const draco_plan* p, const float* G, float2* Z, int64_t len, int64_t ldg, int64_t ldz, int64_t half,
                  cudaStream_t st) {
    using Cfg = StreamCfg<S>;
    constexpr int kThreads = Cfg::kThreads;
    auto kern = cyc_encode_stream_kernel<S, PACKED>;
    static bool configured[64] = {};
    int dev = p->device;
    if (dev < 0 || dev >= 64) dev = 0;
    if (!configured[dev]) {
        DRACO_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::kSmem));
        configured[dev] = true;
    }
    int per_sm = 1;
    DRACO_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, Cfg::kSmem));
    if (per_sm < 1) per_sm = 1;
    constexpr int kStrip = PACKED ? 64 : 128;
    const int64_t nstrips = (len + kStrip - 1) / kStrip;
    const int64_t nblocks = (nstrips + kThreads / 32 - 1) / (kThreads / 32);
    int64_t grid = (int64_t)p->sm_count * per_sm;
    if (grid > nblocks) grid = nblocks;
    if (grid < 1) grid = 1;
    kern<<<(int)grid, kThreads, Cfg::kSmem, st>>>(G, Z, len, ldg, ldz, half, p->n, p->taps, p->taps64, p->phase64);
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

template <bool PACKED>
int launch_stream_any(const draco_plan* p, const float* G, float2* Z, int64_t len, int64_t ldg, int64_t ldz, int64_t half,
                      cudaStream_t st) {
    switch (p->s) {
        case 0: return launch_stream<0, PACKED>(p, G, Z, len, ldg, ldz, half, st);
        case 1: return launch_stream<1, PACKED>(p, G, Z, len, ldg, ldz, half, st);
        case 2: return launch_stream<2, PACKED>(p, G, Z, len, ldg, ldz, half, st);
        case 3: return launch_stream<3, PACKED>(p, G, Z, len, ldg, ldz, half, st);
        case 4: return launch_stream<4, PACKED>(p, G, Z, len, ldg, ldz, half, st);
        case 5: return launch_stream<5, PACKED>(p, G, Z, len, ldg, ldz, half, st);
        case 6: return launch_stream<6, PACKED>(p, G, Z, len, ldg, ldz, half, st);
        default: return launch_stream<7, PACKED>(p, G, Z, len, ldg, ldz, half, st);
    }
}

}  // namespace

// half == 0: Z[j][i], i < len, from G[.][i].  half > 0 (packed): Z[j][i], i < len complex coordinates,
// from G[.][i] (real parts) and G[.][half + i] (imaginary parts, zero for half + i >= d_real).
int launch_cyc_encode(const draco_plan* p, const float* G, float2* Z, int64_t len, int64_t ldg, int64_t ldz,
                      int64_t half, int64_t d_real, cudaStream_t st) {
    // the streaming kernel copies 8 bytes and stores 16 bytes at a time: row starts, strip starts and the half offset
    // are multiples of 4 floats
    const bool packed = half > 0;
    bool fast = (ldg % 4 == 0) && (ldz % 2 == 0) && p->s <= 7;
    if (packed) fast = fast && (len % 4 == 0) && (half % 4 == 0) && (half + len <= d_real);
    else fast = fast && (len % 4 == 0);
    if (fast) return packed ? launch_stream_any<true>(p, G, Z, len, ldg, ldz, half, st)
                            : launch_stream_any<false>(p, G, Z, len, ldg, ldz, 0, st);
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

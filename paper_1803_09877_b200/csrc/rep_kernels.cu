// Repetition code (Section 3, "Fractional Repetition Code"): the encoder
// E^Rep_j(Y_j) = Y_j 1_P and the decoder D^Rep(R) = sum over groups of the
// element-wise majority of the group's received vectors, found with the
// streaming majority vote of Algorithm 2 on 32-bit patterns.
//
// Both kernels are single passes over an [n][len] fp32 matrix: a thread owns
// VEC consecutive coordinates, walks the groups, and keeps one group's replicas
// in registers (128-bit loads, one per replica).  HBM-bound: encode moves
// 8 n len bytes, vote 4 n len + 4 len bytes.
#include "draco_internal.cuh"

namespace draco {

namespace {

constexpr int kThreads = 256;

template <int VEC>
struct Pack;
template <>
struct Pack<4> {
    uint4 v;
    __device__ __forceinline__ uint32_t get(int c) const { return c == 0 ? v.x : c == 1 ? v.y : c == 2 ? v.z : v.w; }
};
template <>
struct Pack<2> {
    uint2 v;
    __device__ __forceinline__ uint32_t get(int c) const { return c == 0 ? v.x : v.y; }
};
template <>
struct Pack<1> {
    uint32_t v;
    __device__ __forceinline__ uint32_t get(int) const { return v; }
};

__device__ __forceinline__ void load_pack(Pack<4>& p, const uint32_t* ptr) {
    p.v = __ldcs(reinterpret_cast<const uint4*>(ptr));
}
__device__ __forceinline__ void load_pack(Pack<2>& p, const uint32_t* ptr) {
    p.v = __ldcs(reinterpret_cast<const uint2*>(ptr));
}
__device__ __forceinline__ void load_pack(Pack<1>& p, const uint32_t* ptr) { p.v = __ldcs(ptr); }

__device__ __forceinline__ void store_vals(float* ptr, const float (&x)[4]) {
    __stcs(reinterpret_cast<float4*>(ptr), make_float4(x[0], x[1], x[2], x[3]));
}
__device__ __forceinline__ void store_vals(float* ptr, const float (&x)[2]) {
    __stcs(reinterpret_cast<float2*>(ptr), make_float2(x[0], x[1]));
}
__device__ __forceinline__ void store_vals(float* ptr, const float (&x)[1]) { __stcs(ptr, x[0]); }

// w <- w - scale * x on VEC consecutive entries (the SGD step of Section 2 fused into the decoder's epilogue)
__device__ __forceinline__ void update_vals(float* ptr, const float (&x)[4], float scale) {
    float4 w = *reinterpret_cast<const float4*>(ptr);
    w.x = fmaf(-scale, x[0], w.x); w.y = fmaf(-scale, x[1], w.y); w.z = fmaf(-scale, x[2], w.z); w.w = fmaf(-scale, x[3], w.w);
    *reinterpret_cast<float4*>(ptr) = w;
}
__device__ __forceinline__ void update_vals(float* ptr, const float (&x)[2], float scale) {
    float2 w = *reinterpret_cast<const float2*>(ptr);
    w.x = fmaf(-scale, x[0], w.x); w.y = fmaf(-scale, x[1], w.y);
    *reinterpret_cast<float2*>(ptr) = w;
}
__device__ __forceinline__ void update_vals(float* ptr, const float (&x)[1], float scale) { ptr[0] = fmaf(-scale, x[0], ptr[0]); }

// ---------------------------------------------------------------- encode
// MMAX > 0: groups of at most MMAX members, GB groups fetched together so that about 16 rows are in flight per
// thread whatever the group size (as in the vote kernel); MMAX == 0: larger groups, members streamed.
template <int MMAX, int VEC, int GB>
__global__ void __launch_bounds__(kThreads)
rep_encode_kernel(const float* __restrict__ G, float* __restrict__ Z, int64_t len, int64_t ldg, int64_t ldz,
                  GroupTable gt) {
    const int64_t nvec = len / VEC;
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    for (int64_t v = (int64_t)blockIdx.x * kThreads + threadIdx.x; v < nvec; v += stride) {
        const int64_t col = v * VEC;
        if constexpr (MMAX > 0) {
            for (int g0 = 0; g0 < gt.num_groups; g0 += GB) {
                Pack<VEC> val[GB][MMAX];
#pragma unroll
                for (int b = 0; b < GB; ++b)
                    if (g0 + b < gt.num_groups) {
                        const int first = gt.first[g0 + b], m = gt.size[g0 + b];
#pragma unroll
                        for (int k = 0; k < MMAX; ++k)
                            if (k < m) load_pack(val[b][k], reinterpret_cast<const uint32_t*>(G + (int64_t)(first + k) * ldg + col));
                    }
#pragma unroll
                for (int b = 0; b < GB; ++b)
                    if (g0 + b < gt.num_groups) {
                        const int first = gt.first[g0 + b], m = gt.size[g0 + b];
                        float acc[VEC];
#pragma unroll
                        for (int c = 0; c < VEC; ++c) acc[c] = __uint_as_float(val[b][0].get(c));
#pragma unroll
                        for (int k = 1; k < MMAX; ++k)
                            if (k < m) {
#pragma unroll
                                for (int c = 0; c < VEC; ++c) acc[c] = __fadd_rn(acc[c], __uint_as_float(val[b][k].get(c)));
                            }
                        for (int k = 0; k < m; ++k) store_vals(Z + (int64_t)(first + k) * ldz + col, acc);
                    }
            }
        } else {
            for (int g = 0; g < gt.num_groups; ++g) {
                const int first = gt.first[g], m = gt.size[g];
                float acc[VEC];
                Pack<VEC> x;
                load_pack(x, reinterpret_cast<const uint32_t*>(G + (int64_t)first * ldg + col));
#pragma unroll
                for (int c = 0; c < VEC; ++c) acc[c] = __uint_as_float(x.get(c));
                for (int k = 1; k < m; ++k) {
                    load_pack(x, reinterpret_cast<const uint32_t*>(G + (int64_t)(first + k) * ldg + col));
#pragma unroll
                    for (int c = 0; c < VEC; ++c) acc[c] = __fadd_rn(acc[c], __uint_as_float(x.get(c)));
                }
                for (int k = 0; k < m; ++k) store_vals(Z + (int64_t)(first + k) * ldz + col, acc);
            }
        }
    }
}

// ---------------------------------------------------------------- vote
struct RepScratch {
    uint32_t mask[kMaxN];             // per group: bit k set <=> member k disagreed somewhere
    unsigned long long no_majority;
};

// One step of Algorithm 2 for item x.
__device__ __forceinline__ void vote_step(uint32_t x, uint32_t& ma, int& counter) {
    const bool empty = counter == 0;
    const bool same = ma == x;
    ma = empty ? x : ma;
    counter = empty ? 1 : (same ? counter + 1 : counter - 1);
}

// Majority of one group whose m <= MMAX replicas sit in registers.  Returns the selected bit
// patterns in sel[], adds the members that disagree somewhere to `dis` and the coordinates
// without a strict majority to `nomaj`.
template <int MMAX, int VEC>
__device__ __forceinline__ void vote_group(const Pack<VEC> (&val)[MMAX], int m, uint32_t (&sel)[VEC], uint32_t& dis,
                                           unsigned int& nomaj) {
    uint32_t differ = 0;
#pragma unroll
    for (int k = 1; k < MMAX; ++k)
        if (k < m) {
#pragma unroll
            for (int c = 0; c < VEC; ++c) differ |= val[k].get(c) ^ val[0].get(c);
        }
    if (differ == 0) {                                   // all replicas bit-identical: they are the majority
#pragma unroll
        for (int c = 0; c < VEC; ++c) sel[c] = val[0].get(c);
        return;
    }
    // Some replica differs.  A value held by strictly more than half of the group IS what
    // Algorithm 2 returns, so first count the votes for member 0's value, then for member 1's
    // (member 0 may be the adversary); only if neither has a strict majority on all VEC
    // coordinates is the streaming vote itself run.
    bool settled = false;
#pragma unroll
    for (int ref = 0; ref < 2 && ref < MMAX; ++ref) {
        if (!settled && ref < m) {
            uint32_t d_ref = 0;
            bool all_major = true;
#pragma unroll
            for (int c = 0; c < VEC; ++c) {
                const uint32_t cand = val[ref].get(c);
                uint32_t ne = 0;
#pragma unroll
                for (int k = 0; k < MMAX; ++k)
                    if (k < m) ne |= (val[k].get(c) != cand ? 1u : 0u) << k;
                all_major &= (2 * (m - __popc(ne)) > m);
                d_ref |= ne;
            }
            if (all_major) {
#pragma unroll
                for (int c = 0; c < VEC; ++c) sel[c] = val[ref].get(c);
                dis |= d_ref;
                settled = true;
            }
        }
    }
    if (!settled) {
#pragma unroll
        for (int c = 0; c < VEC; ++c) {
            uint32_t ma = val[0].get(c);
            int counter = 0;
#pragma unroll
            for (int k = 0; k < MMAX; ++k)
                if (k < m) vote_step(val[k].get(c), ma, counter);
            uint32_t ne = 0;
#pragma unroll
            for (int k = 0; k < MMAX; ++k)
                if (k < m) ne |= (val[k].get(c) != ma ? 1u : 0u) << k;
            nomaj += (2 * (m - __popc(ne)) <= m);
            dis |= ne;
            sel[c] = ma;
        }
    }
}

// MMAX > 0: groups of at most MMAX members, GB groups fetched together so that about 16 rows
// (128-bit or 64-bit loads) are in flight per thread whatever the group size.
// MMAX == 0: groups larger than the register budget, members streamed twice (GB ignored).
template <int MMAX, int VEC, int GB, int TPB>
__global__ void __launch_bounds__(TPB)
rep_vote_kernel(const uint32_t* __restrict__ R, int64_t len, int64_t ld, GroupTable gt, float* __restrict__ u,
                float* __restrict__ maj, RepScratch* scratch, float* __restrict__ w, float scale) {
    __shared__ uint32_t smask[kMaxN][MMAX > 0 ? 1 : 4];   // generic path: up to 128 members = 4 words
    for (int i = threadIdx.x; i < kMaxN * (MMAX > 0 ? 1 : 4); i += TPB) (&smask[0][0])[i] = 0;
    __syncthreads();

    unsigned int nomaj = 0;
    const int64_t nvec = len / VEC;
    const int64_t stride = (int64_t)gridDim.x * TPB;
    for (int64_t v = (int64_t)blockIdx.x * TPB + threadIdx.x; v < nvec; v += stride) {
        const int64_t col = v * VEC;
        float acc[VEC];
#pragma unroll
        for (int c = 0; c < VEC; ++c) acc[c] = 0.0f;
        if constexpr (MMAX > 0) {
            for (int g0 = 0; g0 < gt.num_groups; g0 += GB) {
                Pack<VEC> val[GB][MMAX];
#pragma unroll
                for (int b = 0; b < GB; ++b)
                    if (g0 + b < gt.num_groups) {
                        const int first = gt.first[g0 + b], m = gt.size[g0 + b];
                        const uint32_t* base = R + (int64_t)first * ld + col;
#pragma unroll
                        for (int k = 0; k < MMAX; ++k)
                            if (k < m) load_pack(val[b][k], base + (int64_t)k * ld);
                    }
#pragma unroll
                for (int b = 0; b < GB; ++b)
                    if (g0 + b < gt.num_groups) {
                        const int g = g0 + b, m = gt.size[g];
                        uint32_t sel[VEC];
                        uint32_t dis = 0;
                        vote_group<MMAX, VEC>(val[b], m, sel, dis, nomaj);
                        if (dis & ~smask[g][0]) atomicOr(&smask[g][0], dis);
                        float selv[VEC];
#pragma unroll
                        for (int c = 0; c < VEC; ++c) {
                            selv[c] = __uint_as_float(sel[c]);
                            acc[c] = __fadd_rn(acc[c], selv[c]);
                        }
                        if (maj != nullptr) store_vals(maj + (int64_t)g * len + col, selv);
                    }
            }
        } else {
            for (int g = 0; g < gt.num_groups; ++g) {
                const int first = gt.first[g], m = gt.size[g];
                const uint32_t* base = R + (int64_t)first * ld + col;
                uint32_t ma[VEC];
                int counter[VEC];
                Pack<VEC> x;
                load_pack(x, base);
#pragma unroll
                for (int c = 0; c < VEC; ++c) { ma[c] = x.get(c); counter[c] = 0; }
                for (int k = 0; k < m; ++k) {
                    load_pack(x, base + (int64_t)k * ld);
#pragma unroll
                    for (int c = 0; c < VEC; ++c) vote_step(x.get(c), ma[c], counter[c]);
                }
                int votes[VEC];
#pragma unroll
                for (int c = 0; c < VEC; ++c) votes[c] = 0;
                for (int k = 0; k < m; ++k) {
                    load_pack(x, base + (int64_t)k * ld);
                    bool any_diff = false;
#pragma unroll
                    for (int c = 0; c < VEC; ++c) {
                        const bool same = x.get(c) == ma[c];
                        votes[c] += same;
                        any_diff |= !same;
                    }
                    if (any_diff && !(smask[g][k >> 5] & (1u << (k & 31)))) atomicOr(&smask[g][k >> 5], 1u << (k & 31));
                }
                float selv[VEC];
#pragma unroll
                for (int c = 0; c < VEC; ++c) {
                    nomaj += (2 * votes[c] <= m);
                    selv[c] = __uint_as_float(ma[c]);
                    acc[c] = __fadd_rn(acc[c], selv[c]);
                }
                if (maj != nullptr) store_vals(maj + (int64_t)g * len + col, selv);
            }
        }
        if (u != nullptr) store_vals(u + col, acc);
        if (w != nullptr) update_vals(w + col, acc, scale);
    }

    // block totals -> global scratch (integer OR / add: order-independent, hence deterministic)
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) nomaj += __shfl_xor_sync(0xffffffffu, nomaj, off);
    if ((threadIdx.x & 31) == 0 && nomaj) atomicAdd(&scratch->no_majority, (unsigned long long)nomaj);
    __syncthreads();
    if constexpr (MMAX > 0) {
        for (int g = threadIdx.x; g < gt.num_groups; g += TPB)
            if (smask[g][0]) atomicOr(&scratch->mask[gt.first[g]], smask[g][0]);
    } else {
        // generic path keeps one word per 32 members; spread them over the members' own slots
        for (int g = threadIdx.x; g < gt.num_groups; g += TPB)
            for (int w = 0; w < 4; ++w)
                if (smask[g][w]) atomicOr(&scratch->mask[gt.first[g] + w], smask[g][w]);
    }
}

// mask words -> flag bytes and the info block (one block).
__global__ void rep_finish_kernel(GroupTable gt, const RepScratch* scratch, uint8_t* flags, uint8_t* flags2,
                                  DeviceInfo* info, bool generic) {
    __shared__ int count;
    if (threadIdx.x == 0) count = 0;
    __syncthreads();
    for (int g = threadIdx.x; g < gt.num_groups; g += blockDim.x) {
        const int first = gt.first[g], m = gt.size[g];
        int c = 0;
        for (int k = 0; k < m; ++k) {
            const uint32_t word = generic ? scratch->mask[first + (k >> 5)] : scratch->mask[first];
            const uint8_t bit = (word >> (k & 31)) & 1u;
            if (flags) flags[first + k] = bit;
            if (flags2) flags2[first + k] = bit;
            c += bit;
        }
        atomicAdd(&count, c);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        info->n_flagged = count;
        info->no_majority = scratch->no_majority;
        info->status = scratch->no_majority ? DRACO_ENOMAJ : DRACO_OK;
        info->locator_rank = 0;
        info->n_active = 0;
        info->scale = 0.0;
        info->max_syndrome = 0.0;
    }
}

int grid_for(int64_t nvec, int sm_count, int blocks_per_sm) {
    int64_t want = (nvec + kThreads - 1) / kThreads;
    int64_t cap = (int64_t)sm_count * blocks_per_sm;
    if (want < 1) want = 1;
    return (int)(want < cap ? want : cap);
}

}  // namespace

int launch_rep_encode(const draco_plan* p, const float* G, float* Z, int64_t len, int64_t ldg, int64_t ldz,
                      cudaStream_t st) {
    const GroupTable& gt = p->groups;
    const bool vec4 = (len % 4 == 0) && (ldg % 4 == 0) && (ldz % 4 == 0);
    const int64_t nvec = vec4 ? len / 4 : len;
    const int grid = grid_for(nvec, p->sm_count, 8);
#define DRACO_ENC(MM, VV, GG) rep_encode_kernel<MM, VV, GG><<<grid, kThreads, 0, st>>>(G, Z, len, ldg, ldz, gt)
    if (vec4) {
        if (gt.max_size <= 3) DRACO_ENC(3, 4, 5);
        else if (gt.max_size <= 4) DRACO_ENC(4, 4, 4);
        else if (gt.max_size <= 5) DRACO_ENC(5, 4, 2);
        else if (gt.max_size <= 8) DRACO_ENC(8, 4, 1);
        else if (gt.max_size <= 16) DRACO_ENC(16, 4, 1);
        else DRACO_ENC(0, 4, 1);
    } else {
        if (gt.max_size <= 8) DRACO_ENC(8, 1, 2);
        else if (gt.max_size <= 16) DRACO_ENC(16, 1, 1);
        else DRACO_ENC(0, 1, 1);
    }
#undef DRACO_ENC
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

int launch_rep_vote(draco_plan* p, const float* R, int64_t len, int64_t ld, float* u, float* maj, uint8_t* flags,
                    bool reset, cudaStream_t st, float* w, float scale) {
    const GroupTable& gt = p->groups;
    RepScratch* scratch = reinterpret_cast<RepScratch*>(p->mask_dev);
    if (reset) DRACO_CUDA(cudaMemsetAsync(scratch, 0, sizeof(RepScratch), st));
    const bool vec4 = (len % 4 == 0) && (ld % 4 == 0);
    const uint32_t* Rb = reinterpret_cast<const uint32_t*>(R);
    const bool generic = gt.max_size > 16;
#define DRACO_VOTE(MM, VV, GG, TT)                                                                                 \
    rep_vote_kernel<MM, VV, GG, TT><<<grid_for(len / VV, p->sm_count, 8) * (kThreads / TT), TT, 0, st>>>(Rb, len, ld, gt, u, \
                                                                                                        maj, scratch, w, scale)
    if (vec4) {
        if (gt.max_size <= 3) DRACO_VOTE(3, 4, 5, 256);             // s = 1: five groups of three = 15 rows in flight
        else if (gt.max_size <= 4) DRACO_VOTE(4, 4, 4, 256);
        else if (gt.max_size <= 5) DRACO_VOTE(5, 4, 3, 256);        // s = 2: three groups of five
        else if (gt.max_size <= 8) DRACO_VOTE(8, 4, 2, 256);
        else if (gt.max_size <= 16) DRACO_VOTE(16, 4, 1, 128);      // 16 x 128-bit loads per thread: small blocks keep 3 per SM
        else DRACO_VOTE(0, 4, 1, 256);
    } else {
        if (gt.max_size <= 4) DRACO_VOTE(4, 1, 4, 256);
        else if (gt.max_size <= 8) DRACO_VOTE(8, 1, 2, 256);
        else if (gt.max_size <= 16) DRACO_VOTE(16, 1, 1, 256);
        else DRACO_VOTE(0, 1, 1, 256);
    }
#undef DRACO_VOTE
    DRACO_CUDA(cudaGetLastError());
    rep_finish_kernel<<<1, 128, 0, st>>>(gt, scratch, flags, p->flags_dev, p->info_dev, generic);
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

size_t rep_scratch_bytes() { return sizeof(RepScratch); }

}  // namespace draco

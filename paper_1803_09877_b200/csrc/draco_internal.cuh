// Internal declarations shared by the translation units of libdraco.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "draco.h"

namespace draco {

constexpr int kMaxN = DRACO_MAX_N;
constexpr int kMaxTaps = 15;          // 2 s + 1 for the register-window encoder (s <= 7)
constexpr int kProjectTile = 2048;    // coordinates per tile of the projection kernel
constexpr int kProjectWarps = 8;
constexpr double kMarginBar = 10.0;        // locator_margin below this, or ..
constexpr double kImResidualBar = 1e-2;    // .. im_residual above this fraction of re_max: status DRACO_EUNSURE
constexpr int kJacobiSweepLimit = 60;

struct GroupTable {                   // repetition code: consecutive groups
    int num_groups;
    int max_size;
    uint8_t first[kMaxN];
    uint8_t size[kMaxN];
};

struct EncodeTaps {                   // cyclic encoder: z_j = phase[j] * sum_t tap[t] * g_{(j-t) mod n}
    float2 tap[kMaxTaps];
};

struct EncodePhase {
    float2 phase[kMaxN];
};

struct EncodeTaps64 {                 // the same taps / phases in fp64 (centre taps and the final rotation)
    double2 tap[kMaxTaps];
};

struct EncodePhase64 {
    double2 phase[kMaxN];
};

// Device-resident state of the cyclic decoder (lives in the plan's scratch).
struct CycDevice {
    double2 twiddle[kMaxN];           // w^k, w = exp(2 pi i / n)
    double2 e[kMaxN];                 // projection f R
    double2 h[kMaxN];                 // syndromes, then the full DFT of gamma
    double2 t[kMaxN];                 // IDFT(h)
    double2 b[kMaxN];                 // decode vector (zero on flagged nodes)
    double2 b_active[kMaxN];          // b_j of the active rows, packed
    int32_t active[kMaxN];            // their node indices
    double2 work[kMaxN * (kMaxN + 1)];  // elimination work space
    double2 vec[4 * kMaxN];
    int32_t perm[kMaxN];
    double record[3 * kMaxN];         // the plan's own projection record: n (re, im) pairs, then n values q_j
};

struct DeviceInfo {                   // mirrors draco_info
    int32_t status;
    int32_t n_flagged;
    int32_t locator_rank;
    int32_t n_active;
    unsigned long long no_majority;
    double scale;
    double max_syndrome;
    int32_t internal_error;
    int32_t svd_sweeps;
    double locator_margin;
    unsigned long long im_residual_bits;   // bit patterns of non-negative doubles: they order like integers, so the
    unsigned long long re_max_bits;        // blocks of the recovery kernel merge their maxima with atomicMax
};

}  // namespace draco

struct draco_plan {
    int n, s, code;
    int64_t d;
    int device;
    int sm_count;
    double theta;
    // repetition
    draco::GroupTable groups;
    // cyclic (host copies)
    double* W_host;                   // [n][n][2]
    draco::EncodeTaps taps;
    draco::EncodePhase phase;
    draco::EncodeTaps64 taps64;
    draco::EncodePhase64 phase64;
    double2* taps_full_dev;           // generic encoder: fp64 taps for any s, device [2s+1]
    // device scratch
    draco::CycDevice* cyc_dev;
    draco::DeviceInfo* info_dev;
    double2* partial_dev;             // [project_grid][n]
    int project_grid;                 // capacity of partial_dev in blocks
    int project_used;                 // blocks whose partials the plan's last projection (all its chunks) filled
    uint8_t* flags_dev;               // [n] internal flags
    uint32_t* mask_dev;               // repetition: disagreement bits, [n] words
    // host-buffer pipeline (allocated on its first call)
    float* stage_dev;                 // two [n][stage_chunk] slices of G (double buffer)
    cudaStream_t copy_stream, work_stream;
    cudaEvent_t ev_copied[2], ev_consumed[2];
    int64_t stage_chunk;
    float* f_dev;                     // [d]
    float* u_dev;                     // [d]
};

namespace draco {

// Set the thread's last CUDA error text; returns DRACO_ECUDA.
int cuda_fail(cudaError_t err, const char* what);

#define DRACO_CUDA(call)                                              \
    do {                                                              \
        cudaError_t err__ = (call);                                   \
        if (err__ != cudaSuccess) return draco::cuda_fail(err__, #call); \
    } while (0)

// kernels / launchers (one per translation unit)
int launch_rep_encode(const draco_plan* p, const float* G, float* Z, int64_t len, int64_t ldg, int64_t ldz,
                      cudaStream_t st);
int launch_rep_vote(draco_plan* p, const float* R, int64_t len, int64_t ld, float* u, float* maj, uint8_t* flags,
                    bool reset, cudaStream_t st, float* w = nullptr, float scale = 0.0f);
int launch_cyc_encode(const draco_plan* p, const float* G, float2* Z, int64_t len, int64_t ldg, int64_t ldz,
                      int64_t half, int64_t d_real, cudaStream_t st);
int launch_cyc_project(draco_plan* p, const float2* R, const float* f, int64_t len, int64_t ld, bool accumulate,
                       cudaStream_t st);
int launch_cyc_project_finish(draco_plan* p, double2* e_out, cudaStream_t st);
int launch_cyc_solve(draco_plan* p, const double2* e, uint8_t* flags, bool with_b, cudaStream_t st);
int launch_cyc_decode_vector(draco_plan* p, const uint8_t* flags, cudaStream_t st);
int launch_cyc_recover(draco_plan* p, const float2* R, int64_t len, int64_t ld, float* u, int64_t d_packed,
                       cudaStream_t st, float* w = nullptr, float scale = 0.0f);
int launch_generate(float* out, int rows, int64_t len, int64_t ld, int64_t i0, int row0, float mean, float std,
                    uint64_t seed, cudaStream_t st);
int launch_corrupt(float* R, int64_t row_pitch, int64_t nvals, int64_t v0, const int* node, const int* model,
                   const float* param, int n_adv, uint64_t seed, bool is_complex, int sm_count, cudaStream_t st);
int project_grid_size(int sm_count);
int project_grid_size(int sm_count, int n);

}  // namespace draco

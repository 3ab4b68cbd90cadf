// C ABI of libdraco: plans, code tables, argument checks and launch sequencing.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <complex>
#include <new>
#include <vector>

#include "draco_internal.cuh"

namespace draco {

static thread_local char g_cuda_error[256] = "";

int cuda_fail(cudaError_t err, const char* what) {
    snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", what, cudaGetErrorString(err));
    return DRACO_ECUDA;
}

size_t rep_scratch_bytes();

namespace {

typedef std::complex<long double> cld;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool is_cyc(const draco_plan* p) { return p->code == DRACO_CYC || p->code == DRACO_CYC_PACKED; }
inline bool is_packed(const draco_plan* p) { return p->code == DRACO_CYC_PACKED; }
// entries per worker vector: d, or ceil(d / 2) complex entries in packed mode
inline int64_t vec_len(const draco_plan* p) { return is_packed(p) ? (p->d + 1) / 2 : p->d; }
inline int64_t half_off(const draco_plan* p) { return is_packed(p) ? (p->d + 1) / 2 : 0; }

cld root_of_unity(int n, long long e) {
    const long double pi = 3.141592653589793238462643383279502884L;
    long long k = e % n;
    if (k < 0) k += n;
    const long double ang = 2.0L * pi * (long double)k / (long double)n;
    return cld(cosl(ang), sinl(ang));
}

// Repetition code: n / r groups of r consecutive nodes; when r does not divide n,
// floor(n / r) groups whose sizes differ by at most one, larger groups first.
void build_groups(int n, int s, GroupTable* gt) {
    const int r = 2 * s + 1;
    const int g = n / r;
    const int base = n / g, extra = n % g;
    gt->num_groups = g;
    gt->max_size = 0;
    int first = 0;
    for (int ell = 0; ell < g; ++ell) {
        const int size = base + (ell < extra ? 1 : 0);
        gt->first[ell] = (uint8_t)first;
        gt->size[ell] = (uint8_t)size;
        if (size > gt->max_size) gt->max_size = size;
        first += size;
    }
}

// Cyclic code tables.  W[j][k] = n^(-1/2) prod_{m in alpha_j} (w^k - w^m) with
// alpha_j = {j+2s+1 .. j+n-1} (mod n): the monic polynomial of degree n-2s-1 that the
// construction [q_j 1][C_L]_{.,alpha_j} = 0 defines, evaluated at w^k.
int build_cyclic_tables(draco_plan* p, std::vector<double2>* taps_full, std::vector<double2>* twiddle) {
    const int n = p->n, s = p->s, M = n - 2 * s - 1;
    std::vector<cld> w0(2 * s + 1);
    const long double rsn = 1.0L / sqrtl((long double)n);
    for (int t = 0; t <= 2 * s; ++t) {
        cld prod(rsn, 0.0L);
        for (int m = 2 * s + 1; m < n; ++m) prod *= (root_of_unity(n, t) - root_of_unity(n, m));
        w0[t] = prod;
    }
    p->W_host = (double*)calloc((size_t)n * n * 2, sizeof(double));
    if (!p->W_host) return DRACO_ENOMEM;
    for (int j = 0; j < n; ++j) {
        const cld rot = root_of_unity(n, (long long)j * M);
        for (int t = 0; t <= 2 * s; ++t) {
            const int k = (j + t) % n;
            const cld v = rot * w0[t];
            p->W_host[((size_t)j * n + k) * 2 + 0] = (double)v.real();
            p->W_host[((size_t)j * n + k) * 2 + 1] = (double)v.imag();
        }
    }
    taps_full->resize(2 * s + 1);
    memset(&p->taps, 0, sizeof(p->taps));
    memset(&p->taps64, 0, sizeof(p->taps64));
    memset(&p->phase64, 0, sizeof(p->phase64));
    for (int t = 0; t <= 2 * s; ++t) {
        const cld v = root_of_unity(n, -(long long)t * M) * w0[t];
        (*taps_full)[t] = make_double2((double)v.real(), (double)v.imag());
        if (t < kMaxTaps) {
            p->taps.tap[t] = make_float2((float)v.real(), (float)v.imag());
            p->taps64.tap[t] = (*taps_full)[t];
        }
    }
    memset(&p->phase, 0, sizeof(p->phase));
    twiddle->resize(kMaxN);
    for (int j = 0; j < kMaxN; ++j) (*twiddle)[j] = make_double2(0.0, 0.0);
    for (int j = 0; j < n; ++j) {
        const cld ph = root_of_unity(n, (long long)j * M);
        p->phase.phase[j] = make_float2((float)ph.real(), (float)ph.imag());
        p->phase64.phase[j] = make_double2((double)ph.real(), (double)ph.imag());
        const cld tw = root_of_unity(n, j);
        (*twiddle)[j] = make_double2((double)tw.real(), (double)tw.imag());
    }
    return DRACO_OK;
}

void free_plan(draco_plan* p) {
    if (!p) return;
    free(p->W_host);
    if (p->taps_full_dev) cudaFree(p->taps_full_dev);
    if (p->cyc_dev) cudaFree(p->cyc_dev);
    if (p->info_dev) cudaFree(p->info_dev);
    if (p->partial_dev) cudaFree(p->partial_dev);
    if (p->flags_dev) cudaFree(p->flags_dev);
    if (p->mask_dev) cudaFree(p->mask_dev);
    if (p->stage_dev) cudaFree(p->stage_dev);
    if (p->copy_stream) cudaStreamDestroy(p->copy_stream);
    if (p->work_stream) cudaStreamDestroy(p->work_stream);
    for (int b = 0; b < 2; ++b) {
        if (p->ev_copied[b]) cudaEventDestroy(p->ev_copied[b]);
        if (p->ev_consumed[b]) cudaEventDestroy(p->ev_consumed[b]);
    }
    if (p->f_dev) cudaFree(p->f_dev);
    if (p->u_dev) cudaFree(p->u_dev);
    delete p;
}

}  // namespace
}  // namespace draco

using namespace draco;

extern "C" {

int draco_plan_create(int n, int s, int64_t d, int code, draco_plan** out) {
    if (!out) return DRACO_EINVAL;
    *out = nullptr;
    if (n < 1 || n > DRACO_MAX_N || s < 0 || 2 * s + 1 > n || d < 1) return DRACO_EINVAL;
    if (code != DRACO_REP && code != DRACO_CYC && code != DRACO_CYC_PACKED) return DRACO_EINVAL;
    draco_plan* p = new (std::nothrow) draco_plan();
    if (!p) return DRACO_ENOMEM;
    memset(p, 0, sizeof(*p));
    p->n = n; p->s = s; p->d = d; p->code = code; p->theta = 1e-6;
    cudaError_t err = cudaGetDevice(&p->device);
    if (err == cudaSuccess) err = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device);
    if (err != cudaSuccess) { free_plan(p); return cuda_fail(err, "cudaGetDevice"); }

    int rc = DRACO_OK;
    std::vector<double2> taps_full;
    std::vector<double2> twiddle;
    if (code == DRACO_REP) {
        build_groups(n, s, &p->groups);
    } else {
        rc = build_cyclic_tables(p, &taps_full, &twiddle);
        if (rc != DRACO_OK) { free_plan(p); return rc; }
    }
#define DRACO_TRY(call)                                                          \
    do {                                                                         \
        cudaError_t e__ = (call);                                                \
        if (e__ != cudaSuccess) { free_plan(p); return cuda_fail(e__, #call); }  \
    } while (0)
    DRACO_TRY(cudaMalloc(&p->info_dev, sizeof(DeviceInfo)));
    DRACO_TRY(cudaMemset(p->info_dev, 0, sizeof(DeviceInfo)));
    DRACO_TRY(cudaMalloc(&p->flags_dev, kMaxN));
    DRACO_TRY(cudaMemset(p->flags_dev, 0, kMaxN));
    if (code == DRACO_REP) {
        DRACO_TRY(cudaMalloc(&p->mask_dev, rep_scratch_bytes()));
        DRACO_TRY(cudaMemset(p->mask_dev, 0, rep_scratch_bytes()));
    } else {
        DRACO_TRY(cudaMalloc(&p->cyc_dev, sizeof(CycDevice)));
        DRACO_TRY(cudaMemset(p->cyc_dev, 0, sizeof(CycDevice)));
        DRACO_TRY(cudaMemcpy(p->cyc_dev, twiddle.data(), sizeof(double2) * kMaxN, cudaMemcpyHostToDevice));
        DRACO_TRY(cudaMalloc(&p->taps_full_dev, sizeof(double2) * taps_full.size()));
        DRACO_TRY(cudaMemcpy(p->taps_full_dev, taps_full.data(), sizeof(double2) * taps_full.size(),
                             cudaMemcpyHostToDevice));
        p->project_grid = project_grid_size(p->sm_count, n);
        // per block and node: a double2 partial of e_j, then (after all of those) a double partial of q_j
        const size_t partial_bytes = (sizeof(double2) + sizeof(double)) * (size_t)p->project_grid * n;
        DRACO_TRY(cudaMalloc(&p->partial_dev, partial_bytes));
        DRACO_TRY(cudaMemset(p->partial_dev, 0, partial_bytes));
    }
#undef DRACO_TRY
    *out = p;
    return DRACO_OK;
}

int draco_plan_destroy(draco_plan* plan) {
    free_plan(plan);
    return DRACO_OK;
}

int draco_plan_set_theta(draco_plan* plan, double theta) {
    if (!plan || !(theta > 0.0)) return DRACO_EINVAL;
    plan->theta = theta;
    return DRACO_OK;
}

int draco_num_groups(const draco_plan* plan) {
    if (!plan) return DRACO_EINVAL;
    return plan->code == DRACO_REP ? plan->groups.num_groups : 0;
}

int draco_groups(const draco_plan* plan, int* first, int* size) {
    if (!plan || plan->code != DRACO_REP) return DRACO_EINVAL;
    for (int g = 0; g < plan->groups.num_groups; ++g) {
        if (first) first[g] = plan->groups.first[g];
        if (size) size[g] = plan->groups.size[g];
    }
    return DRACO_OK;
}

int draco_cyc_W(const draco_plan* plan, double* W_host) {
    if (!plan || !is_cyc(plan) || !W_host) return DRACO_EINVAL;
    // stored by rows of the construction (row j = node j's allocation); hand out W itself
    memcpy(W_host, plan->W_host, sizeof(double) * 2 * (size_t)plan->n * plan->n);
    return DRACO_OK;
}

int draco_encode(const draco_plan* plan, const float* G, void* Z, void* stream) {
    if (!plan || !G || !Z || !aligned16(G) || !aligned16(Z)) return DRACO_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    if (plan->code == DRACO_REP) return launch_rep_encode(plan, G, (float*)Z, plan->d, plan->d, plan->d, st);
    return launch_cyc_encode(plan, G, (float2*)Z, vec_len(plan), plan->d, vec_len(plan), half_off(plan), plan->d, st);
}

int draco_rep_vote(draco_plan* plan, const void* R, float* u, float* maj, uint8_t* flags, void* stream) {
    if (!plan || plan->code != DRACO_REP || !R || !aligned16(R) || !aligned16(u) || !aligned16(maj)) return DRACO_EINVAL;
    return launch_rep_vote(plan, (const float*)R, plan->d, plan->d, u, maj, flags, true, (cudaStream_t)stream);
}

int draco_cyc_project(draco_plan* plan, const void* R, const float* f, double* e, void* stream) {
    if (!plan || !is_cyc(plan) || !R || !f || !e || !aligned16(R) || !aligned16(f) || !aligned16(e))
        return DRACO_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    int rc = launch_cyc_project(plan, (const float2*)R, f, vec_len(plan), vec_len(plan), false, st);
    if (rc != DRACO_OK) return rc;
    return launch_cyc_project_finish(plan, (double2*)e, st);
}

int draco_cyc_locate_from_projection(draco_plan* plan, const double* e, uint8_t* flags, void* stream) {
    if (!plan || !is_cyc(plan) || !e || !flags || !aligned16(e)) return DRACO_EINVAL;
    return launch_cyc_solve(plan, (const double2*)e, flags, false, (cudaStream_t)stream);
}

int draco_locate(draco_plan* plan, const void* R, const float* f, uint8_t* flags, void* stream) {
    if (!plan || !R || !aligned16(R)) return DRACO_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    if (plan->code == DRACO_REP)
        return launch_rep_vote(plan, (const float*)R, plan->d, plan->d, nullptr, nullptr, flags, true, st);
    if (!f || !aligned16(f)) return DRACO_EINVAL;
    int rc = launch_cyc_project(plan, (const float2*)R, f, vec_len(plan), vec_len(plan), false, st);
    if (rc != DRACO_OK) return rc;
    return launch_cyc_solve(plan, nullptr, flags, false, st);
}

int draco_decode(draco_plan* plan, const void* R, const uint8_t* flags, float* u, void* stream) {
    if (!plan || !R || !u || !aligned16(R) || !aligned16(u)) return DRACO_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    if (plan->code == DRACO_REP)
        return launch_rep_vote(plan, (const float*)R, plan->d, plan->d, u, nullptr, nullptr, true, st);
    if (!flags) flags = plan->flags_dev;                 // the plan's own copy of its last locate's flags
    int rc = launch_cyc_decode_vector(plan, flags, st);
    if (rc != DRACO_OK) return rc;
    return launch_cyc_recover(plan, (const float2*)R, vec_len(plan), vec_len(plan), u, is_packed(plan) ? plan->d : 0, st);
}

int draco_decode_update(draco_plan* plan, const void* R, const uint8_t* flags, float* w, float scale, void* stream) {
    if (!plan || !R || !w || !aligned16(R) || !aligned16(w)) return DRACO_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    if (plan->code == DRACO_REP)
        return launch_rep_vote(plan, (const float*)R, plan->d, plan->d, nullptr, nullptr, nullptr, true, st, w, scale);
    if (!flags) flags = plan->flags_dev;
    int rc = launch_cyc_decode_vector(plan, flags, st);
    if (rc != DRACO_OK) return rc;
    return launch_cyc_recover(plan, (const float2*)R, vec_len(plan), vec_len(plan), nullptr, is_packed(plan) ? plan->d : 0, st, w,
                              scale);
}

int draco_locate_decode(draco_plan* plan, const void* R, const float* f, uint8_t* flags, float* u, void* stream) {
    if (!plan || !R || !u || !flags || !aligned16(R) || !aligned16(u)) return DRACO_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    if (plan->code == DRACO_REP)
        return launch_rep_vote(plan, (const float*)R, plan->d, plan->d, u, nullptr, flags, true, st);
    // projection, then syndromes / solve / support / decode vector in one launch, then the recovery
    if (!f || !aligned16(f)) return DRACO_EINVAL;
    int rc = launch_cyc_project(plan, (const float2*)R, f, vec_len(plan), vec_len(plan), false, st);
    if (rc == DRACO_OK) rc = launch_cyc_solve(plan, nullptr, flags, true, st);
    if (rc != DRACO_OK) return rc;
    return launch_cyc_recover(plan, (const float2*)R, vec_len(plan), vec_len(plan), u, is_packed(plan) ? plan->d : 0, st);
}

int draco_cyc_decode_vector(draco_plan* plan, double* b_host, void* stream) {
    if (!plan || !is_cyc(plan) || !b_host) return DRACO_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    DRACO_CUDA(cudaMemcpyAsync(b_host, plan->cyc_dev->b, sizeof(double2) * plan->n, cudaMemcpyDeviceToHost, st));
    DRACO_CUDA(cudaStreamSynchronize(st));
    return DRACO_OK;
}

int draco_get_info(draco_plan* plan, draco_info* info, void* stream) {
    if (!plan || !info) return DRACO_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    DeviceInfo h;
    DRACO_CUDA(cudaMemcpyAsync(&h, plan->info_dev, sizeof(h), cudaMemcpyDeviceToHost, st));
    DRACO_CUDA(cudaStreamSynchronize(st));
    info->status = h.status;
    info->n_flagged = h.n_flagged;
    info->locator_rank = h.locator_rank;
    info->n_active = h.n_active;
    info->no_majority = h.no_majority;
    info->scale = h.scale;
    info->max_syndrome = h.max_syndrome;
    info->internal_error = h.internal_error;
    info->svd_sweeps = h.svd_sweeps;
    info->locator_margin = h.locator_margin;
    memcpy(&info->im_residual, &h.im_residual_bits, sizeof(double));
    memcpy(&info->re_max, &h.re_max_bits, sizeof(double));
    // The recovery kernel's blocks only merge their maxima; the verdict on them is formed here.  u-hat = G 1_P is
    // real: an imaginary part beyond rounding means an adversary is still among the rows that were combined.
    // (NaN from an adversary compares false with everything and so counts as a failed check.)
    if (is_cyc(plan) && (info->status == DRACO_OK || info->status == DRACO_EUNSURE)) {
        const bool decoded = info->re_max > 0.0 || info->im_residual > 0.0 || info->re_max != info->re_max;   // since the last locate
        const bool residual_ok = info->im_residual <= kImResidualBar * info->re_max;
        if (decoded && !residual_ok) {
            info->status = DRACO_EUNSURE;
        } else if (decoded && info->status == DRACO_EUNSURE && info->svd_sweeps >= 0 && !is_packed(plan)) {
            // the only open point was the first pass's margin, and the decode's own check came out clean: the
            // locator's later passes closed it (adversaries side by side; V then holds them all)
            info->status = DRACO_OK;
        }
    }
    return h.internal_error ? DRACO_EINTERNAL : DRACO_OK;
}

int draco_generate(float* out, int rows, int64_t len, int row0, float mean, float std, uint64_t seed, void* stream) {
    if (!out || rows < 1 || len < 1 || row0 < 0) return DRACO_EINVAL;
    return launch_generate(out, rows, len, len, 0, row0, mean, std, seed, (cudaStream_t)stream);
}

static int corrupt_range(const draco_plan* plan, void* R, int64_t c0, int64_t len, int64_t ld, const int* adv_idx,
                         const int* adv_model, const float* adv_param, int n_adv, uint64_t seed, cudaStream_t st) {
    const bool cplx = is_cyc(plan);
    const int64_t per = cplx ? 2 : 1;
    if (n_adv > plan->n) return DRACO_EINVAL;
    bool seen[kMaxN] = {};
    for (int a = 0; a < n_adv; ++a) {
        if (adv_idx[a] < 0 || adv_idx[a] >= plan->n || seen[adv_idx[a]]) return DRACO_EINVAL;   // all rows go in one launch
        seen[adv_idx[a]] = true;
        if (adv_model[a] < DRACO_ADV_REVGRAD || adv_model[a] > DRACO_ADV_GAUSS) return DRACO_EINVAL;
    }
    return launch_corrupt((float*)R, ld * per, len * per, c0 * per, adv_idx, adv_model, adv_param, n_adv, seed, cplx,
                          plan->sm_count, st);
}

int draco_corrupt(const draco_plan* plan, void* R, const int* adv_idx, const int* adv_model, const float* adv_param,
                  int n_adv, uint64_t seed, void* stream) {
    if (!plan || !R || n_adv < 0 || (n_adv > 0 && (!adv_idx || !adv_model || !adv_param))) return DRACO_EINVAL;
    return corrupt_range(plan, R, 0, vec_len(plan), vec_len(plan), adv_idx, adv_model, adv_param, n_adv, seed,
                         (cudaStream_t)stream);
}

int draco_pipeline_host(draco_plan* plan, const float* G_host, const float* f_host, const int* adv_idx,
                        const int* adv_model, const float* adv_param, int n_adv, uint64_t adv_seed, void* Z,
                        float* u_host, uint8_t* flags_host, draco_info* info) {
    if (!plan || !G_host || !Z || !u_host || !flags_host || !aligned16(Z)) return DRACO_EINVAL;
    if (n_adv < 0 || (n_adv > 0 && (!adv_idx || !adv_model || !adv_param))) return DRACO_EINVAL;
    const bool cyc = is_cyc(plan), packed = is_packed(plan);
    if (cyc && !f_host) return DRACO_EINVAL;
    const int n = plan->n;
    const int64_t d = plan->d;
    const int64_t vlen = vec_len(plan);              // entries per worker vector (complex entries when packed)
    // column chunk: about 256 MB of G per copy, a multiple of the projection tile
    int64_t chunk = ((int64_t)64 << 20) / n;
    chunk = (chunk / (2 * kProjectTile)) * (2 * kProjectTile);
    if (chunk < 2 * kProjectTile) chunk = 2 * kProjectTile;
    if (!plan->stage_dev) {                            // two staging buffers: the copy of chunk i+1 overlaps the kernels of chunk i
        DRACO_CUDA(cudaMalloc(&plan->stage_dev, sizeof(float) * (size_t)n * chunk * 2));
        plan->stage_chunk = chunk;
        DRACO_CUDA(cudaStreamCreateWithFlags(&plan->copy_stream, cudaStreamNonBlocking));
        DRACO_CUDA(cudaStreamCreateWithFlags(&plan->work_stream, cudaStreamNonBlocking));
        for (int b = 0; b < 2; ++b) {
            DRACO_CUDA(cudaEventCreateWithFlags(&plan->ev_copied[b], cudaEventDisableTiming));
            DRACO_CUDA(cudaEventCreateWithFlags(&plan->ev_consumed[b], cudaEventDisableTiming));
        }
    }
    if (!plan->u_dev) DRACO_CUDA(cudaMalloc(&plan->u_dev, sizeof(float) * (size_t)d));
    if (cyc && !plan->f_dev) DRACO_CUDA(cudaMalloc(&plan->f_dev, sizeof(float) * (size_t)vlen));
    chunk = plan->stage_chunk;
    const int64_t step = packed ? chunk / 2 : chunk;   // vector entries per chunk
    DRACO_CUDA(cudaDeviceSynchronize());               // earlier work of the caller that touches Z or the plan
    cudaStream_t st = plan->work_stream, cst = plan->copy_stream;
    if (cyc) DRACO_CUDA(cudaMemcpyAsync(plan->f_dev, f_host, sizeof(float) * (size_t)vlen, cudaMemcpyHostToDevice, st));
    bool first = true;
    int64_t chunk_no = 0;
    for (int64_t c0 = 0; c0 < vlen; c0 += step, ++chunk_no) {
        const int64_t len = (vlen - c0) < step ? (vlen - c0) : step;
        const int buf = (int)(chunk_no & 1);
        float* stage = plan->stage_dev + (size_t)buf * n * chunk;
        if (chunk_no >= 2) DRACO_CUDA(cudaStreamWaitEvent(cst, plan->ev_consumed[buf], 0));
        DRACO_CUDA(cudaMemcpy2DAsync(stage, sizeof(float) * (size_t)chunk, G_host + c0, sizeof(float) * (size_t)d,
                                     sizeof(float) * (size_t)len, n, cudaMemcpyHostToDevice, cst));
        int rc;
        if (cyc) {
            int64_t half = 0, d_stage = len;
            if (packed) {                              // second half of the gradient next to the first in the stage
                const int64_t len_b = (d - vlen - c0) < len ? (d - vlen - c0) : len;
                if (len_b > 0)
                    DRACO_CUDA(cudaMemcpy2DAsync(stage + step, sizeof(float) * (size_t)chunk, G_host + vlen + c0,
                                                 sizeof(float) * (size_t)d, sizeof(float) * (size_t)len_b, n,
                                                 cudaMemcpyHostToDevice, cst));
                half = step;
                d_stage = step + (len_b > 0 ? len_b : 0);
            }
            DRACO_CUDA(cudaEventRecord(plan->ev_copied[buf], cst));
            DRACO_CUDA(cudaStreamWaitEvent(st, plan->ev_copied[buf], 0));
            float2* Zc = (float2*)Z + c0;
            rc = launch_cyc_encode(plan, stage, Zc, len, chunk, vlen, half, d_stage, st);
            if (rc == DRACO_OK) rc = corrupt_range(plan, Z, c0, len, vlen, adv_idx, adv_model, adv_param, n_adv, adv_seed, st);
            if (rc == DRACO_OK) rc = launch_cyc_project(plan, Zc, plan->f_dev + c0, len, vlen, !first, st);
        } else {
            DRACO_CUDA(cudaEventRecord(plan->ev_copied[buf], cst));
            DRACO_CUDA(cudaStreamWaitEvent(st, plan->ev_copied[buf], 0));
            float* Zc = (float*)Z + c0;
            rc = launch_rep_encode(plan, stage, Zc, len, chunk, d, st);
            if (rc == DRACO_OK) rc = corrupt_range(plan, Z, c0, len, d, adv_idx, adv_model, adv_param, n_adv, adv_seed, st);
        }
        if (rc != DRACO_OK) return rc;
        DRACO_CUDA(cudaEventRecord(plan->ev_consumed[buf], st));
        first = false;
    }
    int rc;
    if (cyc) {
        rc = launch_cyc_solve(plan, nullptr, nullptr, true, st);
        if (rc == DRACO_OK) rc = launch_cyc_recover(plan, (const float2*)Z, vlen, vlen, plan->u_dev, packed ? d : 0, st);
    } else {
        rc = launch_rep_vote(plan, (const float*)Z, d, d, plan->u_dev, nullptr, nullptr, true, st);
    }
    if (rc != DRACO_OK) return rc;
    DRACO_CUDA(cudaMemcpyAsync(u_host, plan->u_dev, sizeof(float) * (size_t)d, cudaMemcpyDeviceToHost, st));
    DRACO_CUDA(cudaMemcpyAsync(flags_host, plan->flags_dev, n, cudaMemcpyDeviceToHost, st));
    if (info) return draco_get_info(plan, info, st);
    DRACO_CUDA(cudaStreamSynchronize(st));
    return DRACO_OK;
}

const char* draco_strerror(int code) {
    switch (code) {
        case DRACO_OK: return "ok";
        case DRACO_EINVAL: return "invalid argument";
        case DRACO_ECUDA: return "CUDA runtime error";
        case DRACO_ETOOMANY: return "more than 2 s nodes flagged: no decode vector exists";
        case DRACO_ENOMEM: return "out of memory";
        case DRACO_EINTERNAL: return "a bounded wait inside a kernel expired";
        case DRACO_ELIMIT: return "size exceeds a fixed capacity of this entry point";
        case DRACO_ENOMAJ: return "no strict majority at some coordinate";
        case DRACO_EUNSURE: return "a self-check of the cyclic decoder failed: the flags or the sum may be wrong";
        default: return "unknown code";
    }
}

const char* draco_last_cuda_error(void) { return g_cuda_error; }

}  // extern "C"

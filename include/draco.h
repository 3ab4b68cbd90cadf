/*
 * draco.h - C ABI of the B200 (sm_100a) implementation of the parameter-server
 * hot path of Draco (arXiv 1803.09877): redundant-gradient encoding, adversary
 * location and exact decoding for the repetition code and the cyclic code.
 *
 * Notation (the paper's, Section 3):  n = P compute nodes (= B gradients),
 * s = number of adversarial nodes tolerated, r = 2 s + 1 the redundancy ratio,
 * d = gradient dimension, G = [g_1 .. g_P], z_j = E_j(Y_j) what node j sends,
 * R = Z + N what the parameter server receives, u = D(R).
 *
 * Layout.  Every matrix is worker-major and dense: row k of G is gradient g_k
 * (d contiguous fp32), row j of Z / R is node j's vector: d fp32 for the
 * repetition code, d interleaved (re, im) fp32 pairs (complex64) for the cyclic
 * code (DRACO_CYC_PACKED: ceil(d / 2) such pairs, entry i holding gradient coordinates i and
 * ceil(d / 2) + i; the decoder returns [Re(u-hat); Im(u-hat)] cut to d entries).  u is d fp32.
 * Indices are 0-based.  Row stride = the row length.
 *
 * Ownership.  The caller owns every buffer it passes (device buffers unless a
 * parameter says "host"); the library never frees or keeps them.  A plan owns
 * its code tables and a small device scratch area allocated by
 * draco_plan_create (kilobytes to a few hundred kilobytes), released by
 * draco_plan_destroy.  Device pointers must be 16-byte aligned.
 *
 * Streams.  `stream` is a cudaStream_t passed as void* (NULL = the default
 * stream).  Calls enqueue work and return without synchronising unless stated.
 * Calls on one plan must not overlap on the device (they share its scratch).
 *
 * Errors.  Functions return DRACO_OK (0) or a negative DRACO_E* code; nothing
 * throws or aborts.  Conditions found on the device (too many nodes flagged, no
 * strict majority somewhere) are reported through draco_get_info.
 */
#ifndef DRACO_H_
#define DRACO_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct draco_plan draco_plan;

/* code type */
enum {
    DRACO_REP = 0,        /* repetition code, fp32 vectors of d entries */
    DRACO_CYC = 1,        /* cyclic code, complex64 vectors of d entries */
    DRACO_CYC_PACKED = 2  /* cyclic code on the packed gradient (Section 3, last paragraph): complex64 vectors of
                             ceil(d / 2) entries, entry i = (G_i, G_{ceil(d/2)+i}); f has ceil(d / 2) entries; u has d */
};
/* adversary models of the corruptor (Section 4, "Adversarial Attack Models", plus Gaussian noise) */
enum { DRACO_ADV_REVGRAD = 0, DRACO_ADV_CONST = 1, DRACO_ADV_GAUSS = 2 };
/* return codes */
enum {
    DRACO_OK = 0,
    DRACO_EINVAL = -1,   /* bad argument: n < 1, s < 0, 2 s + 1 > n (Corollary of Theorem 1), null or misaligned pointer */
    DRACO_ECUDA = -2,    /* a CUDA runtime call failed (see draco_last_cuda_error) */
    DRACO_ETOOMANY = -3, /* more than 2 s nodes flagged: no decode vector exists (u is written as zeros) */
    DRACO_ENOMEM = -4,
    DRACO_EINTERNAL = -5, /* a bounded wait inside a kernel expired (reported by draco_get_info); results are invalid.
                             Kept for ABI stability: the current kernels contain no such wait and never report it */
    DRACO_ELIMIT = -6,   /* a size exceeds a fixed capacity of the entry point called (see draco_cyc_project_noalloc) */
    DRACO_ENOMAJ = 1,    /* warning: some (group, coordinate) had no strict majority; u holds Algorithm 2's candidate */
    DRACO_EUNSURE = 2    /* warning (cyclic): a self-check of the decoder failed, so V or u may be wrong: the flagged and
                            the unflagged |t_j| are less than a factor 10 apart (locator_margin), or the recovered u-hat has
                            an imaginary part above 1e-2 of its real part (im_residual, re_max), or the singular-value
                            iteration of the syndrome system stopped at its sweep limit (svd_sweeps < 0).  More than s
                            adversaries, or adversaries that the precision of complex64 vectors cannot separate, show up
                            here; u is still written.  Once an unpacked plan has decoded, im_residual decides: a low
                            locator_margin next to a clean residual means that the locator's later passes closed what its
                            first pass left open, and the status is DRACO_OK; packed plans have no residual to go by */
};

#define DRACO_MAX_N 128  /* largest supported number of nodes */

/* Device-side results of the most recent locate / decode on a plan. */
typedef struct draco_info {
    int32_t status;        /* DRACO_OK, DRACO_ETOOMANY, DRACO_ENOMAJ or DRACO_EUNSURE */
    int32_t n_flagged;     /* |V|: nodes flagged by the last locate (or given to the last cyclic decode) */
    int32_t locator_rank;  /* cyclic: adversaries seen = sum over the locator's passes of the numerical rank of the pass's system */
    int32_t n_active;      /* cyclic decode: number of rows with b_j != 0 */
    uint64_t no_majority;  /* repetition: (group, coordinate) pairs without a strict majority */
    double scale;          /* cyclic: median_j q_j^(1/2), q_j = sum_i |R[j][i]|^2: the unit of the rank cutoff */
    double max_syndrome;   /* cyclic: max_m |h_m| over the 2 s syndromes */
    int32_t internal_error; /* non-zero: a kernel gave up a bounded wait (sticky); draco_get_info then returns DRACO_EINTERNAL.
                               Always 0 with the current kernels, none of which spins on a flag */
    int32_t svd_sweeps;    /* cyclic locate: Jacobi sweeps the singular-value iteration of the s x s syndrome system took
                              (0 when it was skipped: s = 0, or all syndromes within the cutoff); negative (minus the
                              limit of 60) when it was still rotating at the limit: rank and V are then not to be trusted */
    double locator_margin; /* cyclic locate: |t| of the weakest flagged node / |t| of the strongest unflagged one (exactly
                              `rank` entries of t are non-zero in exact arithmetic, so this is large when the flags can be
                              trusted and near 1 when they cannot); 1e300 when no node or every node is flagged */
    double im_residual;    /* cyclic decode, unpacked plans: max |Im(u-hat_i)| over the coordinates i with floor(i / 64) mod 8 = 0.
                              u-hat = R_{.,U} b is real when every node of U is honest, so against re_max this tells a decode
                              whose U still holds an adversary (wrong or missing flags, more than s adversaries) from a good
                              one, whose residual is the rounding floor of complex64 vectors; 0 for packed plans */
    double re_max;         /* the same maximum of |Re(u-hat_i)|, the scale for im_residual */
} draco_info;

/*
 * Build the tables for one (n, s, d, code) and allocate the plan's scratch on
 * the current CUDA device.  Repetition code (Section 3, "Fractional Repetition
 * Code"): groups of consecutive nodes; n / r groups of r when r divides n,
 * otherwise floor(n / r) groups whose sizes differ by at most one (all >= r).
 * Cyclic code (Section 3, "Cyclic Code"): the matrix W = [Q 1_P] C_L in closed
 * form, the IDFT twiddles, and the locator / decode-vector work space.
 * Requires 1 <= n <= DRACO_MAX_N, s >= 0, 2 s + 1 <= n, d >= 1.
 */
int draco_plan_create(int n, int s, int64_t d, int code, draco_plan** out);
int draco_plan_destroy(draco_plan* plan);

/* Rank cutoff theta of the cyclic locator (default 1e-6): singular values of the s x s syndrome
 * system below theta * median_j q_j^(1/2) count as zero, q_j = sum_i |R[j][i]|^2 (the size of what
 * node j sent: complex64 rounding perturbs e_j by about 2^-25 (2 q_j)^(1/2) even where e_j itself
 * cancels to something small; the paper's "t_j != 0" needs such a yardstick and names none).
 * The rank found is the number of adversaries seen, and V is the set of that many nodes with the
 * largest |t_j| (exactly that many t_j are non-zero in exact arithmetic). */
int draco_plan_set_theta(draco_plan* plan, double theta);

/* Number of groups of a repetition plan (0 for a cyclic plan); group g covers
 * nodes first[g] .. first[g] + size[g] - 1 (host arrays of draco_num_groups entries, may be NULL). */
int draco_num_groups(const draco_plan* plan);
int draco_groups(const draco_plan* plan, int* first /*host*/, int* size /*host*/);

/* Cyclic plans: copy W (n x n complex, row-major, (re, im) doubles; z_j = sum_k W[k][j] g_k) to host memory. */
int draco_cyc_W(const draco_plan* plan, double* W_host /*host [n][n][2]*/);

/*
 * Encoding: Z[j] = E_j(Y_j) for all n nodes in one pass over G.
 *   repetition: z_j = Y_j 1_P = sum of the gradients of j's group, ascending, fp32
 *               (members of a group produce identical bits);
 *   cyclic:     z_j = G W_{.,j} = sum_{t=0..2s} W[j-t][j] g_{(j-t) mod n}, complex64.
 * G: device [n][d] fp32.  Z: device [n][d] fp32 (repetition) or complex64 (cyclic).
 */
int draco_encode(const draco_plan* plan, const float* G, void* Z, void* stream);

/*
 * Locating the adversaries: flags[j] = 1 iff node j is in V, else 0.
 *   repetition: j is flagged when its vector differs in any bit, at any coordinate,
 *               from the majority of its group (derived from D^Rep; f is ignored);
 *   cyclic:     V = phi(R): e = f R (fp64 accumulation), the 2 s syndromes e C_R^dagger,
 *               the s x s Toeplitz system for beta (pseudo-inverse solution from an SVD),
 *               the recurrence h_l = sum_u beta_u h_{l+u-s}, t = IDFT(h), V = supp(t)
 *               read as the rank-many largest |t_j|.  That is one pass; further passes treat the nodes
 *               flagged so far as erasures (modified syndromes sum_k lambda_k h_{m-k}, lambda(x) =
 *               prod_{v in V} (x - w^v)) and look for more in the same way, until a pass finds nothing:
 *               adversaries side by side, which one pass cannot always separate with complex64 vectors, end
 *               up in V all the same, at times together with an honest neighbour (V then is a superset of
 *               the adversaries, which is all that decoding needs, as long as |V| <= 2 s).  A node whose
 *               vector holds NaN or infinities (its projection is then not finite) is in V from the start.
 * R: device [n][d].  f: device [d] fp32, the caller's draw of N(1_d, I_d) (cyclic only).
 * flags: device [n] bytes.
 */
int draco_locate(draco_plan* plan, const void* R, const float* f, uint8_t* flags, void* stream);

/*
 * Decoding: u = D(R).
 *   repetition: u = sum over groups of Maj(group) (Algorithm 2 on 32-bit patterns), groups
 *               ascending, fp32; flags may be NULL and is ignored;
 *   cyclic:     Algorithm 1, steps 2-4: U = nodes with flags[j] = 0, b = the minimum-norm
 *               solution of W_{.,U} b = 1_P, u = Re(R_{.,U} b), fp64 accumulation, fp32 result.
 * flags: device [n] bytes, or NULL.  Cyclic plans with flags == NULL decode with the set V that the most recent
 * draco_locate / draco_cyc_locate_from_projection on this plan found (the plan keeps its own copy; no node is
 * flagged on a plan that has not located yet), so locate and decode chain without the caller holding V.
 * u: device [d] fp32.
 */
int draco_decode(draco_plan* plan, const void* R, const uint8_t* flags, float* u, void* stream);

/*
 * Decoding fused with the model update of Section 2 (mini-batch SGD, w_k = w_{k-1} - gamma / |S_k| * sum of gradients):
 * w <- w - scale * D(R) in the decoder's epilogue; u is never written.  w: device [d] fp32, read and written.
 * Same arguments and arithmetic as draco_decode; each entry of D(R) is rounded to fp32, then one fused multiply-add.
 * When more than 2 s nodes are flagged (cyclic) D(R) is zero and w is left unchanged.
 */
int draco_decode_update(draco_plan* plan, const void* R, const uint8_t* flags, float* w, float scale, void* stream);

/* locate + decode in one call.  Repetition: one pass over R.  Cyclic: three launches for short vectors (projection;
 * one kernel for the sum of the block partials, the locator and the decode vector; recovery), one more (the
 * reduction of the block partials) when the projection ran on more than 64 blocks.  f as in draco_locate. */
int draco_locate_decode(draco_plan* plan, const void* R, const float* f, uint8_t* flags, float* u, void* stream);

/* Repetition code with the selections exposed: maj (device [groups][d] fp32, may be NULL) receives
 * the value selected for every group and coordinate; u and flags may be NULL. */
int draco_rep_vote(draco_plan* plan, const void* R, float* u, float* maj, uint8_t* flags, void* stream);

/* The two halves of the cyclic locator, for callers that shard d across devices and add the
 * projection records.  e: device, 3 n doubles, 16-byte aligned: e_j = (f R)_j as n (re, im) pairs, then the
 * n values q_j = sum_i |R[j][i]|^2 that set the rank cutoff; both are sums over this plan's d
 * coordinates, so records of disjoint coordinate ranges add up. */
int draco_cyc_project(draco_plan* plan, const void* R, const float* f, double* e, void* stream);
int draco_cyc_locate_from_projection(draco_plan* plan, const double* e, uint8_t* flags, void* stream);

/*
 * The projection e = f R again, for callers that may not allocate.  (The paper has no counterpart:
 * this is a deployment variant of draco_cyc_project, not a step of the method.)
 *
 * Who needs it: a host process whose device memory is owned entirely by another allocator (a
 * serving framework's pool that took the whole GPU at start-up, so a later cudaMalloc fails or
 * splits the pool), or a step loop that cannot tolerate the device-wide synchronisation that an
 * allocation or free may imply.  draco_plan_create allocates; this entry point needs no plan and
 * calls neither cudaMalloc nor cudaFree nor any allocating library routine.  Its only scratch, the
 * per-block partial sums, is a fixed array compiled into the library: 296 blocks x 128 nodes x 24
 * bytes = 888 KB of device memory on every GPU that loads the library, held until the process ends.
 *
 * n nodes, d coordinates; R: device [n][d] complex64; f: device [d] fp32; e: device, 3 n doubles (the
 * projection record of draco_cyc_project: n (re, im) pairs, then n values q_j), written by the call.
 * All three 16-byte aligned; the caller owns them.
 * Limits: n <= DRACO_MAX_N (128) and device ordinal < 64, else DRACO_ELIMIT; d is unbounded
 * (at most 296 blocks are launched, each walking its share of the tiles).
 * The first call on each device looks up the array's device address (with that device current);
 * make that first call before any stream capture begins.  The CUDA runtime may place the library's
 * kernels and this array in device memory only then (lazy module loading), so where another allocator
 * is about to take the whole device, make one call on it (any small input) before that happens: a
 * first call on a device with no memory left fails with DRACO_ECUDA.  All calls on a device share the one
 * array, which keeps the previous call's contents (every call overwrites all entries it reads, so
 * nothing needs clearing); two calls that overlap on the GPU, on any streams, race on it.
 * Same kernel and arithmetic as draco_cyc_project; only the number of fp64 block partials may differ
 * (296 at most here), so the two agree to fp64 rounding (about 1e-15 relative).
 */
int draco_cyc_project_noalloc(int n, int64_t d, const void* R, const float* f, double* e, void* stream);

/* The decode vector b of the last cyclic decode (host [n][2] doubles); synchronises the stream. */
int draco_cyc_decode_vector(draco_plan* plan, double* b_host /*host*/, void* stream);

/* Copies the device-side results of the last calls to host memory; synchronises the stream. */
int draco_get_info(draco_plan* plan, draco_info* info /*host*/, void* stream);

/*
 * Whole path with host buffers (pageable or pinned): copies G and f to the device in
 * column chunks, encodes, applies the given adversaries, locates, decodes, and copies
 * u and flags back.  Synchronous: waits for the device's earlier work on entry, runs on two internal streams (the copy
 * of one chunk overlaps the kernels of the previous one) and returns when u and flags are on the host.  The first call
 * on a plan allocates two staging buffers (n x 2 x chunk floats), u and f on the device.
 * Z (device, one row per node, caller-owned) keeps the received matrix.
 */
int draco_pipeline_host(draco_plan* plan, const float* G_host, const float* f_host,
                        const int* adv_idx /*host*/, const int* adv_model /*host*/, const float* adv_param /*host*/,
                        int n_adv, uint64_t adv_seed, void* Z, float* u_host, uint8_t* flags_host,
                        draco_info* info /*host, may be NULL*/);

/*
 * Seeded synthetic inputs (counter-based; identical bits to the published definition:
 * row key = SplitMix64 output number row+1 from state seed; element i of a row sums the eight
 * 16-bit fields of outputs 2 i + 1 and 2 i + 2 from state key, S; value =
 * fl32(fl32(fl32(S - 262140) * c) * std) + mean with c = fl32(1 / sqrt(8 (2^32 - 1) / 12))).
 * out: device [rows][len] fp32, rows numbered row0 .. row0 + rows - 1.
 */
int draco_generate(float* out, int rows, int64_t len, int row0, float mean, float std, uint64_t seed, void* stream);

/*
 * The adversary: R = Z + N in place, N non-zero on rows adv_idx[0 .. n_adv-1] (host arrays, distinct
 * node indices; all rows are rewritten by one kernel launch).
 *   DRACO_ADV_REVGRAD: row <- -c * row          (param = c)
 *   DRACO_ADV_CONST:   row <- kappa             (param = kappa; imaginary parts 0)
 *   DRACO_ADV_GAUSS:   row <- row + sigma * x   (param = sigma; x from the generator above with
 *                      seed `seed`, row = node index, over the row's fp32 values)
 */
int draco_corrupt(const draco_plan* plan, void* R, const int* adv_idx, const int* adv_model,
                  const float* adv_param, int n_adv, uint64_t seed, void* stream);

const char* draco_strerror(int code);
/* Text of the last CUDA error seen by this library on the calling thread ("" if none). */
const char* draco_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* DRACO_H_ */

// Cyclic-code adversary locator phi(R) (Section 3, "Cyclic Code"; correctness: Lemmas 4, 6-8).
//
//   cyc_project_kernel   e_j = sum_i f_i R[j][i]: the one O(d P) step, a single pass over R; beside it
//                        q_j = sum_i |R[j][i]|^2, the yardstick of the rank cutoff below.
//   cyc_reduce_partials_kernel   the blocks' partial sums of e and q added up in a fixed order.
//   cyc_solve_kernel     [h_{n-2s} .. h_{n-1}] = e C_R^dagger, the s x s Toeplitz system for
//                        beta (pseudo-inverse by a Jacobi SVD: its rank = the number of
//                        adversaries seen), the recurrence h_l = sum_u beta_u h_{l+u-s}, t = C h,
//                        V = the `rank` nodes with the largest |t_j|.
//   cyc_decode_vector_kernel   b with support in U = [n] \ V and [C_L]_{.,U} b_U = (0,..,0,1)^T
//                        (equivalent to W_{.,U} b = 1_P, proof of Lemma 3), minimum 2-norm.
//
// The small solves run in fp64 in a single thread block; only the projection touches HBM:
// 8 n len + 4 len bytes read.
#include <mutex>

#include "draco_internal.cuh"

namespace draco {

namespace {

constexpr int kThreads = kProjectWarps * 32;
constexpr int kSolveThreads = 512;

__device__ __forceinline__ double2 cmul(double2 a, double2 b) {
    return make_double2(a.x * b.x - a.y * b.y, a.x * b.y + a.y * b.x);
}
__device__ __forceinline__ double2 cmulc(double2 a, double2 b) {   // a * conj(b)
    return make_double2(a.x * b.x + a.y * b.y, a.y * b.x - a.x * b.y);
}
__device__ __forceinline__ double2 cdiv(double2 a, double2 b) {
    const double den = b.x * b.x + b.y * b.y;
    const double2 q = cmulc(a, b);
    return make_double2(q.x / den, q.y / den);
}
__device__ __forceinline__ double cabs2(double2 a) { return a.x * a.x + a.y * a.y; }

// ------------------------------------------------------------------ projection
// Arithmetic.  f_i and R[j][i] are fp32, so their product has at most 48 significant bits and is exact in fp64:
// every term enters an fp64 running sum through one fused multiply-add on the converted operands, and the only
// rounding left is that of fp64 addition (2^-53 per term).  The device's e_j therefore carries the rounding of the
// complex64 vectors themselves and nothing of its own; products or short runs in fp32 would add about as much
// again per term (a 16-term fp32 run: three times as much), which the s x s syndrome system amplifies by about
// sqrt(s): at s = 20 that noise alone reached the rank cutoff and flagged an honest node.
//
// q_j = sum_i |R[j][i]|^2 travels with e_j: it is the yardstick of the locator's rank cutoff (rounding R to
// complex64 perturbs e_j by about 2^-25 (E f^2 q_j)^(1/2), whatever e_j itself cancels to).  It is summed in fp64
// from the converted values as well: squares of fp32 values overflow fp32 from 1.8e19 on, which a node may well
// send (W itself reaches 1e17 at n = 128, s = 20).  Layout of the block partials: [grid][n] double2 (e), then
// [grid][n] double (q).
__device__ __forceinline__ double warp_sum(double a) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
    return a;
}
// Block partials: [cap][n] double2 (e) followed by [cap][n] double (q); cap = the capacity of the buffer in blocks,
// of which a launch fills the first gridDim.x.
__device__ __forceinline__ double* q_partials(double2* partial, int cap, int n) {
    return reinterpret_cast<double*>(partial + (int64_t)cap * n);
}
// Block = 8 warps over one tile of coordinates; warp w owns rows row0 + w, row0 + w + 8, ... of the
// launch's nrows <= 8 RPW rows; f for the tile sits in shared memory as fp64 (converted once per tile, used by
// every row).  More than 64 rows take two launches of half the rows each (rows are
// independent; f is read twice, 1 % more traffic): 16 rows per warp in registers halve the blocks per SM
// (0.79 of the copy bandwidth at n = 105), and per-lane sums in shared memory left the compiler too few
// registers to keep its loads in flight once the squared norms were added (0.98 -> 0.68).
template <int RPW, bool VEC2>
__global__ void __launch_bounds__(kThreads, 4)
cyc_project_kernel(const float2* __restrict__ R, const float* __restrict__ f, int64_t len, int64_t ld, int n,
                   int row0, int nrows, double2* __restrict__ partial, int cap, int accumulate) {
    __shared__ __align__(16) double fs[kProjectTile];
    // Running sums of row warp + r * 8 over this block's tiles, kept by lane 0 of the row's warp: after every tile
    // the warp adds its lanes' sums up (fixed butterfly order) and lane 0 adds the result here.  Keeping them in
    // registers instead (2 RPW doubles per lane) left too few of the 64 registers for eight 128-bit loads in flight.
    __shared__ double2 es[kProjectWarps * RPW];
    __shared__ double qs[kProjectWarps * RPW];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Short vectors have fewer tiles than the device has SMs; the launch then splits the rows over gridDim.y as well
    // (whole multiples of the 8 warps' rows), every (tile, node) partial still being written by exactly one block.
    if (gridDim.y > 1) {
        const int per = (((nrows + (int)gridDim.y - 1) / (int)gridDim.y + kProjectWarps - 1) / kProjectWarps) * kProjectWarps;
        const int skip = (int)blockIdx.y * per;
        if (skip >= nrows) return;
        row0 += skip;
        nrows = (nrows - skip) < per ? (nrows - skip) : per;
    }
    if (lane == 0) {
#pragma unroll
        for (int r = 0; r < RPW; ++r) {
            es[r * kProjectWarps + warp] = make_double2(0.0, 0.0);
            qs[r * kProjectWarps + warp] = 0.0;
        }
    }

    const int64_t ntiles = (len + kProjectTile - 1) / kProjectTile;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const int64_t c0 = tile * kProjectTile;
        const int cnt = (int)((len - c0) < kProjectTile ? (len - c0) : kProjectTile);
        for (int i = threadIdx.x; i < kProjectTile; i += kThreads) fs[i] = (i < cnt) ? (double)__ldcs(f + c0 + i) : 0.0;
        __syncthreads();
#pragma unroll
        for (int r = 0; r < RPW; ++r) {
            const int j = row0 + warp + r * kProjectWarps;
            if (j < row0 + nrows) {
                const float2* row = R + (int64_t)j * ld + c0;
                double eq = 0.0;
                double ar = 0.0, ai = 0.0;
                if (VEC2 && cnt == kProjectTile) {
                    const float4* row4 = reinterpret_cast<const float4*>(row);
#pragma unroll 1
                    for (int step0 = 0; step0 < kProjectTile / 64; step0 += 8) {
                        float4 v[8];
#pragma unroll
                        for (int q = 0; q < 8; ++q) v[q] = __ldcs(row4 + (step0 + q) * 32 + lane);
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            const double2 ff = *reinterpret_cast<const double2*>(&fs[((step0 + q) * 32 + lane) * 2]);
                            const double x0 = (double)v[q].x, y0 = (double)v[q].y, x1 = (double)v[q].z, y1 = (double)v[q].w;
                            ar = fma(ff.x, x0, ar); ai = fma(ff.x, y0, ai);
                            ar = fma(ff.y, x1, ar); ai = fma(ff.y, y1, ai);
                            eq = fma(x0, x0, eq); eq = fma(y0, y0, eq);
                            eq = fma(x1, x1, eq); eq = fma(y1, y1, eq);
                        }
                    }
                } else {
                    for (int i = lane; i < cnt; i += 32) {
                        const float2 v = __ldcs(row + i);
                        const double ff = fs[i], x0 = (double)v.x, y0 = (double)v.y;
                        ar = fma(ff, x0, ar);
                        ai = fma(ff, y0, ai);
                        eq = fma(y0, y0, fma(x0, x0, eq));
                    }
                }
                ar = warp_sum(ar);
                ai = warp_sum(ai);
                eq = warp_sum(eq);
                if (lane == 0) {
                    double2 acc = es[r * kProjectWarps + warp];
                    acc.x += ar;
                    acc.y += ai;
                    es[r * kProjectWarps + warp] = acc;
                    qs[r * kProjectWarps + warp] += eq;
                }
            }
        }
        __syncthreads();
    }
    double* qpartial = q_partials(partial, cap, n);
    if (lane == 0) {
#pragma unroll
        for (int r = 0; r < RPW; ++r) {
            const int j = row0 + warp + r * kProjectWarps;
            if (j < row0 + nrows) {
                double2* dst = partial + (int64_t)blockIdx.x * n + j;
                double* qdst = qpartial + (int64_t)blockIdx.x * n + j;
                double2 a = es[r * kProjectWarps + warp];
                double c = qs[r * kProjectWarps + warp];
                if (accumulate) { a.x += dst->x; a.y += dst->y; c += *qdst; }
                *dst = a;
                *qdst = c;
            }
        }
    }
}

// The same projection for few rows (n <= 16): with one or two rows per warp the block-wide tile
// barriers of the kernel above dominate, so here every warp works alone on 256-coordinate chunks
// of all n rows, with f for its chunk in registers (8 values per lane) and no
// shared memory or barrier in the loop.  Per-lane running sums in fp64 registers (2 n doubles).
template <bool VEC2>
__global__ void __launch_bounds__(kThreads, 2)
cyc_project_fewrows_kernel(const float2* __restrict__ R, const float* __restrict__ f, int64_t len, int64_t ld, int n,
                           double2* __restrict__ partial, int cap, int accumulate) {
    constexpr int NMAX = 16, CH = 256;
    __shared__ double2 wsum[kProjectWarps][NMAX];
    __shared__ double wq[kProjectWarps][NMAX];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double accr[NMAX], acci[NMAX];
#pragma unroll
    for (int j = 0; j < NMAX; ++j) { accr[j] = 0.0; acci[j] = 0.0; }
    if (lane < NMAX) wq[warp][lane] = 0.0;               // q_j of this warp's chunks: summed over the lanes per chunk, kept here
    __syncwarp();
    const int64_t nchunks = (len + CH - 1) / CH;
    const int64_t nwarps = (int64_t)gridDim.x * kProjectWarps;
    for (int64_t chunk = (int64_t)blockIdx.x * kProjectWarps + warp; chunk < nchunks; chunk += nwarps) {
        const int64_t c0 = chunk * CH;
        const int cnt = (int)((len - c0) < CH ? (len - c0) : CH);
        if (VEC2 && cnt == CH) {
            float2 ff[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) ff[q] = __ldcs(reinterpret_cast<const float2*>(f + c0) + q * 32 + lane);
#pragma unroll
            for (int jj = 0; jj < NMAX; jj += 2) {
                if (jj < n) {
                    float4 va[4], vb[4];
                    const float4* ra = reinterpret_cast<const float4*>(R + (int64_t)jj * ld + c0);
                    const bool two = jj + 1 < n;
                    const float4* rb = reinterpret_cast<const float4*>(R + (int64_t)(two ? jj + 1 : jj) * ld + c0);
#pragma unroll
                    for (int q = 0; q < 4; ++q) va[q] = __ldcs(ra + q * 32 + lane);
                    if (two) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) vb[q] = __ldcs(rb + q * 32 + lane);
                    }
                    double qa = 0.0, qb = 0.0;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const double fx = (double)ff[q].x, fy = (double)ff[q].y;     // shared by the two rows
                        double x0 = (double)va[q].x, y0 = (double)va[q].y, x1 = (double)va[q].z, y1 = (double)va[q].w;
                        accr[jj] = fma(fx, x0, accr[jj]); acci[jj] = fma(fx, y0, acci[jj]);
                        accr[jj] = fma(fy, x1, accr[jj]); acci[jj] = fma(fy, y1, acci[jj]);
                        qa = fma(x0, x0, qa); qa = fma(y0, y0, qa); qa = fma(x1, x1, qa); qa = fma(y1, y1, qa);
                        if (two) {
                            x0 = (double)vb[q].x; y0 = (double)vb[q].y; x1 = (double)vb[q].z; y1 = (double)vb[q].w;
                            accr[jj + 1] = fma(fx, x0, accr[jj + 1]); acci[jj + 1] = fma(fx, y0, acci[jj + 1]);
                            accr[jj + 1] = fma(fy, x1, accr[jj + 1]); acci[jj + 1] = fma(fy, y1, acci[jj + 1]);
                            qb = fma(x0, x0, qb); qb = fma(y0, y0, qb); qb = fma(x1, x1, qb); qb = fma(y1, y1, qb);
                        }
                    }
                    qa = warp_sum(qa);
                    qb = warp_sum(qb);
                    if (lane == 0) { wq[warp][jj] += qa; if (two) wq[warp][jj + 1] += qb; }
                }
            }
        } else {
            for (int i0 = 0; i0 < cnt; i0 += 32) {           // every lane takes part in the sums over the lanes below
                const int i = i0 + lane;
                const bool valid = i < cnt;
                const double fi = valid ? (double)__ldcs(f + c0 + i) : 0.0;
#pragma unroll
                for (int j = 0; j < NMAX; ++j)
                    if (j < n) {
                        const float2 v = valid ? __ldcs(R + (int64_t)j * ld + c0 + i) : make_float2(0.f, 0.f);
                        const double x0 = (double)v.x, y0 = (double)v.y;
                        accr[j] = fma(fi, x0, accr[j]);
                        acci[j] = fma(fi, y0, acci[j]);
                        const double qv = warp_sum(fma(y0, y0, x0 * x0));
                        if (lane == 0) wq[warp][j] += qv;
                    }
            }
        }
    }
#pragma unroll
    for (int j = 0; j < NMAX; ++j) {
        double a = accr[j], b = acci[j];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            a += __shfl_xor_sync(0xffffffffu, a, off);
            b += __shfl_xor_sync(0xffffffffu, b, off);
        }
        if (lane == 0) wsum[warp][j] = make_double2(a, b);
    }
    __syncthreads();
    if (threadIdx.x < n) {
        double a = 0.0, b = 0.0, c = 0.0;
        for (int w = 0; w < kProjectWarps; ++w) {            // fixed order: reproducible
            a += wsum[w][threadIdx.x].x;
            b += wsum[w][threadIdx.x].y;
            c += wq[w][threadIdx.x];
        }
        double2* dst = partial + (int64_t)blockIdx.x * n + threadIdx.x;
        double* qdst = q_partials(partial, cap, n) + (int64_t)blockIdx.x * n + threadIdx.x;
        if (accumulate) { a += dst->x; b += dst->y; c += *qdst; }
        *dst = make_double2(a, b);
        *qdst = c;
    }
}

// e_j and q_j = sums over the blocks' partials: one block of 128 threads per node j.  Thread t adds the partials
// of blocks t, t + 128, .. in ascending order, the 128 thread sums are then added by a butterfly inside each warp
// and the four warp sums in ascending order.  The order is fixed, so the sums are reproducible bit for bit.
// record: n (re, im) pairs, then n values q_j (3 n doubles).  (A single block doing this for all nodes took
// 20-40 us: one SM's load latency, serialised.)
constexpr int kReduceThreads = 128;
__global__ void __launch_bounds__(kReduceThreads)
cyc_reduce_partials_kernel(const double2* __restrict__ partial, int grid, int cap, int n, double* __restrict__ record) {
    constexpr int kBatch = 8;
    __shared__ double wsum[3][kReduceThreads / 32];
    const int j = blockIdx.x, tid = threadIdx.x;
    const double* __restrict__ qpartial = reinterpret_cast<const double*>(partial + (int64_t)cap * n);
    double a = 0.0, b = 0.0, c = 0.0;
    for (int base = 0; base < grid; base += kBatch * kReduceThreads) {
        double2 pe[kBatch];
        double pq[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {               // all loads first (beyond the grid: block 0 again, not added)
            const int blk = base + u * kReduceThreads + tid;
            const int64_t at = (int64_t)(blk < grid ? blk : 0) * n + j;
            pe[u] = __ldcg(partial + at);
            pq[u] = __ldcg(qpartial + at);
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            if (base + u * kReduceThreads + tid < grid) {
                a += pe[u].x;
                b += pe[u].y;
                c += pq[u];
            }
        }
    }
    a = warp_sum(a);
    b = warp_sum(b);
    c = warp_sum(c);
    if ((tid & 31) == 0) { wsum[0][tid >> 5] = a; wsum[1][tid >> 5] = b; wsum[2][tid >> 5] = c; }
    __syncthreads();
    if (tid == 0) {
        double x = 0.0, y = 0.0, z = 0.0;
        for (int w = 0; w < kReduceThreads / 32; ++w) { x += wsum[0][w]; y += wsum[1][w]; z += wsum[2][w]; }
        record[2 * j] = x;
        record[2 * j + 1] = y;
        record[2 * n + j] = z;
    }
}

// The small solves below run either on the whole block (WARP = false: block-wide barriers, any size) or on its
// first warp alone (WARP = true: warp barriers only; the matrices then sit in shared memory).  The arithmetic and
// its order are the same in both.
template <bool WARP>
__device__ __forceinline__ void small_sync() {
    if (WARP) __syncwarp(); else __syncthreads();
}

// ------------------------------------------------------------------ small dense solve
// Gauss-Jordan elimination with complete pivoting on the dim x (dim+1) augmented matrix A
// (row stride dim+1).  Pivots with |pivot| <= tol end the elimination (numerical rank); the
// free unknowns are set to zero.  x receives the solution.  WARP: called by warp 0 only, dim <= 32.
template <bool WARP>
__device__ int block_gauss_jordan(double2* A, int dim, double tol, double2* x, int* perm, double* rowbest,
                                  int* rowbestc, int* sh) {
    const int tid = threadIdx.x, ldA = dim + 1;
    const int nthr = WARP ? 32 : blockDim.x;
    for (int i = tid; i < dim; i += nthr) perm[i] = i;
    small_sync<WARP>();
    int rank = 0;
    for (int p = 0; p < dim; ++p) {
        for (int i = p + tid; i < dim; i += nthr) {
            double best = -1.0;
            int bc = p;
            for (int c = p; c < dim; ++c) {
                const double m = cabs2(A[i * ldA + c]);
                if (m > best) { best = m; bc = c; }
            }
            rowbest[i] = best;
            rowbestc[i] = bc;
        }
        small_sync<WARP>();
        if (tid == 0) {
            double best = -1.0;
            int br = p;
            for (int i = p; i < dim; ++i)
                if (rowbest[i] > best) { best = rowbest[i]; br = i; }
            sh[0] = br;
            sh[1] = rowbestc[br];
            sh[2] = (best > tol * tol) ? 1 : 0;
        }
        small_sync<WARP>();
        const int pr = sh[0], pc = sh[1], ok = sh[2];
        if (!ok) break;
        if (pr != p)
            for (int c = tid; c <= dim; c += nthr) {
                const double2 tmp = A[p * ldA + c];
                A[p * ldA + c] = A[pr * ldA + c];
                A[pr * ldA + c] = tmp;
            }
        small_sync<WARP>();
        if (pc != p) {
            for (int i = tid; i < dim; i += nthr) {
                const double2 tmp = A[i * ldA + p];
                A[i * ldA + p] = A[i * ldA + pc];
                A[i * ldA + pc] = tmp;
            }
            if (tid == 0) { const int tmp = perm[p]; perm[p] = perm[pc]; perm[pc] = tmp; }
        }
        small_sync<WARP>();
        const double2 piv = A[p * ldA + p];
        for (int i = tid; i < dim; i += nthr) {
            if (i == p) continue;
            const double2 factor = cdiv(A[i * ldA + p], piv);
            for (int c = p + 1; c <= dim; ++c) {
                const double2 q = cmul(factor, A[p * ldA + c]);
                A[i * ldA + c].x -= q.x;
                A[i * ldA + c].y -= q.y;
            }
            A[i * ldA + p] = make_double2(0.0, 0.0);
        }
        small_sync<WARP>();
        rank = p + 1;
    }
    small_sync<WARP>();
    for (int i = tid; i < dim; i += nthr) x[i] = make_double2(0.0, 0.0);
    small_sync<WARP>();
    for (int k = tid; k < rank; k += nthr) x[perm[k]] = cdiv(A[k * ldA + dim], A[k * ldA + k]);
    small_sync<WARP>();
    return rank;
}

// Rotation of one Jacobi pair from alpha = |a_p|^2, beta = |a_q|^2 and gamma = a_p^H a_q (g2 = |gamma|^2 > 0): the
// unitary [[c, st], [-conj(st), c]] (c real, st complex) that makes the new columns a_p' = c a_p - conj(st) a_q and
// a_q' = st a_p + c a_q orthogonal, the smaller of the two angles.  With delta = beta - alpha, h = (delta^2 +
// 4 |gamma|^2)^(1/2) and x = |delta| / h:  c^2 = (1 + x) / 2,  st = sign(delta) gamma / (h c).  (The textbook form
// first turns a_q by exp(-i arg gamma) and then rotates by a real angle; the result differs by a unit factor on the
// second column, which one-sided Jacobi does not care about.)  Two reciprocal square roots and no division or square
// root: the chain of long-latency operations is serial and is most of a Jacobi step.
__device__ __forceinline__ void jacobi_rotation(double alpha, double bet, double gr, double gi, double g2, double& c,
                                                double2& st) {
    const double delta = bet - alpha;
    const double rh = rsqrt(fma(delta, delta, 4.0 * g2));
    const double c2 = fma(0.5 * fabs(delta), rh, 0.5);
    const double rc = rsqrt(c2);
    c = c2 * rc;
    const double k = copysign(rh * rc, delta);
    st = make_double2(gr * k, gi * k);
}

// one column pair, rows i0, i0 + step, ..: (x, y) <- (c x - conj(st) y, st x + c y)
__device__ __forceinline__ void rotate_pair(double2* xp, double2* yp, int i0, int step, int rows, double c, double2 st) {
    for (int i = i0; i < rows; i += step) {
        const double2 x = xp[i], y = yp[i];
        xp[i] = make_double2(c * x.x - (st.x * y.x + st.y * y.y), c * x.y - (st.x * y.y - st.y * y.x));
        yp[i] = make_double2(st.x * x.x - st.y * x.y + c * y.x, st.x * x.y + st.y * x.x + c * y.y);
    }
}

// ------------------------------------------------------------------ small SVD solve
// Pseudo-inverse solution of the s x s complex system A beta = rhs by one-sided (Hestenes)
// Jacobi: columns of [A; V] are rotated in pairs until the columns of A are orthogonal; then
// A = U Sigma, sigma_k = |a_k|, and beta = sum_{sigma_k > tol} v_k (a_k^H rhs) / sigma_k^2.
// Singular values come out to high relative accuracy, so the rank decision (sigma_k > tol)
// matches a LAPACK SVD except on a knife edge.  A, V: column-major with column stride ld
// (ld = s rounded up to even; a zero pad column never rotates).  One thread per column pair,
// pairs of a step disjoint (round-robin schedule).  Returns the rank.
__device__ int block_jacobi_pinv(double2* A, double2* V, const double2* rhs, int s, double tol, double2* beta,
                                 double2* coef, int* sh) {
    const int tid = threadIdx.x;
    const int nthr = blockDim.x;
    const int sp = s + (s & 1);
    for (int idx = tid; idx < sp * sp; idx += nthr) {
        const int c = idx / sp, i = idx % sp;
        V[idx] = make_double2(c == i ? 1.0 : 0.0, 0.0);
    }
    __syncthreads();
    int sweeps = 0;
    bool converged = false;
    for (int sweep = 0; sweep < kJacobiSweepLimit; ++sweep) {
        if (tid == 0) sh[0] = 0;
        __syncthreads();
        for (int step = 0; step < sp - 1; ++step) {
            if (tid < sp / 2) {
                int a, b;
                if (tid == 0) { a = sp - 1; b = step; }
                else {                                    // (step +- tid) mod (sp - 1); both step and tid are below sp - 1
                    a = step + tid;
                    if (a >= sp - 1) a -= sp - 1;
                    b = step - tid;
                    if (b < 0) b += sp - 1;
                }
                const int p = a < b ? a : b, q = a < b ? b : a;
                double2* ap = A + p * sp;
                double2* aq = A + q * sp;
                double alpha = 0.0, bet = 0.0, gr = 0.0, gi = 0.0;
                for (int i = 0; i < s; ++i) {
                    const double2 x = ap[i], y = aq[i];
                    alpha += x.x * x.x + x.y * x.y;
                    bet += y.x * y.x + y.y * y.y;
                    gr += x.x * y.x + x.y * y.y;          // conj(x) * y
                    gi += x.x * y.y - x.y * y.x;
                }
                const double g2 = gr * gr + gi * gi;
                if (g2 > 1e-30 * alpha * bet && g2 > 0.0) {
                    double c;
                    double2 st;
                    jacobi_rotation(alpha, bet, gr, gi, g2, c, st);
                    rotate_pair(ap, aq, 0, 1, s, c, st);
                    rotate_pair(V + p * sp, V + q * sp, 0, 1, sp, c, st);
                    sh[0] = 1;
                }
            }
            __syncthreads();
        }
        const int rotated = sh[0];
        __syncthreads();
        ++sweeps;
        if (!rotated) { converged = true; break; }
    }
    if (tid == 0) { sh[1] = 0; sh[3] = converged ? sweeps : -sweeps; }
    __syncthreads();
    if (tid < sp) {
        const double2* ak = A + tid * sp;
        double sig2 = 0.0, pr = 0.0, pi = 0.0;
        for (int i = 0; i < s; ++i) {
            const double2 x = ak[i], r = rhs[i];
            sig2 += x.x * x.x + x.y * x.y;
            pr += x.x * r.x + x.y * r.y;                  // conj(x) * r
            pi += x.x * r.y - x.y * r.x;
        }
        const bool keep = sqrt(sig2) > tol;
        coef[tid] = keep ? make_double2(pr / sig2, pi / sig2) : make_double2(0.0, 0.0);
        if (keep) atomicAdd(&sh[1], 1);
    }
    __syncthreads();
    if (tid < s) {
        double re = 0.0, im = 0.0;
        for (int k = 0; k < sp; ++k) {
            const double2 q = cmul(V[k * sp + tid], coef[k]);
            re += q.x;
            im += q.y;
        }
        beta[tid] = make_double2(re, im);
    }
    __syncthreads();
    return sh[1];
}


// The same solve by one warp for s <= 16 (A, V in shared memory): the pairs of a step sit side by side in the
// warp, LP lanes per pair (a power of two), each lane holding the rows sub, sub + LP, .. of its pair's columns;
// the three inner products of a pair are reduced with shuffles inside its LP lanes, every lane of the pair then
// forms the same rotation and applies it to its own rows.  Only warp barriers.  Called by all 32 lanes of warp 0.
__device__ int warp_jacobi_pinv(double2* A, double2* V, const double2* rhs, int s, double tol, double2* beta,
                                double2* coef, int* sh) {
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int sp = s + (s & 1), npairs = sp / 2;
    int lp = 1;
    while (lp * 2 * npairs <= 32) lp *= 2;
    const int pair = lane / lp, sub = lane % lp;
    const bool act = pair < npairs;
    for (int idx = lane; idx < sp * sp; idx += 32) {
        const int c = idx / sp, i = idx % sp;
        V[idx] = make_double2(c == i ? 1.0 : 0.0, 0.0);
    }
    __syncwarp();
    int sweeps = 0;
    bool converged = false;
    for (int sweep = 0; sweep < kJacobiSweepLimit; ++sweep) {
        bool rotated = false;
        for (int step = 0; step < sp - 1; ++step) {
            int p = 0, q = 1;
            if (act) {
                int a, b;
                if (pair == 0) { a = sp - 1; b = step; }
                else {                                    // (step +- pair) mod (sp - 1); both are below sp - 1
                    a = step + pair;
                    if (a >= sp - 1) a -= sp - 1;
                    b = step - pair;
                    if (b < 0) b += sp - 1;
                }
                p = a < b ? a : b;
                q = a < b ? b : a;
            }
            double2* ap = A + p * sp;
            double2* aq = A + q * sp;
            double alpha = 0.0, bet = 0.0, gr = 0.0, gi = 0.0;
            if (act)
                for (int i = sub; i < s; i += lp) {
                    const double2 x = ap[i], y = aq[i];
                    alpha += x.x * x.x + x.y * x.y;
                    bet += y.x * y.x + y.y * y.y;
                    gr += x.x * y.x + x.y * y.y;          // conj(x) * y
                    gi += x.x * y.y - x.y * y.x;
                }
            for (int off = lp >> 1; off > 0; off >>= 1) {
                alpha += __shfl_xor_sync(full, alpha, off);
                bet += __shfl_xor_sync(full, bet, off);
                gr += __shfl_xor_sync(full, gr, off);
                gi += __shfl_xor_sync(full, gi, off);
            }
            const double g2 = gr * gr + gi * gi;
            if (act && g2 > 1e-30 * alpha * bet && g2 > 0.0) {
                double c;
                double2 st;
                jacobi_rotation(alpha, bet, gr, gi, g2, c, st);
                rotate_pair(ap, aq, sub, lp, s, c, st);
                rotate_pair(V + p * sp, V + q * sp, sub, lp, sp, c, st);
                rotated = true;
            }
            __syncwarp();
        }
        ++sweeps;
        if (!__any_sync(full, rotated)) { converged = true; break; }
    }
    bool keep = false;
    if (lane < sp) {
        const double2* ak = A + lane * sp;
        double sig2 = 0.0, pr = 0.0, pi = 0.0;
        for (int i = 0; i < s; ++i) {
            const double2 x = ak[i], r = rhs[i];
            sig2 += x.x * x.x + x.y * x.y;
            pr += x.x * r.x + x.y * r.y;                  // conj(x) * r
            pi += x.x * r.y - x.y * r.x;
        }
        keep = sqrt(sig2) > tol;
        coef[lane] = keep ? make_double2(pr / sig2, pi / sig2) : make_double2(0.0, 0.0);
    }
    const int rank = __popc(__ballot_sync(full, keep));
    __syncwarp();
    if (lane < s) {
        double re = 0.0, im = 0.0;
        for (int k = 0; k < sp; ++k) {
            const double2 q = cmul(V[k * sp + lane], coef[k]);
            re += q.x;
            im += q.y;
        }
        beta[lane] = make_double2(re, im);
    }
    if (lane == 0) { sh[1] = rank; sh[3] = converged ? sweeps : -sweeps; }
    __syncwarp();
    return rank;
}

constexpr int kSmallDim = 16;         // systems up to this size are solved in shared memory by one warp
constexpr int kFusedReduceMax = 64;   // up to this many block partials are added up by the locator kernel itself

// ------------------------------------------------------------------ decode vector
// With B = [C_L]_{.,V} and A = [C_L]_{.,U}: A A^H = I - B B^H, so the minimum-norm solution of
// A b_U = e_last is b_U = A^H y, y = e_last + B (I - B^H B)^{-1} B^H e_last, and
// I - B^H B = [C_R]_{.,V}^H [C_R]_{.,V} is only |V| x |V| (|V| <= 2 s).
// Called by every thread of a block of kSolveThreads threads; flags may point to global or to shared memory.
__device__ void decode_vector_body(CycDevice* cd, const uint8_t* flags, int n, int s, DeviceInfo* info) {
    __shared__ int vlist[kMaxN], rowbestc[kMaxN], perm_s[kMaxN], sh[4], a_s;
    __shared__ uint8_t fl[kMaxN];
    __shared__ double rowbest[kMaxN];
    __shared__ double2 y[kMaxN], tw[kMaxN], x_s[kMaxN], b_s[kMaxN];
    __shared__ double2 As[kSmallDim * (kSmallDim + 1)];
    const int tid = threadIdx.x;
    const int rows = n - 2 * s, L = rows - 1;
    const double rsn = 1.0 / sqrt((double)n);
    if (tid < n) {
        tw[tid] = cd->twiddle[tid];
        fl[tid] = flags[tid];
    }
    __syncthreads();
    if (tid == 0) {
        int a = 0;
        for (int j = 0; j < n; ++j)
            if (fl[j]) vlist[a++] = j;
        a_s = a;
    }
    __syncthreads();
    const int a = a_s;
    if (a > 2 * s) {                                       // fewer than n - 2 s rows left: no b exists
        if (tid < n) cd->b[tid] = make_double2(0.0, 0.0);
        if (tid == 0) {
            info->n_active = 0; info->n_flagged = a; info->status = DRACO_ETOOMANY;
            info->im_residual_bits = 0ull; info->re_max_bits = 0ull;
        }
        return;
    }
    double2* x = x_s;
    if (a > 0) {
        const bool small = a <= kSmallDim;
        double2* A = small ? As : cd->work;
        for (int idx = tid; idx < a * (a + 1); idx += blockDim.x) {
            const int p = idx / (a + 1), q = idx % (a + 1);
            double2 val;
            if (q < a) {                                   // (1/n) sum_{m >= n-2s} w^(m (v_q - v_p))
                int dv = vlist[q] - vlist[p];
                if (dv < 0) dv += n;
                double re = 0.0, im = 0.0;
                int k = ((n - 2 * s) * dv) % n;
                for (int m = n - 2 * s; m < n; ++m) {
                    const double2 w = tw[k];
                    re += w.x;
                    im += w.y;
                    k += dv;
                    if (k >= n) k -= n;
                }
                val = make_double2(re / n, im / n);
            } else {                                       // conj(C[L][v_p])
                const double2 w = tw[(L * vlist[p]) % n];
                val = make_double2(w.x * rsn, -w.y * rsn);
            }
            A[idx] = val;
        }
        __syncthreads();
        if (small) {
            if (tid < 32) block_gauss_jordan<true>(A, a, 0.0, x, perm_s, rowbest, rowbestc, sh);
            __syncthreads();
        } else {
            block_gauss_jordan<false>(A, a, 0.0, x, perm_s, rowbest, rowbestc, sh);
        }
    }
    if (tid < rows) {
        double re = (tid == L) ? 1.0 : 0.0, im = 0.0;
        for (int p = 0; p < a; ++p) {
            const double2 w = tw[(tid * vlist[p]) % n];
            const double2 q = cmul(w, x[p]);
            re += q.x * rsn;
            im += q.y * rsn;
        }
        y[tid] = make_double2(re, im);
    }
    __syncthreads();
    if (tid < n) {
        double2 b = make_double2(0.0, 0.0);
        if (!fl[tid]) {
            double re = 0.0, im = 0.0;
            int k = 0;                                     // (m tid) mod n
            for (int m = 0; m < rows; ++m) {
                const double2 q = cmulc(y[m], tw[k]);
                re += q.x;
                im += q.y;
                k += tid;
                if (k >= n) k -= n;
            }
            b = make_double2(re * rsn, im * rsn);
        }
        cd->b[tid] = b;
        b_s[tid] = b;
    }
    __syncthreads();
    // the active rows in ascending order: position = number of unflagged nodes before this one
    if (tid < n && !fl[tid]) {
        int k = 0;
        for (int j = 0; j < tid; ++j) k += fl[j] ? 0 : 1;
        cd->active[k] = tid;
        cd->b_active[k] = b_s[tid];
    }
    if (tid == 0) {
        info->n_active = n - a;
        info->n_flagged = a;
        info->im_residual_bits = 0ull;                     // the recovery kernel's blocks merge their maxima into these
        info->re_max_bits = 0ull;
        if (info->status == DRACO_ETOOMANY) info->status = DRACO_OK;
    }
}


__global__ void __launch_bounds__(kSolveThreads)
cyc_decode_vector_kernel(CycDevice* cd, const uint8_t* __restrict__ flags, int n, int s, DeviceInfo* info) {
    decode_vector_body(cd, flags, n, s, info);
}

// ------------------------------------------------------------------ locator after the projection
__global__ void __launch_bounds__(kSolveThreads)
cyc_solve_kernel(CycDevice* cd, const double2* __restrict__ e_in, const double2* __restrict__ partial, int used, int cap,
                 int n, int s, double theta, uint8_t* flags, uint8_t* flags2, DeviceInfo* info, int with_b) {
    __shared__ double2 e[kMaxN], h[kMaxN], tw[kMaxN];
    __shared__ double2 As[kSmallDim * kSmallDim], Vs[kSmallDim * kSmallDim];
    __shared__ double2 rhs_s[kMaxN / 2], beta_s[kMaxN / 2], coef_s[kMaxN / 2];
    __shared__ double mag[kMaxN], sorted[kMaxN], qv[kMaxN];
    __shared__ int sh[4], count;
    __shared__ double scale_s, maxsyn_s;
    const int tid = threadIdx.x;
    const double rsn = 1.0 / sqrt((double)n);

    if (tid < n) tw[tid] = cd->twiddle[tid];
    if (e_in != nullptr) {                                 // the projection record: n (re, im) pairs, then n values q_j
        if (tid < n) {
            e[tid] = e_in[tid];
            qv[tid] = reinterpret_cast<const double*>(e_in + n)[tid];
        }
    } else {
        // the projection's block partials, few enough to add up here: thread (j, part) takes one of the three sums of
        // node j over the blocks in ascending order, four running sums in rotation (all loads of a round are in flight
        // together), combined in a fixed order: reproducible
        const double* __restrict__ qpartial = reinterpret_cast<const double*>(partial + (int64_t)cap * n);
        for (int idx = tid; idx < 3 * n; idx += blockDim.x) {
            const int part = idx / n, j = idx - part * n;
            double acc[4] = {0.0, 0.0, 0.0, 0.0};
            for (int b0 = 0; b0 < used; b0 += 4) {
                double v[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int b = (b0 + k < used) ? b0 + k : 0;
                    const int64_t at = (int64_t)b * n + j;
                    v[k] = part == 2 ? __ldcg(qpartial + at) : (part == 0 ? __ldcg(&partial[at].x) : __ldcg(&partial[at].y));
                }
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (b0 + k < used) acc[k] += v[k];
            }
            const double sum = (acc[0] + acc[1]) + (acc[2] + acc[3]);
            if (part == 0) e[j].x = sum;
            else if (part == 1) e[j].y = sum;
            else qv[j] = sum;
        }
    }
    __syncthreads();
    // A node whose record is not finite sent NaN or infinities: no honest vector does.  It is flagged outright and
    // its record taken as zero, which keeps the arithmetic below finite (the node then looks to the locator as if it
    // had sent a vector with f R_j = 0: one of the at most s errors it locates anyway).
    __shared__ uint8_t nonfinite[kMaxN];
    if (tid < n) {
        const bool bad = !(isfinite(e[tid].x) && isfinite(e[tid].y) && isfinite(qv[tid]));
        nonfinite[tid] = bad ? 1 : 0;
        if (bad) {
            e[tid] = make_double2(0.0, 0.0);
            qv[tid] = 0.0;
        }
        cd->e[tid] = e[tid];
        mag[tid] = sqrt(qv[tid]);
        h[tid] = make_double2(0.0, 0.0);
    }
    if (tid == 0) { count = 0; sh[3] = 0; }
    __syncthreads();
    // scale = median of q_j^(1/2) by rank counting
    if (tid < n) {
        int rank = 0;
        for (int k = 0; k < n; ++k) rank += (mag[k] < mag[tid]) || (mag[k] == mag[tid] && k < tid);
        sorted[rank] = mag[tid];
    }
    __syncthreads();
    if (tid == 0) scale_s = (n & 1) ? sorted[n / 2] : 0.5 * (sorted[n / 2 - 1] + sorted[n / 2]);
    // syndromes h_m = n^(-1/2) sum_j e_j w^(-m j), m = n-2s .. n-1
    if (tid < 2 * s) {
        const int m = n - 2 * s + tid;
        double a = 0.0, b = 0.0;
        int idx = 0;                                       // (m j) mod n
        for (int j = 0; j < n; ++j) {
            const double2 q = cmulc(e[j], tw[idx]);
            a += q.x;
            b += q.y;
            idx += m;
            if (idx >= n) idx -= n;
        }
        h[m] = make_double2(a * rsn, b * rsn);
    }
    __syncthreads();
    if (tid == 0) {
        double mx = 0.0;
        for (int m = n - 2 * s; m < n; ++m) mx = fmax(mx, sqrt(cabs2(h[m])));
        maxsyn_s = mx;
    }
    __syncthreads();
    const double tol = theta * scale_s;
    // The locator runs in passes.  The first is the paper's phi.  Each further pass treats the set E of nodes flagged
    // so far (nodes with a non-finite record from the start) as erasures: with lambda(x) = prod_{v in E} (x - w^v) =
    // sum_k lambda_k x^k the sequence T_m = sum_k lambda_k h_{m-k} no longer contains the nodes of E and is again a sum
    // of exponentials, one per adversary not yet flagged, so its last 2 s2 values, s2 = floor((2 s - |E|) / 2), go
    // through the same Toeplitz system, recurrence and IDFT with s2 in place of s.  A pass that finds nothing (the
    // usual second pass: rounding noise) ends the search.  Adversaries that sit side by side make one pass miss some of
    // them with complex64 vectors; the passes then still end with a set that contains them all.
    __shared__ double2 syn[kMaxN];                         // h_{n-2s+i}: every pass rewrites h
    __shared__ double2 lam[kMaxN + 2];
    __shared__ uint8_t fl_s[kMaxN];                        // V so far
    __shared__ int elist[kMaxN];
    __shared__ int eps_s, rank_total_s, sweeps_s;
    __shared__ double lam1_s, margin_s;
    if (tid < 2 * s) syn[tid] = h[n - 2 * s + tid];
    if (tid < n) {
        fl_s[tid] = nonfinite[tid];
        cd->t[tid] = make_double2(0.0, 0.0);
        cd->h[tid] = h[tid];
    }
    if (tid == 0) { rank_total_s = 0; sweeps_s = 0; margin_s = 1e300; }
    __syncthreads();
    double2* beta = beta_s;
    bool first = true;
    for (int pass = 0; pass <= 2 * s && s > 0; ++pass) {
        if (tid == 0) {
            int a = 0;
            for (int j = 0; j < n; ++j)
                if (fl_s[j]) elist[a++] = j;
            eps_s = a;
        }
        __syncthreads();
        const int eps = eps_s;
        const int s2 = (2 * s - eps) / 2;
        if (s2 < 1) break;
        // lambda: one factor (x - w^v) at a time, new_k = old_{k-1} - w^v old_k
        if (tid <= eps) lam[tid] = make_double2(tid == 0 ? 1.0 : 0.0, 0.0);
        __syncthreads();
        for (int a = 0; a < eps; ++a) {
            double2 nv = make_double2(0.0, 0.0);
            if (tid <= a + 1) {
                const double2 wv = tw[elist[a]];
                const double2 prev = tid > 0 ? lam[tid - 1] : make_double2(0.0, 0.0);
                const double2 cur = tid <= a ? lam[tid] : make_double2(0.0, 0.0);
                const double2 q = cmul(wv, cur);
                nv = make_double2(prev.x - q.x, prev.y - q.y);
            }
            __syncthreads();
            if (tid <= a + 1) lam[tid] = nv;
            __syncthreads();
        }
        if (tid < 32) {
            double acc = 0.0;
            for (int k = tid; k <= eps; k += 32) acc += sqrt(cabs2(lam[k]));
            acc = warp_sum(acc);
            if (tid == 0) lam1_s = acc;
        }
        if (tid < n) {                                     // T_m on its window m = n - 2 s2 .. n - 1, zero before it
            double a = 0.0, b = 0.0;
            if (tid >= n - 2 * s2)
                for (int k = 0; k <= eps; ++k) {
                    const double2 q = cmul(lam[k], syn[tid - k - (n - 2 * s)]);
                    a += q.x;
                    b += q.y;
                }
            h[tid] = make_double2(a, b);
        }
        __syncthreads();
        const double cut = tol * lam1_s;                   // the rounding noise of h enters T through |lambda_k|
        int rank = 0;
        {
            // row i: [h_{n-s2-1-i} .. h_{n-2-i}] beta = h_{n-1-i}; stored by columns
            const int sp = s2 + (s2 & 1);
            const bool small = sp <= kSmallDim;
            double2* A = small ? As : cd->work;
            double2* V = small ? Vs : cd->work + sp * sp;
            for (int idx = tid; idx < sp * sp; idx += blockDim.x) {
                const int c = idx / sp, i = idx % sp;
                A[idx] = (c < s2 && i < s2) ? h[n - s2 - 1 - i + c] : make_double2(0.0, 0.0);
            }
            if (tid < s2) rhs_s[tid] = h[n - 1 - tid];
            __syncthreads();
            // No singular value exceeds the Frobenius norm: when that is within the cutoff (the usual step without any
            // adversary, and the usual last pass: rounding noise) the rank is 0 and the SVD is skipped.
            if (tid < 32) {
                double fro2 = 0.0;
                for (int idx = tid; idx < sp * sp; idx += 32) fro2 += cabs2(A[idx]);
                fro2 = warp_sum(fro2);
                if (tid == 0) sh[2] = (fro2 > cut * cut) ? 1 : 0;
            }
            __syncthreads();
            if (sh[2]) {
                if (small) {
                    if (tid < 32) warp_jacobi_pinv(A, V, rhs_s, s2, cut, beta_s, coef_s, sh);
                    __syncthreads();
                    rank = sh[1];
                } else {
                    rank = block_jacobi_pinv(A, V, rhs_s, s2, cut, beta_s, coef_s, sh);
                }
                if (tid == 0) {                            // sweeps of the longest iteration; negative once one hit the limit
                    if (sh[3] < 0) sweeps_s = sh[3];
                    else if (sweeps_s >= 0 && sh[3] > sweeps_s) sweeps_s = sh[3];
                }
            }
        }
        if (rank == 0) break;
        if (tid == 0) {
            for (int l = 0; l < n - 2 * s2; ++l) {
                double a = 0.0, b = 0.0;
                for (int u = 0; u < s2; ++u) {
                    int idx = l + u - s2;
                    if (idx < 0) idx += n;
                    const double2 q = cmul(beta[u], h[idx]);
                    a += q.x;
                    b += q.y;
                }
                h[l] = make_double2(a, b);
            }
        }
        __syncthreads();
        if (tid < n) {
            double a = 0.0, b = 0.0;
            int idx = 0;                                   // (tid m) mod n
            for (int m = 0; m < n; ++m) {
                const double2 q = cmul(h[m], tw[idx]);
                a += q.x;
                b += q.y;
                idx += tid;
                if (idx >= n) idx -= n;
            }
            const double2 t = make_double2(a * rsn, b * rsn);
            if (first) {
                cd->t[tid] = t;
                cd->h[tid] = h[tid];
            }
            mag[tid] = fl_s[tid] ? -1.0 : cabs2(t);        // nodes already in V are not candidates
        }
        __syncthreads();
        // exactly `rank` entries of t are non-zero in exact arithmetic: the rank largest |t_j| join V
        bool found = false;
        if (tid < n) {
            int pos = 0;
            for (int k = 0; k < n; ++k) pos += (mag[k] > mag[tid]) || (mag[k] == mag[tid] && k < tid);
            found = pos < rank;
            if (first && pos == rank - 1) sorted[0] = mag[tid];     // |t|^2 of the weakest flagged node ..
            if (first && pos == rank) sorted[1] = mag[tid];         // .. and of the strongest unflagged one
        }
        __syncthreads();
        if (found) fl_s[tid] = 1;
        if (tid == 0) {
            rank_total_s += rank;
            if (first && rank < n - eps) margin_s = sqrt(sorted[0] / fmax(sorted[1], 1e-300));
        }
        first = false;
        __syncthreads();
    }
    __syncthreads();
    bool flagged = false;
    if (tid < n) {
        flagged = fl_s[tid] != 0;
        if (flags) flags[tid] = flagged ? 1 : 0;
        if (flags2) flags2[tid] = flagged ? 1 : 0;
        if (flagged) atomicAdd(&count, 1);
    }
    __syncthreads();
    if (tid == 0) {
        info->n_flagged = count;
        info->locator_rank = rank_total_s;
        info->scale = scale_s;
        info->max_syndrome = maxsyn_s;
        const double margin = margin_s;
        // exactly `rank` entries of t are non-zero in exact arithmetic: where the weakest flagged and the strongest
        // unflagged |t_j| of the first pass are less than a decade apart the choice of V is not to be trusted, nor is a
        // rank that comes from an iteration that was stopped at its sweep limit
        info->status = (margin >= kMarginBar && sweeps_s >= 0) ? DRACO_OK : DRACO_EUNSURE;
        info->no_majority = 0;
        info->locator_margin = margin;
        info->svd_sweeps = sweeps_s;
        info->im_residual_bits = 0ull;                     // a decode's self-check belongs to the locate before it
        info->re_max_bits = 0ull;
    }
    if (with_b) {                                          // the decode vector for the V just found, same launch
        __syncthreads();
        decode_vector_body(cd, fl_s, n, s, info);
    }
}

}  // namespace

// Blocks of the projection: four per SM (six measured slower at n = 15).
int project_grid_size(int sm_count, int) { return sm_count * 4; }
int project_grid_size(int sm_count) { return sm_count * 4; }

// All launches of one projection: n <= 16 the few-rows kernel, n <= 64 one launch of the tile kernel, otherwise two
// launches of it over half the rows each.  partial: [cap][n] double2 followed by [cap][n] double.  No more blocks
// are launched than have work (a tile each, or eight 256-coordinate chunks each in the few-rows kernel): short
// vectors then leave a handful of partials instead of several hundred zeros.  Returns the grid used in *grid_used.
static cudaError_t launch_project_kernels(int cap, cudaStream_t st, const float2* R, const float* f, int64_t len,
                                          int64_t ld, int n, double2* partial, int accumulate, int* grid_used) {
    const bool vec2 = (ld % 2 == 0);
    const int64_t work = n <= 16 ? (len + 256 * kProjectWarps - 1) / (256 * kProjectWarps)
                                 : (len + kProjectTile - 1) / kProjectTile;
    int grid = cap;
    if (work < grid) grid = (int)(work < 1 ? 1 : work);
    *grid_used = grid;
    if (n <= 16) {
        if (vec2) cyc_project_fewrows_kernel<true><<<grid, kThreads, 0, st>>>(R, f, len, ld, n, partial, cap, accumulate);
        else cyc_project_fewrows_kernel<false><<<grid, kThreads, 0, st>>>(R, f, len, ld, n, partial, cap, accumulate);
        return cudaGetLastError();
    }
    const int parts = n <= 64 ? 1 : 2;
    const int per = (n + parts - 1) / parts;
    // fewer tiles than an eighth of the blocks the device takes: spread the rows over gridDim.y too (latency of short vectors)
    int ysplit = 1;
    if (grid * 8 <= cap) {
        ysplit = (per + kProjectWarps - 1) / kProjectWarps;
        const int room = cap / (2 * grid);
        if (ysplit > room) ysplit = room;
        if (ysplit < 1) ysplit = 1;
    }
    const dim3 grid2(grid, ysplit);
    for (int row0 = 0; row0 < n; row0 += per) {
        const int nrows = (n - row0) < per ? (n - row0) : per;
        if (nrows <= 32) {
            if (vec2) cyc_project_kernel<4, true><<<grid2, kThreads, 0, st>>>(R, f, len, ld, n, row0, nrows, partial, cap, accumulate);
            else cyc_project_kernel<4, false><<<grid2, kThreads, 0, st>>>(R, f, len, ld, n, row0, nrows, partial, cap, accumulate);
        } else {
            if (vec2) cyc_project_kernel<8, true><<<grid2, kThreads, 0, st>>>(R, f, len, ld, n, row0, nrows, partial, cap, accumulate);
            else cyc_project_kernel<8, false><<<grid2, kThreads, 0, st>>>(R, f, len, ld, n, row0, nrows, partial, cap, accumulate);
        }
        const cudaError_t err = cudaGetLastError();
        if (err != cudaSuccess) return err;
    }
    return cudaSuccess;
}

// accumulate: add to the partials of the plan's earlier launches (column chunks of one vector).  A chunk that needs
// more blocks than any before it finds the extra slots cleared first.
int launch_cyc_project(draco_plan* p, const float2* R, const float* f, int64_t len, int64_t ld, bool accumulate,
                       cudaStream_t st) {
    const int cap = p->project_grid;
    const int64_t work = p->n <= 16 ? (len + 256 * kProjectWarps - 1) / (256 * kProjectWarps)
                                    : (len + kProjectTile - 1) / kProjectTile;
    const int want = (int)(work < cap ? (work < 1 ? 1 : work) : cap);
    if (!accumulate) p->project_used = 0;
    if (accumulate && want > p->project_used) {
        const size_t n = (size_t)p->n;
        DRACO_CUDA(cudaMemsetAsync(p->partial_dev + (size_t)p->project_used * n, 0,
                                   sizeof(double2) * n * (size_t)(want - p->project_used), st));
        double* q = reinterpret_cast<double*>(p->partial_dev + (size_t)cap * n);
        DRACO_CUDA(cudaMemsetAsync(q + (size_t)p->project_used * n, 0, sizeof(double) * n * (size_t)(want - p->project_used), st));
    }
    int used = 0;
    DRACO_CUDA(launch_project_kernels(cap, st, R, f, len, ld, p->n, p->partial_dev, accumulate ? 1 : 0, &used));
    if (used > p->project_used) p->project_used = used;
    return DRACO_OK;
}

int launch_cyc_project_finish(draco_plan* p, double2* e_out, cudaStream_t st) {
    cyc_reduce_partials_kernel<<<p->n, kReduceThreads, 0, st>>>(p->partial_dev, p->project_used, p->project_grid, p->n,
                                                                reinterpret_cast<double*>(e_out));
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

// e == nullptr: the record of the plan's own projection (launch_cyc_project) is formed first: by the locator kernel
// itself when the projection left few block partials (short vectors, where every launch counts), by the reduction
// kernel otherwise.  with_b: the decode vector for the set V just found is formed in the same launch.
int launch_cyc_solve(draco_plan* p, const double2* e, uint8_t* flags, bool with_b, cudaStream_t st) {
    const double2* partial = nullptr;
    int used = 0;
    if (!e) {
        if (p->project_used <= kFusedReduceMax) {
            partial = p->partial_dev;
            used = p->project_used;
        } else {
            double2* own = reinterpret_cast<double2*>(p->cyc_dev->record);  // address arithmetic only: cyc_dev is a device pointer
            const int rc = launch_cyc_project_finish(p, own, st);
            if (rc != DRACO_OK) return rc;
            e = own;
        }
    }
    cyc_solve_kernel<<<1, kSolveThreads, 0, st>>>(p->cyc_dev, e, partial, used, p->project_grid, p->n, p->s, p->theta, flags,
                                                  p->flags_dev, p->info_dev, with_b ? 1 : 0);
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

int launch_cyc_decode_vector(draco_plan* p, const uint8_t* flags, cudaStream_t st) {
    cyc_decode_vector_kernel<<<1, kSolveThreads, 0, st>>>(p->cyc_dev, flags, p->n, p->s, p->info_dev);
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

}  // namespace draco

// ------------------------------------------------------------------ projection without any allocation
// Some callers must not allocate device memory at all: a parameter server embedded in a host
// process whose memory pool owner has handed out the whole device up front (a later cudaMalloc
// fails or fragments the pool), or a step loop that cannot afford the implicit device-wide
// synchronisation an allocation or a free may cause.  For them the block partials of the
// projection live in this fixed array instead of in a plan.  Every GPU that loads the library
// carries its 888 KB until the process exits.
namespace draco {
namespace {
constexpr int kStaticGridMax = 296;                                   // blocks whose partials fit
// per block and node one double2 (partial of e_j) and, after all of those, one double (partial of q_j)
static __device__ __align__(256) double2 g_static_partial[kStaticGridMax * kMaxN * 3 / 2];
constexpr int kMaxDevices = 64;
double2* g_static_partial_ptr[kMaxDevices] = {};                      // device address per device, set once
int g_static_sm_count[kMaxDevices] = {};
std::mutex g_static_mutex;
}  // namespace
}  // namespace draco

extern "C" int draco_cyc_project_noalloc(int n, int64_t d, const void* R, const float* f, double* e, void* stream) {
    using namespace draco;
    if (n < 1 || d < 1 || !R || !f || !e) return DRACO_EINVAL;
    if (n > kMaxN) return DRACO_ELIMIT;                               // the static array holds at most kMaxN rows per block
    if ((reinterpret_cast<uintptr_t>(R) & 15u) || (reinterpret_cast<uintptr_t>(f) & 15u) ||
        (reinterpret_cast<uintptr_t>(e) & 15u))
        return DRACO_EINVAL;
    int dev = 0;
    DRACO_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return DRACO_ELIMIT;
    double2* partial = nullptr;
    int sms = 0;
    {
        // Set-up, once per device, with that device current.  In host code the array's name is only a
        // stand-in for the symbol; the kernel needs the device address, which the runtime looks up here.
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_partial_ptr[dev]) {
            double2* ptr = nullptr;
            DRACO_CUDA(cudaGetSymbolAddress((void**)&ptr, g_static_partial));
            int count = 0;
            DRACO_CUDA(cudaDeviceGetAttribute(&count, cudaDevAttrMultiProcessorCount, dev));
            g_static_sm_count[dev] = count;
            g_static_partial_ptr[dev] = ptr;
        }
        partial = g_static_partial_ptr[dev];
        sms = g_static_sm_count[dev];
    }
    int grid = project_grid_size(sms);
    if (grid > kStaticGridMax) grid = kStaticGridMax;
    if (grid < 1) grid = 1;
    cudaStream_t st = (cudaStream_t)stream;
    const float2* Rc = static_cast<const float2*>(R);
    // Every block that is launched writes its n partials and only those are read back, so nothing has
    // to be cleared between calls even though the array keeps the previous call's contents.
    int used = 0;
    DRACO_CUDA(launch_project_kernels(grid, st, Rc, f, d, d, n, partial, 0, &used));
    cyc_reduce_partials_kernel<<<n, kReduceThreads, 0, st>>>(partial, used, grid, n, e);
    DRACO_CUDA(cudaGetLastError());
    return DRACO_OK;
}

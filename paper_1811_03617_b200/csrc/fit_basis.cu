// Basis refresh (Section 2, PCA paragraph): per layer, sample mean and 1/n covariance of the
// n = L * S_l stored slices, then the symmetric eigendecomposition of the d x d covariance
// and the selection of the k leading eigenvectors.
//
// Covariance, shapes with a tensor-core kernel (d = 64, 128, 192, 256): the history is read once --
//   shift_kernel      -> a centre m near the mean (mean of <= 256 slices spread over the layer)
//   cov_tc_kernel     -> per-tile partial sums of (x - m)(x - m)^T and the sums of (x - m)   (cov_tc.cu, tcgen05)
//   cov_reduce_kernel -> C = S2 / n - delta delta^T in a fixed order in fp64, delta = sum (x - m) / n
//   mean_kernel       -> mean = m + delta, mu = (N / c) mean
// other shapes: colsum_kernel -> mean_kernel -> cov_partial_kernel (FP32 pipe, about the mean) -> cov_reduce_kernel.
// A fit spread over several participants stops after the partial sums (moments_kernel: n, sum (x - m), S2 in
// fp64, additive over participants) and resumes from their sum (cov_from_moments_kernel).
//
// Eigendecomposition, default (d <= 256, k <= 32): eigenvalues and the k leading eigenvectors only --
//   chol_kernel       -> L with L L^T = C + ridge I
//   hestenes_kernel   -> one-sided Jacobi on the columns of L, in shared memory on a thread-block cluster, without
//                        accumulated rotations: squared column norms - ridge = eigenvalues, accurate also where
//                        they are tiny; the k longest columns span the leading eigenspace
//   topk_start_kernel -> eigenvalues sorted, the k longest columns normalised
//   subspace_kernel x2, jacobi_kernel on the k x k problem, ritz_kernel -> the k leading eigenpairs polished on the
//                        untouched covariance (fp64 Rayleigh quotients); merge_evals_kernel joins the two lists
// With the rotations kept (every eigenvector; gvq_set_fit_path(1), and shapes the above does not serve):
//   hestenes_kernel on C with V accumulated (or jacobi_kernel, two-sided, in global memory for d > 256)
//   rayleigh_kernel   -> eigenvalues re-evaluated as w^T C w against the untouched covariance (fp64):
//                        thousands of fp32 rotations leave ~1e-5 relative drift on the diagonal, the
//                        eigenvectors are good to ~1e-6 and the quotient's error is quadratic in that
//   finalize_kernel   -> eigenvalues descending, sign convention, Ut rows
// The cheap refresh (gvq_refresh_basis) replaces the eigen-solve by subspace_kernel + the k x k solver + ritz_kernel.
#include <algorithm>
#include <cooperative_groups.h>
#include <mutex>

#include "gvq_internal.h"

namespace gvq {
namespace {

constexpr int NTC = 256;  // threads of the covariance kernels
constexpr int RC = 32;    // sample rows staged per step
constexpr int NTJ = 512;  // threads of the Jacobi kernel

__host__ __device__ inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

struct FitWs {
    double *colsum;   // [n_layers][d]
    float *mean;      // [n_layers][d]
    float *partial;   // [n_fit_tiles][d][d]
    float *C;         // [n_layers][d][d]   covariance, then (in place) the rotated matrix
    float *W;         // [n_layers][d][d]   eigenvectors as ROWS
    float *C0;        // [n_layers][d][d]   the covariance, kept for the Rayleigh quotients
    float *lam;       // [n_layers][d]      eigenvalue of row j of W
    int32_t *status;  // [1] != 0 when some layer hit the sweep limit
    int32_t *sweeps;  // [n_layers]
    size_t bytes;
};

FitWs carve(void *base, int d, int n_layers, int n_fit_tiles)
{
    FitWs w;
    size_t o = 0;
    char *b = (char *)base;
    w.colsum = (double *)(b + o); o = align256(o + sizeof(double) * (size_t)n_layers * d);
    w.mean = (float *)(b + o);    o = align256(o + sizeof(float) * (size_t)n_layers * d);
    w.partial = (float *)(b + o); o = align256(o + sizeof(float) * (size_t)n_fit_tiles * d * d);
    w.C = (float *)(b + o);       o = align256(o + sizeof(float) * (size_t)n_layers * d * d);
    w.W = (float *)(b + o);       o = align256(o + sizeof(float) * (size_t)n_layers * d * d);
    w.C0 = (float *)(b + o);      o = align256(o + sizeof(float) * (size_t)n_layers * d * d);
    w.lam = (float *)(b + o);     o = align256(o + sizeof(float) * (size_t)n_layers * d);
    w.status = (int32_t *)(b + o); o = align256(o + sizeof(int32_t));
    w.sweeps = (int32_t *)(b + o); o = align256(o + sizeof(int32_t) * (size_t)n_layers);
    w.bytes = o;
    return w;
}

// ---- column sums --------------------------------------------------------------------------------
// grid (n_fit_tiles, L).  Thread (rl, c4) sums rows rl, rl + RL, ... of 4 adjacent columns.
__global__ void __launch_bounds__(NTC) colsum_kernel(int d, const float *__restrict__ hist, int64_t hist_stride,
                                                      const int32_t *tile_layer, const int32_t *tile_row0,
                                                      const int64_t *layer_off, const int32_t *layer_S,
                                                      double *colsum)
{
    __shared__ float4 red[NTC];
    const int tile = blockIdx.x, h = blockIdx.y;
    const int layer = tile_layer[tile], row0 = tile_row0[tile];
    const int count = min(kFitRows, layer_S[layer] - row0);
    const int d4 = d / 4;
    const int RL = NTC / d4;  // d <= 512 -> RL >= 2
    const int c4 = threadIdx.x % d4, rl = threadIdx.x / d4;
    const float *src = hist + (size_t)h * hist_stride + layer_off[layer] + (int64_t)row0 * d;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (rl < RL)
        for (int r = rl; r < count; r += RL) {
            const float4 v = *reinterpret_cast<const float4 *>(src + (size_t)r * d + c4 * 4);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
    red[threadIdx.x] = acc;
    __syncthreads();
    if (threadIdx.x < d4) {
        double s0 = 0, s1 = 0, s2 = 0, s3 = 0;
        for (int r = 0; r < RL; ++r) {
            const float4 v = red[r * d4 + threadIdx.x];
            s0 += v.x; s1 += v.y; s2 += v.z; s3 += v.w;
        }
        double *dst = colsum + (size_t)layer * d + threadIdx.x * 4;
        atomicAdd(dst + 0, s0); atomicAdd(dst + 1, s1); atomicAdd(dst + 2, s2); atomicAdd(dst + 3, s3);
    }
}

// mean = shift + colsum / n ; mu = (N / c) * mean.  One thread per (layer, t).  shift (may be null, may alias mean):
// the point the column sums were taken about.
__global__ void mean_kernel(int d, int n_layers, int L, int N, int c, const int32_t *layer_S,
                            const double *colsum, const float *shift, float *mean, float *mu)
{
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n_layers * d) return;
    const int layer = idx / d;
    const double n = (double)L * (double)layer_S[layer];
    const double m = n > 0 ? (shift ? (double)shift[idx] : 0.0) + colsum[idx] / n : 0.0;
    mean[idx] = (float)m;
    mu[idx] = (float)(m * (double)N / (double)c);
}

// An approximate mean to centre by: the mean of <= 256 slices spread evenly over the layer, in the first and in the
// last stored gradient (a centre far from the mean would cost digits in S2 / n - delta delta^T).
// grid n_layers, d * G threads: thread (q, t) sums entry t of every G-th sampled slice (rows read coalesced, four
// loads in flight per thread), the G partial sums meet in shared memory.
__global__ void __launch_bounds__(1024) shift_kernel(int d, int L, const float *__restrict__ hist, int64_t hist_stride,
                                                     const int64_t *layer_off, const int32_t *layer_S, float *shift)
{
    __shared__ float part[1024];
    const int layer = blockIdx.x, t = threadIdx.x % d, q = threadIdx.x / d, G = blockDim.x / d;
    const int S = layer_S[layer];
    const int rows = min(S, 256), step = rows > 0 ? S / rows : 0;       // slices 0, step, 2 step, ...
    const int passes = L > 1 ? 2 : 1;
    float acc = 0.0f;
    for (int pass = 0; pass < passes; ++pass) {
        const float *src = hist + (size_t)(pass == 0 ? 0 : L - 1) * hist_stride + layer_off[layer] + t;
#pragma unroll 4
        for (int i = q; i < rows; i += G) acc += src[(size_t)i * step * d];
    }
    part[threadIdx.x] = acc;
    __syncthreads();
    if (q == 0) {
        for (int g = 1; g < G; ++g) acc += part[g * d + t];
        const int used = rows * passes;
        shift[(size_t)layer * d + t] = used > 0 ? acc / (float)used : 0.0f;
    }
}

// ---- covariance partials ------------------------------------------------------------------------
// grid (n_fit_tiles * n_pairs).  A CTA owns one tile (<= 512 slices, all L stored gradients) and
// one BS x BS block (bi <= bj) of X^T X; thread (ti, tj) owns a 4 x 4 patch of it.
__global__ void __launch_bounds__(NTC) cov_partial_kernel(int d, int BS, int L, const float *__restrict__ hist,
                                                          int64_t hist_stride, const int32_t *tile_layer,
                                                          const int32_t *tile_row0, const int64_t *layer_off,
                                                          const int32_t *layer_S, const float *__restrict__ mean,
                                                          float *__restrict__ partial)
{
    __shared__ __align__(16) float Xa[RC][64];
    __shared__ __align__(16) float Xb[RC][64];
    const int nb = d / BS, n_pairs = nb * (nb + 1) / 2;
    const int tile = blockIdx.x / n_pairs;
    int pi = blockIdx.x - tile * n_pairs;
    int bi = 0;
    while (pi >= nb - bi) { pi -= nb - bi; ++bi; }
    const int bj = bi + pi;
    const int layer = tile_layer[tile], row0 = tile_row0[tile];
    const int count = min(kFitRows, layer_S[layer] - row0);
    const int B4 = BS / 4;
    const int ti = threadIdx.x / B4, tj = threadIdx.x % B4;
    const bool worker = threadIdx.x < B4 * B4;
    const float *m = mean + (size_t)layer * d;

    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.0f;

    for (int h = 0; h < L; ++h) {
        const float *src = hist + (size_t)h * hist_stride + layer_off[layer] + (int64_t)row0 * d;
        for (int r0 = 0; r0 < count; r0 += RC) {
            __syncthreads();
            for (int u = threadIdx.x; u < RC * B4; u += NTC) {
                const int r = u / B4, c4 = u - r * B4;
                float4 va = make_float4(0.f, 0.f, 0.f, 0.f), vb = va;
                if (r0 + r < count) {
                    const float *row = src + (size_t)(r0 + r) * d;
                    va = *reinterpret_cast<const float4 *>(row + bi * BS + c4 * 4);
                    vb = *reinterpret_cast<const float4 *>(row + bj * BS + c4 * 4);
                    const float4 ma = *reinterpret_cast<const float4 *>(m + bi * BS + c4 * 4);
                    const float4 mb = *reinterpret_cast<const float4 *>(m + bj * BS + c4 * 4);
                    va.x -= ma.x; va.y -= ma.y; va.z -= ma.z; va.w -= ma.w;
                    vb.x -= mb.x; vb.y -= mb.y; vb.z -= mb.z; vb.w -= mb.w;
                }
                *reinterpret_cast<float4 *>(&Xa[r][c4 * 4]) = va;
                *reinterpret_cast<float4 *>(&Xb[r][c4 * 4]) = vb;
            }
            __syncthreads();
            if (worker) {
#pragma unroll 8
                for (int r = 0; r < RC; ++r) {
                    const float4 a4 = *reinterpret_cast<const float4 *>(&Xa[r][ti * 4]);
                    const float4 b4 = *reinterpret_cast<const float4 *>(&Xb[r][tj * 4]);
                    const float a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
                    for (int x = 0; x < 4; ++x)
#pragma unroll
                        for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(a[x], b[y], acc[x][y]);
                }
            }
        }
    }
    if (worker) {
        float *dst = partial + (size_t)tile * d * d;
#pragma unroll
        for (int x = 0; x < 4; ++x)
            *reinterpret_cast<float4 *>(dst + (size_t)(bi * BS + ti * 4 + x) * d + bj * BS + tj * 4) =
                make_float4(acc[x][0], acc[x][1], acc[x][2], acc[x][3]);
    }
}

// C_l[a][b] = C_l[b][a] = (1/n) * sum over the layer's tiles of partial[a][b], a <= b (the blocks
// below the diagonal blocks are never written), and W_l = identity.  grid (d, n_layers), d threads.
// shift_sum (may be null): the partial sums were taken about a point m near the mean and shift_sum holds
// sum (x - m); then C = S2 / n - delta delta^T with delta = shift_sum / n.
__global__ void cov_reduce_kernel(int d, int L, const int32_t *layer_first_tile, const int32_t *layer_S,
                                  const float *__restrict__ partial, const double *shift_sum, float *C, float *C0, float *W)
{
    const int layer = blockIdx.y, a = blockIdx.x, b = threadIdx.x;
    W[((size_t)layer * d + a) * d + b] = (a == b) ? 1.0f : 0.0f;
    if (a > b) return;
    const double n = (double)L * (double)layer_S[layer];
    double s = 0.0;
    for (int t = layer_first_tile[layer]; t < layer_first_tile[layer + 1]; ++t)
        s += (double)partial[((size_t)t * d + a) * d + b];
    if (shift_sum && a / 128 == b / 128) {
        // the tensor-core kernel leaves X = hh + 2 hl in a diagonal block (hl^T stands for lh): (X + X^T) / 2
        double st = 0.0;
        for (int t = layer_first_tile[layer]; t < layer_first_tile[layer + 1]; ++t)
            st += (double)partial[((size_t)t * d + b) * d + a];
        s = 0.5 * (s + st);
    }
    if (shift_sum && n > 0) s -= shift_sum[(size_t)layer * d + a] * shift_sum[(size_t)layer * d + b] / n;
    const float v = n > 0 ? (float)(s / n) : 0.0f;
    C[((size_t)layer * d + a) * d + b] = v;
    C[((size_t)layer * d + b) * d + a] = v;
    C0[((size_t)layer * d + a) * d + b] = v;
    C0[((size_t)layer * d + b) * d + a] = v;
}

// ---- a fit whose samples are spread over several participants ------------------------------------
// Second moments are additive over samples once every participant centres by the SAME point m:
//   n, sum (x - m), sum (x - m)(x - m)^T   summed over the participants give   C = S2 / n - delta delta^T,
//   mean = m + delta,  delta = sum (x - m) / n   -- the very formula the one-pass covariance uses on one GPU.
// moments_kernel writes one participant's share in fp64, [layer][1 + d + d * d]: n, sum (x - m), the full
// symmetric S2.  grid (d, n_layers), d threads.  tc: the partials come from the tensor-core kernel (its diagonal
// blocks hold X with S2 = (X + X^T) / 2, and shift_sum = sum (x - m)); otherwise they were taken about `centre`
// by the FP32-pipe kernel, which fills the blocks on and above the diagonal, and colsum = sum x.
__global__ void moments_kernel(int d, int L, int tc, const int32_t *layer_first_tile, const int32_t *layer_S,
                               const float *__restrict__ partial, const double *colsum, const float *centre, double *moments)
{
    const int layer = blockIdx.y, a = blockIdx.x, b = threadIdx.x;
    const int lo = a < b ? a : b, hi = a < b ? b : a;
    const double n = (double)L * (double)layer_S[layer];
    double s = 0.0;
    for (int t = layer_first_tile[layer]; t < layer_first_tile[layer + 1]; ++t)
        s += (double)partial[((size_t)t * d + lo) * d + hi];
    if (tc && lo / 128 == hi / 128) {
        double st = 0.0;
        for (int t = layer_first_tile[layer]; t < layer_first_tile[layer + 1]; ++t)
            st += (double)partial[((size_t)t * d + hi) * d + lo];
        s = 0.5 * (s + st);
    }
    double *M = moments + (size_t)layer * (1 + d + (size_t)d * d);
    M[1 + d + (size_t)a * d + b] = s;
    if (a == 0) {
        const size_t i = (size_t)layer * d + b;
        M[1 + b] = tc ? colsum[i] : colsum[i] - n * (double)centre[i];
        if (b == 0) M[0] = n;
    }
}

// From the summed moments: C (and its untouched copy C0), W = identity, the mean and mu = (N / c) mean.
__global__ void cov_from_moments_kernel(int d, int N, int c, const double *__restrict__ moments, const float *centre,
                                        float *C, float *C0, float *W, float *mean, float *mu)
{
    const int layer = blockIdx.y, a = blockIdx.x, b = threadIdx.x;
    const double *M = moments + (size_t)layer * (1 + d + (size_t)d * d);
    const double n = M[0];
    const double da = n > 0 ? M[1 + a] / n : 0.0, db = n > 0 ? M[1 + b] / n : 0.0;
    const float v = n > 0 ? (float)(M[1 + d + (size_t)a * d + b] / n - da * db) : 0.0f;
    const size_t e = ((size_t)layer * d + a) * d + b;
    C[e] = v;
    C0[e] = v;
    W[e] = (a == b) ? 1.0f : 0.0f;
    if (a == 0) {
        const size_t i = (size_t)layer * d + b;
        const double m = n > 0 ? (double)centre[i] + db : 0.0;
        mean[i] = (float)m;
        mu[i] = (float)(m * (double)N / (double)c);
    }
}

// ---- eigendecomposition -------------------------------------------------------------------------
// Parallel-ordered cyclic Jacobi.  A round pairs the d indices into d/2 disjoint (p, q) by the
// round-robin tournament schedule; all d/2 rotations of a round commute, so
//   A <- J^T A J   becomes an independent 2 x 2 update  B_ij <- J_i^T B_ij J_j  of every block
// (rows p_i, q_i; columns p_j, q_j), and  W <- J^T W  rotates row pairs.  d - 1 rounds visit
// every pair once (one sweep).  A rotation is skipped when |a_pq| <= tol * sqrt(|a_pp a_qq|);
// the loop ends after a sweep without rotations or at the sweep limit.
// in_smem: both matrices are first copied into shared memory (small d: the k x k problem of the cheap refresh),
// which takes the L2 round trips out of every round.
__global__ void __launch_bounds__(NTJ) jacobi_kernel(int d, float *C, float *W, int max_sweeps, float tol,
                                                     int32_t *status, int32_t *sweeps, int in_smem)
{
    extern __shared__ __align__(16) unsigned char jsm[];
    const int half = d / 2;
    int *pp = reinterpret_cast<int *>(jsm);
    int *qq = pp + half;
    float *cc = reinterpret_cast<float *>(qq + half);
    float *ss = cc + half;
    __shared__ int rotated;
    float *A_glob = C + (size_t)blockIdx.x * d * d;
    float *W_glob = W + (size_t)blockIdx.x * d * d;
    float *A = A_glob, *Wl = W_glob;
    const int tid = threadIdx.x;
    if (in_smem) {
        A = ss + half;
        Wl = A + d * d;
        for (int e = tid; e < d * d; e += NTJ) { A[e] = A_glob[e]; Wl[e] = W_glob[e]; }
        __syncthreads();
    }

    int sweep = 0;
    bool converged = false;
    for (; sweep < max_sweeps; ++sweep) {
        if (tid == 0) rotated = 0;
        __syncthreads();
        for (int r = 0; r < d - 1; ++r) {
            for (int i = tid; i < half; i += NTJ) {
                int p, q;
                if (i == 0) { p = d - 1; q = r; }
                else { p = (r + i) % (d - 1); q = (r - i + d - 1) % (d - 1); }
                if (p > q) { const int t = p; p = q; q = t; }
                const float app = A[(size_t)p * d + p], aqq = A[(size_t)q * d + q], apq = A[(size_t)p * d + q];
                float c = 1.0f, s = 0.0f;
                if (fabsf(apq) > tol * sqrtf(fabsf(app * aqq)) && fabsf(apq) > 1e-37f) {
                    const float theta = (aqq - app) / (2.0f * apq);
                    const float t = copysignf(1.0f, theta) / (fabsf(theta) + sqrtf(theta * theta + 1.0f));
                    c = 1.0f / sqrtf(t * t + 1.0f);
                    s = t * c;
                    if (s != 0.0f) rotated = 1;
                }
                pp[i] = p; qq[i] = q; cc[i] = c; ss[i] = s;
            }
            __syncthreads();
            for (int b = tid; b < half * half; b += NTJ) {
                const int i = b / half, j = b - i * half;
                const float ci = cc[i], si = ss[i], cj = cc[j], sj = ss[j];
                if (si == 0.0f && sj == 0.0f) continue;
                const int pi = pp[i], qi = qq[i], pj = pp[j], qj = qq[j];
                float *r0 = A + (size_t)pi * d, *r1 = A + (size_t)qi * d;
                const float b00 = r0[pj], b01 = r0[qj], b10 = r1[pj], b11 = r1[qj];
                // rows: J_i^T B
                const float t00 = ci * b00 - si * b10, t01 = ci * b01 - si * b11;
                const float t10 = si * b00 + ci * b10, t11 = si * b01 + ci * b11;
                // columns: (.) J_j
                float n00 = cj * t00 - sj * t01, n01 = sj * t00 + cj * t01;
                float n10 = cj * t10 - sj * t11, n11 = sj * t10 + cj * t11;
                if (i == j) { n01 = 0.0f; n10 = 0.0f; }  // the rotation annihilates a_pq exactly
                r0[pj] = n00; r0[qj] = n01; r1[pj] = n10; r1[qj] = n11;
            }
            for (int e = tid; e < half * d; e += NTJ) {
                const int j = e / d, t = e - j * d;
                const float c = cc[j], s = ss[j];
                if (s == 0.0f) continue;
                float *w0 = Wl + (size_t)pp[j] * d + t, *w1 = Wl + (size_t)qq[j] * d + t;
                const float a = *w0, b = *w1;
                *w0 = c * a - s * b;
                *w1 = s * a + c * b;
            }
            __syncthreads();
        }
        if (rotated == 0) { converged = true; ++sweep; break; }
        __syncthreads();
    }
    if (in_smem) {
        __syncthreads();
        for (int e = tid; e < d * d; e += NTJ) { A_glob[e] = A[e]; W_glob[e] = Wl[e]; }
    }
    if (tid == 0) {
        sweeps[blockIdx.x] = sweep;
        if (!converged) atomicOr(status, 1);
    }
}

// ---- square-root factor of the covariance ---------------------------------------------------------
// L L^T = C + ridge I (unpivoted Cholesky, left-looking; ridge = 1e-5 of the largest diagonal entry, so that the
// rounding of C -- whose null eigenvalues come out as +-1e-7 of the largest -- cannot make a pivot negative).
// The one-sided Jacobi solver then orthogonalises the columns of L instead of those of C: the squared column norms
// it converges to are the eigenvalues of L L^T, and an absolute error e in a column of norm sigma moves the
// eigenvalue sigma^2 by 2 sigma e, so the small eigenvalues come out far more accurately than as column norms of
// C itself (the classical reason for running Jacobi on a Cholesky factor).
// One CTA per layer, thread i owns row i; L is kept in shared memory as packed columns (column k = rows k .. d - 1),
// so a warp reads consecutive words of one column.  Output: Lt [layer][c][r] = L[r][c] (row c = column c of L, zero
// above the diagonal), the layout the solver reads; ridge_out [layer].
__global__ void __launch_bounds__(256) chol_kernel(int d, const float *__restrict__ C0, float *Lt, float *ridge_out)
{
    extern __shared__ __align__(16) float chol_sm[];
    __shared__ float s_red[8];
    __shared__ float s_ridge, s_inv;
    const int layer = blockIdx.x, i = threadIdx.x;
    const float *A = C0 + (size_t)layer * d * d;
    float *out = Lt + (size_t)layer * d * d;
    auto col = [&](int k) { return chol_sm + (size_t)k * d - (size_t)k * (k - 1) / 2 - k; };   // col(k)[r] = L[r][k], r >= k
    float dg = i < d ? A[(size_t)i * d + i] : 0.0f;
    for (int o = 16; o >= 1; o >>= 1) dg = fmaxf(dg, __shfl_xor_sync(0xffffffffu, dg, o));
    if ((i & 31) == 0) s_red[i >> 5] = dg;
    __syncthreads();
    if (i == 0) {
        float m = 0.0f;
        for (int w = 0; w < (int)(blockDim.x + 31) / 32; ++w) m = fmaxf(m, s_red[w]);
        s_ridge = 1e-5f * m;
        ridge_out[layer] = s_ridge;
    }
    __syncthreads();
    const float ridge = s_ridge;
    for (int j = 0; j < d; ++j) {
        float v = 0.0f;
        if (i >= j && i < d) {
            v = A[(size_t)j * d + i] + (i == j ? ridge : 0.0f);
            // the dot product of rows i and j of L over columns k < j: four chains, the column pointer stepped
            // along (column k + 1 starts d - k - 1 words after column k in the packed layout)
            float v1 = 0.0f, v2 = 0.0f, v3 = 0.0f;
            const float *ck = chol_sm;           // ck[r] = L[r][k]
            int k = 0, step = d - 1;
            for (; k + 3 < j; k += 4) {
                const float *c1 = ck + step, *c2 = c1 + (step - 1), *c3 = c2 + (step - 2);
                v = fmaf(-ck[i], ck[j], v);
                v1 = fmaf(-c1[i], c1[j], v1);
                v2 = fmaf(-c2[i], c2[j], v2);
                v3 = fmaf(-c3[i], c3[j], v3);
                ck = c3 + (step - 3);
                step -= 4;
            }
            for (; k < j; ++k) {
                v = fmaf(-ck[i], ck[j], v);
                ck += step;
                --step;
            }
            v += (v1 + v2) + v3;
        }
        if (i == j) {
            // a pivot that rounding pushed below the ridge's share is held there (a null layer: ridge 0, column 0)
            const float piv = sqrtf(fmaxf(v, 1e-3f * ridge));
            s_inv = piv > 0.0f ? 1.0f / piv : 0.0f;
            v = piv * piv;
        }
        __syncthreads();
        if (i >= j && i < d) col(j)[i] = v * s_inv;
        __syncthreads();
    }
    for (int c = 0; c < d; ++c)
        if (i < d) out[(size_t)c * d + i] = i >= c ? col(c)[i] : 0.0f;
}

// ---- eigendecomposition in shared memory: one-sided (Hestenes) Jacobi on a thread-block cluster ---
// The global-memory kernel above is bound by L2 latency (two passes over 2 d^2 floats per round).  Here the
// iteration matrix G (starts as C, converges to V diag(lambda)) and the accumulated rotations V live in
// shared memory, split by ROWS over the CL CTAs of a cluster: a rotation of columns (p, q) acts on every
// row alike, so each CTA rotates its own rows; only the three inner products alpha = |g_p|^2,
// beta = |g_q|^2, gamma = g_p . g_q of a pair need all rows -- every CTA pushes its partial sums into
// all CTAs' shared memory, one cluster barrier later everyone adds the CL partials in rank order (so all
// CTAs take bit-identical decisions) and rotates.  Eight lanes own a pair of a round (four pairs per
// warp, so the scalar work of a rotation -- divisions, square roots -- runs for four pairs at once), a lane holds
// chunks of four rows of both columns in registers between the two phases.  A pair is rotated whenever
// |gamma| > tol sqrt(alpha beta); it counts against convergence only when also |gamma| > 5e-7 max_j |g_j|^2
// (below that, gamma of a column that was reduced by cancellation is fp32 noise: rotating on it is harmless
// and keeps polishing, but it would never let the sweep count end).  Column-major shared layout: the eight lanes of a pair read
// 128 contiguous bytes per 128-bit access, conflict-free.
namespace cg = cooperative_groups;
constexpr int HLP = 8;     // lanes per pair: a warp works on 4 pairs at once, a lane on chunks of 4 rows
constexpr int HMAXC = 4;   // chunks per lane (rows per CTA <= 4 * HLP * HMAXC = 128)

// NCH: chunks of four rows per lane when the CTA's R rows fill them exactly (R = 32 NCH), 0 = any R (predicated).
// KEEP_V: accumulate the rotations (eigenvectors for every eigenvalue, however small).  Without it only G is
// kept -- half the shared memory, so a layer needs half the CTAs -- and the kernel returns the columns of G.  Its
// input is then the square-root factor (row c of the input = column c of L with L L^T = C + ridge I): the SQUARED
// norms of the converged columns are the eigenvalues (+ ridge) and their directions the eigenvectors of C.
template <int NCH, bool KEEP_V>
__global__ void __launch_bounds__(1024, 1) hestenes_kernel(int d, int CL, const float *__restrict__ C, float *W,
                                                           int max_sweeps, float tol, int32_t *status, int32_t *sweeps)
{
    constexpr int MC = NCH > 0 ? NCH : HMAXC;
    extern __shared__ __align__(16) float hsm[];
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = CL > 1 ? (int)cluster.block_rank() : 0;
    const int layer = blockIdx.x / CL;
    const int R = d / CL, row0 = rank * R, half = d / 2, nchunk = R / 4;
    float *Gs = hsm;                        // [d][R]  column c, own rows
    float *Vs = Gs + (size_t)d * R;         // [d][R]  (KEEP_V only)
    float *part = Gs + (size_t)(KEEP_V ? 2 : 1) * d * R;   // [2][CL][half][4]  every CTA's partial (alpha, beta, gamma), pushed here
    float *cnorm = part + 2 * CL * half * 4;   // [d] this CTA's partial column norms^2 (start-up only)
    __shared__ float s_amax;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    const float *A = C + (size_t)layer * d * d;

    // G = C (symmetric: column c, rows row0.. = row c of C, columns row0..), V = identity
    for (int idx = tid; idx < d * R; idx += blockDim.x) {
        const int c = idx / R, r = idx - c * R;
        Gs[idx] = A[(size_t)c * d + row0 + r];
        if (KEEP_V) Vs[idx] = (row0 + r == c) ? 1.0f : 0.0f;
    }
    __syncthreads();
    for (int c = warp; c < d; c += nwarps) {
        float a = 0.0f;
        for (int r = lane; r < R; r += 32) a = fmaf(Gs[c * R + r], Gs[c * R + r], a);
        for (int o = 16; o >= 1; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        if (lane == 0) cnorm[c] = a;
    }
    if (CL > 1) cluster.sync(); else __syncthreads();
    if (warp == 0) {
        float m = 0.0f;
        for (int c = lane; c < d; c += 32) {
            float a = 0.0f;
            for (int k = 0; k < CL; ++k) a += (CL > 1 ? cluster.map_shared_rank(cnorm, k) : cnorm)[c];
            m = fmaxf(m, a);
        }
        for (int o = 16; o >= 1; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0) s_amax = m;
    }
    __syncthreads();
    // The scale of the thresholds below: the largest squared column norm seen so far.  At the start that is a
    // column of the input (well below the largest eigenvalue for a Cholesky factor); as the columns turn into
    // eigen-directions it grows towards the largest eigenvalue, so it is brought up to date after every sweep
    // (every CTA of the cluster sees the same sums, hence the same value).
    float amax = s_amax;
    __shared__ float s_wmax[32];
    const float tol2 = tol * tol;

    const int j = lane & (HLP - 1);
    const int i = warp * (32 / HLP) + (lane / HLP);   // this lane group's pair of the round
    const bool has_pair = i < half;
    int sweep = 0;
    bool converged = false;
    for (; sweep < max_sweeps; ++sweep) {
        int rotated = 0;
        float seen = 0.0f;
        const float floor_abs = 5e-7f * amax;
        for (int r = 0; r < d - 1; ++r) {
            const int par = r & 1;
            // round-robin pairing of the d columns: column d - 1 stays, the others rotate (r, i < d - 1)
            int p, q;
            if (i == 0) { p = d - 1; q = r; }
            else {
                p = r + i; if (p >= d - 1) p -= d - 1;
                q = r - i + d - 1; if (q >= d - 1) q -= d - 1;
            }
            if (p > q) { const int t = p; p = q; q = t; }
            float4 x[MC], y[MC];
            float a = 0.0f, b = 0.0f, g = 0.0f;
            if (has_pair) {
                const float4 *gp = reinterpret_cast<const float4 *>(Gs + p * R);
                const float4 *gq = reinterpret_cast<const float4 *>(Gs + q * R);
#pragma unroll
                for (int m = 0; m < MC; ++m) {
                    const int c = j + HLP * m;
                    if (NCH > 0 || c < nchunk) {
                        x[m] = gp[c]; y[m] = gq[c];
                        a = fmaf(x[m].x, x[m].x, a); a = fmaf(x[m].y, x[m].y, a); a = fmaf(x[m].z, x[m].z, a); a = fmaf(x[m].w, x[m].w, a);
                        b = fmaf(y[m].x, y[m].x, b); b = fmaf(y[m].y, y[m].y, b); b = fmaf(y[m].z, y[m].z, b); b = fmaf(y[m].w, y[m].w, b);
                        g = fmaf(x[m].x, y[m].x, g); g = fmaf(x[m].y, y[m].y, g); g = fmaf(x[m].z, y[m].z, g); g = fmaf(x[m].w, y[m].w, g);
                    }
                }
            }
#pragma unroll
            for (int o = HLP / 2; o >= 1; o >>= 1) {
                a += __shfl_xor_sync(0xffffffffu, a, o);
                b += __shfl_xor_sync(0xffffffffu, b, o);
                g += __shfl_xor_sync(0xffffffffu, g, o);
            }
            if (CL > 1) {
                // push the partial sums into every CTA's copy (remote stores do not stall; the reads after the
                // barrier are local)
                if (has_pair && j < CL)
                    *reinterpret_cast<float4 *>(cluster.map_shared_rank(part, j) + ((par * CL + rank) * half + i) * 4) =
                        make_float4(a, b, g, 0.f);
                cluster.sync();
                if (has_pair) {
                    a = 0.0f; b = 0.0f; g = 0.0f;
                    for (int k = 0; k < CL; ++k) {  // rank order: every CTA forms the same sums
                        const float4 pv = *reinterpret_cast<const float4 *>(part + ((par * CL + k) * half + i) * 4);
                        a += pv.x; b += pv.y; g += pv.z;
                    }
                }
            }
            if (has_pair) seen = fmaxf(seen, fmaxf(a, b));
            if (has_pair && g * g > tol2 * (a * b)) {
                // The angle only has to annihilate gamma approximately (the iteration converges quadratically), so
                // zeta and t use the fast division; (c, s) must be a rotation to full fp32 accuracy, so the
                // reciprocal square root gets a Newton step.
                const float zeta = __fdividef(b - a, 2.0f * g);
                const float t = __fdividef(copysignf(1.0f, zeta), fabsf(zeta) + sqrtf(fmaf(zeta, zeta, 1.0f)));
                const float w = fmaf(t, t, 1.0f);
                float c = rsqrtf(w);
                c = c * fmaf(-0.5f * w * c, c, 1.5f);
                const float sn = t * c;
                if (sn != 0.0f) {
                    // Without V only the eigenvalues are wanted from this solver, and they are the squared column
                    // norms (the input is a square-root factor): the rotation moves the two of them by |t gamma|,
                    // and the pair counts only while that exceeds 5e-7 of the largest squared norm.  (Couplings
                    // between a large and a small column shrink only linearly per sweep while the small columns,
                    // nearly degenerate among themselves, keep being rotated by large angles; they stop mattering
                    // for the eigenvalues long before they fall under the floor on gamma.)
                    const bool moves = KEEP_V || fabsf(t * g) > 5e-7f * amax;
                    if (fabsf(g) > floor_abs && moves) rotated = 1;
                    float4 *gp = reinterpret_cast<float4 *>(Gs + p * R);
                    float4 *gq = reinterpret_cast<float4 *>(Gs + q * R);
                    float4 *vp = reinterpret_cast<float4 *>(Vs + p * R);
                    float4 *vq = reinterpret_cast<float4 *>(Vs + q * R);
#pragma unroll
                    for (int m = 0; m < MC; ++m) {
                        const int cc = j + HLP * m;
                        if (NCH > 0 || cc < nchunk) {
                            const float4 xx = x[m], yy = y[m];
                            gp[cc] = make_float4(c * xx.x - sn * yy.x, c * xx.y - sn * yy.y, c * xx.z - sn * yy.z, c * xx.w - sn * yy.w);
                            gq[cc] = make_float4(sn * xx.x + c * yy.x, sn * xx.y + c * yy.y, sn * xx.z + c * yy.z, sn * xx.w + c * yy.w);
                            if (KEEP_V) {
                                const float4 a4 = vp[cc], b4 = vq[cc];
                                vp[cc] = make_float4(c * a4.x - sn * b4.x, c * a4.y - sn * b4.y, c * a4.z - sn * b4.z, c * a4.w - sn * b4.w);
                                vq[cc] = make_float4(sn * a4.x + c * b4.x, sn * a4.y + c * b4.y, sn * a4.z + c * b4.z, sn * a4.w + c * b4.w);
                            }
                        }
                    }
                }
            }
            __syncthreads();  // the next round pairs columns rotated by other warps
        }
        for (int o = 16; o >= 1; o >>= 1) seen = fmaxf(seen, __shfl_xor_sync(0xffffffffu, seen, o));
        if (lane == 0) s_wmax[warp] = seen;
        if (__syncthreads_or(rotated) == 0) { converged = true; ++sweep; break; }
        // (with the rotations kept the scale stays the start's: that path's bars were set with it)
        if (!KEEP_V)
            for (int wv = 0; wv < nwarps; ++wv) amax = fmaxf(amax, s_wmax[wv]);
        __syncthreads();   // s_wmax is written again at the end of the next sweep
    }
    // rows of W = eigenvectors: W[j][row0 + r] = V[row0 + r][j]  (without V: the columns of G, not normalised)
    float *Wl = W + (size_t)layer * d * d;
    for (int idx = tid; idx < d * R; idx += blockDim.x) {
        const int c = idx / R, r = idx - c * R;
        Wl[(size_t)c * d + row0 + r] = KEEP_V ? Vs[idx] : Gs[idx];
    }
    if (tid == 0 && rank == 0) {
        sweeps[layer] = sweep;
        if (!converged) atomicOr(status, 1);
    }
    if (CL > 1) cluster.sync();  // nobody leaves while a neighbour may still address its shared memory
}

// Cluster size for the shared-memory eigen-solver, 0 if the matrices do not fit (the global-memory kernel runs then).
size_t hestenes_smem_bytes(int d, int CL, bool keep_v)
{
    return ((size_t)(keep_v ? 2 : 1) * d * (d / CL) + (size_t)4 * CL * d + d) * sizeof(float);
}

int hestenes_cluster_size(int d, bool keep_v = true)
{
    const int cls[4] = {1, 2, 4, 8};
    for (int CL : cls) {
        if (d % CL) continue;
        const int R = d / CL;
        if (R % 4 || R > 4 * HLP * HMAXC) continue;
        if (d / 2 > 32 * (32 / HLP)) continue;
        if (hestenes_smem_bytes(d, CL, keep_v) <= 200 * 1024) return CL;
    }
    return 0;
}

// The values-only eigen-solve's follow-up: eigenvalue j = |column j of G|^2 - ridge (row j of W; G started as the
// square-root factor of C + ridge I), sorted descending into evals; the k longest columns, normalised, become the
// start of the subspace iteration.  One CTA per layer.
__global__ void __launch_bounds__(256) topk_start_kernel(int d, int k, const float *__restrict__ W,
                                                         const float *__restrict__ ridge, float *evals, float *Ut)
{
    __shared__ float lam[GVQ_MAX_D];
    __shared__ int col_of_rank[GVQ_MAX_D];
    const int layer = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float *Wl = W + (size_t)layer * d * d;
    for (int j = warp; j < d; j += 8) {
        double acc = 0.0;
        for (int t = lane; t < d; t += 32) acc += (double)Wl[(size_t)j * d + t] * (double)Wl[(size_t)j * d + t];
        for (int o = 16; o >= 1; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) lam[j] = (float)fmax(acc - (double)ridge[layer], 0.0);
    }
    __syncthreads();
    for (int t = tid; t < d; t += 256) {
        int rank = 0;
        const float v = lam[t];
        for (int o = 0; o < d; ++o) rank += (lam[o] > v) || (lam[o] == v && o < t);
        col_of_rank[rank] = t;
        evals[(size_t)layer * d + rank] = v;
    }
    __syncthreads();
    for (int j = 0; j < k; ++j) {
        const int c = col_of_rank[j];
        // the column's length is sqrt(lambda + ridge); a vanished column: the unit vector of its rank keeps the start full rank
        const float len = sqrtf(lam[c] + ridge[layer]);
        const float inv = lam[c] > 0.0f ? 1.0f / len : 0.0f;
        for (int t = tid; t < d; t += 256)
            Ut[((size_t)layer * k + j) * d + t] = lam[c] > 0.0f ? Wl[(size_t)c * d + t] * inv : (t == j ? 1.0f : 0.0f);
    }
}

// The k leading eigenvalues come from the Ritz step (fp64 sums), the others stay what the solver gave; the list is kept
// non-increasing where the two meet.
__global__ void merge_evals_kernel(int d, int k, int n_layers, const float *__restrict__ evals_k, float *evals)
{
    const int layer = blockIdx.x * blockDim.x + threadIdx.x;
    if (layer >= n_layers) return;
    float *e = evals + (size_t)layer * d;
    for (int j = 0; j < k; ++j) e[j] = evals_k[(size_t)layer * k + j];
    for (int j = k; j < d; ++j) e[j] = fminf(e[j], e[j - 1]);
}

// lam[layer][j] = (w_j^T C0 w_j) / (w_j^T w_j) for row j of W, in fp64.  grid (d, n_layers), d threads;
// thread b forms column b of w^T C0 (C0 is symmetric, so the reads are coalesced).
__global__ void rayleigh_kernel(int d, const float *__restrict__ C0, const float *__restrict__ W, float *lam)
{
    __shared__ float w[GVQ_MAX_D];
    __shared__ double red[2][32];
    const int layer = blockIdx.y, j = blockIdx.x, b = threadIdx.x;
    const float *A = C0 + (size_t)layer * d * d;
    w[b] = W[((size_t)layer * d + j) * d + b];
    __syncthreads();
    double y = 0.0;
    for (int a = 0; a < d; ++a) y += (double)A[(size_t)a * d + b] * (double)w[a];
    double num = y * (double)w[b], den = (double)w[b] * (double)w[b];
    for (int o = 16; o >= 1; o >>= 1) {
        num += __shfl_xor_sync(0xffffffffu, num, o);
        den += __shfl_xor_sync(0xffffffffu, den, o);
    }
    if ((b & 31) == 0) { red[0][b >> 5] = num; red[1][b >> 5] = den; }
    __syncthreads();
    if (b == 0) {
        double n = 0.0, q = 0.0;
        for (int i = 0; i < (d + 31) / 32; ++i) { n += red[0][i]; q += red[1][i]; }
        lam[(size_t)layer * d + j] = q > 0.0 ? (float)(n / q) : 0.0f;
    }
}

// Eigenvalues descending (equal values: lower index first); the k leading eigenvectors become
// the rows of Ut, each with its largest-magnitude entry (lowest index among equals) positive and
// rescaled to unit length (thousands of fp32 rotations let the norm drift by ~1e-5).
// One CTA per layer, 256 threads, d <= 512.
__global__ void __launch_bounds__(256) finalize_kernel(int d, int k, const float *lam_in, const float *W, float *Ut,
                                                       float *evals)
{
    __shared__ float lam[GVQ_MAX_D];
    __shared__ int col_of_rank[GVQ_MAX_D];
    __shared__ float red_v[256];
    __shared__ int red_i[256];
    __shared__ float red_q[256];
    const int layer = blockIdx.x, tid = threadIdx.x;
    const float *Wl = W + (size_t)layer * d * d;
    for (int t = tid; t < d; t += 256) lam[t] = lam_in[(size_t)layer * d + t];
    __syncthreads();
    for (int t = tid; t < d; t += 256) {
        int rank = 0;
        const float v = lam[t];
        for (int o = 0; o < d; ++o) rank += (lam[o] > v) || (lam[o] == v && o < t);
        col_of_rank[rank] = t;
        evals[(size_t)layer * d + rank] = v;
    }
    __syncthreads();
    for (int j = 0; j < k; ++j) {
        const float *row = Wl + (size_t)col_of_rank[j] * d;
        float best = -1.0f, sq = 0.0f;
        int besti = 0;
        for (int t = tid; t < d; t += 256) {
            const float a = fabsf(row[t]);
            if (a > best) { best = a; besti = t; }
            sq = fmaf(a, a, sq);
        }
        red_v[tid] = best; red_i[tid] = besti; red_q[tid] = sq;
        __syncthreads();
        for (int s = 128; s >= 1; s >>= 1) {
            if (tid < s) {
                const float ov = red_v[tid + s];
                const int oi = red_i[tid + s];
                if (ov > red_v[tid] || (ov == red_v[tid] && oi < red_i[tid])) { red_v[tid] = ov; red_i[tid] = oi; }
                red_q[tid] += red_q[tid + s];
            }
            __syncthreads();
        }
        const float scale = (row[red_i[0]] < 0.0f ? -1.0f : 1.0f) / sqrtf(red_q[0]);
        for (int t = tid; t < d; t += 256) Ut[((size_t)layer * k + j) * d + t] = scale * row[t];
        __syncthreads();
    }
}

// ---- the k leading eigenvectors by subspace iteration (the cheap refresh) --------------------------------------
// One CTA per layer; thread t owns column t of the k x d iterate (d <= 256, k <= 32).  A round multiplies the
// iterate by C (thread t forms column t of Q C from C's column t, read coalesced, and Q in shared memory) and
// orthonormalises the rows again (classical Gram-Schmidt, two passes; a row that vanishes -- C of rank < k -- is
// replaced by a pseudo-random one).  After the last round B = Q C Q^T (k x k, fp64 sums) goes to the small Jacobi
// solver; ritz_kernel rotates Q by its eigenvectors.
constexpr int SUB_T = 256, SUB_K = 32;

__device__ __forceinline__ float sub_noise(int layer, int j, int t, int salt)
{
    uint32_t x = (uint32_t)layer * 0x9E3779B9u ^ ((uint32_t)j * 0x85EBCA6Bu + (uint32_t)t * 0xC2B2AE35u + (uint32_t)salt * 0x27D4EB2Fu);
    x ^= x >> 16; x *= 0x7FEB352Du; x ^= x >> 15; x *= 0x846CA68Bu; x ^= x >> 16;
    return (float)(x >> 8) * (1.0f / 8388608.0f) - 1.0f;   // [-1, 1)
}

struct SubSmem {
    float Q[SUB_K][SUB_T];
    float Y[SUB_K][SUB_T];
    float dots[SUB_K];
    float red[8];
};

// rows [0, k) of X (entries [0, d)) -> orthonormal rows, in place
__device__ void sub_orthonormalise(float (*X)[SUB_T], int d, int k, int layer, float *dots, float *red)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int j = 0; j < k; ++j) {
        for (int attempt = 0; attempt < 4; ++attempt) {
            // the norm before and after tells whether the row lay in the span of the earlier ones
            float before = 0.0f, after = 0.0f;
            for (int pass = 0; pass < 3; ++pass) {   // pass 0: norm before; 1, 2: project out rows < j
                if (pass > 0) {
                    for (int i = warp; i < j; i += SUB_T / 32) {
                        float acc = 0.0f;
                        for (int t = lane; t < d; t += 32) acc = fmaf(X[j][t], X[i][t], acc);
                        for (int o = 16; o >= 1; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
                        if (lane == 0) dots[i] = acc;
                    }
                    __syncthreads();
                    if (tid < d) {
                        float v = X[j][tid];
                        for (int i = 0; i < j; ++i) v = fmaf(-dots[i], X[i][tid], v);
                        X[j][tid] = v;
                    }
                    __syncthreads();
                }
                float sq = tid < d ? X[j][tid] * X[j][tid] : 0.0f;
                for (int o = 16; o >= 1; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
                if (lane == 0) red[warp] = sq;
                __syncthreads();
                float tot = 0.0f;
                for (int wv = 0; wv < SUB_T / 32; ++wv) tot += red[wv];
                __syncthreads();
                if (pass == 0) before = tot; else after = tot;
            }
            if (after > 1e-10f * before && after > 0.0f) {
                const float inv = rsqrtf(after);
                if (tid < d) X[j][tid] *= inv;
                __syncthreads();
                break;
            }
            if (tid < d) X[j][tid] = sub_noise(layer, j, tid, attempt + 1);   // a fresh direction
            __syncthreads();
        }
    }
}

// Y = X C (C symmetric, [d][d] in global memory)
__device__ void sub_multiply(const float (*X)[SUB_T], float (*Y)[SUB_T], const float *__restrict__ C, int d, int k)
{
    const int t = threadIdx.x;
    if (t < d) {
        float acc[SUB_K];
#pragma unroll
        for (int j = 0; j < SUB_K; ++j) acc[j] = 0.0f;
        for (int a = 0; a < d; a += 4) {
            const float c0 = C[(size_t)a * d + t], c1 = C[(size_t)(a + 1) * d + t];
            const float c2 = C[(size_t)(a + 2) * d + t], c3 = C[(size_t)(a + 3) * d + t];
#pragma unroll
            for (int j = 0; j < SUB_K; ++j) {
                if (j < k) {
                    const float4 q = *reinterpret_cast<const float4 *>(&X[j][a]);
                    acc[j] = fmaf(q.x, c0, fmaf(q.y, c1, fmaf(q.z, c2, fmaf(q.w, c3, acc[j]))));
                }
            }
        }
#pragma unroll
        for (int j = 0; j < SUB_K; ++j)
            if (j < k) Y[j][t] = acc[j];
    }
    __syncthreads();
}

// kp = k rounded up to even: the small solver pairs indices.  Bk, B0: [layers][kp][kp], Wk likewise (identity),
// Qk: [layers][k][d], trace: [layers].
__global__ void __launch_bounds__(SUB_T) subspace_kernel(int d, int k, int kp, int iters, int warm,
                                                         const float *__restrict__ C, const float *Ut_in, float *Qk,
                                                         float *Bk, float *B0, float *Wk, float *trace)
{
    extern __shared__ __align__(16) unsigned char sub_raw[];
    SubSmem &sm = *reinterpret_cast<SubSmem *>(sub_raw);
    const int layer = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float *A = C + (size_t)layer * d * d;
    __shared__ float s_trace;
    if (warp == 0) {
        double tr = 0.0;
        for (int t = lane; t < d; t += 32) tr += (double)A[(size_t)t * d + t];
        for (int o = 16; o >= 1; o >>= 1) tr += __shfl_xor_sync(0xffffffffu, tr, o);
        if (lane == 0) { s_trace = (float)tr; trace[layer] = (float)tr; }
    }
    __syncthreads();
    const bool null_matrix = !(s_trace > 0.0f);   // a layer without samples: the unit vectors, as the full fit gives
    for (int j = 0; j < k; ++j)
        if (tid < d)
            sm.Q[j][tid] = null_matrix ? (tid == j ? 1.0f : 0.0f)
                                       : warm ? Ut_in[((size_t)layer * k + j) * d + tid] : sub_noise(layer, j, tid, 0);
    __syncthreads();
    if (!null_matrix) {
        sub_orthonormalise(sm.Q, d, k, layer, sm.dots, sm.red);
        for (int it = 0; it < iters; ++it) {
            sub_multiply(sm.Q, sm.Y, A, d, k);
            for (int j = 0; j < k; ++j)
                if (tid < d) sm.Q[j][tid] = sm.Y[j][tid];
            __syncthreads();
            // two multiplications per orthonormalisation: the rows drift towards the leading eigenvector by
            // (lambda_1 / lambda_k)^2 in between, far from what fp32 would lose
            if ((it & 1) || it == iters - 1) sub_orthonormalise(sm.Q, d, k, layer, sm.dots, sm.red);
        }
    }
    sub_multiply(sm.Q, sm.Y, A, d, k);
    // B = Q (Q C)^T, symmetrised; the padding index gets a negative diagonal entry so that it sorts last
    float *Bl = Bk + (size_t)layer * kp * kp, *B0l = B0 + (size_t)layer * kp * kp, *Wl = Wk + (size_t)layer * kp * kp;
    for (int pi = warp; pi < kp * kp; pi += SUB_T / 32) {
        const int i = pi / kp, j = pi - i * kp;
        if (j < i) continue;
        double acc = 0.0;
        if (i < k && j < k) {
            for (int t = lane; t < d; t += 32)
                acc += 0.5 * ((double)sm.Q[i][t] * (double)sm.Y[j][t] + (double)sm.Q[j][t] * (double)sm.Y[i][t]);
            for (int o = 16; o >= 1; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        } else if (i == j) {
            acc = -1.0;
        }
        if (lane == 0) {
            Bl[i * kp + j] = (float)acc; Bl[j * kp + i] = (float)acc;
            B0l[i * kp + j] = (float)acc; B0l[j * kp + i] = (float)acc;
        }
    }
    for (int e = tid; e < kp * kp; e += SUB_T) Wl[e] = (e / kp == e % kp) ? 1.0f : 0.0f;
    for (int j = 0; j < k; ++j)
        if (tid < d) Qk[((size_t)layer * k + j) * d + tid] = sm.Q[j][tid];
}

// Eigenvalues of the small problem as fp64 Rayleigh quotients against the untouched B0, descending; the k leading
// Ritz vectors u_j = sum_m w_j[m] Q_m, unit length, largest-magnitude entry positive.  One CTA per layer.
__global__ void __launch_bounds__(SUB_T) ritz_kernel(int d, int k, int kp, const float *__restrict__ B0,
                                                     const float *__restrict__ Wk, const float *__restrict__ Qk, float *Ut,
                                                     float *evals_k)
{
    __shared__ float lam[SUB_K + 2];
    __shared__ int col_of_rank[SUB_K + 2];
    __shared__ float red_v[SUB_T];
    __shared__ int red_i[SUB_T];
    __shared__ float red_q[SUB_T];
    const int layer = blockIdx.x, tid = threadIdx.x;
    const float *Bl = B0 + (size_t)layer * kp * kp, *Wl = Wk + (size_t)layer * kp * kp;
    if (tid < kp) {
        double num = 0.0, den = 0.0;
        for (int a = 0; a < kp; ++a) {
            double y = 0.0;
            for (int b = 0; b < kp; ++b) y += (double)Bl[a * kp + b] * (double)Wl[tid * kp + b];
            num += y * (double)Wl[tid * kp + a];
            den += (double)Wl[tid * kp + a] * (double)Wl[tid * kp + a];
        }
        lam[tid] = den > 0.0 ? (float)(num / den) : -2.0f;
    }
    __syncthreads();
    if (tid < kp) {
        int rank = 0;
        const float v = lam[tid];
        for (int o = 0; o < kp; ++o) rank += (lam[o] > v) || (lam[o] == v && o < tid);
        col_of_rank[rank] = tid;
        if (rank < k) evals_k[(size_t)layer * k + rank] = fmaxf(v, 0.0f);
    }
    __syncthreads();
    for (int j = 0; j < k; ++j) {
        const float *wrow = Wl + (size_t)col_of_rank[j] * kp;
        float u = 0.0f;
        if (tid < d)
            for (int m = 0; m < k; ++m) u = fmaf(wrow[m], Qk[((size_t)layer * k + m) * d + tid], u);
        red_v[tid] = tid < d ? fabsf(u) : -1.0f; red_i[tid] = tid; red_q[tid] = tid < d ? u * u : 0.0f;
        __syncthreads();
        for (int s = SUB_T / 2; s >= 1; s >>= 1) {
            if (tid < s) {
                const float ov = red_v[tid + s];
                const int oi = red_i[tid + s];
                if (ov > red_v[tid] || (ov == red_v[tid] && oi < red_i[tid])) { red_v[tid] = ov; red_i[tid] = oi; }
                red_q[tid] += red_q[tid + s];
            }
            __syncthreads();
        }
        __shared__ float s_sign;
        if (tid == red_i[0]) s_sign = u < 0.0f ? -1.0f : 1.0f;
        __syncthreads();
        if (tid < d) Ut[((size_t)layer * k + j) * d + tid] = u * s_sign * rsqrtf(red_q[0]);
        __syncthreads();
    }
}

}  // namespace

size_t fit_workspace_bytes(int d, int n_layers, int n_fit_tiles)
{
    return carve(nullptr, d, n_layers, n_fit_tiles).bytes;
}

static cudaError_t launch_eigen_stage(cudaStream_t st, const FitArgs &a, const FitWs &w);

// The sampled centre of every layer (what the one-pass covariance centres by), for fits spread over participants.
cudaError_t launch_fit_centre(cudaStream_t st, int d, int n_layers, int L, const float *hist, int64_t hist_stride,
                              const LayerTables &lt, float *centre)
{
    shift_kernel<<<n_layers, d * (1024 / d), 0, st>>>(d, L, hist, hist_stride, lt.off, lt.S, centre);
    return cudaGetLastError();
}

cudaError_t launch_fit_basis(cudaStream_t st, int num_sms, const FitArgs &a, const TileTable &tiles,
                             const LayerTables &lt, int32_t **status_dev, int32_t **sweeps_dev)
{
    const int d = a.d;
    FitWs w = carve(a.ws, d, a.n_layers, tiles.n_tiles);
    *status_dev = w.status;
    *sweeps_dev = w.sweeps;
    cudaError_t e;
    if ((e = cudaMemsetAsync(w.status, 0, sizeof(int32_t), st)) != cudaSuccess) return e;
    if (a.stage == 2) {   // the covariance comes from moments summed over the participants
        cov_from_moments_kernel<<<dim3(d, a.n_layers), d, 0, st>>>(d, a.N, a.c, a.moments, a.centre, w.C, w.C0, w.W, w.mean, a.mu);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        return launch_eigen_stage(st, a, w);
    }
    if ((e = cudaMemsetAsync(w.colsum, 0, sizeof(double) * (size_t)a.n_layers * d, st)) != cudaSuccess) return e;
    const bool one_pass = tiles.n_tiles > 0 && a.hist_maps != nullptr;   // tensor-core covariance: the history is read once
    if (a.stage == 1) {
        // one participant's moments about the given centre: the same covariance kernels, no reduction to C
        if (tiles.n_tiles > 0) {
            if (one_pass) {
                if ((e = launch_cov_tc(st, num_sms, d, a.L, tiles, lt, a.centre, a.hist_maps, a.cov_order, w.partial, w.colsum,
                                       a.error_word, a.wait_kcycles, a.test_drop)) != cudaSuccess)
                    return e;
            } else {
                colsum_kernel<<<dim3(tiles.n_tiles, a.L), NTC, 0, st>>>(d, a.hist, a.hist_stride, tiles.layer, tiles.row0,
                                                                         lt.off, lt.S, w.colsum);
                if ((e = cudaGetLastError()) != cudaSuccess) return e;
                const int BS = d < 64 ? d : 64;
                const int nb = d / BS, n_pairs = nb * (nb + 1) / 2;
                cov_partial_kernel<<<tiles.n_tiles * n_pairs, NTC, 0, st>>>(d, BS, a.L, a.hist, a.hist_stride, tiles.layer,
                                                                            tiles.row0, lt.off, lt.S, a.centre, w.partial);
                if ((e = cudaGetLastError()) != cudaSuccess) return e;
            }
        }
        moments_kernel<<<dim3(d, a.n_layers), d, 0, st>>>(d, a.L, one_pass ? 1 : 0, tiles.layer_first, lt.S, w.partial, w.colsum,
                                                           a.centre, a.moments);
        return cudaGetLastError();
    }
    if (one_pass) {
        shift_kernel<<<a.n_layers, d * (1024 / d), 0, st>>>(d, a.L, a.hist, a.hist_stride, lt.off, lt.S, w.mean);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        if ((e = launch_cov_tc(st, num_sms, d, a.L, tiles, lt, w.mean, a.hist_maps, a.cov_order, w.partial, w.colsum,
                               a.error_word, a.wait_kcycles, a.test_drop)) != cudaSuccess)
            return e;
    } else if (tiles.n_tiles > 0) {
        colsum_kernel<<<dim3(tiles.n_tiles, a.L), NTC, 0, st>>>(d, a.hist, a.hist_stride, tiles.layer, tiles.row0,
                                                                 lt.off, lt.S, w.colsum);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    if (one_pass) {   // the reduction corrects for the approximate centre; mean_kernel then replaces it by the mean
        cov_reduce_kernel<<<dim3(d, a.n_layers), d, 0, st>>>(d, a.L, tiles.layer_first, lt.S, w.partial, w.colsum, w.C,
                                                             w.C0, w.W);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    mean_kernel<<<(a.n_layers * d + 255) / 256, 256, 0, st>>>(d, a.n_layers, a.L, a.N, a.c, lt.S, w.colsum,
                                                               one_pass ? w.mean : nullptr, w.mean, a.mu);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (!one_pass) {
        if (tiles.n_tiles > 0) {
            const int BS = d < 64 ? d : 64;
            const int nb = d / BS, n_pairs = nb * (nb + 1) / 2;
            cov_partial_kernel<<<tiles.n_tiles * n_pairs, NTC, 0, st>>>(d, BS, a.L, a.hist, a.hist_stride, tiles.layer,
                                                                        tiles.row0, lt.off, lt.S, w.mean, w.partial);
            if ((e = cudaGetLastError()) != cudaSuccess) return e;
        }
        cov_reduce_kernel<<<dim3(d, a.n_layers), d, 0, st>>>(d, a.L, tiles.layer_first, lt.S, w.partial, nullptr, w.C,
                                                             w.C0, w.W);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    return launch_eigen_stage(st, a, w);
}

// Everything after the covariance: w.C / w.C0 hold it, w.W the identity.
static cudaError_t launch_eigen_stage(cudaStream_t st, const FitArgs &a, const FitWs &w)
{
    const int d = a.d;
    cudaError_t e;
    const float tol = 6e-8f * sqrtf((float)d);
    const int max_sweeps = a.max_sweeps > 0 ? a.max_sweeps : kJacobiMaxSweeps;
    const int k = a.k, kp = (k + 1) & ~1;
    // scratch of the subspace iteration, inside the W region (after anything the eigen-solver left there was used)
    float *Qk = w.W, *Bk = Qk + (size_t)a.n_layers * k * d, *B0 = Bk + (size_t)a.n_layers * kp * kp;
    float *Wk = B0 + (size_t)a.n_layers * kp * kp, *evk = Wk + (size_t)a.n_layers * kp * kp;
    float *trc = evk + (size_t)a.n_layers * k;
    int32_t *sweeps_small = reinterpret_cast<int32_t *>(trc + a.n_layers);   // sweep counts of the k x k problems
    const bool sub_ok = d <= SUB_T && k <= SUB_K && (int64_t)k * d + 3 * (int64_t)kp * kp + k + 2 <= (int64_t)d * d;
    // k leading eigenpairs by subspace iteration from Ut_start (or a pseudo-random start), into a.Ut / ev_out / tr_out
    auto subspace_stage = [&](int iters, int warm, float *ev_out, float *tr_out, int32_t *sweeps_out) -> cudaError_t {
        cudaError_t err = cudaFuncSetAttribute(subspace_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(SubSmem));
        if (err != cudaSuccess) return err;
        subspace_kernel<<<a.n_layers, SUB_T, sizeof(SubSmem), st>>>(d, k, kp, iters, warm, w.C0, a.Ut, Qk, Bk, B0, Wk, tr_out);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        jacobi_kernel<<<a.n_layers, NTJ, (size_t)(kp / 2) * 16 + (size_t)2 * kp * kp * sizeof(float), st>>>(
            kp, Bk, Wk, kJacobiMaxSweeps, 6e-8f * sqrtf((float)kp), w.status, sweeps_out, 1);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        ritz_kernel<<<a.n_layers, SUB_T, 0, st>>>(d, k, kp, B0, Wk, Qk, a.Ut, ev_out);
        return cudaGetLastError();
    };
    if (a.topk_iters > 0) return subspace_stage(a.topk_iters, a.warm_start, a.evals_k, a.trace, w.sweeps);   // the cheap refresh

    // the shared-memory eigen-solver, with or without the accumulated rotations
    auto hestenes = [&](int CL, bool keep_v) -> cudaError_t {
        const int R = d / CL;
        const size_t smem = hestenes_smem_bytes(d, CL, keep_v);
        using Kernel = void (*)(int, int, const float *, float *, int, float, int32_t *, int32_t *);
        Kernel kernel = keep_v ? (Kernel)hestenes_kernel<0, true> : (Kernel)hestenes_kernel<0, false>;
        if (R % 32 == 0) {
            switch (R / 32) {
            case 1: kernel = keep_v ? (Kernel)hestenes_kernel<1, true> : (Kernel)hestenes_kernel<1, false>; break;
            case 2: kernel = keep_v ? (Kernel)hestenes_kernel<2, true> : (Kernel)hestenes_kernel<2, false>; break;
            case 3: kernel = keep_v ? (Kernel)hestenes_kernel<3, true> : (Kernel)hestenes_kernel<3, false>; break;
            default: kernel = keep_v ? (Kernel)hestenes_kernel<4, true> : (Kernel)hestenes_kernel<4, false>; break;
            }
        }
        cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        int nw = (d / 2 + 32 / HLP - 1) / (32 / HLP);   // four pairs per warp
        if (nw < 1) nw = 1;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(a.n_layers * CL);
        cfg.blockDim = dim3(nw * 32);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = CL; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, kernel, d, CL, (const float *)w.C, w.W, max_sweeps, tol, w.status, w.sweeps);
    };
    const int CL = hestenes_cluster_size(d, true), CLv = hestenes_cluster_size(d, false);
    // Only the k leading eigenvectors are ever used, so wherever the subspace iteration serves the shape the
    // eigenvalues come from the solver without accumulated rotations -- half the shared memory per layer (fewer CTAs
    // per cluster, so more layers resident at once), half the data moved per round, and sweeps that end once the
    // eigenvalues have settled -- and the k leading eigenvectors from two rounds of subspace iteration started at the
    // k longest columns it returns.  Measured full fits, rotations kept -> not: 14.3 -> 8.9 ms (ResNet-50 shape),
    // 2.7 -> 1.6 ms (VGG-16 shape), 0.58 -> 0.55 ms (ResNet-32 shape).
    const bool values_only = (a.fit_path == 2 || a.fit_path == 0) && sub_ok && CLv > 0;
    if (a.fit_path == 2 && !values_only) return cudaErrorNotSupported;
    if (values_only) {
        // the solver works on the square-root factor of the covariance (written over w.C; w.C0 keeps the covariance)
        const size_t chol_smem = sizeof(float) * (size_t)d * (d + 1) / 2;
        if ((e = cudaFuncSetAttribute(chol_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)chol_smem)) != cudaSuccess)
            return e;
        chol_kernel<<<a.n_layers, std::max(32, (d + 31) / 32 * 32), chol_smem, st>>>(d, w.C0, w.C, w.lam);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        if ((e = hestenes(CLv, false)) != cudaSuccess) return e;
        topk_start_kernel<<<a.n_layers, 256, 0, st>>>(d, k, w.W, w.lam, a.evals, a.Ut);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        if ((e = subspace_stage(2, 1, evk, trc, sweeps_small)) != cudaSuccess) return e;
        merge_evals_kernel<<<(a.n_layers + 127) / 128, 128, 0, st>>>(d, k, a.n_layers, evk, a.evals);
        return cudaGetLastError();
    }
    if (CL > 0) {
        if ((e = hestenes(CL, true)) != cudaSuccess) return e;
    } else {
        jacobi_kernel<<<a.n_layers, NTJ, (size_t)(d / 2) * 16, st>>>(d, w.C, w.W, max_sweeps, tol, w.status,
                                                                     w.sweeps, 0);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    rayleigh_kernel<<<dim3(d, a.n_layers), d, 0, st>>>(d, w.C0, w.W, w.lam);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    finalize_kernel<<<a.n_layers, 256, 0, st>>>(d, a.k, w.lam, w.W, a.Ut, a.evals);
    return cudaGetLastError();
}

using EncodeTiledFn3 = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

cudaError_t prepare_fit_maps(gvq_ctx *ctx, const float *hist, int64_t hist_stride, int L, const CUtensorMap **maps_out)
{
    *maps_out = nullptr;
    if (!ctx->fit_maps_dev || !ctx->encode_fn || !cov_tc_supported(ctx->d)) return cudaSuccess;
    EncodeTiledFn3 enc = (EncodeTiledFn3)ctx->encode_fn;
    for (int l = 0; l < ctx->n_layers; ++l) {
        const int64_t S = ctx->layer_len[l] / ctx->d;
        // dims: entries of a slice, slices of the layer, stored gradients; a layer without a full slice has no tile
        cuuint64_t dims[3] = {(cuuint64_t)ctx->d, (cuuint64_t)(S > 0 ? S : 1), (cuuint64_t)L};
        cuuint64_t strides[2] = {(cuuint64_t)ctx->d * sizeof(float),
                                 (cuuint64_t)(L > 1 ? hist_stride : (int64_t)ctx->d * (S > 0 ? S : 1)) * sizeof(float)};
        cuuint32_t box[3] = {32, 32, 1};
        cuuint32_t estr[3] = {1, 1, 1};
        CUresult r = enc(&ctx->fit_maps_host[l], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, (void *)(hist + ctx->layer_off[l]),
                         dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    // pageable source: staged before the call returns; ordered on the stream before the kernel that reads it
    cudaError_t e = cudaMemcpyAsync(ctx->fit_maps_dev, ctx->fit_maps_host.data(), sizeof(CUtensorMap) * (size_t)ctx->n_layers,
                                    cudaMemcpyHostToDevice, ctx->stream);
    if (e != cudaSuccess) return e;
    *maps_out = ctx->fit_maps_dev;
    return cudaSuccess;
}

}  // namespace gvq

// ---- basis fit without a caller-provided workspace ------------------------------------------------
// The scratch of gvq_fit_basis_static: a fixed device array that every GPU loading the library holds
// until the process exits.  In host code `g_static_fit_scratch` is only a stand-in for the symbol; the
// device address comes from cudaGetSymbolAddress, asked once per device with that device current.
static __device__ __align__(256) unsigned char g_static_fit_scratch[GVQ_STATIC_FIT_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_addr[kMaxDevices] = {};

// Device address of the static scratch on `device` (which must be current); looked up on first use.
cudaError_t static_scratch_address(int device, void **out)
{
    if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_addr[device]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_fit_scratch);
        if (e != cudaSuccess) return e;
        g_static_addr[device] = p;
    }
    *out = g_static_addr[device];
    return cudaSuccess;
}
}  // namespace

extern "C" gvq_status gvq_fit_basis_static(gvq_ctx *ctx, const float *hist, int64_t hist_stride, int L, int N,
                                           int samples_are_sums_of, float *Ut, float *mu, float *evals,
                                           int32_t *info)
{
    using namespace gvq;
    if (!ctx || !hist || !Ut || !mu || !evals) return GVQ_ERR_NULL;
    if (L < 1 || N < 1 || N > GVQ_MAX_NODES || samples_are_sums_of < 1) return GVQ_ERR_SHAPE;
    if (hist_stride < ctx->M && L > 1) return GVQ_ERR_SHAPE;
    auto misaligned = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
    if (hist_stride % 4 != 0 || misaligned(hist) || misaligned(Ut) || misaligned(mu) || misaligned(evals))
        return GVQ_ERR_ALIGN;
    if (fit_workspace_bytes(ctx->d, ctx->n_layers, ctx->fit_tiles.n_tiles) > (size_t)GVQ_STATIC_FIT_BYTES)
        return GVQ_ERR_WORKSPACE;  // this layout needs more scratch than the fixed array holds

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(ctx->device) != cudaSuccess) {
        ctx->last_cuda_error = (int)cudaGetLastError();
        return GVQ_ERR_CUDA;
    }
    gvq_status result = GVQ_OK;
    cudaError_t e;
    void *scratch = nullptr;
    int32_t *status_dev = nullptr, *sweeps_dev = nullptr;
    int32_t gave_up = 0;   // a tensor-core kernel of the fit whose bounded wait ran out
    int32_t status = 0;
    FitArgs a;
    a.d = ctx->d; a.k = ctx->k; a.n_layers = ctx->n_layers; a.L = L; a.N = N; a.c = samples_are_sums_of;
    a.hist = hist; a.hist_stride = hist_stride; a.Ut = Ut; a.mu = mu; a.evals = evals;
    a.fit_path = ctx->fit_path;
    a.max_sweeps = ctx->max_sweeps; a.wait_kcycles = ctx->wait_kcycles; a.test_drop = ctx->drop_last_load;
    if ((e = static_scratch_address(ctx->device, &scratch)) != cudaSuccess) goto cuda_failed;
    a.ws = scratch;
    if ((e = prepare_fit_maps(ctx, hist, hist_stride, L, &a.hist_maps)) != cudaSuccess) goto cuda_failed;
    a.error_word = ctx->error_word;
    a.cov_order = ctx->cov_unit_order;
    // launch_fit_basis clears what must start at zero (column sums, convergence word); everything else in
    // the scratch is written before it is read, so the previous call's contents do not matter
    if ((e = launch_fit_basis(ctx->stream, ctx->num_sms, a, ctx->fit_tiles, ctx->lt, &status_dev, &sweeps_dev)) !=
        cudaSuccess)
        goto cuda_failed;
    if ((e = cudaMemcpyAsync(&status, status_dev, sizeof(status), cudaMemcpyDeviceToHost, ctx->stream)) != cudaSuccess)
        goto cuda_failed;
    if (info && (e = cudaMemcpyAsync(info, sweeps_dev, sizeof(int32_t) * (size_t)ctx->n_layers,
                                     cudaMemcpyDeviceToHost, ctx->stream)) != cudaSuccess)
        goto cuda_failed;
    if ((e = cudaMemcpyAsync(&gave_up, ctx->error_word, sizeof(gave_up), cudaMemcpyDeviceToHost, ctx->stream)) != cudaSuccess)
        goto cuda_failed;
    if ((e = cudaStreamSynchronize(ctx->stream)) != cudaSuccess) goto cuda_failed;
    result = gave_up ? GVQ_ERR_TIMEOUT : status ? GVQ_ERR_NOT_CONVERGED : GVQ_OK;
    if (gave_up) {   // leave the word clear for the next call, as gvq_fit_basis does
        cudaMemsetAsync(ctx->error_word, 0, sizeof(int32_t), ctx->stream);
        if (ctx->tc_tile_counter)
            cudaMemsetAsync(ctx->tc_tile_counter, 0,
                            sizeof(int32_t) * (size_t)(ctx->project_tc_tiles.n_tiles > 0 ? ctx->project_tc_tiles.n_tiles : 1),
                            ctx->stream);
    }
    cudaSetDevice(prev);
    return result;

cuda_failed:
    ctx->last_cuda_error = (int)e;
    (void)cudaGetLastError();
    cudaSetDevice(prev);
    return GVQ_ERR_CUDA;
}

/*
 * GradiVeQ oracle -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, obviously-correct CPU statement of what the GradiVeQ hot path
 * computes, written from the paper's equations.  Floating point is fp64 on the
 * fp32 input bytes (the quantizer is the one exception: it is defined in fp32 so
 * that its integer levels can be compared bit for bit).  There is no blocking,
 * fusion or reordering beyond what the equations state; OpenMP "parallel for"
 * over independent slices / layers is the only parallelism.  Nothing here is
 * shared with, or imported by, the CUDA library; only tests, the smoke check and
 * the benchmark's cpu_baseline / reference legs may call it.
 *
 * Notation (the paper's symbols in brackets):
 *   d  slice length [K]          k  compressed length [d]        N  nodes
 *   M  gradient entries          S  = number of full slices      L  stored gradients [L_t]
 *   Ut compressor transposed, [layer][k][d] row-major (row j = j-th eigenvector) [U_{d,m}^T]
 *   mu whitening vector of the AGGREGATED gradient, [layer][d]   [mu_m]
 *
 * A flat gradient is a sequence of layers; layer l occupies layer_len[l] floats
 * starting at layer_off[l].  Its first S_l = layer_len[l] / d runs of d entries are
 * the slices (Section 2, "every slice of K adjacent gradients"); the remaining
 * layer_len[l] % d entries ("tail") are not compressed and are summed as they are
 * (Algorithm 1 without compression is the plain sum).  Compressed buffers are
 * [S_total][k], the layers' slices following one another.
 *
 * Pins (tests/test_oracle_pins.py): linearity Eq. 1 / Eq. 4, U^T U = I, exact
 * reconstruction at k = d, fit-set residual = discarded eigenvalue mass (Eq. 6),
 * Jacobi against closed forms / constructed spectra / a library eigensolver,
 * quantizer unbiasedness and bounds.  Parity unpinned: nothing in this file.
 * (The paper's figures that carry numbers need recorded ResNet-32 gradients and
 * are not reproduced.)
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define GVQO_OK 0
#define GVQO_ERR_ARG 1
#define GVQO_ERR_NOT_CONVERGED 2
#define GVQO_ERR_NOMEM 3

/* ------------------------------------------------------------------------- */
/* Symmetric eigendecomposition: cyclic two-sided Jacobi (Section 2: "applies */
/* SVD to obtain the eigen matrix and eigen vector of C" -- for a symmetric   */
/* PSD matrix that is its eigendecomposition).                                */
/* A is n x n row-major, symmetric, overwritten (diagonal -> eigenvalues,     */
/* unsorted).  V (n x n row-major) receives the eigenvectors as COLUMNS.      */
/* ------------------------------------------------------------------------- */
int gvqo_jacobi_eig(int n, double *A, double *V, int max_sweeps, int *sweeps_used)
{
    if (n <= 0 || !A || !V) return GVQO_ERR_ARG;
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j) V[(size_t)i * n + j] = (i == j) ? 1.0 : 0.0;

    double fro2 = 0.0;
    for (size_t i = 0; i < (size_t)n * n; ++i) fro2 += A[i] * A[i];
    const double tol2 = 1e-28 * fro2; /* off(A) <= 1e-14 * ||A||_F */

    int sweep = 0;
    for (;; ++sweep) {
        double off2 = 0.0;
        for (int p = 0; p < n; ++p)
            for (int q = 0; q < n; ++q)
                if (p != q) off2 += A[(size_t)p * n + q] * A[(size_t)p * n + q];
        if (off2 <= tol2) break;
        if (sweep >= max_sweeps) {
            if (sweeps_used) *sweeps_used = sweep;
            return GVQO_ERR_NOT_CONVERGED;
        }
        for (int p = 0; p < n - 1; ++p) {
            for (int q = p + 1; q < n; ++q) {
                const double apq = A[(size_t)p * n + q];
                if (apq == 0.0) continue;
                const double app = A[(size_t)p * n + p], aqq = A[(size_t)q * n + q];
                /* rotation angle that zeroes A[p][q]: tan(2 phi) = 2 apq / (aqq - app) */
                const double theta = (aqq - app) / (2.0 * apq);
                const double t = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
                const double c = 1.0 / sqrt(t * t + 1.0), s = t * c;
                /* A <- J^T A J, J = rotation in the (p,q) plane */
                for (int r = 0; r < n; ++r) { /* columns p, q */
                    const double arp = A[(size_t)r * n + p], arq = A[(size_t)r * n + q];
                    A[(size_t)r * n + p] = c * arp - s * arq;
                    A[(size_t)r * n + q] = s * arp + c * arq;
                }
                for (int r = 0; r < n; ++r) { /* rows p, q */
                    const double apr = A[(size_t)p * n + r], aqr = A[(size_t)q * n + r];
                    A[(size_t)p * n + r] = c * apr - s * aqr;
                    A[(size_t)q * n + r] = s * apr + c * aqr;
                }
                for (int r = 0; r < n; ++r) { /* V <- V J */
                    const double vrp = V[(size_t)r * n + p], vrq = V[(size_t)r * n + q];
                    V[(size_t)r * n + p] = c * vrp - s * vrq;
                    V[(size_t)r * n + q] = s * vrp + c * vrq;
                }
            }
        }
    }
    if (sweeps_used) *sweeps_used = sweep;
    return GVQO_OK;
}

/* ------------------------------------------------------------------------- */
/* Mean and covariance of the n = L * S_l sample slices of one layer          */
/* (Section 2: the whitening vector is the average of the samples; then "the  */
/* covariance matrix of the K gradients using these samples").  Two passes,   */
/* 1/n normalisation.  hist holds L stored flat gradients, hist_stride floats */
/* apart.  mean[d], cov[d*d] in double.                                       */
/* ------------------------------------------------------------------------- */
int gvqo_mean_cov(int d, int64_t layer_off, int64_t layer_len, const float *hist, int64_t hist_stride,
                  int L, double *mean, double *cov)
{
    if (d <= 0 || L <= 0 || !hist || !mean || !cov) return GVQO_ERR_ARG;
    const int64_t S = layer_len / d;
    const double n = (double)L * (double)S;
    for (int t = 0; t < d; ++t) mean[t] = 0.0;
    for (size_t e = 0; e < (size_t)d * d; ++e) cov[e] = 0.0;
    if (S == 0) return GVQO_OK;

    for (int h = 0; h < L; ++h)
        for (int64_t i = 0; i < S; ++i) {
            const float *x = hist + (size_t)h * hist_stride + layer_off + i * d;
            for (int t = 0; t < d; ++t) mean[t] += (double)x[t];
        }
    for (int t = 0; t < d; ++t) mean[t] /= n;

    /* rows of the covariance are independent: split them over threads, each
       thread summing the samples in the same order */
#pragma omp parallel for schedule(dynamic, 1)
    for (int a = 0; a < d; ++a) {
        double *row = cov + (size_t)a * d;
        for (int h = 0; h < L; ++h)
            for (int64_t i = 0; i < S; ++i) {
                const float *x = hist + (size_t)h * hist_stride + layer_off + i * d;
                const double xa = (double)x[a] - mean[a];
                for (int b = 0; b < d; ++b) row[b] += xa * ((double)x[b] - mean[b]);
            }
        for (int b = 0; b < d; ++b) row[b] /= n;
    }
    return GVQO_OK;
}

/* ------------------------------------------------------------------------- */
/* From eigenpairs to the compressor: eigenvalues descending (equal values:   */
/* lower original index first), first k eigenvectors, each with its largest-  */
/* magnitude entry made positive (equal magnitudes: lowest index decides).    */
/* evals[n] (double, sorted), Ut[k*n] (double, row j = j-th eigenvector).     */
/* ------------------------------------------------------------------------- */
int gvqo_sort_eigs(int n, int k, const double *diagA, const double *V, double *evals, double *Ut)
{
    if (n <= 0 || k < 0 || k > n) return GVQO_ERR_ARG;
    int *order = (int *)malloc(sizeof(int) * (size_t)n);
    if (!order) return GVQO_ERR_NOMEM;
    for (int i = 0; i < n; ++i) order[i] = i;
    for (int i = 1; i < n; ++i) { /* stable insertion sort, descending */
        const int oi = order[i];
        int j = i - 1;
        while (j >= 0 && diagA[(size_t)order[j] * n + order[j]] < diagA[(size_t)oi * n + oi]) {
            order[j + 1] = order[j];
            --j;
        }
        order[j + 1] = oi;
    }
    for (int j = 0; j < n; ++j) evals[j] = diagA[(size_t)order[j] * n + order[j]];
    for (int j = 0; j < k; ++j) {
        const int col = order[j];
        int big = 0;
        for (int t = 1; t < n; ++t)
            if (fabs(V[(size_t)t * n + col]) > fabs(V[(size_t)big * n + col])) big = t;
        const double sgn = V[(size_t)big * n + col] < 0.0 ? -1.0 : 1.0;
        for (int t = 0; t < n; ++t) Ut[(size_t)j * n + t] = sgn * V[(size_t)t * n + col];
    }
    free(order);
    return GVQO_OK;
}

/* ------------------------------------------------------------------------- */
/* Basis fit for every layer (Section 2, the PCA paragraph).                  */
/*   mu (aggregate convention) = (N / samples_are_sums_of) * sample mean:     */
/*   the paper's samples are N-node aggregates (samples_are_sums_of = N), so  */
/*   mu is their plain average; per-node samples pass 1.                      */
/* Outputs in double: Ut [layers][k][d], mu [layers][d], evals [layers][d];   */
/* sweeps [layers].  A layer with no full slice gets Ut = first k unit        */
/* vectors, mu = 0, evals = 0.                                                */
/* ------------------------------------------------------------------------- */
int gvqo_fit_basis(int d, int k, int n_layers, const int64_t *layer_off, const int64_t *layer_len,
                   const float *hist, int64_t hist_stride, int L, int N, int samples_are_sums_of,
                   double *Ut, double *mu, double *evals, int32_t *sweeps)
{
    if (d <= 0 || k <= 0 || k > d || n_layers < 0 || L <= 0 || N <= 0 || samples_are_sums_of <= 0)
        return GVQO_ERR_ARG;
    /* pass 1, layer after layer (each call is parallel inside): sample mean and covariance */
    double *means = (double *)malloc(sizeof(double) * (size_t)n_layers * d);
    double *covs = (double *)malloc(sizeof(double) * (size_t)n_layers * d * d);
    if (!means || !covs) { free(means); free(covs); return GVQO_ERR_NOMEM; }
    int rc_all = GVQO_OK;
    for (int l = 0; l < n_layers && rc_all == GVQO_OK; ++l)
        rc_all = gvqo_mean_cov(d, layer_off[l], layer_len[l], hist, hist_stride, L,
                               means + (size_t)l * d, covs + (size_t)l * d * d);
    /* pass 2, layers independent: eigendecomposition, ordering, sign */
    if (rc_all == GVQO_OK) {
#pragma omp parallel for schedule(dynamic, 1)
        for (int l = 0; l < n_layers; ++l) {
            double *C = covs + (size_t)l * d * d;
            double *V = (double *)malloc(sizeof(double) * (size_t)d * d);
            int sw = 0;
            int rc = V ? GVQO_OK : GVQO_ERR_NOMEM;
            if (rc == GVQO_OK) rc = gvqo_jacobi_eig(d, C, V, 100, &sw);
            if (rc == GVQO_OK)
                rc = gvqo_sort_eigs(d, k, C, V, evals + (size_t)l * d, Ut + (size_t)l * k * d);
            if (rc == GVQO_OK) {
                const double scale = (double)N / (double)samples_are_sums_of;
                for (int t = 0; t < d; ++t) mu[(size_t)l * d + t] = scale * means[(size_t)l * d + t];
                if (sweeps) sweeps[l] = sw;
            } else {
#pragma omp critical
                rc_all = rc;
            }
            free(V);
        }
    }
    free(means); free(covs);
    return rc_all;
}

/* total number of full slices */
int64_t gvqo_total_slices(int d, int n_layers, const int64_t *layer_len)
{
    int64_t S = 0;
    for (int l = 0; l < n_layers; ++l) S += layer_len[l] / d;
    return S;
}

/* ------------------------------------------------------------------------- */
/* Eq. 3:  s_{n,i} = U^T (x_{n,i} - mu / N)  for every slice of one node.     */
/* Ut and mu are the fp32 arrays the CUDA path is given.  s_node [S_total][k] */
/* in double.                                                                 */
/* ------------------------------------------------------------------------- */
int gvqo_compress(int d, int k, int n_layers, const int64_t *layer_off, const int64_t *layer_len,
                  const float *g_node, const float *Ut, const float *mu, int N, double *s_node)
{
    if (d <= 0 || k <= 0 || N <= 0) return GVQO_ERR_ARG;
    int64_t soff = 0;
    for (int l = 0; l < n_layers; ++l) {
        const int64_t S = layer_len[l] / d;
        const float *U = Ut + (size_t)l * k * d, *m = mu + (size_t)l * d;
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < S; ++i) {
            const float *x = g_node + layer_off[l] + i * d;
            for (int j = 0; j < k; ++j) {
                double acc = 0.0;
                for (int t = 0; t < d; ++t)
                    acc += (double)U[(size_t)j * d + t] * ((double)x[t] - (double)m[t] / (double)N);
                s_node[(size_t)(soff + i) * k + j] = acc;
            }
        }
        soff += S;
    }
    return GVQO_OK;
}

/* Eq. 4 (left-hand side):  s_i = sum_{n=0}^{N-1} s_{n,i}. */
int gvqo_aggregate(int64_t count, int N, const double *const *s_nodes, double *s_sum)
{
    if (count < 0 || N <= 0) return GVQO_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < count; ++e) {
        double acc = 0.0;
        for (int n = 0; n < N; ++n) acc += s_nodes[n][e];
        s_sum[e] = acc;
    }
    return GVQO_OK;
}

/* ------------------------------------------------------------------------- */
/* Eq. 5:  g_hat_i = U s_i + mu  for every slice; the uncompressed tail of    */
/* each layer is the plain sum over the nodes.  g_hat is a flat gradient in   */
/* double; entries outside every layer are left untouched.  g_nodes may be    */
/* NULL when no layer has a tail.                                             */
/* ------------------------------------------------------------------------- */
int gvqo_decompress(int d, int k, int n_layers, const int64_t *layer_off, const int64_t *layer_len,
                    const double *s_sum, const float *Ut, const float *mu,
                    const float *const *g_nodes, int N, double *g_hat)
{
    if (d <= 0 || k <= 0 || N <= 0) return GVQO_ERR_ARG;
    int64_t soff = 0;
    for (int l = 0; l < n_layers; ++l) {
        const int64_t S = layer_len[l] / d, tail = layer_len[l] % d;
        const float *U = Ut + (size_t)l * k * d, *m = mu + (size_t)l * d;
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < S; ++i) {
            const double *s = s_sum + (size_t)(soff + i) * k;
            double *out = g_hat + layer_off[l] + i * d;
            for (int t = 0; t < d; ++t) {
                double acc = 0.0;
                for (int j = 0; j < k; ++j) acc += (double)U[(size_t)j * d + t] * s[j];
                out[t] = acc + (double)m[t];
            }
        }
        if (tail > 0) {
            if (!g_nodes) return GVQO_ERR_ARG;
            for (int64_t e = S * d; e < layer_len[l]; ++e) {
                double acc = 0.0;
                for (int n = 0; n < N; ++n) acc += (double)g_nodes[n][layer_off[l] + e];
                g_hat[layer_off[l] + e] = acc;
            }
        }
        soff += S;
    }
    return GVQO_OK;
}

/* Eq. 6: the smallest k with (sum of the k largest eigenvalues) / (sum of all) >= 1 - lambda.
   evals sorted descending.  Returns k in [1, d]; 0 when the spectrum sums to zero or less. */
int gvqo_select_k(int d, const double *evals, double lambda_loss)
{
    double total = 0.0;
    for (int j = 0; j < d; ++j) total += evals[j];
    if (!(total > 0.0)) return 0;
    double head = 0.0;
    for (int j = 0; j < d; ++j) {
        head += evals[j];
        if (head / total >= 1.0 - lambda_loss) return j + 1;
    }
    return d;
}

/* Section 2, the figure on flattening and slicing: a convolutional layer with F filters of size (H, W, D) is
   flattened with the F gradients of one position (h, w, dep) next to each other, positions visited depth first,
   then width, then height.  With the framework's layout [F][D][H][W] (x = h * W + w the spatial index, X = H * W):
       flat[(x * D + dep) * F + f] = framework[(f * D + dep) * X + x].
   inverse != 0 applies the inverse map. */
int gvqo_flatten(int F, int D, int X, const float *src, float *dst, int inverse)
{
    if (F < 1 || D < 1 || X < 1 || !src || !dst) return GVQO_ERR_ARG;
    for (int f = 0; f < F; ++f)
        for (int dep = 0; dep < D; ++dep)
            for (int x = 0; x < X; ++x) {
                const size_t fw = ((size_t)f * D + dep) * X + x, fl = ((size_t)x * D + dep) * F + f;
                if (inverse) dst[fw] = src[fl]; else dst[fl] = src[fw];
            }
    return GVQO_OK;
}

/* Eq. 7: local compression loss of one node,
   sum over slices of || x_{n,i} - (U s_{n,i} + mu / N) ||^2, with s_{n,i} from Eq. 3. */
double gvqo_local_loss(int d, int k, int n_layers, const int64_t *layer_off, const int64_t *layer_len,
                       const float *g_node, const float *Ut, const float *mu, int N)
{
    double total = 0.0;
    double *s = (double *)malloc(sizeof(double) * (size_t)k);
    if (!s) return -1.0;
    for (int l = 0; l < n_layers; ++l) {
        const int64_t S = layer_len[l] / d;
        const float *U = Ut + (size_t)l * k * d, *m = mu + (size_t)l * d;
        for (int64_t i = 0; i < S; ++i) {
            const float *x = g_node + layer_off[l] + i * d;
            for (int j = 0; j < k; ++j) {
                double acc = 0.0;
                for (int t = 0; t < d; ++t)
                    acc += (double)U[(size_t)j * d + t] * ((double)x[t] - (double)m[t] / (double)N);
                s[j] = acc;
            }
            for (int t = 0; t < d; ++t) {
                double rec = (double)m[t] / (double)N;
                for (int j = 0; j < k; ++j) rec += (double)U[(size_t)j * d + t] * s[j];
                const double r = (double)x[t] - rec;
                total += r * r;
            }
        }
    }
    free(s);
    return total;
}

/* ------------------------------------------------------------------------- */
/* Stochastic scalar quantizer for compressed slices (the paper cites QSGD    */
/* for this and does not define it; this is the definition the library        */
/* documents).  Everything below is fp32 with one rounding per operation and  */
/* no fused multiply-add (build with -ffp-contract=off), because the integer  */
/* levels are compared bit for bit.                                           */
/*                                                                            */
/* Counter-based generator: u = 24 hashed bits of                             */
/* (seed, node, global slice index, coordinate), times 2^-24.                 */
/* ------------------------------------------------------------------------- */
static uint64_t gvqo_mix64(uint64_t z)
{
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ULL;
    z ^= z >> 27; z *= 0x94D049BB133111EBULL;
    z ^= z >> 31;
    return z;
}

/* 24 random bits for (seed, node, slice, coordinate): two rounds of the 64-bit mixer over (seed, node) and
   the slice, then one cheap 32-bit finalizer per coordinate (multiply / xor-shift), top 24 bits. */
uint32_t gvqo_hash24(uint64_t seed, uint32_t node, uint64_t slice, uint32_t coord)
{
    uint64_t h = gvqo_mix64(seed + 0x9E3779B97F4A7C15ULL * ((uint64_t)node + 1ULL));
    h = gvqo_mix64(h ^ (0xD1B54A32D192ED03ULL * (slice + 1ULL)));
    uint32_t x = (uint32_t)(h >> 32) ^ ((uint32_t)h + 0x9E3779B9u * (coord + 1u));
    x ^= x >> 16; x *= 0x7FEB352Du;
    x ^= x >> 15; x *= 0x846CA68Bu;
    x ^= x >> 16;
    return x >> 8;
}

/* One bucket = one compressed slice (k coordinates) of one node.
     sq_j   = v_j * v_j
     total  = pairwise "butterfly" sum over the next power of two kp >= k (padding +0):
              for stride = kp/2, kp/4, ..., 1:  a[j] <- a[j] + a[j xor stride]  (all j at once)
     norm   = sqrt(total)
     scale  = levels / norm ;  r_j = |v_j| * scale ;  lo = floor(r_j) ;  p = r_j - lo
     level  = min(levels, lo + (u < p)) ;  q_j = sign(v_j) * level ;  norm = 0 -> q = 0
   q [count][k] int8, norms [count] fp32.  slice0 = global index of the first slice passed. */
int gvqo_quantize(int k, int64_t count, int64_t slice0, const float *s_node, int levels, uint64_t seed,
                  uint32_t node, int8_t *q, float *norms)
{
    if (k <= 0 || k > 1024 || levels < 1 || levels > 127 || count < 0) return GVQO_ERR_ARG;
    int kp = 1;
    while (kp < k) kp <<= 1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) {
        float a[1024], b[1024];
        const float *v = s_node + (size_t)i * k;
        for (int j = 0; j < kp; ++j) a[j] = (j < k) ? v[j] * v[j] : 0.0f;
        for (int stride = kp / 2; stride >= 1; stride /= 2) {
            for (int j = 0; j < kp; ++j) b[j] = a[j] + a[j ^ stride];
            memcpy(a, b, sizeof(float) * (size_t)kp);
        }
        const float norm = sqrtf(a[0]);
        norms[i] = norm;
        const float scale = (norm > 0.0f) ? (float)levels / norm : 0.0f;   /* once per bucket */
        for (int j = 0; j < k; ++j) {
            int level = 0;
            if (norm > 0.0f) {
                const float r = fabsf(v[j]) * scale;
                const float lo = floorf(r);
                const float p = r - lo;
                const float u = (float)gvqo_hash24(seed, node, (uint64_t)(slice0 + i), (uint32_t)j) * (1.0f / 16777216.0f);
                level = (int)lo + ((u < p) ? 1 : 0);
                if (level > levels) level = levels;
            }
            q[(size_t)i * k + j] = (int8_t)((v[j] < 0.0f) ? -level : level);
        }
    }
    return GVQO_OK;
}

/* "4-bit" packing of signed levels in [-7, 7]: two's-complement nibbles, the even coordinate in the low half of
   the byte.  count levels (even) -> count / 2 bytes; unpack is the inverse. */
int gvqo_pack4(int64_t count, const int8_t *q, uint8_t *packed)
{
    if (count < 0 || (count & 1)) return GVQO_ERR_ARG;
    for (int64_t i = 0; i < count; i += 2) {
        if (q[i] < -7 || q[i] > 7 || q[i + 1] < -7 || q[i + 1] > 7) return GVQO_ERR_ARG;
        packed[i / 2] = (uint8_t)(((uint8_t)q[i] & 0x0F) | (((uint8_t)q[i + 1] & 0x0F) << 4));
    }
    return GVQO_OK;
}

int gvqo_unpack4(int64_t count, const uint8_t *packed, int8_t *q)
{
    if (count < 0 || (count & 1)) return GVQO_ERR_ARG;
    for (int64_t i = 0; i < count; i += 2) {
        const int lo = packed[i / 2] & 0x0F, hi = packed[i / 2] >> 4;
        q[i] = (int8_t)(lo >= 8 ? lo - 16 : lo);
        q[i + 1] = (int8_t)(hi >= 8 ? hi - 16 : hi);
    }
    return GVQO_OK;
}

/* Aggregate of the dequantised vectors:  s_i[j] = sum_n norm_{n,i} * q_{n,i}[j] / levels  (double). */
int gvqo_dequantize_aggregate(int k, int64_t count, int N, const int8_t *const *q_nodes,
                              const float *const *norms_nodes, int levels, double *s_sum)
{
    if (k <= 0 || levels < 1 || N <= 0) return GVQO_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i)
        for (int j = 0; j < k; ++j) {
            double acc = 0.0;
            for (int n = 0; n < N; ++n)
                acc += (double)norms_nodes[n][i] * (double)q_nodes[n][(size_t)i * k + j] / (double)levels;
            s_sum[(size_t)i * k + j] = acc;
        }
    return GVQO_OK;
}

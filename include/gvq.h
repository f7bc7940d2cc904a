/*
 * gvq.h -- C ABI of the GradiVeQ hot path on one B200 (sm_100a).
 *
 * GradiVeQ (arXiv 1811.03617) compresses CNN gradients with a linear PCA
 * compressor that commutes with summation (Eq. 1), so N nodes' compressed
 * gradients are summed directly in the compressed domain and decompressed once.
 *
 * Notation (the paper's symbol in brackets):
 *   d  slice length [K]            k  compressed length [d], 1 <= k <= d
 *   N  nodes                       M  entries of a flat gradient
 *   S  total number of full slices over all layers
 *   L  stored gradients used by a basis fit [L_t]
 *   Ut [n_layers][k][d]  the compressor transposed, row j = j-th eigenvector [U_{d,m}^T]
 *   mu [n_layers][d]     whitening vector of the AGGREGATED gradient [mu_m]
 *
 * Layout of a flat gradient: layer l is layer_len[l] floats at offset
 * layer_off[l] (in floats, a multiple of 4; layers must not overlap).  Its first
 * S_l = layer_len[l] / d runs of d floats are the slices of Section 2; one
 * compressor (Ut_l, mu_l) serves every slice of a layer (the paper's compressor
 * reuse factor s = infinity).  The layer_len[l] % d floats after the last full
 * slice ("tail") are not compressed: they are summed over the nodes as they are.
 * A compressed buffer is [S][k] floats, the layers' slices in layer order.
 *
 * Conventions for every entry point unless stated otherwise:
 *  - "device pointer" = memory of the context's GPU, owned by the caller,
 *    16-byte aligned (else GVQ_ERR_ALIGN); "host pointer" = ordinary host memory.
 *  - Arrays OF pointers (g_nodes, s_nodes, ...) are host arrays of device
 *    pointers; they are read during the call only.  N <= GVQ_MAX_NODES.
 *  - Work is enqueued on the context's stream and the call returns without
 *    waiting (gvq_fit_basis, gvq_fit_basis_static, gvq_refresh_basis and
 *    gvq_allreduce_host are the exceptions: they wait for their result).
 *  - Inputs are never modified, outputs are fully overwritten, and an output
 *    must not alias an input.  Hot calls allocate nothing.
 *  - Errors are return codes; nothing throws, exits or traps.  On a CUDA error
 *    the call returns GVQ_ERR_CUDA and gvq_last_cuda_error() gives the code.
 *  - The library is the only implementation: there is no CPU fallback.
 *  - A context serves one host thread at a time (its calls update per-context caches); different
 *    contexts are independent, except for gvq_fit_basis_static's shared scratch (see there).
 *  - A context's calls are ordered on ONE stream at a time: its scratch (pieces of tiles that two CTAs
 *    share, the fault word, cached tensor maps) is ordered by the stream alone.  gvq_set_stream makes
 *    the new stream wait for what the old one was given, so switching streams is safe; issuing calls
 *    of one context concurrently on two streams is not.
 *  - CUDA graphs: on tensor-core shapes (k 16 or 32, d 64 / 128 / 192 / 256) the first call that sees
 *    a gradient buffer uploads its tensor maps.  That upload cannot be part of a graph, so a call
 *    that meets a NEW buffer while its stream is being captured returns GVQ_ERR_CAPTURE and records
 *    nothing: pass every buffer to one ordinary call first, then capture.  The context caches the maps
 *    of the 2 * GVQ_MAX_NODES most recently used buffers; a captured graph stays valid as long as no
 *    later call brings in so many other buffers that the graph's are evicted (replaying it then reads
 *    another buffer's maps) -- keep the set of buffers of a context within that number, or use one
 *    context per set.
 */
#ifndef GVQ_H
#define GVQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GVQ_MAX_NODES 64
#define GVQ_MAX_D 1024

typedef enum {
    GVQ_OK = 0,
    GVQ_ERR_NULL = 1,          /* a required pointer is NULL */
    GVQ_ERR_SHAPE = 2,         /* a size or count is out of range, or buffers overlap */
    GVQ_ERR_ALIGN = 3,         /* a device pointer or layer offset is not 16-byte aligned */
    GVQ_ERR_UNSUPPORTED = 4,   /* (d, k) has no compiled kernel */
    GVQ_ERR_WORKSPACE = 5,     /* workspace missing or too small */
    GVQ_ERR_CUDA = 6,          /* a CUDA call failed */
    GVQ_ERR_NOT_CONVERGED = 7, /* the eigen-solver hit its sweep limit (outputs are still written) */
    GVQ_ERR_DEGENERATE = 8,    /* a spectrum sums to zero where a ratio of it is needed */
    GVQ_ERR_TIMEOUT = 9,       /* a bounded wait inside a kernel ran out (reported by gvq_device_status) */
    GVQ_ERR_CAPTURE = 10       /* a buffer new to the context was passed while its stream is being captured */
} gvq_status;

/* Host struct, caller-owned, copied by gvq_create. */
typedef struct {
    int32_t d;                /* slice length, multiple of 4, 4 <= d <= GVQ_MAX_D */
    int32_t k;                /* compressed length, 1 <= k <= d */
    int32_t n_layers;         /* >= 1 */
    const int64_t *layer_off; /* [n_layers] offset of layer l in floats, multiple of 4 */
    const int64_t *layer_len; /* [n_layers] entries of layer l, >= 0 */
} gvq_layout;

typedef struct gvq_ctx gvq_ctx;

/* ---- host-only helpers (no CUDA call, usable without a GPU) ---------------------------- */

const char *gvq_status_string(gvq_status s);

/* Validates a layout: ranges, alignment, non-overlap (layers sorted by offset),
   and that (d, k) has a kernel.  */
gvq_status gvq_layout_check(const gvq_layout *layout);

/* S: total number of full slices; -1 on a NULL / invalid layout. */
int64_t gvq_total_slices(const gvq_layout *layout);

/* M: one past the last entry of the last layer; -1 on a NULL / invalid layout. */
int64_t gvq_total_entries(const gvq_layout *layout);

/* Floats of an exchange buffer of Algorithm 1 for this layout: the S * k compressed entries followed by the
   T = sum_l layer_len[l] % d uncompressed tail entries (layer order); -1 on a NULL / invalid layout. */
int64_t gvq_exchange_floats(const gvq_layout *layout);

/* Algorithm 1, "partitions its g_n into N equal segments, each containing several gradient slices": the part of
   a layout that segment j of n_segments covers.  Segment j holds the global slices [floor(j S / G),
   floor((j + 1) S / G)), G = n_segments, counted through the layers in order; a layer cut by a boundary gives a
   piece to both segments; the tail of a layer (and a layer shorter than a slice) goes with the slice just before
   it in that order (segment 0 if there is none).  Outputs (host arrays of n_layers elements, the first *n_pieces
   written; *n_pieces = 0 for an empty segment): piece p is piece_len[p] floats at offset piece_off[p] of a flat
   gradient and lies in layer piece_layer[p] (increasing).  {d, k, *n_pieces, piece_off, piece_len} is itself a
   layout: a context made from it runs the segment, given the rows piece_layer[] of Ut and mu. */
gvq_status gvq_segment_layout(const gvq_layout *layout, int n_segments, int j, int32_t *n_pieces,
                              int32_t *piece_layer, int64_t *piece_off, int64_t *piece_len);

/* Bytes of device scratch gvq_fit_basis needs for L stored gradients (0 on an invalid layout). */
size_t gvq_fit_workspace_bytes(const gvq_layout *layout, int L);

/* Bytes of device scratch gvq_allreduce_host needs for N nodes (0 on an invalid layout). */
size_t gvq_host_workspace_bytes(const gvq_layout *layout, int N);

/* How the tensor-core kernels split their work over n_parts CTAs (host-only; for inspection and tests; the
   paper has no counterpart).  kind 0: the projection, whose units are (tile of 128 slices, node), n_nodes per
   tile; kind 1: the decompression, whose units are (tile, block of 128 output columns).  Units are numbered tile
   by tile, tiles layer by layer; part b works on units [start[b], start[b+1]).  The split minimises the largest
   cost of a part under a model that charges a part for every layer it touches (the kernels drain their pipeline
   and stage the layer's basis there).  start: HOST array [n_parts + 1]; *n_units_out: total units. */
gvq_status gvq_work_partition(const gvq_layout *layout, int kind, int n_nodes, int n_parts, int32_t *start,
                              int64_t *n_units_out);

/* Eq. 6 (Section 3, "Compressor dimension"): the smallest k with
   (sum of the k largest eigenvalues) / (sum of all d) >= 1 - lambda_loss.
   evals: HOST pointer, d values sorted descending (one layer's row of gvq_fit_basis' evals).
   Writes k to *k_out.  GVQ_ERR_DEGENERATE (and *k_out = 1) when the spectrum sums to <= 0. */
gvq_status gvq_select_k(const float *evals, int d, double lambda_loss, int32_t *k_out);

/* ---- context --------------------------------------------------------------------------- */

/* Creates a context for one layout on `device`; `cuda_stream` is a cudaStream_t (NULL =
   the legacy default stream).  Allocates the context's device memory once: tile -> layer maps,
   room for the TMA descriptors of up to 128 gradient buffers and of one history buffer, two
   partial tiles per SM and a counter per tile for the tensor-core projection.  These are the
   only device allocations the library makes, apart from what gvq_host_prepare adds when asked
   (on the host, the first call with a new node count keeps that count's work split: a few
   hundred integers). */
gvq_status gvq_create(gvq_ctx **out, const gvq_layout *layout, int device, void *cuda_stream);
gvq_status gvq_destroy(gvq_ctx *ctx);
/* The stream the context's later calls are enqueued on.  When it differs from the current one, the new stream is
   first made to wait (an event) for everything the old one was given by this context -- unless one of the two is
   being captured, when no dependency can be added: start a capture only after the context's earlier work on other
   streams has been waited for. */
gvq_status gvq_set_stream(gvq_ctx *ctx, void *cuda_stream);

/* Hands the context a device scratch buffer (256-byte aligned) that gvq_fit_basis and
   gvq_allreduce_host use; the caller keeps ownership and must keep it alive while such a
   call is in flight.  (ptr = NULL, bytes = 0) takes it away again. */
gvq_status gvq_set_workspace(gvq_ctx *ctx, void *device_ptr, size_t bytes);

/* The cudaError_t of the last failed CUDA call made through this context (0 if none). */
int gvq_last_cuda_error(const gvq_ctx *ctx);

/* Which kernels compute Eq. 3 / Eq. 4 and Eq. 5:  0 = automatic (default), 1 = the FP32-pipe
   kernels, 2 = the tensor-core kernels (split TF32; GVQ_ERR_UNSUPPORTED unless k is 16 or 32
   and d is 64, 128, 192 or 256).  Automatic picks the tensor cores where they exist.  Both
   meet the same tolerance; this exists for tests and measurements. */
gvq_status gvq_set_projection_path(gvq_ctx *ctx, int path);

/* How gvq_fit_basis gets its eigenpairs:  1 = the Jacobi eigen-solver works on the covariance and accumulates its
   rotations (every eigenvector, however small its eigenvalue);  2 = the solver works on the Cholesky factor of the
   covariance (+ a small ridge) without accumulating rotations (eigenvalues only: the squared column norms it
   converges to; half the shared memory, so twice as many layers fit the GPU at once) and the k leading eigenvectors
   come from two rounds of subspace iteration started at the solver's k longest columns (d <= 256, k <= 32, else
   GVQ_ERR_UNSUPPORTED);  0 (default) = 2 wherever it is supported (it is the faster one: only the k leading
   eigenvectors are ever used), else 1.  Both meet the same tolerances: every eigenvalue to 1e-5 of the largest,
   orthonormality, the subspace of the k leading eigenvectors. */
gvq_status gvq_set_fit_path(gvq_ctx *ctx, int path);

/* Waits for the context's stream and reports whether a kernel recorded a fault since the last
   call: the tensor-core kernel bounds every wait on its internal barriers and, should one run
   out, gives up cleanly and sets a device word (GVQ_ERR_TIMEOUT; its outputs are then invalid).
   The word is cleared by the call (and by a fit entry point that returns GVQ_ERR_TIMEOUT). */
gvq_status gvq_device_status(gvq_ctx *ctx);

/* ---- testing hooks (the paper has no counterpart; off by default) ------------------------------------
   gvq_set_limits: max_sweeps > 0 replaces the sweep limit of the eigen-solvers of gvq_fit_basis (30), so that a
   test can see GVQ_ERR_NOT_CONVERGED with its outputs still written; wait_cycles > 0 replaces the limit of every
   bounded wait inside the tensor-core kernels (about 4e9 SM clocks, ~2 s), rounded up to a multiple of 1024.
   0 restores a default.
   gvq_test_drop_load(on != 0): the next tensor-core kernels each leave out one hand-over in their first CTA -- the
   projection the very last load of its run, the decompression the hand-over of its first tile to the tensor core,
   the covariance kernel of a fit its first load -- so that the wait for it runs out: the kernel returns, its
   outputs are invalid, gvq_device_status (or the fit entry point) reports GVQ_ERR_TIMEOUT.  Nothing faults or
   hangs: every wait in those kernels is bounded.  Use it with a short wait_cycles. */
gvq_status gvq_set_limits(gvq_ctx *ctx, int max_sweeps, int64_t wait_cycles);
gvq_status gvq_test_drop_load(gvq_ctx *ctx, int on);

/* ---- the hot path ---------------------------------------------------------------------- */

/* Eq. 3:  s_{n,i} = Ut (x_{n,i} - mu / N)  for every slice i of ONE node's gradient.
   g_node: device [M]; Ut, mu: device; N: the number of nodes the aggregate will have (it
   scales the mean and must equal the N later given to gvq_decompress); s_node: device [S][k]. */
gvq_status gvq_compress(gvq_ctx *ctx, const float *g_node, const float *Ut, const float *mu, int N,
                        float *s_node);

/* Eq. 4, left-hand side:  s_i = sum_{n<N} s_{n,i}  (fp32, n ascending).
   s_nodes: host array of N device pointers [S][k]; s_sum: device [S][k]. */
gvq_status gvq_aggregate(gvq_ctx *ctx, const float *const *s_nodes, int N, float *s_sum);

/* Eq. 3 fused with Eq. 4: each node's raw gradient is read once and the N compressed
   vectors of a slice are summed on chip;  s_sum_i = sum_n Ut (x_{n,i} - mu / N).
   Every node's projection is computed (N * S * d * k multiply-adds); the raw gradients are
   never summed first.  g_nodes: host array of N device pointers [M]; s_sum: device [S][k];
   s_nodes_opt: NULL, or a host array of N device pointers [S][k] that also receive each
   node's own s_n (needed when the compressed vectors are quantized before summation). */
gvq_status gvq_compress_aggregate(gvq_ctx *ctx, const float *const *g_nodes, int N, const float *Ut,
                                  const float *mu, float *s_sum, float *const *s_nodes_opt);

/* Eq. 5:  g_hat_i = U s_i + mu  for every slice, fused with the mean add; and the
   uncompressed tails:  g_hat_tail = sum_{n<N} g_{n,tail}  (fp32, n ascending).
   s_sum: device [S][k]; g_nodes_for_tails: host array of N device pointers [M], may be NULL
   when no layer has a tail; g_hat: device [M] -- entries outside every layer are not written. */
gvq_status gvq_decompress(gvq_ctx *ctx, const float *s_sum, const float *Ut, const float *mu,
                          const float *const *g_nodes_for_tails, int N, float *g_hat);

/* ---- Algorithm 1: one node's share of the ring ------------------------------------------ */

/* A node's compressed segment, ready to send (Algorithm 1: "compresses g_n(j) to g'_n(j) as in Eq. 3"):
     x[0 .. S k)           = sum over the n_local local nodes of Ut (x_{n,i} - mu / N)
     x[S k .. S k + T)     = sum over the local nodes of the layers' uncompressed tails (layer order)
   for the layout of the context, which is normally one segment (gvq_segment_layout).  N = nodes of the whole job
   (>= n_local; it scales the mean), n_local = gradients held here (1 in the paper's setting; more when one GPU
   stands for several nodes).  The sum of all participants' x over the job is what gvq_compress_aggregate would
   give on all N gradients, up to the fp32 summation order.  x: device, gvq_exchange_floats() floats. */
gvq_status gvq_compress_aggregate_partial(gvq_ctx *ctx, const float *const *g_nodes, int n_local, int N,
                                          const float *Ut, const float *mu, float *x);

/* Algorithm 1, "adds g'_n(j) to g'(j)":  x_acc += x_in  over a whole exchange buffer (compressed part and
   tails).  Both device, gvq_exchange_floats() floats, distinct. */
gvq_status gvq_exchange_accumulate(gvq_ctx *ctx, float *x_acc, const float *x_in);

/* Algorithm 1, "decompresses g'(j) into g''(j)": Eq. 5 on the compressed part of a completely aggregated
   exchange buffer, and its tail entries copied to their places.  g_hat: device [M], written inside the layout's
   layers only. */
gvq_status gvq_decompress_exchanged(gvq_ctx *ctx, const float *x, const float *Ut, const float *mu, float *g_hat);

/* Basis refresh (Section 2, the PCA paragraph): for every layer, the mean and covariance
   (1/n normalisation) of its n = L * S_l sample slices, the symmetric eigendecomposition of
   the covariance (parallel-ordered Jacobi rotations, fp32), eigenvalues sorted descending
   (equal values: lower index first), the first k eigenvectors with their largest-magnitude
   entry made positive.
   hist: device, L stored gradients laid out like flat gradients, hist_stride floats apart
   (multiple of 4).  samples_are_sums_of = c: each stored gradient is the sum of c nodes'
   gradients (c = N for the paper's aggregated samples, 1 for single-node samples);
   mu = (N / c) * sample mean, i.e. always the mean of an N-node aggregate.
   Outputs (device): Ut [n_layers][k][d], mu [n_layers][d], evals [n_layers][d].
   info: HOST pointer [n_layers] or NULL, receives the sweeps each layer used.
   A layer without a full slice gets Ut = the first k unit vectors, mu = 0, evals = 0.
   Needs the workspace (gvq_fit_workspace_bytes).  Synchronises the stream once, to read the
   convergence word; returns GVQ_ERR_NOT_CONVERGED if any layer hit the sweep limit (the outputs
   are written all the same: the solver's state at the limit), and GVQ_ERR_TIMEOUT if a bounded
   wait inside the tensor-core covariance kernel (d = 64, 128, 192, 256) ran out (the fault word
   is cleared before the call returns; the outputs are invalid). */
gvq_status gvq_fit_basis(gvq_ctx *ctx, const float *hist, int64_t hist_stride, int L, int N,
                         int samples_are_sums_of, float *Ut, float *mu, float *evals, int32_t *info);

/* ---- a basis fit whose stored gradients are spread over several participants (Section 2: every node computes
   the covariance of the samples; with the samples sharded over GPUs the covariance is assembled from additive
   moments).  All participants centre by ONE point m per layer (gvq_fit_centre on one participant, broadcast):
     moments[l] = { n_l,  sum_i (x_i - m_l),  sum_i (x_i - m_l)(x_i - m_l)^T }      (fp64, 1 + d + d * d numbers)
   over the participant's own L stored gradients; the element-wise SUM of all participants' moments (one all-reduce)
   goes to gvq_fit_from_moments, which forms  C = S2 / n - delta delta^T,  mean = m + delta  (delta = sum (x - m) / n)
   and continues exactly as gvq_fit_basis does after its covariance (same outputs, same return codes; it
   synchronises the stream once).  The result does not depend on how the samples were split, up to fp64 rounding
   of the sums.  centre: device [n_layers][d]; moments: device double [gvq_fit_moments_count()]; both calls that
   read the history need the workspace of gvq_fit_basis.  gvq_fit_centre: the mean of up to 256 slices spread over
   each layer, in the first and the last of the L stored gradients (any point near the mean serves). */
int64_t gvq_fit_moments_count(const gvq_layout *layout);
gvq_status gvq_fit_centre(gvq_ctx *ctx, const float *hist, int64_t hist_stride, int L, float *centre);
gvq_status gvq_fit_moments(gvq_ctx *ctx, const float *hist, int64_t hist_stride, int L, const float *centre,
                           double *moments);
gvq_status gvq_fit_from_moments(gvq_ctx *ctx, const double *moments, const float *centre, int N,
                                int samples_are_sums_of, float *Ut, float *mu, float *evals, int32_t *info);

/* gvq_fit_basis for callers that have no device workspace to hand over and may not allocate one
   (the paper has no counterpart: this is an addition of this library).  Such callers exist: code
   hosted inside an application whose own allocator has already claimed the device's memory, or
   whose rules forbid cudaMalloc / cudaFree on the training thread because those calls can
   synchronise the whole device.  The entry point computes exactly what gvq_fit_basis computes
   (same arguments, same outputs, same return codes) but takes its scratch from a fixed array of
   GVQ_STATIC_FIT_BYTES that is part of the library image, so every GPU that loads the library
   holds that much memory until the process exits.  It calls no cudaMalloc, no cudaFree and no
   allocating library routine, and ignores the context's workspace.
   Limits and rules:
    - a layout whose fit needs more than GVQ_STATIC_FIT_BYTES of scratch
      (gvq_fit_workspace_bytes tells) is refused with GVQ_ERR_WORKSPACE;
    - the first call on a device looks up the array's device address (one cudaGetSymbolAddress);
      make that first call before any stream capture begins;
    - all calls on a device share the one array and it keeps the last call's contents; the entry
      point clears what must start at zero itself, but two calls that overlap on the GPU (two
      contexts or two streams) race on it -- serialise them;
    - like gvq_fit_basis it synchronises the stream once before returning. */
#define GVQ_STATIC_FIT_BYTES (4u << 20)
gvq_status gvq_fit_basis_static(gvq_ctx *ctx, const float *hist, int64_t hist_stride, int L, int N,
                                int samples_are_sums_of, float *Ut, float *mu, float *evals, int32_t *info);

/* gvq_compress_aggregate with the monitor of Eq. 7 (Section 3, "Number of compressed iterations"): besides
   s_sum (and the optional s_n) the call returns, for every layer l and node n, over the layer's full slices,
     monitor[l][0][n] = sum_i || x_{n,i} - mu_l / N ||^2          (energy of the centred slices)
     monitor[l][1][n] = sum_i || s_{n,i} ||^2                     (energy the basis captures)
   Eq. 7's local compression loss || g_n - (U s_n + mu / N) ||^2 of node n on layer l is their difference: for
   a basis with orthonormal columns the residual of the projection is orthogonal to it.  The caller compares
   loss / energy with its threshold and counts the nodes above it (the paper stops compressing when the
   majority is).  fp32 partial sums, fp64 totals; absolute accuracy about 1e-5 of the energy (the loss is a
   difference).  On tensor-core shapes (k 16 or 32, d 64 / 128 / 192 / 256) the sums are formed inside the
   projection kernel at no extra memory traffic; on other shapes s_nodes_opt must be given (GVQ_ERR_UNSUPPORTED
   otherwise) and a second kernel reads g_n and s_n again.
   monitor: device double [n_layers][2][N], overwritten.  Other arguments as gvq_compress_aggregate. */
gvq_status gvq_compress_aggregate_monitored(gvq_ctx *ctx, const float *const *g_nodes, int N, const float *Ut,
                                            const float *mu, float *s_sum, float *const *s_nodes_opt, double *monitor);

/* The quantizer of gvq_quantize applied to RAW gradient slices, 4 bits per entry -- what a node sends in the
   iterations that aggregate without the PCA compressor (Section 3: those iterations use a scalar quantizer such as
   QSGD; the experiments use its 4-bit form).  Bucket = one full slice (d entries) of one node; (q, norm) exactly as
   gvq_quantize defines them with k := d (butterfly over the next power of two >= d) and the slice's global index
   (its row in a compressed buffer) as the counter i of hash24(seed, node, i, j); levels in [1, 7]; the signed
   levels are packed two per byte, two's-complement nibbles, entry 2b in the low half of byte b.  The uncompressed
   tails are not quantized.  g_node: device [M]; q4: device bytes [S][d / 2]; norms: device [S]. */
gvq_status gvq_quantize_raw4(gvq_ctx *ctx, const float *g_node, int levels, uint64_t seed, uint32_t node, uint8_t *q4,
                             float *norms);

/* The aggregate of N nodes' quantized gradients, i.e. the sample the basis fit stores in those iterations:
   full slices: g_sum = sum_{n<N} q_n * (norm_n / levels)  (fp32, one rounding per operation, n ascending);
   tails: the plain sum of the raw tails (g_nodes_for_tails, may be NULL when the layout has none).
   q4_nodes / norms_nodes / g_nodes_for_tails: host arrays of N device pointers; g_sum: device [M], entries outside
   every layer are not written. */
gvq_status gvq_dequantize_raw4_aggregate(gvq_ctx *ctx, const uint8_t *const *q4_nodes, const float *const *norms_nodes,
                                         const float *const *g_nodes_for_tails, int levels, int N, float *g_sum);

/* gvq_quantize_raw4 for all N nodes and gvq_dequantize_raw4_aggregate in ONE launch (plus the tails): every node's
   gradient is read once and g_sum written once; bit-identical to the N + 1 separate calls.  q4_nodes_opt /
   norms_nodes_opt: NULL, or host arrays of N device pointers that receive what each node would send. */
gvq_status gvq_quantize_raw4_aggregate(gvq_ctx *ctx, const float *const *g_nodes, int N, int levels, uint64_t seed,
                                       float *g_sum, uint8_t *const *q4_nodes_opt, float *const *norms_nodes_opt);

/* The flatten order of one convolutional layer (Section 2, figure on flattening and slicing): the F gradients of one
   position next to each other, positions visited depth first, then width, then height, so that d = a multiple of
   F * D entries is a natural slice.  Against the framework's layout [F][D][H][W] (x = h * W + w, X = H * W):
       flat[(x * D + dep) * F + f] = framework[(f * D + dep) * X + x].
   gvq_flatten_layer writes `flat` (X * D * F floats) from `framework`; gvq_unflatten_layer is the inverse (to hand
   the aggregate back).  Device pointers, not aliased; launched on the context's stream.  These are separate
   passes over the layer (read + write), not part of the timed path: a framework that can emit the gradient in
   channels-last order needs neither. */
gvq_status gvq_flatten_layer(gvq_ctx *ctx, const float *framework, float *flat, int F, int D, int X);
gvq_status gvq_unflatten_layer(gvq_ctx *ctx, const float *flat, float *framework, int F, int D, int X);

/* A cheaper refresh than gvq_fit_basis, for slices too long for a full eigendecomposition every time (Section 3
   notes that the cost of the "SVD" grows with the slice size) and for bases that move slowly (Section 1, "time
   domain invariance"): mean and covariance as in gvq_fit_basis, then only the k leading eigenpairs, by `iters`
   rounds of subspace iteration (multiply the k x d iterate by the covariance, orthonormalise) and a Rayleigh-Ritz
   step.  warm_start != 0: the iteration starts from the rows of Ut (the previous basis; any k x d matrix of full
   rank); 0: from a fixed pseudo-random matrix.  The error of the subspace shrinks by lambda_{k+1} / lambda_k per
   round: a handful of rounds when the spectrum has a gap after k, many when it has none -- the caller chooses.
   Outputs: Ut [n_layers][k][d] (same order, sign and normalisation rules as gvq_fit_basis), mu [n_layers][d],
   evals_k [n_layers][k] descending, trace [n_layers] = the sum of all d eigenvalues (Eq. 6's denominator).
   d <= 256, k <= 32, k d + 3 k^2 <= d^2 (GVQ_ERR_UNSUPPORTED otherwise); workspace as gvq_fit_basis; synchronises. */
gvq_status gvq_refresh_basis(gvq_ctx *ctx, const float *hist, int64_t hist_stride, int L, int N, int samples_are_sums_of,
                             int warm_start, int iters, float *Ut, float *mu, float *evals_k, float *trace);

/* Per-layer compressed length (Eq. 6 gives each layer its own minimum k_l for a loss threshold; the buffers of
   this library have one k): rows k_l .. k-1 of layer l's basis are set to zero, so coordinates k_l .. k-1 of every
   compressed vector of that layer are exactly 0 and Eq. 3 - Eq. 5 compute what a basis of k_l columns would.
   k_per_layer: HOST array [n_layers], 0 <= k_l <= k.  Ut: device, modified in place (stream-ordered). */
gvq_status gvq_mask_basis(gvq_ctx *ctx, float *Ut, const int32_t *k_per_layer);

/* What crosses a link when every layer has its own compressed length (Eq. 6 layer by layer): with the basis masked
   by gvq_mask_basis the coordinates k_l .. k - 1 of layer l's compressed vectors are exact zeros, and an exchange
   buffer (gvq_exchange_floats: S * k + T floats) carries sum_l S_l * k_l + T numbers that matter.
   gvq_set_layer_k tells the context the lengths (HOST array [n_layers], 0 <= k_l <= k; NULL = all k again) -- it
   uploads two small tables, so call it outside a stream capture; gvq_packed_floats is that count (host only; -1 on
   bad arguments); gvq_exchange_pack copies an exchange buffer x into the packed form x_packed (layer after layer,
   k_l floats per slice, then the T tail entries), gvq_exchange_unpack is the inverse, with zeros in the dropped
   places.  Sums commute with the packing, so a collective may run on packed buffers:
     mask -> compress (partial) -> pack -> all-reduce of gvq_packed_floats() floats -> unpack -> decompress.
   Device pointers, not aliased.  The kernels of Eq. 3 / Eq. 5 still work k wide: they are bound by the raw
   gradient's bytes, which do not depend on k; the saving is in the bytes exchanged. */
int64_t gvq_packed_floats(const gvq_layout *layout, const int32_t *k_per_layer);
gvq_status gvq_set_layer_k(gvq_ctx *ctx, const int32_t *k_per_layer);
gvq_status gvq_exchange_pack(gvq_ctx *ctx, const float *x, float *x_packed);
gvq_status gvq_exchange_unpack(gvq_ctx *ctx, const float *x_packed, float *x);

/* ---- when to collect samples, refit and compress (Section 3, "Parameter selection") -------------------
   The paper's iteration plan: L_t iterations with uncompressed aggregation, whose aggregated gradients are the
   PCA samples; one fit; then compressed iterations, at most L_c of them, ended early when the majority of the
   nodes see a local compression loss (Eq. 7) above a threshold.  This is a host-side state machine without any
   device work: the training loop calls gvq_schedule_step once after every iteration and does what it returns.
   loss_threshold is relative: a node is "over" when sum_l loss > loss_threshold * sum_l energy, both from the
   monitor array of gvq_compress_aggregate_monitored copied to the host. */
typedef struct gvq_schedule gvq_schedule;
enum { GVQ_PHASE_COLLECT = 0, GVQ_PHASE_COMPRESS = 1 };
enum {
    GVQ_ACT_NONE = 0,    /* carry on in the current phase */
    GVQ_ACT_FIT = 1,     /* L_t samples are stored: call gvq_fit_basis on them; compressed iterations follow */
    GVQ_ACT_RESTART = 2  /* stop compressing: the next L_t iterations aggregate uncompressed and store samples */
};
gvq_status gvq_schedule_create(gvq_schedule **out, int L_t, int L_c, int n_nodes, double loss_threshold);
gvq_status gvq_schedule_destroy(gvq_schedule *s);
/* Phase of the NEXT iteration. */
int gvq_schedule_phase(const gvq_schedule *s);
/* Call after every iteration.  monitor_host: NULL (no loss check this iteration; always NULL in the collect
   phase), or HOST double [n_layers][2][n_nodes] as gvq_compress_aggregate_monitored lays it out. */
gvq_status gvq_schedule_step(gvq_schedule *s, const double *monitor_host, int n_layers, int *action);
/* Nodes over the threshold at the last monitored step. */
int gvq_schedule_nodes_over(const gvq_schedule *s);
gvq_status gvq_schedule_counters(const gvq_schedule *s, int64_t *iteration, int64_t *refreshes, int64_t *early_stops);

/* Stochastic scalar quantizer applied to ONE node's compressed vectors (the paper cites
   QSGD for this step and does not define it; this header is the definition).  One bucket =
   one compressed slice v = s_{n,i} (k floats).  All arithmetic is fp32, one rounding per
   operation, no fused multiply-add:
     sq_j  = v_j * v_j
     total = butterfly sum over kp = next power of two >= k (padding +0):
             for stride = kp/2, ..., 1:  a[j] <- a[j] + a[j xor stride]   (all j at once)
     norm  = sqrt(total)
     scale = levels / norm                                    (one division per bucket)
     r_j   = |v_j| * scale ;  lo = floor(r_j) ;  p = r_j - lo
     u     = hash24(seed, node, i, j) * 2^-24                (i = global slice index)
     level = min(levels, lo + (u < p)) ;  q_j = sign(v_j) * level ;  norm == 0 -> q = 0
   hash24: with mix(z) = { z ^= z >> 30; z *= 0xBF58476D1CE4E5B9; z ^= z >> 27;
                           z *= 0x94D049BB133111EB; z ^= z >> 31; } on 64-bit words,
     h = mix(seed + 0x9E3779B97F4A7C15 * (node + 1));   h = mix(h ^ (0xD1B54A32D192ED03 * (i + 1)));
   and then on 32-bit words, per coordinate,
     x = (h >> 32) ^ (low32(h) + 0x9E3779B9 * (j + 1));
     x ^= x >> 16; x *= 0x7FEB352D; x ^= x >> 15; x *= 0x846CA68B; x ^= x >> 16;   hash24 = x >> 8.
   levels in [1, 127] ("4-bit" = sign + 3 magnitude bits = 7).  k <= 32 here.
   s_node: device [S][k]; q: device int8 [S][k]; norms: device [S]. */
gvq_status gvq_quantize(gvq_ctx *ctx, const float *s_node, int levels, uint64_t seed, uint32_t node,
                        int8_t *q, float *norms);

/* Aggregate of the dequantised vectors:  s_i[j] = sum_{n<N} q_{n,i}[j] * (norm_{n,i} / levels)
   (fp32, one rounding per operation: the step norm / levels once per bucket, then the product, then the sum;
   n ascending).  q_nodes / norms_nodes: host arrays of N device pointers. */
gvq_status gvq_dequantize_aggregate(gvq_ctx *ctx, const int8_t *const *q_nodes,
                                    const float *const *norms_nodes, int levels, int N, float *s_sum);

/* gvq_quantize for all N nodes and gvq_dequantize_aggregate in ONE launch:
     s_sum_i = sum_{n<N} q_{n,i} * (norm_{n,i} / levels),   (q, norm) = gvq_quantize(s_{n,i}, node n)
   (fp32, n ascending; bit-identical to the N + 1 separate calls).  s_nodes: host array of N device pointers
   [S][k] (e.g. the s_nodes_opt outputs of gvq_compress_aggregate); q_nodes_opt / norms_nodes_opt: NULL, or
   host arrays of N device pointers that receive what each node would transmit.  k <= 32. */
gvq_status gvq_quantize_aggregate(gvq_ctx *ctx, const float *const *s_nodes, int N, int levels, uint64_t seed,
                                  float *s_sum, int8_t *const *q_nodes_opt, float *const *norms_nodes_opt);

/* Eq. 3, the quantizer and the sum in one pass over the raw gradients (tensor-core shapes only: k 16 or 32,
   d 64 / 128 / 192 / 256; GVQ_ERR_UNSUPPORTED otherwise -- use the three separate calls then).  For every node n
   and slice i: s_{n,i} by Eq. 3, then (q, norm) exactly as gvq_quantize defines them with node index n, and
     s_sum_i = sum_{n<N} q_{n,i} * (norm_{n,i} / levels)        (the aggregate of the dequantised vectors).
   The per-node compressed vectors never leave the chip (no N * S * k scratch).  q_nodes_opt / norms_nodes_opt: NULL, or host arrays
   of N device pointers (int8 [S][k], fp32 [S]) that receive what each node would transmit; their contents are
   bit-identical to gvq_quantize applied to the s_n this library computes (s_nodes_opt of
   gvq_compress_aggregate).  g_nodes: host array of N device pointers [M]; s_sum: device [S][k]. */
gvq_status gvq_compress_quantize_aggregate(gvq_ctx *ctx, const float *const *g_nodes, int N, const float *Ut,
                                           const float *mu, int levels, uint64_t seed, float *s_sum,
                                           int8_t *const *q_nodes_opt, float *const *norms_nodes_opt);

/* The whole path for callers whose gradients live in HOST memory (Eq. 3 + Eq. 4 + Eq. 5):
   copies the N gradients to the device scratch, runs gvq_compress_aggregate and
   gvq_decompress there, copies g_hat back and waits for it.
   g_nodes_host: host array of N HOST pointers [M] (pinned memory makes the copies fast);
   Ut, mu: device; g_hat_host: HOST [M].  Needs the workspace (gvq_host_workspace_bytes).
   After gvq_host_prepare a gradient of more than 16 M entries is worked through in 8 chunks of slices, so that
   a chunk's part of g_hat travels back while the next chunk's inputs arrive; without it the whole gradient goes
   in one piece.  The call itself allocates nothing.  Values as from the device calls, up to the fp32 order of the
   sum over nodes inside a tile. */
gvq_status gvq_allreduce_host(gvq_ctx *ctx, const float *const *g_nodes_host, int N, const float *Ut,
                              const float *mu, float *g_hat_host);

/* The same with every node's compressed vectors quantized before the sum (gvq_compress_quantize_aggregate in
   place of gvq_compress_aggregate; tensor-core shapes only, GVQ_ERR_UNSUPPORTED otherwise).  The quantizer's
   counter of a slice is its index in the whole layout, in chunks too, so the result does not depend on whether
   gvq_host_prepare was called. */
gvq_status gvq_allreduce_host_quantized(gvq_ctx *ctx, const float *const *g_nodes_host, int N, const float *Ut,
                                        const float *mu, int levels, uint64_t seed, float *g_hat_host);

/* Creates, once, what the chunked form of gvq_allreduce_host needs for this context's layout (a context per
   chunk, two copy streams, events; kept until gvq_destroy) -- the only device allocations outside gvq_create.
   Does nothing for gradients of at most 16 M entries and for layouts whose chunks would not be runs of consecutive
   layers.  Call it outside the training loop. */
gvq_status gvq_host_prepare(gvq_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* GVQ_H */

// Internal declarations shared by the translation units of libgvq.so.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <vector>

#include "gvq.h"

namespace gvq {

// A tiling of all layers' slices into runs of at most `rows` slices of ONE layer.
// Device arrays; tile t covers slices [row0, row0 + min(rows, S_layer - row0)) of layer `layer`.
struct TileTable {
    int rows = 0;
    int n_tiles = 0;
    int32_t *layer = nullptr;  // [n_tiles]
    int32_t *row0 = nullptr;   // [n_tiles]
    int32_t *layer_first = nullptr;  // [n_layers + 1] first tile of each layer (tiles are in layer order)
    // host copies (owned by the context) for the work partitions computed on the host
    const int32_t *host_layer = nullptr;   // [n_tiles]
    const int32_t *host_count = nullptr;   // [n_tiles] slices in the tile (<= rows)
};

// Splits the sequence of work units -- per_tile units for every tile, tiles in order -- into n_parts contiguous
// runs of about equal cost.  A unit of tile t costs max(count_t / rows, min_unit_cost); a run pays stage_cost
// (in units) whenever it starts work on another layer than the one before, its first included: what the
// tensor-core kernels pay to drain their pipeline and stage a layer's basis.  start: [n_parts + 1] unit indices.
void partition_units(const TileTable &tiles, int per_tile, int n_parts, float stage_cost, float min_unit_cost,
                     int32_t *start);
constexpr int kMaxPartitionCtas = 192;
// Cost model of the tensor-core projection, in units of one full (tile, node) unit: a change of layer (pipeline
// drained, basis staged) and the floor under the cost of a tile with few slices (its 128 rows are still processed, in about the time a full tile takes to arrive).
// The decompression's unit is a (tile, 128-column block); measured on the ResNet-50 shape: 0 / 2 / 4 / 6 -> 37 / 29 / 25 / 25 us.
constexpr float kDecompressTcStageCost = 4.0f, kDecompressTcMinUnitCost = 1.0f;
constexpr float kProjectTcStageCost = 2.0f, kProjectTcMinUnitCost = 1.0f;   // measured: 0 / 0.8 / 2.0 / 3.0 -> 274 / 266 / 262 / 263 us

// Per-layer device tables.
struct LayerTables {
    int64_t *off = nullptr;   // [n_layers] offset of the layer in a flat gradient (floats)
    int64_t *soff = nullptr;  // [n_layers] index of the layer's first slice in a compressed buffer
    int32_t *S = nullptr;     // [n_layers] full slices
    // layers that have an uncompressed tail
    int n_tails = 0;
    int64_t *tail_off = nullptr;  // [n_tails] offset of the tail in a flat gradient
    int32_t *tail_len = nullptr;  // [n_tails] < d
    int64_t *tail_pos = nullptr;  // [n_tails] offset of the tail in the tail part of an exchange buffer
};

// Node pointers travel to the kernels by value.
template <typename T>
struct NodePtrs {
    T *p[GVQ_MAX_NODES];
};

constexpr int kProjectRows = 256;     // slices per tile of the FP32-pipe projection kernel
constexpr int kProjectTcRows = 128;   // slices per tile of the tensor-core projection kernel
constexpr int kDecompressRows = 64;   // slices per tile of the decompression kernel
constexpr int kFitRows = 512;         // slices (per stored gradient) per tile of the covariance kernels
constexpr int kJacobiMaxSweeps = 30;

// ---- launchers (each returns the cudaError_t of its launch) ---------------------------------

// Eq. 3 (+ Eq. 4 when n_nodes > 1): s_sum = sum_n Ut (x_n - mu / mean_div); optional per-node outputs.
cudaError_t launch_project_sum(cudaStream_t st, int num_sms, int d, int k, const TileTable &tiles,
                               const LayerTables &lt, const NodePtrs<const float> &g, int n_nodes,
                               int mean_div, const float *Ut, const float *mu, float *s_sum,
                               const NodePtrs<float> *s_nodes);
size_t project_sum_smem_bytes(int d, int k);
// The same on the tensor cores (split TF32); only for the (d, k) project_sum_tc_supported accepts.
// error_word: device int32, set non-zero if a bounded wait inside the kernel ran out.
bool project_sum_tc_supported(int d, int k);
// Optional quantizing step inside the tensor-core projection (levels, seed as gvq_quantize; outputs may be null).
struct TcQuant {
    int levels;
    uint64_t seed;
    const NodePtrs<int8_t> *q_nodes;
    const NodePtrs<float> *norms;
};
cudaError_t launch_project_sum_tc(cudaStream_t st, int num_sms, int d, int k, const TileTable &tiles,
                                  const LayerTables &lt, const NodePtrs<const float> &g, int n_nodes, int mean_div,
                                  const float *Ut, const float *mu, float *s_sum, int32_t *error_word,
                                  const CUtensorMap *tmaps, int n_layers, const int *slots,
                                  const NodePtrs<float> *s_nodes, float *partial, int32_t *tile_counter,
                                  const int32_t *unit_start, int n_ctas, const TcQuant *quant = nullptr,
                                  double *monitor = nullptr, int wait_kcycles = 0, int drop_last_load = 0,
                                  int64_t slice_base = 0);
size_t project_sum_tc_smem_bytes(int d, int k);
size_t project_sum_tc_partial_bytes(int num_sms, int k);

// Eq. 4 on materialised buffers.
cudaError_t launch_aggregate(cudaStream_t st, int num_sms, const NodePtrs<const float> &s, int n_nodes,
                             int64_t count, float *out);

// Eq. 5 fused with the mean add, and the raw tails.
cudaError_t launch_decompress(cudaStream_t st, int num_sms, int d, int k, const TileTable &tiles,
                              const LayerTables &lt, const float *s_sum, const float *Ut, const float *mu,
                              float *g_hat);
size_t decompress_smem_bytes(int d, int k);
// The same on the tensor cores, for the shapes project_sum_tc_supported accepts; the output is written by
// tiled TMA stores through the tensor maps of g_hat's layers.  With g_for_tails the same launch also sums the
// uncompressed tails (otherwise launch_tail_sum does).
cudaError_t launch_decompress_tc(cudaStream_t st, int num_sms, int d, int k, const TileTable &tiles,
                                 const LayerTables &lt, const float *s_sum, const float *Ut, const float *mu,
                                 const CUtensorMap *tmaps_of_g_hat, int32_t *error_word,
                                 const NodePtrs<const float> *g_for_tails, int n_nodes, const int32_t *unit_start,
                                 int n_ctas, float *g_hat, int wait_kcycles, int test_drop);
// Exchange buffers of Algorithm 1 (exchange.cu): tails of the local nodes summed into / copied out of the tail
// part of a buffer, and x_acc += x_in over a whole buffer.
cudaError_t launch_tail_pack(cudaStream_t st, const LayerTables &lt, const NodePtrs<const float> &g, int n_nodes,
                             float *x_tail);
cudaError_t launch_tail_unpack(cudaStream_t st, const LayerTables &lt, const float *x_tail, float *g_hat);
cudaError_t launch_exchange_accumulate(cudaStream_t st, int num_sms, float *x_acc, const float *x_in, int64_t n);
// The exchange buffer with / without the coordinates past each layer's own compressed length (pack = true drops them).
cudaError_t launch_exchange_pack(cudaStream_t st, int num_sms, int k, int n_layers, const LayerTables &lt,
                                 const int32_t *layer_k, const int64_t *packed_off, int64_t S_total, int64_t n_tail,
                                 const float *src, float *dst, bool pack);
cudaError_t launch_tail_sum(cudaStream_t st, const LayerTables &lt, int d, const NodePtrs<const float> &g,
                            int n_nodes, float *g_hat);

// Eq. 7's sums (|x - mu / N|^2 and |s_n|^2 per layer and node) from materialised s_n; tiles of kProjectRows slices.
cudaError_t launch_monitor(cudaStream_t st, int d, int k, const TileTable &tiles, const LayerTables &lt,
                           const NodePtrs<const float> &g, const NodePtrs<const float> &s, int n_nodes, int mean_div,
                           const float *mu, double *monitor);

// The quantizer on raw gradient slices (bucket = slice), 4 bits per entry; tiles of kProjectRows slices.
cudaError_t launch_quantize_raw4(cudaStream_t st, int d, const TileTable &tiles, const LayerTables &lt, const float *g,
                                 int levels, uint64_t seed, uint32_t node, uint8_t *q4, float *norms);
cudaError_t launch_quantize_raw4_aggregate(cudaStream_t st, int d, const TileTable &tiles, const LayerTables &lt,
                                           const NodePtrs<const float> &g, int n_nodes, int levels, uint64_t seed,
                                           const NodePtrs<uint8_t> &q4, const NodePtrs<float> &norms, float *out);
cudaError_t launch_dequantize_raw4(cudaStream_t st, int d, const TileTable &tiles, const LayerTables &lt,
                                   const NodePtrs<const uint8_t> &q4, const NodePtrs<const float> &norms, int n_nodes,
                                   int levels, float *out);

// The paper's flatten order of one layer, framework [F][D][X] <-> flat [X][D][F].
cudaError_t launch_flatten(cudaStream_t st, int F, int D, int X, const float *src, float *dst, bool inverse);

// Quantizer.
cudaError_t launch_quantize(cudaStream_t st, int num_sms, int k, int64_t S, const float *s_node, int levels,
                            uint64_t seed, uint32_t node, int8_t *q, float *norms);
// All nodes quantized and the dequantised vectors summed in one launch (q / norms entries may be null).
cudaError_t launch_quantize_aggregate(cudaStream_t st, int num_sms, int k, int64_t S, const NodePtrs<const float> &s,
                                      int n_nodes, int levels, uint64_t seed, const NodePtrs<int8_t> &q,
                                      const NodePtrs<float> &norms, float *s_sum);
cudaError_t launch_dequantize_aggregate(cudaStream_t st, int num_sms, int k, int64_t S,
                                        const NodePtrs<const int8_t> &q, const NodePtrs<const float> &norms,
                                        int n_nodes, int levels, float *s_sum);

// Basis fit.  Workspace layout is private to fit_basis.cu.
size_t fit_workspace_bytes(int d, int n_layers, int n_fit_tiles);
struct FitArgs {
    int d, k, n_layers, L, N, c;
    const float *hist;
    int64_t hist_stride;
    float *Ut, *mu, *evals;
    void *ws;
    const CUtensorMap *hist_maps = nullptr;   // per layer, 3-D view of the history: the covariance runs on the tensor cores
    int32_t *error_word = nullptr;            // set by a kernel whose bounded wait ran out
    const int32_t *cov_order = nullptr;       // units of the tensor-core covariance, longest first
    // the cheap refresh: topk_iters > 0 replaces the full eigen-solve by subspace iteration (d <= 256, k <= 32);
    // Ut is then also an input when warm_start is set; evals_k [n_layers][k], trace [n_layers]
    int topk_iters = 0, warm_start = 0;
    float *evals_k = nullptr, *trace = nullptr;
    int fit_path = 0;   // full fit: 0 = automatic, 1 = eigen-solver with accumulated rotations, 2 = values + subspace
    // a fit spread over participants: stage 1 = this participant's moments about `centre` only (-> moments),
    // stage 2 = the fit from summed moments (no history read); 0 = the whole fit on one GPU
    int stage = 0;
    const float *centre = nullptr;   // [n_layers][d]
    double *moments = nullptr;       // [n_layers][1 + d + d * d]: n, sum (x - centre), sum (x - centre)(x - centre)^T
    int max_sweeps = 0;     // sweep limit of the eigen-solvers (0 = kJacobiMaxSweeps)
    int wait_kcycles = 0;   // limit of the bounded waits of the tensor-core covariance (0 = default)
    int test_drop = 0;      // test hook: the covariance kernel's first CTA leaves out its first load
};
// Covariance partial sums on the tensor cores (d = 64, 128, 192, 256).
bool cov_tc_supported(int d);
cudaError_t launch_cov_tc(cudaStream_t st, int num_sms, int d, int L, const TileTable &tiles, const LayerTables &lt,
                          const float *mean, const CUtensorMap *maps, const int32_t *unit_order, float *partial,
                          double *shift_sum, int32_t *error_word, int wait_kcycles, int test_drop);
// Enqueues the whole fit; *status_dev / *sweeps_dev (inside the workspace) are then read by the caller.
cudaError_t launch_fit_basis(cudaStream_t st, int num_sms, const FitArgs &a, const TileTable &tiles,
                             const LayerTables &lt, int32_t **status_dev, int32_t **sweeps_dev);
cudaError_t launch_fit_centre(cudaStream_t st, int d, int n_layers, int L, const float *hist, int64_t hist_stride,
                              const LayerTables &lt, float *centre);
}  // namespace gvq
struct gvq_ctx;
namespace gvq {
// Encodes the fit's tensor maps for this history buffer and queues their copy to the device; *maps_out is null
// when the shape has no tensor-core covariance (the FP32-pipe kernel runs then).
cudaError_t prepare_fit_maps(gvq_ctx *ctx, const float *hist, int64_t hist_stride, int L, const CUtensorMap **maps_out);

}  // namespace gvq

struct gvq_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    int num_sms = 0;
    int d = 0, k = 0, n_layers = 0;
    std::vector<int64_t> layer_off, layer_len;
    int64_t S = 0, M = 0, T = 0;   // full slices, entries of a flat gradient, tail entries
    bool has_tails = false;
    gvq::LayerTables lt;
    gvq::TileTable project_tiles, project_tc_tiles, decompress_tiles, fit_tiles;
    int32_t *error_word = nullptr;  // device word inside table_block, set by a kernel whose wait ran out
    int32_t *cov_unit_order = nullptr;  // inside table_block: units of the tensor-core covariance, longest first
    std::vector<int32_t> tile_layer_host[4], tile_count_host[4];   // host copies of the four tile tables
    // unit partitions of the tensor-core projection, one per node count seen (index N), and of the decompression
    std::vector<int32_t> tc_project_parts[GVQ_MAX_NODES + 1];
    std::vector<int32_t> tc_decompress_parts;
    int projection_path = 0;        // 0 = automatic, 1 = FP32 pipe, 2 = tensor cores
    int fit_path = 0;               // 0 = automatic, 1 = rotations accumulated, 2 = eigenvalues only + subspace iteration
    // Tensor maps of the tensor-core projection: slot s holds the n_layers maps of one gradient buffer
    // (a 2-D view, d entries x S_l slices, of every layer).  Slots are reused while a caller keeps
    // passing the same buffers, least recently used first otherwise.
    static constexpr int kTmapSlots = 2 * GVQ_MAX_NODES;
    CUtensorMap *tmaps_dev = nullptr;            // [kTmapSlots][n_layers]
    const float *slot_ptr[kTmapSlots] = {};
    uint64_t slot_tick[kTmapSlots] = {};
    uint64_t tick = 0;
    void *encode_fn = nullptr;                   // cuTensorMapEncodeTiled, looked up at create
    std::vector<CUtensorMap> slot_host;          // [kTmapSlots][n_layers] host images the uploads are made from (kept: an
                                                 // asynchronous copy may read its source after the call has returned)
    // Tensor maps of the basis fit: one 3-D map (entries, slices, stored gradients) per layer, re-encoded by
    // every fit call for its history buffer (host image and device copy both sized at create).
    CUtensorMap *fit_maps_dev = nullptr;         // [n_layers]
    std::vector<CUtensorMap> fit_maps_host;
    // Scratch of the tensor-core projection: pieces of tiles whose nodes are split between two CTAs, and
    // one arrival counter per tile (zero between launches).  Inside the tmaps_dev allocation.
    float *tc_partial = nullptr;
    int32_t *tc_tile_counter = nullptr;
    void *table_block = nullptr;  // one device allocation holding every table above
    void *ws = nullptr;
    size_t ws_bytes = 0;
    int last_cuda_error = 0;
    // per-layer compressed lengths (gvq_set_layer_k): host images and their device copies inside table_block
    std::vector<int32_t> layer_k_host;       // [n_layers]
    std::vector<int64_t> packed_off_host;    // [n_layers + 1] start of a layer in a packed exchange buffer; total
    int32_t *layer_k_dev = nullptr;
    int64_t *packed_off_dev = nullptr;
    cudaEvent_t stream_switch = nullptr;   // orders the work of the previous stream before the next one's (gvq_set_stream)
    // test hooks (gvq_set_limits, gvq_test_drop_load): 0 = the defaults
    int max_sweeps = 0;              // sweep limit of the eigen-solvers
    int wait_kcycles = 0;            // limit of the bounded waits inside the tensor-core kernels, units of 1024 clocks
    int drop_last_load = 0;          // the projection's CTA 0 leaves out its last load
    int64_t slice_index_base = 0;    // contexts over a part of a layout: index of their first slice in the whole layout
    // gvq_allreduce_host on a large gradient works through the layout in chunks (contexts over runs of slices, as
    // gvq_segment_layout cuts them) so that a chunk's result travels back while the next chunk's inputs arrive.
    struct HostChunk {
        gvq_ctx *sub = nullptr;      // context over the chunk's pieces
        int64_t begin = 0, end = 0;  // the chunk's extent in a flat gradient (floats)
        int64_t slice0 = 0;          // its first row in a compressed buffer
        int layer0 = 0;              // layer of its first piece (the pieces lie in consecutive layers)
        cudaEvent_t arrived = nullptr, computed = nullptr;
    };
    std::vector<HostChunk> host_chunks;
    cudaStream_t host_in = nullptr, host_out = nullptr;
    cudaEvent_t host_start = nullptr;
    int host_pipe_state = 0;         // 0 = not built yet, 1 = in use, -1 = not applicable to this layout
};

// Host side of the C ABI: argument validation, the context and its device tables, dispatch.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>

#include "gvq_internal.h"

using namespace gvq;

namespace {

constexpr size_t kMaxSmem = 227 * 1024;

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

gvq_status check_layout(const gvq_layout *l)
{
    if (!l || !l->layer_off || !l->layer_len) return GVQ_ERR_NULL;
    if (l->d < 4 || l->d > GVQ_MAX_D || l->k < 1 || l->k > l->d || l->n_layers < 1) return GVQ_ERR_SHAPE;
    if (l->d % 4 != 0) return GVQ_ERR_ALIGN;
    int64_t end = 0;
    for (int i = 0; i < l->n_layers; ++i) {
        if (l->layer_len[i] < 0 || l->layer_off[i] < 0) return GVQ_ERR_SHAPE;
        if (l->layer_off[i] % 4 != 0) return GVQ_ERR_ALIGN;
        if (l->layer_off[i] < end) return GVQ_ERR_SHAPE;  // sorted, no overlap
        end = l->layer_off[i] + l->layer_len[i];
        if (l->layer_len[i] / l->d > INT32_MAX) return GVQ_ERR_SHAPE;
    }
    // kernels exist for d a multiple of 4 up to 32, or a multiple of 64, with the basis of a layer
    // and the staging ring fitting one SM's shared memory
    if (!(l->d <= 32 || l->d % 64 == 0)) return GVQ_ERR_UNSUPPORTED;
    if (l->k > 128) return GVQ_ERR_UNSUPPORTED;
    if (project_sum_smem_bytes(l->d, l->k) > kMaxSmem || decompress_smem_bytes(l->d, l->k) > kMaxSmem)
        return GVQ_ERR_UNSUPPORTED;
    return GVQ_OK;
}

int count_tiles(const gvq_layout *l, int rows)
{
    int64_t n = 0;
    for (int i = 0; i < l->n_layers; ++i) n += (l->layer_len[i] / l->d + rows - 1) / rows;
    return (int)n;
}

gvq_status cuda_fail(gvq_ctx *ctx, cudaError_t e)
{
    if (ctx) ctx->last_cuda_error = (int)e;
    (void)cudaGetLastError();
    // tmap_slot's refusal to upload tensor maps while the stream is being captured
    return e == cudaErrorStreamCaptureUnsupported ? GVQ_ERR_CAPTURE : GVQ_ERR_CUDA;
}

#define GVQ_CUDA(ctx, call)                                    \
    do {                                                       \
        cudaError_t e__ = (call);                              \
        if (e__ != cudaSuccess) return cuda_fail((ctx), e__);  \
    } while (0)

template <typename T>
gvq_status gather_nodes(const T *const *src, int N, NodePtrs<const T> &dst, bool need_align = true)
{
    if (!src) return GVQ_ERR_NULL;
    if (N < 1 || N > GVQ_MAX_NODES) return GVQ_ERR_SHAPE;
    for (int n = 0; n < GVQ_MAX_NODES; ++n) dst.p[n] = nullptr;
    for (int n = 0; n < N; ++n) {
        if (!src[n]) return GVQ_ERR_NULL;
        if (need_align && !aligned16(src[n])) return GVQ_ERR_ALIGN;
        dst.p[n] = src[n];
    }
    return GVQ_OK;
}

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Finds (or makes) the slot that holds the tensor maps of gradient buffer `ptr`: one 2-D map per layer,
// inner dimension = the d entries of a slice, outer = the layer's S_l slices, box = 32 entries x 128
// slices, 128-byte swizzle, zero fill outside.  `busy` marks slots already taken by this call.
cudaError_t tmap_slot(gvq_ctx *ctx, const float *ptr, bool *busy, int *slot_out)
{
    int hit = -1, lru = -1;
    for (int s = 0; s < gvq_ctx::kTmapSlots; ++s) {
        if (ctx->slot_ptr[s] == ptr && !busy[s]) { hit = s; break; }
        if (!busy[s] && (lru < 0 || ctx->slot_tick[s] < ctx->slot_tick[lru])) lru = s;
    }
    if (hit < 0) {
        // A buffer the context has not seen: its maps have to be uploaded.  Not while the stream is being captured:
        // the copy would become a node of the graph that reads this context's host image at every replay, long
        // after the image has been reused for another buffer.
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        cudaError_t ce = cudaStreamIsCapturing(ctx->stream, &cap);
        if (ce != cudaSuccess) return ce;
        if (cap != cudaStreamCaptureStatusNone) return cudaErrorStreamCaptureUnsupported;
        hit = lru;
        CUtensorMap *maps = ctx->slot_host.data() + (size_t)hit * ctx->n_layers;
        EncodeTiledFn enc = (EncodeTiledFn)ctx->encode_fn;
        for (int l = 0; l < ctx->n_layers; ++l) {
            const int64_t S = ctx->layer_len[l] / ctx->d;
            cuuint64_t dims[2] = {(cuuint64_t)ctx->d, (cuuint64_t)(S > 0 ? S : 1)};
            cuuint64_t strides[1] = {(cuuint64_t)ctx->d * sizeof(float)};
            cuuint32_t box[2] = {32, (cuuint32_t)kProjectTcRows};
            cuuint32_t estr[2] = {1, 1};
            CUresult r = enc(&maps[l], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, (void *)(ptr + ctx->layer_off[l]), dims,
                             strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) { ctx->slot_ptr[hit] = nullptr; return cudaErrorInvalidValue; }
        }
        // the source is the slot's own host image, which lives as long as the context; the copy is ordered on the
        // stream after every kernel that still reads the slot's previous maps
        cudaError_t e = cudaMemcpyAsync(ctx->tmaps_dev + (size_t)hit * ctx->n_layers, maps,
                                        sizeof(CUtensorMap) * (size_t)ctx->n_layers, cudaMemcpyHostToDevice,
                                        ctx->stream);
        if (e != cudaSuccess) { ctx->slot_ptr[hit] = nullptr; return e; }
        ctx->slot_ptr[hit] = ptr;
    }
    busy[hit] = true;
    ctx->slot_tick[hit] = ++ctx->tick;
    *slot_out = hit;
    return cudaSuccess;
}

}  // namespace

void gvq::partition_units(const TileTable &tiles, int per_tile, int n_parts, float stage_cost, float min_unit_cost,
                          int32_t *start)
{
    const int nt = tiles.n_tiles;
    auto unit_cost = [&](int t) { return std::max((float)tiles.host_count[t] / (float)tiles.rows, min_unit_cost); };
    // how many runs a cost limit needs (greedy: fill a run up to the limit)
    auto fill = [&](double limit, int32_t *out) {
        int part = 0, layer = -1;
        double load = 0.0;
        if (out) out[0] = 0;
        for (int t = 0; t < nt; ++t) {
            const double c = unit_cost(t);
            int left = per_tile;
            while (left > 0) {
                const double entry = tiles.host_layer[t] != layer ? stage_cost : 0.0;
                int fit = (int)std::floor((limit - load - entry) / c + 1e-9);
                if (fit <= 0 && load == 0.0) fit = 1;   // a run takes at least one unit
                if (fit <= 0) {                          // close the run
                    ++part;
                    if (out && part <= n_parts) out[std::min(part, n_parts)] = t * per_tile + (per_tile - left);
                    load = 0.0;
                    layer = -1;
                    continue;
                }
                fit = std::min(fit, left);
                load += entry + fit * c;
                layer = tiles.host_layer[t];
                left -= fit;
            }
        }
        return part + 1;
    };
    double total = 0.0, biggest = 0.0;
    for (int t = 0; t < nt; ++t) { total += per_tile * (double)unit_cost(t); biggest = std::max(biggest, (double)unit_cost(t)); }
    double lo = total / n_parts, hi = total + (double)stage_cost * (nt + n_parts) + biggest;
    for (int it = 0; it < 40; ++it) {   // smallest limit that n_parts runs can meet
        const double mid = 0.5 * (lo + hi);
        if (fill(mid, nullptr) <= n_parts) hi = mid; else lo = mid;
    }
    for (int b = 0; b <= n_parts; ++b) start[b] = nt * per_tile;
    fill(hi, start);
    start[0] = 0;
    start[n_parts] = nt * per_tile;
    for (int b = 1; b <= n_parts; ++b) start[b] = std::max(start[b], start[b - 1]);
}

namespace {

// Eq. 3 (+ Eq. 4): on the tensor cores where the shape has such a kernel.
cudaError_t project(gvq_ctx *ctx, const NodePtrs<const float> &g, int n_nodes, int mean_div, const float *Ut,
                    const float *mu, float *s_sum, const NodePtrs<float> *s_nodes, const TcQuant *quant = nullptr,
                    double *monitor = nullptr)
{
    const bool tc_ok = project_sum_tc_supported(ctx->d, ctx->k) && ctx->encode_fn;
    if (quant && !tc_ok) return cudaErrorNotSupported;
    if (monitor) {
        cudaError_t e = cudaMemsetAsync(monitor, 0, sizeof(double) * 2 * (size_t)ctx->n_layers * n_nodes, ctx->stream);
        if (e != cudaSuccess) return e;
    }
    if (monitor && !(tc_ok && ctx->projection_path != 1)) {
        // no fused form for this shape: the FP32-pipe projection with per-node outputs, then the sums from them
        if (!s_nodes) return cudaErrorNotSupported;
        cudaError_t e = launch_project_sum(ctx->stream, ctx->num_sms, ctx->d, ctx->k, ctx->project_tiles, ctx->lt, g,
                                           n_nodes, mean_div, Ut, mu, s_sum, s_nodes);
        if (e != cudaSuccess) return e;
        NodePtrs<const float> sc;
        for (int n = 0; n < GVQ_MAX_NODES; ++n) sc.p[n] = s_nodes->p[n];
        return launch_monitor(ctx->stream, ctx->d, ctx->k, ctx->project_tiles, ctx->lt, g, sc, n_nodes, mean_div, mu,
                              monitor);
    }
    if (tc_ok && (ctx->projection_path != 1 || quant)) {
        bool busy[gvq_ctx::kTmapSlots] = {};
        int slots[GVQ_MAX_NODES] = {};
        for (int n = 0; n < n_nodes; ++n) {
            cudaError_t e = tmap_slot(ctx, g.p[n], busy, &slots[n]);
            if (e != cudaSuccess) return e;
        }
        // the split of the (tile, node) units over the CTAs depends on the node count only: computed once per count
        const int n_ctas = std::min(ctx->num_sms, kMaxPartitionCtas);
        std::vector<int32_t> &parts = ctx->tc_project_parts[n_nodes];
        if (parts.empty()) {
            parts.resize((size_t)n_ctas + 1);
            partition_units(ctx->project_tc_tiles, n_nodes, n_ctas, kProjectTcStageCost, kProjectTcMinUnitCost, parts.data());
        }
        return launch_project_sum_tc(ctx->stream, ctx->num_sms, ctx->d, ctx->k, ctx->project_tc_tiles, ctx->lt, g,
                                     n_nodes, mean_div, Ut, mu, s_sum, ctx->error_word, ctx->tmaps_dev, ctx->n_layers,
                                     slots, s_nodes, ctx->tc_partial, ctx->tc_tile_counter, parts.data(), n_ctas, quant,
                                     monitor, ctx->wait_kcycles, ctx->drop_last_load, ctx->slice_index_base);
    }
    return launch_project_sum(ctx->stream, ctx->num_sms, ctx->d, ctx->k, ctx->project_tiles, ctx->lt, g, n_nodes,
                              mean_div, Ut, mu, s_sum, s_nodes);
}

// Eq. 5 and the tails: on the tensor cores where the shape has such a kernel (one launch does both), else the
// FP32-pipe kernel followed by the tail kernel.  g is read only when the layout has tails; with_tails = false leaves
// the tails alone (the caller fills them from an exchange buffer).
cudaError_t decompress(gvq_ctx *ctx, const float *s_sum, const float *Ut, const float *mu, float *g_hat,
                       const NodePtrs<const float> &g, int n_nodes, bool with_tails = true)
{
    const bool tails = ctx->has_tails && with_tails;
    const bool tc_ok = project_sum_tc_supported(ctx->d, ctx->k) && ctx->encode_fn;
    if (tc_ok && ctx->projection_path != 1) {
        bool busy[gvq_ctx::kTmapSlots] = {};
        int slot = 0;
        cudaError_t e = tmap_slot(ctx, g_hat, busy, &slot);
        if (e != cudaSuccess) return e;
        if (ctx->project_tc_tiles.n_tiles > 0) {
            const int n_ctas = std::min(ctx->num_sms, kMaxPartitionCtas);
            std::vector<int32_t> &parts = ctx->tc_decompress_parts;
            if (parts.empty()) {
                parts.resize((size_t)n_ctas + 1);
                partition_units(ctx->project_tc_tiles, (ctx->d + 127) / 128, n_ctas, kDecompressTcStageCost,
                                kDecompressTcMinUnitCost, parts.data());
            }
            return launch_decompress_tc(ctx->stream, ctx->num_sms, ctx->d, ctx->k, ctx->project_tc_tiles, ctx->lt, s_sum,
                                        Ut, mu, ctx->tmaps_dev + (size_t)slot * ctx->n_layers, ctx->error_word,
                                        tails ? &g : nullptr, n_nodes, parts.data(), n_ctas, g_hat, ctx->wait_kcycles, ctx->drop_last_load);
        }
    }
    cudaError_t e = launch_decompress(ctx->stream, ctx->num_sms, ctx->d, ctx->k, ctx->decompress_tiles, ctx->lt, s_sum, Ut,
                                      mu, g_hat);
    if (e != cudaSuccess || !tails) return e;
    return launch_tail_sum(ctx->stream, ctx->lt, ctx->d, g, n_nodes, g_hat);
}

// After a kernel reported that one of its bounded waits ran out: the error word back to zero, and the arrival
// tickets of shared tiles too (a projection that gave up may have left some behind), so that the next call starts
// clean.
cudaError_t clear_device_fault(gvq_ctx *ctx)
{
    cudaError_t e = cudaMemsetAsync(ctx->error_word, 0, sizeof(int32_t), ctx->stream);
    if (e == cudaSuccess && ctx->tc_tile_counter)
        e = cudaMemsetAsync(ctx->tc_tile_counter, 0, sizeof(int32_t) * (size_t)std::max(1, ctx->project_tc_tiles.n_tiles),
                            ctx->stream);
    return e;
}

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) == cudaSuccess) ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard()
    {
        if (ok && prev >= 0) cudaSetDevice(prev);
    }
};

}  // namespace

extern "C" {

const char *gvq_status_string(gvq_status s)
{
    switch (s) {
    case GVQ_OK: return "ok";
    case GVQ_ERR_NULL: return "a required pointer is NULL";
    case GVQ_ERR_SHAPE: return "a size or count is out of range, or buffers overlap";
    case GVQ_ERR_ALIGN: return "a pointer or offset is not 16-byte aligned";
    case GVQ_ERR_UNSUPPORTED: return "no kernel for this (d, k)";
    case GVQ_ERR_WORKSPACE: return "workspace missing or too small";
    case GVQ_ERR_CUDA: return "a CUDA call failed";
    case GVQ_ERR_NOT_CONVERGED: return "the eigen-solver hit its sweep limit";
    case GVQ_ERR_DEGENERATE: return "degenerate spectrum";
    case GVQ_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case GVQ_ERR_CAPTURE: return "a buffer new to the context was passed while its stream is being captured";
    }
    return "unknown status";
}

gvq_status gvq_layout_check(const gvq_layout *layout) { return check_layout(layout); }

int64_t gvq_total_slices(const gvq_layout *l)
{
    if (check_layout(l) != GVQ_OK) return -1;
    int64_t S = 0;
    for (int i = 0; i < l->n_layers; ++i) S += l->layer_len[i] / l->d;
    return S;
}

int64_t gvq_total_entries(const gvq_layout *l)
{
    if (check_layout(l) != GVQ_OK) return -1;
    return l->layer_off[l->n_layers - 1] + l->layer_len[l->n_layers - 1];
}

int64_t gvq_exchange_floats(const gvq_layout *l)
{
    if (check_layout(l) != GVQ_OK) return -1;
    int64_t n = 0;
    for (int i = 0; i < l->n_layers; ++i) n += (l->layer_len[i] / l->d) * l->k + l->layer_len[i] % l->d;
    return n;
}

gvq_status gvq_segment_layout(const gvq_layout *l, int n_segments, int j, int32_t *n_pieces, int32_t *piece_layer,
                              int64_t *piece_off, int64_t *piece_len)
{
    if (!l || !piece_layer || !n_pieces || !piece_off || !piece_len) return GVQ_ERR_NULL;
    gvq_status st = check_layout(l);
    if (st != GVQ_OK) return st;
    if (n_segments < 1 || j < 0 || j >= n_segments) return GVQ_ERR_SHAPE;
    const int64_t S = gvq_total_slices(l), G = n_segments, d = l->d;
    // segment of global slice g: the j with floor(j S / G) <= g < floor((j + 1) S / G)
    auto seg_of = [&](int64_t g) {
        int64_t jj = (g * G) / S;                       // within one of the answer
        while (jj + 1 < G && ((jj + 1) * S) / G <= g) ++jj;
        while (jj > 0 && (jj * S) / G > g) --jj;
        return jj;
    };
    const int64_t lo = ((int64_t)j * S) / G, hi = ((int64_t)(j + 1) * S) / G;
    int np = 0;
    int64_t base = 0;
    for (int i = 0; i < l->n_layers; ++i) {
        const int64_t Sl = l->layer_len[i] / d, tail = l->layer_len[i] % d;
        const int64_t a = std::max(lo, base), b = std::min(hi, base + Sl);
        const int64_t n_here = std::max<int64_t>(0, b - a);
        // a tail travels with the slice just before it in layer order (segment 0 if there is none)
        const bool tail_here = tail > 0 && (base + Sl - 1 >= 0 ? seg_of(base + Sl - 1) : 0) == j;
        if (n_here > 0 || tail_here) {
            piece_layer[np] = i;
            piece_off[np] = l->layer_off[i] + (n_here > 0 ? (a - base) * d : Sl * d);
            piece_len[np] = n_here * d + (tail_here ? tail : 0);
            ++np;
        }
        base += Sl;
    }
    *n_pieces = np;
    return GVQ_OK;
}

size_t gvq_fit_workspace_bytes(const gvq_layout *l, int L)
{
    if (check_layout(l) != GVQ_OK || L < 1) return 0;
    return fit_workspace_bytes(l->d, l->n_layers, count_tiles(l, kFitRows));
}

size_t gvq_host_workspace_bytes(const gvq_layout *l, int N)
{
    if (check_layout(l) != GVQ_OK || N < 1 || N > GVQ_MAX_NODES) return 0;
    const size_t M = (size_t)gvq_total_entries(l), S = (size_t)gvq_total_slices(l);
    auto a256 = [](size_t x) { return (x + 255) & ~(size_t)255; };
    return a256(M * 4) * (size_t)(N + 1) + a256(S * l->k * 4);
}

gvq_status gvq_work_partition(const gvq_layout *l, int kind, int n_nodes, int n_parts, int32_t *start, int64_t *n_units_out)
{
    if (!l || !start || !n_units_out) return GVQ_ERR_NULL;
    gvq_status st = check_layout(l);
    if (st != GVQ_OK) return st;
    if ((kind != 0 && kind != 1) || n_parts < 1 || (kind == 0 && (n_nodes < 1 || n_nodes > GVQ_MAX_NODES))) return GVQ_ERR_SHAPE;
    std::vector<int32_t> layer, count;
    for (int i = 0; i < l->n_layers; ++i) {
        const int64_t S = l->layer_len[i] / l->d;
        for (int64_t r = 0; r < S; r += kProjectTcRows) {
            layer.push_back(i);
            count.push_back((int32_t)std::min<int64_t>(kProjectTcRows, S - r));
        }
    }
    TileTable t;
    t.rows = kProjectTcRows; t.n_tiles = (int)layer.size();
    t.host_layer = layer.data(); t.host_count = count.data();
    const int per_tile = kind == 0 ? n_nodes : (l->d + 127) / 128;
    partition_units(t, per_tile, n_parts, kind == 0 ? kProjectTcStageCost : kDecompressTcStageCost,
                    kind == 0 ? kProjectTcMinUnitCost : kDecompressTcMinUnitCost, start);
    *n_units_out = (int64_t)t.n_tiles * per_tile;
    return GVQ_OK;
}

gvq_status gvq_select_k(const float *evals, int d, double lambda_loss, int32_t *k_out)
{
    if (!evals || !k_out) return GVQ_ERR_NULL;
    if (d < 1 || !(lambda_loss >= 0.0) || !(lambda_loss < 1.0)) return GVQ_ERR_SHAPE;
    double total = 0.0;
    for (int j = 0; j < d; ++j) total += (double)evals[j];
    if (!(total > 0.0)) { *k_out = 1; return GVQ_ERR_DEGENERATE; }
    double head = 0.0;
    for (int j = 0; j < d; ++j) {
        head += (double)evals[j];
        if (head / total >= 1.0 - lambda_loss) { *k_out = j + 1; return GVQ_OK; }
    }
    *k_out = d;
    return GVQ_OK;
}

gvq_status gvq_create(gvq_ctx **out, const gvq_layout *layout, int device, void *cuda_stream)
{
    if (!out) return GVQ_ERR_NULL;
    *out = nullptr;
    gvq_status s = check_layout(layout);
    if (s != GVQ_OK) return s;
    gvq_ctx *ctx = new (std::nothrow) gvq_ctx();
    if (!ctx) return GVQ_ERR_CUDA;
    ctx->device = device;
    ctx->stream = (cudaStream_t)cuda_stream;
    ctx->d = layout->d; ctx->k = layout->k; ctx->n_layers = layout->n_layers;
    ctx->layer_off.assign(layout->layer_off, layout->layer_off + layout->n_layers);
    ctx->layer_len.assign(layout->layer_len, layout->layer_len + layout->n_layers);
    ctx->S = gvq_total_slices(layout);
    ctx->M = gvq_total_entries(layout);

    DeviceGuard guard(device);
    cudaError_t e = guard.ok ? cudaSuccess : cudaErrorInvalidDevice;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) { delete ctx; (void)cudaGetLastError(); return GVQ_ERR_CUDA; }

    // host images of every table, packed into one block
    const int nl = ctx->n_layers, d = ctx->d;
    std::vector<int64_t> off(ctx->layer_off), soff(nl), tail_off, tail_pos;
    std::vector<int32_t> Sl(nl), tail_len;
    int64_t acc = 0;
    for (int l = 0; l < nl; ++l) {
        Sl[l] = (int32_t)(ctx->layer_len[l] / d);
        soff[l] = acc;
        acc += Sl[l];
        const int tl = (int)(ctx->layer_len[l] % d);
        if (tl > 0) {
            tail_off.push_back(ctx->layer_off[l] + (int64_t)Sl[l] * d);
            tail_len.push_back(tl);
            tail_pos.push_back(ctx->T);
            ctx->T += tl;
        }
    }
    ctx->has_tails = !tail_len.empty();
    struct HostTiles { std::vector<int32_t> layer, row0, first; };
    auto build = [&](int rows) {
        HostTiles t;
        for (int l = 0; l < nl; ++l) {
            t.first.push_back((int32_t)t.layer.size());
            for (int r = 0; r < Sl[l]; r += rows) { t.layer.push_back(l); t.row0.push_back(r); }
        }
        t.first.push_back((int32_t)t.layer.size());
        return t;
    };
    HostTiles tp = build(kProjectRows), td = build(kDecompressRows), tf = build(kFitRows), tt = build(kProjectTcRows);

    std::vector<unsigned char> image;
    auto put = [&](const void *src, size_t bytes) {
        const size_t o = (image.size() + 255) & ~(size_t)255;
        image.resize(o + std::max<size_t>(bytes, 1));
        if (bytes) std::memcpy(image.data() + o, src, bytes);
        return o;
    };
    const size_t o_off = put(off.data(), off.size() * 8), o_soff = put(soff.data(), soff.size() * 8);
    const size_t o_S = put(Sl.data(), Sl.size() * 4);
    const size_t o_toff = put(tail_off.data(), tail_off.size() * 8), o_tlen = put(tail_len.data(), tail_len.size() * 4);
    const size_t o_tpos = put(tail_pos.data(), tail_pos.size() * 8);
    const int32_t zero = 0;
    const size_t o_err = put(&zero, sizeof(zero));
    // per-layer compressed lengths, all k until gvq_set_layer_k says otherwise
    ctx->layer_k_host.assign((size_t)nl, ctx->k);
    ctx->packed_off_host.assign((size_t)nl + 1, 0);
    for (int l = 0; l < nl; ++l) ctx->packed_off_host[l + 1] = ctx->packed_off_host[l] + (int64_t)Sl[l] * ctx->k;
    const size_t o_lk = put(ctx->layer_k_host.data(), (size_t)nl * 4);
    const size_t o_po = put(ctx->packed_off_host.data(), ((size_t)nl + 1) * 8);
    // units of the tensor-core covariance, (fit tile, pair of 128-entry blocks), longest first: the kernel deals
    // them out in that order so that its CTAs finish together
    std::vector<int32_t> cov_order;
    if (cov_tc_supported(d)) {
        const int nb = (d + 127) / 128, n_pairs = nb * (nb + 1) / 2;
        const int n_units = (int)tf.layer.size() * n_pairs;
        std::vector<int32_t> cost((size_t)n_units);
        for (int u = 0; u < n_units; ++u) {
            const int t = u / n_pairs;
            cost[u] = (std::min<int32_t>(kFitRows, Sl[tf.layer[t]] - tf.row0[t]) + 31) / 32;
        }
        cov_order.resize((size_t)n_units);
        for (int u = 0; u < n_units; ++u) cov_order[u] = u;
        std::stable_sort(cov_order.begin(), cov_order.end(), [&](int32_t a, int32_t b) { return cost[a] > cost[b]; });
    }
    const size_t o_cov = put(cov_order.data(), cov_order.size() * 4);
    size_t o_t[4][3];
    HostTiles *hts[4] = {&tp, &td, &tf, &tt};
    for (int i = 0; i < 4; ++i) {
        o_t[i][0] = put(hts[i]->layer.data(), hts[i]->layer.size() * 4);
        o_t[i][1] = put(hts[i]->row0.data(), hts[i]->row0.size() * 4);
        o_t[i][2] = put(hts[i]->first.data(), hts[i]->first.size() * 4);
    }
    e = cudaMalloc(&ctx->table_block, image.size());
    if (e == cudaSuccess) e = cudaMemcpy(ctx->table_block, image.data(), image.size(), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        if (ctx->table_block) cudaFree(ctx->table_block);
        delete ctx;
        (void)cudaGetLastError();
        return GVQ_ERR_CUDA;
    }
    const int tt_n_tiles = (int)tt.layer.size();
    if (project_sum_tc_supported(ctx->d, ctx->k) || cov_tc_supported(ctx->d)) {
        cudaDriverEntryPointQueryResult qres;
        void *fn = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            ctx->encode_fn = fn;
        (void)cudaGetLastError();
    }
    if (ctx->encode_fn && cov_tc_supported(ctx->d)) {
        ctx->fit_maps_host.resize((size_t)ctx->n_layers);
        if (cudaMalloc((void **)&ctx->fit_maps_dev, sizeof(CUtensorMap) * (size_t)ctx->n_layers) != cudaSuccess) {
            ctx->fit_maps_dev = nullptr;   // the FP32-pipe covariance kernel serves then
            (void)cudaGetLastError();
        }
    }
    if (project_sum_tc_supported(ctx->d, ctx->k)) {
        if (ctx->encode_fn) {
            const size_t map_bytes = (sizeof(CUtensorMap) * (size_t)gvq_ctx::kTmapSlots * ctx->n_layers + 255) & ~(size_t)255;
            const size_t part_bytes = (project_sum_tc_partial_bytes(ctx->num_sms, ctx->k) + 255) & ~(size_t)255;
            const size_t cnt_bytes = sizeof(int32_t) * (size_t)std::max(1, tt_n_tiles);
            ctx->slot_host.resize((size_t)gvq_ctx::kTmapSlots * ctx->n_layers);
            e = cudaMalloc((void **)&ctx->tmaps_dev, map_bytes + part_bytes + cnt_bytes);
            if (e == cudaSuccess) {
                ctx->tc_partial = (float *)((char *)ctx->tmaps_dev + map_bytes);
                ctx->tc_tile_counter = (int32_t *)((char *)ctx->tmaps_dev + map_bytes + part_bytes);
                e = cudaMemset(ctx->tc_tile_counter, 0, cnt_bytes);
            }
            if (e != cudaSuccess) {
                cudaFree(ctx->table_block);
                delete ctx;
                (void)cudaGetLastError();
                return GVQ_ERR_CUDA;
            }
        }
    }
    if (cudaEventCreateWithFlags(&ctx->stream_switch, cudaEventDisableTiming) != cudaSuccess) {
        ctx->stream_switch = nullptr;
        (void)cudaGetLastError();
    }
    char *base = (char *)ctx->table_block;
    ctx->lt.off = (int64_t *)(base + o_off); ctx->lt.soff = (int64_t *)(base + o_soff);
    ctx->lt.S = (int32_t *)(base + o_S);
    ctx->lt.n_tails = (int)tail_len.size();
    ctx->lt.tail_off = (int64_t *)(base + o_toff); ctx->lt.tail_len = (int32_t *)(base + o_tlen);
    ctx->lt.tail_pos = (int64_t *)(base + o_tpos);
    ctx->error_word = (int32_t *)(base + o_err);
    ctx->layer_k_dev = (int32_t *)(base + o_lk);
    ctx->packed_off_dev = (int64_t *)(base + o_po);
    ctx->cov_unit_order = cov_order.empty() ? nullptr : (int32_t *)(base + o_cov);
    TileTable *tts[4] = {&ctx->project_tiles, &ctx->decompress_tiles, &ctx->fit_tiles, &ctx->project_tc_tiles};
    const int rows[4] = {kProjectRows, kDecompressRows, kFitRows, kProjectTcRows};
    for (int i = 0; i < 4; ++i) {
        ctx->tile_layer_host[i] = hts[i]->layer;
        ctx->tile_count_host[i].resize(hts[i]->layer.size());
        for (size_t t = 0; t < hts[i]->layer.size(); ++t)
            ctx->tile_count_host[i][t] = std::min<int32_t>(rows[i], Sl[hts[i]->layer[t]] - hts[i]->row0[t]);
        tts[i]->host_layer = ctx->tile_layer_host[i].data();
        tts[i]->host_count = ctx->tile_count_host[i].data();
        tts[i]->rows = rows[i];
        tts[i]->n_tiles = (int)hts[i]->layer.size();
        tts[i]->layer = (int32_t *)(base + o_t[i][0]);
        tts[i]->row0 = (int32_t *)(base + o_t[i][1]);
        tts[i]->layer_first = (int32_t *)(base + o_t[i][2]);
    }
    *out = ctx;
    return GVQ_OK;
}

gvq_status gvq_destroy(gvq_ctx *ctx)
{
    if (!ctx) return GVQ_ERR_NULL;
    DeviceGuard guard(ctx->device);
    for (auto &c : ctx->host_chunks) {
        if (c.sub) gvq_destroy(c.sub);
        if (c.arrived) cudaEventDestroy(c.arrived);
        if (c.computed) cudaEventDestroy(c.computed);
    }
    if (ctx->stream_switch) cudaEventDestroy(ctx->stream_switch);
    if (ctx->host_start) cudaEventDestroy(ctx->host_start);
    if (ctx->host_in) cudaStreamDestroy(ctx->host_in);
    if (ctx->host_out) cudaStreamDestroy(ctx->host_out);
    if (ctx->table_block) cudaFree(ctx->table_block);
    if (ctx->tmaps_dev) cudaFree(ctx->tmaps_dev);
    if (ctx->fit_maps_dev) cudaFree(ctx->fit_maps_dev);
    delete ctx;
    return GVQ_OK;
}

gvq_status gvq_set_stream(gvq_ctx *ctx, void *cuda_stream)
{
    if (!ctx) return GVQ_ERR_NULL;
    cudaStream_t next = (cudaStream_t)cuda_stream;
    if (next == ctx->stream) return GVQ_OK;
    // The context's scratch (pieces and tickets of shared tiles, the error word, the tensor-map slots) is ordered by
    // the stream alone, so work already enqueued on the old stream must come before what the new one gets.  While
    // either stream is being captured no dependency is added (an event recorded outside a capture cannot be waited
    // for inside it): a capture has to begin after the context has settled on the capturing stream's predecessor.
    if (ctx->stream_switch) {
        DeviceGuard guard(ctx->device);
        cudaStreamCaptureStatus a = cudaStreamCaptureStatusNone, b = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(ctx->stream, &a) == cudaSuccess && cudaStreamIsCapturing(next, &b) == cudaSuccess &&
            a == cudaStreamCaptureStatusNone && b == cudaStreamCaptureStatusNone) {
            GVQ_CUDA(ctx, cudaEventRecord(ctx->stream_switch, ctx->stream));
            GVQ_CUDA(ctx, cudaStreamWaitEvent(next, ctx->stream_switch, 0));
        } else {
            (void)cudaGetLastError();
        }
    }
    ctx->stream = next;
    return GVQ_OK;
}

gvq_status gvq_set_limits(gvq_ctx *ctx, int max_sweeps, int64_t wait_cycles)
{
    if (!ctx) return GVQ_ERR_NULL;
    if (max_sweeps < 0 || max_sweeps > 1000 || wait_cycles < 0) return GVQ_ERR_SHAPE;
    ctx->max_sweeps = max_sweeps;
    const int64_t kc = (wait_cycles + 1023) >> 10;
    ctx->wait_kcycles = (int)std::min<int64_t>(kc, INT32_MAX);
    return GVQ_OK;
}

gvq_status gvq_test_drop_load(gvq_ctx *ctx, int on)
{
    if (!ctx) return GVQ_ERR_NULL;
    ctx->drop_last_load = on ? 1 : 0;
    return GVQ_OK;
}

gvq_status gvq_set_workspace(gvq_ctx *ctx, void *device_ptr, size_t bytes)
{
    if (!ctx) return GVQ_ERR_NULL;
    if ((device_ptr == nullptr) != (bytes == 0)) return GVQ_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(device_ptr) & 255u) return GVQ_ERR_ALIGN;
    ctx->ws = device_ptr;
    ctx->ws_bytes = bytes;
    return GVQ_OK;
}

int gvq_last_cuda_error(const gvq_ctx *ctx) { return ctx ? ctx->last_cuda_error : 0; }

gvq_status gvq_set_projection_path(gvq_ctx *ctx, int path)
{
    if (!ctx) return GVQ_ERR_NULL;
    if (path < 0 || path > 2) return GVQ_ERR_SHAPE;
    if (path == 2 && !(project_sum_tc_supported(ctx->d, ctx->k) && ctx->encode_fn)) return GVQ_ERR_UNSUPPORTED;
    ctx->projection_path = path;
    return GVQ_OK;
}

gvq_status gvq_set_fit_path(gvq_ctx *ctx, int path)
{
    if (!ctx) return GVQ_ERR_NULL;
    if (path < 0 || path > 2) return GVQ_ERR_SHAPE;
    const int kp = (ctx->k + 1) & ~1;
    if (path == 2 && (ctx->d > 256 || ctx->k > 32 || (int64_t)ctx->k * ctx->d + 3 * (int64_t)kp * kp + ctx->k + 2 > (int64_t)ctx->d * ctx->d))
        return GVQ_ERR_UNSUPPORTED;
    ctx->fit_path = path;
    return GVQ_OK;
}

gvq_status gvq_device_status(gvq_ctx *ctx)
{
    if (!ctx) return GVQ_ERR_NULL;
    DeviceGuard guard(ctx->device);
    int32_t word = 0;
    GVQ_CUDA(ctx, cudaMemcpyAsync(&word, ctx->error_word, sizeof(word), cudaMemcpyDeviceToHost, ctx->stream));
    GVQ_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (word != 0) {
        GVQ_CUDA(ctx, clear_device_fault(ctx));
        return GVQ_ERR_TIMEOUT;
    }
    return GVQ_OK;
}

gvq_status gvq_compress(gvq_ctx *ctx, const float *g_node, const float *Ut, const float *mu, int N, float *s_node)
{
    if (!ctx || !g_node || !Ut || !mu || !s_node) return GVQ_ERR_NULL;
    if (N < 1 || N > GVQ_MAX_NODES) return GVQ_ERR_SHAPE;
    if (!aligned16(g_node) || !aligned16(Ut) || !aligned16(mu) || !aligned16(s_node)) return GVQ_ERR_ALIGN;
    NodePtrs<const float> g;
    for (int n = 0; n < GVQ_MAX_NODES; ++n) g.p[n] = nullptr;
    g.p[0] = g_node;
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, project(ctx, g, 1, N, Ut, mu, s_node, nullptr));
    return GVQ_OK;
}

gvq_status gvq_aggregate(gvq_ctx *ctx, const float *const *s_nodes, int N, float *s_sum)
{
    if (!ctx || !s_sum) return GVQ_ERR_NULL;
    NodePtrs<const float> s;
    gvq_status st = gather_nodes(s_nodes, N, s);
    if (st != GVQ_OK) return st;
    if (!aligned16(s_sum)) return GVQ_ERR_ALIGN;
    for (int n = 0; n < N; ++n)
        if (s.p[n] == s_sum) return GVQ_ERR_SHAPE;
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, launch_aggregate(ctx->stream, ctx->num_sms, s, N, ctx->S * ctx->k, s_sum));
    return GVQ_OK;
}

gvq_status gvq_compress_aggregate(gvq_ctx *ctx, const float *const *g_nodes, int N, const float *Ut, const float *mu,
                                  float *s_sum, float *const *s_nodes_opt)
{
    if (!ctx || !Ut || !mu || !s_sum) return GVQ_ERR_NULL;
    NodePtrs<const float> g;
    gvq_status st = gather_nodes(g_nodes, N, g);
    if (st != GVQ_OK) return st;
    if (!aligned16(Ut) || !aligned16(mu) || !aligned16(s_sum)) return GVQ_ERR_ALIGN;
    NodePtrs<float> sn;
    for (int n = 0; n < GVQ_MAX_NODES; ++n) sn.p[n] = nullptr;
    if (s_nodes_opt)
        for (int n = 0; n < N; ++n) {
            if (!s_nodes_opt[n]) return GVQ_ERR_NULL;
            if (!aligned16(s_nodes_opt[n])) return GVQ_ERR_ALIGN;
            if (s_nodes_opt[n] == s_sum) return GVQ_ERR_SHAPE;
            sn.p[n] = s_nodes_opt[n];
        }
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, project(ctx, g, N, N, Ut, mu, s_sum, s_nodes_opt ? &sn : nullptr));
    return GVQ_OK;
}

gvq_status gvq_compress_aggregate_partial(gvq_ctx *ctx, const float *const *g_nodes, int n_local, int N, const float *Ut,
                                          const float *mu, float *x)
{
    if (!ctx || !Ut || !mu || !x) return GVQ_ERR_NULL;
    NodePtrs<const float> g;
    gvq_status st = gather_nodes(g_nodes, n_local, g);
    if (st != GVQ_OK) return st;
    if (N < n_local) return GVQ_ERR_SHAPE;
    if (!aligned16(Ut) || !aligned16(mu) || !aligned16(x)) return GVQ_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, launch_tail_pack(ctx->stream, ctx->lt, g, n_local, x + ctx->S * ctx->k));   // first: see exchange.cu
    GVQ_CUDA(ctx, project(ctx, g, n_local, N, Ut, mu, x, nullptr));
    return GVQ_OK;
}

gvq_status gvq_exchange_accumulate(gvq_ctx *ctx, float *x_acc, const float *x_in)
{
    if (!ctx || !x_acc || !x_in) return GVQ_ERR_NULL;
    if (!aligned16(x_acc) || !aligned16(x_in)) return GVQ_ERR_ALIGN;
    if (x_acc == x_in) return GVQ_ERR_SHAPE;
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, launch_exchange_accumulate(ctx->stream, ctx->num_sms, x_acc, x_in, ctx->S * ctx->k + ctx->T));
    return GVQ_OK;
}

gvq_status gvq_decompress_exchanged(gvq_ctx *ctx, const float *x, const float *Ut, const float *mu, float *g_hat)
{
    if (!ctx || !x || !Ut || !mu || !g_hat) return GVQ_ERR_NULL;
    if (!aligned16(x) || !aligned16(Ut) || !aligned16(mu) || !aligned16(g_hat)) return GVQ_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    NodePtrs<const float> none;
    for (int n = 0; n < GVQ_MAX_NODES; ++n) none.p[n] = nullptr;
    GVQ_CUDA(ctx, launch_tail_unpack(ctx->stream, ctx->lt, x + ctx->S * ctx->k, g_hat));   // the tails come from the buffer
    GVQ_CUDA(ctx, decompress(ctx, x, Ut, mu, g_hat, none, 1, false));
    return GVQ_OK;
}

int64_t gvq_packed_floats(const gvq_layout *l, const int32_t *k_per_layer)
{
    if (check_layout(l) != GVQ_OK || !k_per_layer) return -1;
    int64_t n = 0;
    for (int i = 0; i < l->n_layers; ++i) {
        if (k_per_layer[i] < 0 || k_per_layer[i] > l->k) return -1;
        n += (l->layer_len[i] / l->d) * k_per_layer[i] + l->layer_len[i] % l->d;
    }
    return n;
}

gvq_status gvq_set_layer_k(gvq_ctx *ctx, const int32_t *k_per_layer)
{
    if (!ctx) return GVQ_ERR_NULL;
    if (k_per_layer)
        for (int l = 0; l < ctx->n_layers; ++l)
            if (k_per_layer[l] < 0 || k_per_layer[l] > ctx->k) return GVQ_ERR_SHAPE;
    for (int l = 0; l < ctx->n_layers; ++l) {
        ctx->layer_k_host[l] = k_per_layer ? k_per_layer[l] : ctx->k;
        ctx->packed_off_host[l + 1] = ctx->packed_off_host[l] + (ctx->layer_len[l] / ctx->d) * ctx->layer_k_host[l];
    }
    DeviceGuard guard(ctx->device);
    // the sources are the context's own host images; ordered on the stream behind the kernels that read the old tables
    GVQ_CUDA(ctx, cudaMemcpyAsync(ctx->layer_k_dev, ctx->layer_k_host.data(), sizeof(int32_t) * (size_t)ctx->n_layers,
                                  cudaMemcpyHostToDevice, ctx->stream));
    GVQ_CUDA(ctx, cudaMemcpyAsync(ctx->packed_off_dev, ctx->packed_off_host.data(),
                                  sizeof(int64_t) * ((size_t)ctx->n_layers + 1), cudaMemcpyHostToDevice, ctx->stream));
    return GVQ_OK;
}

static gvq_status exchange_pack_call(gvq_ctx *ctx, const float *src, float *dst, bool pack)
{
    if (!ctx || !src || !dst) return GVQ_ERR_NULL;
    if (!aligned16(src) || !aligned16(dst)) return GVQ_ERR_ALIGN;
    if (src == dst) return GVQ_ERR_SHAPE;
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, launch_exchange_pack(ctx->stream, ctx->num_sms, ctx->k, ctx->n_layers, ctx->lt, ctx->layer_k_dev,
                                       ctx->packed_off_dev, ctx->S, ctx->T, src, dst, pack));
    return GVQ_OK;
}

gvq_status gvq_exchange_pack(gvq_ctx *ctx, const float *x, float *x_packed) { return exchange_pack_call(ctx, x, x_packed, true); }

gvq_status gvq_exchange_unpack(gvq_ctx *ctx, const float *x_packed, float *x) { return exchange_pack_call(ctx, x_packed, x, false); }

gvq_status gvq_quantize_raw4(gvq_ctx *ctx, const float *g_node, int levels, uint64_t seed, uint32_t node, uint8_t *q4,
                             float *norms)
{
    if (!ctx || !g_node || !q4 || !norms) return GVQ_ERR_NULL;
    if (levels < 1 || levels > 7) return GVQ_ERR_SHAPE;
    if (!aligned16(g_node) || !aligned16(q4) || !aligned16(norms)) return GVQ_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, launch_quantize_raw4(ctx->stream, ctx->d, ctx->project_tiles, ctx->lt, g_node, levels, seed, node, q4, norms));
    return GVQ_OK;
}

gvq_status gvq_quantize_raw4_aggregate(gvq_ctx *ctx, const float *const *g_nodes, int N, int levels, uint64_t seed,
                                       float *g_sum, uint8_t *const *q4_nodes_opt, float *const *norms_nodes_opt)
{
    if (!ctx || !g_sum) return GVQ_ERR_NULL;
    if (levels < 1 || levels > 7) return GVQ_ERR_SHAPE;
    NodePtrs<const float> g;
    gvq_status st = gather_nodes(g_nodes, N, g);
    if (st != GVQ_OK) return st;
    if (!aligned16(g_sum)) return GVQ_ERR_ALIGN;
    NodePtrs<uint8_t> qn;
    NodePtrs<float> nn;
    for (int n = 0; n < GVQ_MAX_NODES; ++n) { qn.p[n] = nullptr; nn.p[n] = nullptr; }
    for (int n = 0; n < N; ++n) {
        if (g.p[n] == g_sum) return GVQ_ERR_SHAPE;
        if (q4_nodes_opt) {
            if (!q4_nodes_opt[n]) return GVQ_ERR_NULL;
            if (!aligned16(q4_nodes_opt[n])) return GVQ_ERR_ALIGN;
            qn.p[n] = q4_nodes_opt[n];
        }
        if (norms_nodes_opt) {
            if (!norms_nodes_opt[n]) return GVQ_ERR_NULL;
            if (!aligned16(norms_nodes_opt[n])) return GVQ_ERR_ALIGN;
            nn.p[n] = norms_nodes_opt[n];
        }
    }
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, launch_quantize_raw4_aggregate(ctx->stream, ctx->d, ctx->project_tiles, ctx->lt, g, N, levels, seed, qn, nn,
                                                 g_sum));
    if (ctx->has_tails) GVQ_CUDA(ctx, launch_tail_sum(ctx->stream, ctx->lt, ctx->d, g, N, g_sum));
    return GVQ_OK;
}

gvq_status gvq_dequantize_raw4_aggregate(gvq_ctx *ctx, const uint8_t *const *q4_nodes, const float *const *norms_nodes,
                                         const float *const *g_nodes_for_tails, int levels, int N, float *g_sum)
{
    if (!ctx || !q4_nodes || !norms_nodes || !g_sum) return GVQ_ERR_NULL;
    if (levels < 1 || levels > 7 || N < 1 || N > GVQ_MAX_NODES) return GVQ_ERR_SHAPE;
    if (!aligned16(g_sum)) return GVQ_ERR_ALIGN;
    NodePtrs<const uint8_t> q;
    NodePtrs<const float> nn;
    for (int n = 0; n < GVQ_MAX_NODES; ++n) { q.p[n] = nullptr; nn.p[n] = nullptr; }
    for (int n = 0; n < N; ++n) {
        if (!q4_nodes[n] || !norms_nodes[n]) return GVQ_ERR_NULL;
        if (!aligned16(q4_nodes[n]) || !aligned16(norms_nodes[n])) return GVQ_ERR_ALIGN;
        q.p[n] = q4_nodes[n]; nn.p[n] = norms_nodes[n];
    }
    NodePtrs<const float> g;
    if (ctx->has_tails) {
        gvq_status st = gather_nodes(g_nodes_for_tails, N, g);
        if (st != GVQ_OK) return st;
        for (int n = 0; n < N; ++n)
            if (g.p[n] == g_sum) return GVQ_ERR_SHAPE;
    }
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, launch_dequantize_raw4(ctx->stream, ctx->d, ctx->project_tiles, ctx->lt, q, nn, N, levels, g_sum));
    if (ctx->has_tails) GVQ_CUDA(ctx, launch_tail_sum(ctx->stream, ctx->lt, ctx->d, g, N, g_sum));
    return GVQ_OK;
}

static gvq_status flatten_call(gvq_ctx *ctx, const float *src, float *dst, int F, int D, int X, bool inverse)
{
    if (!ctx || !src || !dst) return GVQ_ERR_NULL;
    if (F < 1 || D < 1 || X < 1 || (int64_t)D * X > (int64_t)2000000000 || (F + 63) / 64 > 65535) return GVQ_ERR_SHAPE;
    if ((int64_t)F * D * X > (int64_t)1 << 40) return GVQ_ERR_SHAPE;
    if (src == dst) return GVQ_ERR_SHAPE;
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, launch_flatten(ctx->stream, F, D, X, src, dst, inverse));
    return GVQ_OK;
}

gvq_status gvq_flatten_layer(gvq_ctx *ctx, const float *framework, float *flat, int F, int D, int X)
{
    return flatten_call(ctx, framework, flat, F, D, X, false);
}

gvq_status gvq_unflatten_layer(gvq_ctx *ctx, const float *flat, float *framework, int F, int D, int X)
{
    return flatten_call(ctx, flat, framework, F, D, X, true);
}

gvq_status gvq_mask_basis(gvq_ctx *ctx, float *Ut, const int32_t *k_per_layer)
{
    if (!ctx || !Ut || !k_per_layer) return GVQ_ERR_NULL;
    for (int l = 0; l < ctx->n_layers; ++l)
        if (k_per_layer[l] < 0 || k_per_layer[l] > ctx->k) return GVQ_ERR_SHAPE;
    DeviceGuard guard(ctx->device);
    for (int l = 0; l < ctx->n_layers; ++l) {
        const int kl = k_per_layer[l];
        if (kl == ctx->k) continue;
        GVQ_CUDA(ctx, cudaMemsetAsync(Ut + ((size_t)l * ctx->k + kl) * ctx->d, 0,
                                      sizeof(float) * (size_t)(ctx->k - kl) * ctx->d, ctx->stream));
    }
    return GVQ_OK;
}

gvq_status gvq_compress_aggregate_monitored(gvq_ctx *ctx, const float *const *g_nodes, int N, const float *Ut,
                                            const float *mu, float *s_sum, float *const *s_nodes_opt, double *monitor)
{
    if (!ctx || !Ut || !mu || !s_sum || !monitor) return GVQ_ERR_NULL;
    NodePtrs<const float> g;
    gvq_status st = gather_nodes(g_nodes, N, g);
    if (st != GVQ_OK) return st;
    if (!aligned16(Ut) || !aligned16(mu) || !aligned16(s_sum) || ((uintptr_t)monitor & 7)) return GVQ_ERR_ALIGN;
    const bool fused = project_sum_tc_supported(ctx->d, ctx->k) && ctx->encode_fn && ctx->projection_path != 1;
    if (!fused && !s_nodes_opt) return GVQ_ERR_UNSUPPORTED;
    NodePtrs<float> sn;
    for (int n = 0; n < GVQ_MAX_NODES; ++n) sn.p[n] = nullptr;
    if (s_nodes_opt)
        for (int n = 0; n < N; ++n) {
            if (!s_nodes_opt[n]) return GVQ_ERR_NULL;
            if (!aligned16(s_nodes_opt[n])) return GVQ_ERR_ALIGN;
            if (s_nodes_opt[n] == s_sum) return GVQ_ERR_SHAPE;
            sn.p[n] = s_nodes_opt[n];
        }
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, project(ctx, g, N, N, Ut, mu, s_sum, s_nodes_opt ? &sn : nullptr, nullptr, monitor));
    return GVQ_OK;
}

gvq_status gvq_compress_quantize_aggregate(gvq_ctx *ctx, const float *const *g_nodes, int N, const float *Ut,
                                           const float *mu, int levels, uint64_t seed, float *s_sum,
                                           int8_t *const *q_nodes_opt, float *const *norms_nodes_opt)
{
    if (!ctx || !Ut || !mu || !s_sum) return GVQ_ERR_NULL;
    if (levels < 1 || levels > 127) return GVQ_ERR_SHAPE;
    if (!(project_sum_tc_supported(ctx->d, ctx->k) && ctx->encode_fn)) return GVQ_ERR_UNSUPPORTED;
    NodePtrs<const float> g;
    gvq_status st = gather_nodes(g_nodes, N, g);
    if (st != GVQ_OK) return st;
    if (!aligned16(Ut) || !aligned16(mu) || !aligned16(s_sum)) return GVQ_ERR_ALIGN;
    NodePtrs<int8_t> qn;
    NodePtrs<float> nn;
    for (int n = 0; n < GVQ_MAX_NODES; ++n) { qn.p[n] = nullptr; nn.p[n] = nullptr; }
    for (int n = 0; n < N; ++n) {
        if (q_nodes_opt) {
            if (!q_nodes_opt[n]) return GVQ_ERR_NULL;
            if (!aligned16(q_nodes_opt[n])) return GVQ_ERR_ALIGN;
            qn.p[n] = q_nodes_opt[n];
        }
        if (norms_nodes_opt) {
            if (!norms_nodes_opt[n]) return GVQ_ERR_NULL;
            if (!aligned16(norms_nodes_opt[n])) return GVQ_ERR_ALIGN;
            nn.p[n] = norms_nodes_opt[n];
        }
    }
    TcQuant quant{levels, seed, q_nodes_opt ? &qn : nullptr, norms_nodes_opt ? &nn : nullptr};
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, project(ctx, g, N, N, Ut, mu, s_sum, nullptr, &quant));
    return GVQ_OK;
}

gvq_status gvq_decompress(gvq_ctx *ctx, const float *s_sum, const float *Ut, const float *mu,
                          const float *const *g_nodes_for_tails, int N, float *g_hat)
{
    if (!ctx || !s_sum || !Ut || !mu || !g_hat) return GVQ_ERR_NULL;
    if (N < 1 || N > GVQ_MAX_NODES) return GVQ_ERR_SHAPE;
    if (!aligned16(s_sum) || !aligned16(Ut) || !aligned16(mu) || !aligned16(g_hat)) return GVQ_ERR_ALIGN;
    NodePtrs<const float> g;
    if (ctx->has_tails) {
        gvq_status st = gather_nodes(g_nodes_for_tails, N, g);
        if (st != GVQ_OK) return st;
        for (int n = 0; n < N; ++n)
            if (g.p[n] == g_hat) return GVQ_ERR_SHAPE;
    }
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, decompress(ctx, s_sum, Ut, mu, g_hat, g, N));
    return GVQ_OK;
}

gvq_status gvq_fit_basis(gvq_ctx *ctx, const float *hist, int64_t hist_stride, int L, int N, int samples_are_sums_of,
                         float *Ut, float *mu, float *evals, int32_t *info)
{
    if (!ctx || !hist || !Ut || !mu || !evals) return GVQ_ERR_NULL;
    if (L < 1 || N < 1 || N > GVQ_MAX_NODES || samples_are_sums_of < 1) return GVQ_ERR_SHAPE;
    if (hist_stride < ctx->M && L > 1) return GVQ_ERR_SHAPE;
    if (hist_stride % 4 != 0 || !aligned16(hist) || !aligned16(Ut) || !aligned16(mu) || !aligned16(evals))
        return GVQ_ERR_ALIGN;
    const size_t need = fit_workspace_bytes(ctx->d, ctx->n_layers, ctx->fit_tiles.n_tiles);
    if (!ctx->ws || ctx->ws_bytes < need) return GVQ_ERR_WORKSPACE;
    FitArgs a;
    a.d = ctx->d; a.k = ctx->k; a.n_layers = ctx->n_layers; a.L = L; a.N = N; a.c = samples_are_sums_of;
    a.hist = hist; a.hist_stride = hist_stride; a.Ut = Ut; a.mu = mu; a.evals = evals; a.ws = ctx->ws;
    a.fit_path = ctx->fit_path;
    a.max_sweeps = ctx->max_sweeps; a.wait_kcycles = ctx->wait_kcycles; a.test_drop = ctx->drop_last_load;
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, prepare_fit_maps(ctx, hist, hist_stride, L, &a.hist_maps));
    a.error_word = ctx->error_word;
    a.cov_order = ctx->cov_unit_order;
    int32_t *status_dev = nullptr, *sweeps_dev = nullptr;
    GVQ_CUDA(ctx, launch_fit_basis(ctx->stream, ctx->num_sms, a, ctx->fit_tiles, ctx->lt, &status_dev, &sweeps_dev));
    int32_t status = 0;
    GVQ_CUDA(ctx, cudaMemcpyAsync(&status, status_dev, sizeof(status), cudaMemcpyDeviceToHost, ctx->stream));
    if (info)
        GVQ_CUDA(ctx, cudaMemcpyAsync(info, sweeps_dev, sizeof(int32_t) * (size_t)ctx->n_layers,
                                      cudaMemcpyDeviceToHost, ctx->stream));
    int32_t gave_up = 0;   // a tensor-core kernel of the fit whose bounded wait ran out
    GVQ_CUDA(ctx, cudaMemcpyAsync(&gave_up, ctx->error_word, sizeof(gave_up), cudaMemcpyDeviceToHost, ctx->stream));
    GVQ_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (gave_up) {
        GVQ_CUDA(ctx, clear_device_fault(ctx));
        return GVQ_ERR_TIMEOUT;
    }
    return status ? GVQ_ERR_NOT_CONVERGED : GVQ_OK;
}

int64_t gvq_fit_moments_count(const gvq_layout *l)
{
    if (check_layout(l) != GVQ_OK) return -1;
    return (int64_t)l->n_layers * (1 + (int64_t)l->d + (int64_t)l->d * l->d);
}

gvq_status gvq_fit_centre(gvq_ctx *ctx, const float *hist, int64_t hist_stride, int L, float *centre)
{
    if (!ctx || !hist || !centre) return GVQ_ERR_NULL;
    if (L < 1 || (hist_stride < ctx->M && L > 1)) return GVQ_ERR_SHAPE;
    if (hist_stride % 4 != 0 || !aligned16(hist) || !aligned16(centre)) return GVQ_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, launch_fit_centre(ctx->stream, ctx->d, ctx->n_layers, L, hist, hist_stride, ctx->lt, centre));
    return GVQ_OK;
}

gvq_status gvq_fit_moments(gvq_ctx *ctx, const float *hist, int64_t hist_stride, int L, const float *centre, double *moments)
{
    if (!ctx || !hist || !centre || !moments) return GVQ_ERR_NULL;
    if (L < 1 || (hist_stride < ctx->M && L > 1)) return GVQ_ERR_SHAPE;
    if (hist_stride % 4 != 0 || !aligned16(hist) || !aligned16(centre) || !aligned16(moments)) return GVQ_ERR_ALIGN;
    const size_t need = fit_workspace_bytes(ctx->d, ctx->n_layers, ctx->fit_tiles.n_tiles);
    if (!ctx->ws || ctx->ws_bytes < need) return GVQ_ERR_WORKSPACE;
    FitArgs a;
    a.d = ctx->d; a.k = ctx->k; a.n_layers = ctx->n_layers; a.L = L; a.N = 1; a.c = 1;
    a.hist = hist; a.hist_stride = hist_stride; a.Ut = nullptr; a.mu = nullptr; a.evals = nullptr; a.ws = ctx->ws;
    a.stage = 1; a.centre = centre; a.moments = moments; a.wait_kcycles = ctx->wait_kcycles; a.test_drop = ctx->drop_last_load;
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, prepare_fit_maps(ctx, hist, hist_stride, L, &a.hist_maps));
    a.error_word = ctx->error_word;
    a.cov_order = ctx->cov_unit_order;
    int32_t *status_dev = nullptr, *sweeps_dev = nullptr;
    GVQ_CUDA(ctx, launch_fit_basis(ctx->stream, ctx->num_sms, a, ctx->fit_tiles, ctx->lt, &status_dev, &sweeps_dev));
    return GVQ_OK;
}

gvq_status gvq_fit_from_moments(gvq_ctx *ctx, const double *moments, const float *centre, int N, int samples_are_sums_of,
                                float *Ut, float *mu, float *evals, int32_t *info)
{
    if (!ctx || !moments || !centre || !Ut || !mu || !evals) return GVQ_ERR_NULL;
    if (N < 1 || N > GVQ_MAX_NODES || samples_are_sums_of < 1) return GVQ_ERR_SHAPE;
    if (!aligned16(moments) || !aligned16(centre) || !aligned16(Ut) || !aligned16(mu) || !aligned16(evals)) return GVQ_ERR_ALIGN;
    const size_t need = fit_workspace_bytes(ctx->d, ctx->n_layers, ctx->fit_tiles.n_tiles);
    if (!ctx->ws || ctx->ws_bytes < need) return GVQ_ERR_WORKSPACE;
    FitArgs a;
    a.d = ctx->d; a.k = ctx->k; a.n_layers = ctx->n_layers; a.L = 1; a.N = N; a.c = samples_are_sums_of;
    a.hist = nullptr; a.hist_stride = 0; a.Ut = Ut; a.mu = mu; a.evals = evals; a.ws = ctx->ws;
    a.fit_path = ctx->fit_path; a.max_sweeps = ctx->max_sweeps;
    a.stage = 2; a.centre = centre; a.moments = const_cast<double *>(moments);
    DeviceGuard guard(ctx->device);
    int32_t *status_dev = nullptr, *sweeps_dev = nullptr;
    GVQ_CUDA(ctx, launch_fit_basis(ctx->stream, ctx->num_sms, a, ctx->fit_tiles, ctx->lt, &status_dev, &sweeps_dev));
    int32_t status = 0;
    GVQ_CUDA(ctx, cudaMemcpyAsync(&status, status_dev, sizeof(status), cudaMemcpyDeviceToHost, ctx->stream));
    if (info)
        GVQ_CUDA(ctx, cudaMemcpyAsync(info, sweeps_dev, sizeof(int32_t) * (size_t)ctx->n_layers,
                                      cudaMemcpyDeviceToHost, ctx->stream));
    GVQ_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return status ? GVQ_ERR_NOT_CONVERGED : GVQ_OK;
}

gvq_status gvq_refresh_basis(gvq_ctx *ctx, const float *hist, int64_t hist_stride, int L, int N, int samples_are_sums_of,
                             int warm_start, int iters, float *Ut, float *mu, float *evals_k, float *trace)
{
    if (!ctx || !hist || !Ut || !mu || !evals_k || !trace) return GVQ_ERR_NULL;
    if (L < 1 || N < 1 || N > GVQ_MAX_NODES || samples_are_sums_of < 1 || iters < 1 || iters > 1000) return GVQ_ERR_SHAPE;
    if (hist_stride < ctx->M && L > 1) return GVQ_ERR_SHAPE;
    if (hist_stride % 4 != 0 || !aligned16(hist) || !aligned16(Ut) || !aligned16(mu) || !aligned16(evals_k) ||
        ((uintptr_t)trace & 3))
        return GVQ_ERR_ALIGN;
    const int kp = (ctx->k + 1) & ~1;
    if (ctx->d > 256 || ctx->k > 32 || (int64_t)ctx->k * ctx->d + 3 * (int64_t)kp * kp > (int64_t)ctx->d * ctx->d)
        return GVQ_ERR_UNSUPPORTED;
    const size_t need = fit_workspace_bytes(ctx->d, ctx->n_layers, ctx->fit_tiles.n_tiles);
    if (!ctx->ws || ctx->ws_bytes < need) return GVQ_ERR_WORKSPACE;
    FitArgs a;
    a.d = ctx->d; a.k = ctx->k; a.n_layers = ctx->n_layers; a.L = L; a.N = N; a.c = samples_are_sums_of;
    a.hist = hist; a.hist_stride = hist_stride; a.Ut = Ut; a.mu = mu; a.evals = nullptr; a.ws = ctx->ws;
    a.topk_iters = iters; a.warm_start = warm_start ? 1 : 0; a.evals_k = evals_k; a.trace = trace;
    a.max_sweeps = ctx->max_sweeps; a.wait_kcycles = ctx->wait_kcycles; a.test_drop = ctx->drop_last_load;
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, prepare_fit_maps(ctx, hist, hist_stride, L, &a.hist_maps));
    a.error_word = ctx->error_word;
    a.cov_order = ctx->cov_unit_order;
    int32_t *status_dev = nullptr, *sweeps_dev = nullptr;
    GVQ_CUDA(ctx, launch_fit_basis(ctx->stream, ctx->num_sms, a, ctx->fit_tiles, ctx->lt, &status_dev, &sweeps_dev));
    int32_t status = 0, gave_up = 0;
    GVQ_CUDA(ctx, cudaMemcpyAsync(&status, status_dev, sizeof(status), cudaMemcpyDeviceToHost, ctx->stream));
    GVQ_CUDA(ctx, cudaMemcpyAsync(&gave_up, ctx->error_word, sizeof(gave_up), cudaMemcpyDeviceToHost, ctx->stream));
    GVQ_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (gave_up) {
        GVQ_CUDA(ctx, clear_device_fault(ctx));
        return GVQ_ERR_TIMEOUT;
    }
    return status ? GVQ_ERR_NOT_CONVERGED : GVQ_OK;
}

gvq_status gvq_quantize(gvq_ctx *ctx, const float *s_node, int levels, uint64_t seed, uint32_t node, int8_t *q,
                        float *norms)
{
    if (!ctx || !s_node || !q || !norms) return GVQ_ERR_NULL;
    if (levels < 1 || levels > 127) return GVQ_ERR_SHAPE;
    if (ctx->k > 32) return GVQ_ERR_UNSUPPORTED;
    if (!aligned16(s_node) || !aligned16(q) || !aligned16(norms)) return GVQ_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, launch_quantize(ctx->stream, ctx->num_sms, ctx->k, ctx->S, s_node, levels, seed, node, q, norms));
    return GVQ_OK;
}

gvq_status gvq_quantize_aggregate(gvq_ctx *ctx, const float *const *s_nodes, int N, int levels, uint64_t seed,
                                  float *s_sum, int8_t *const *q_nodes_opt, float *const *norms_nodes_opt)
{
    if (!ctx || !s_sum) return GVQ_ERR_NULL;
    if (levels < 1 || levels > 127) return GVQ_ERR_SHAPE;
    if (ctx->k > 32) return GVQ_ERR_UNSUPPORTED;
    NodePtrs<const float> s;
    gvq_status st = gather_nodes(s_nodes, N, s);
    if (st != GVQ_OK) return st;
    if (!aligned16(s_sum)) return GVQ_ERR_ALIGN;
    NodePtrs<int8_t> qn;
    NodePtrs<float> nn;
    for (int n = 0; n < GVQ_MAX_NODES; ++n) { qn.p[n] = nullptr; nn.p[n] = nullptr; }
    for (int n = 0; n < N; ++n) {
        if (s.p[n] == s_sum) return GVQ_ERR_SHAPE;
        if (q_nodes_opt) {
            if (!q_nodes_opt[n]) return GVQ_ERR_NULL;
            if (!aligned16(q_nodes_opt[n])) return GVQ_ERR_ALIGN;
            qn.p[n] = q_nodes_opt[n];
        }
        if (norms_nodes_opt) {
            if (!norms_nodes_opt[n]) return GVQ_ERR_NULL;
            if (!aligned16(norms_nodes_opt[n])) return GVQ_ERR_ALIGN;
            nn.p[n] = norms_nodes_opt[n];
        }
    }
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, launch_quantize_aggregate(ctx->stream, ctx->num_sms, ctx->k, ctx->S, s, N, levels, seed, qn, nn, s_sum));
    return GVQ_OK;
}

gvq_status gvq_dequantize_aggregate(gvq_ctx *ctx, const int8_t *const *q_nodes, const float *const *norms_nodes,
                                    int levels, int N, float *s_sum)
{
    if (!ctx || !s_sum) return GVQ_ERR_NULL;
    if (levels < 1 || levels > 127) return GVQ_ERR_SHAPE;
    NodePtrs<const int8_t> q;
    NodePtrs<const float> nr;
    gvq_status st = gather_nodes(q_nodes, N, q);
    if (st == GVQ_OK) st = gather_nodes(norms_nodes, N, nr);
    if (st != GVQ_OK) return st;
    if (!aligned16(s_sum)) return GVQ_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    GVQ_CUDA(ctx, launch_dequantize_aggregate(ctx->stream, ctx->num_sms, ctx->k, ctx->S, q, nr, N, levels, s_sum));
    return GVQ_OK;
}

// Builds the chunk pipeline of gvq_allreduce_host: kHostChunks runs of slices, each a context of its own, two copy
// streams and the events that order them.  Left out (state -1) for small gradients, where a copy is short
// against the fixed cost of a chunk, and for layouts whose chunks would skip a layer (their basis rows would not
// be contiguous).
static constexpr int kHostChunks = 8;
static constexpr int64_t kHostChunkMinFloats = 2 << 20;   // per chunk

static void build_host_pipe(gvq_ctx *ctx)
{
    ctx->host_pipe_state = -1;
    if (ctx->M < kHostChunks * kHostChunkMinFloats) return;
    gvq_layout lay{ctx->d, ctx->k, ctx->n_layers, ctx->layer_off.data(), ctx->layer_len.data()};
    std::vector<int32_t> pl((size_t)ctx->n_layers);
    std::vector<int64_t> po((size_t)ctx->n_layers), pn((size_t)ctx->n_layers);
    std::vector<gvq_ctx::HostChunk> chunks;
    bool ok = true;
    for (int j = 0; j < kHostChunks && ok; ++j) {
        int32_t np = 0;
        if (gvq_segment_layout(&lay, kHostChunks, j, &np, pl.data(), po.data(), pn.data()) != GVQ_OK) { ok = false; break; }
        if (np == 0) continue;
        for (int p = 1; p < np; ++p) ok = ok && pl[p] == pl[p - 1] + 1;
        if (!ok) break;
        gvq_ctx::HostChunk c;
        gvq_layout sub{ctx->d, ctx->k, np, po.data(), pn.data()};
        if (gvq_create(&c.sub, &sub, ctx->device, ctx->stream) != GVQ_OK) { ok = false; break; }
        c.begin = po[0];
        c.end = po[np - 1] + pn[np - 1];
        c.layer0 = pl[0];
        c.slice0 = 0;
        for (int l = 0; l < pl[0]; ++l) c.slice0 += ctx->layer_len[l] / ctx->d;
        c.slice0 += (po[0] - ctx->layer_off[pl[0]]) / ctx->d;
        c.sub->slice_index_base = c.slice0;   // the quantizer's hash is keyed on the slice's index in the whole layout
        ok = cudaEventCreateWithFlags(&c.arrived, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&c.computed, cudaEventDisableTiming) == cudaSuccess;
        chunks.push_back(c);
    }
    ok = ok && chunks.size() > 1;
    ok = ok && cudaStreamCreateWithFlags(&ctx->host_in, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&ctx->host_out, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&ctx->host_start, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
        (void)cudaGetLastError();
        for (auto &c : chunks) {
            if (c.sub) gvq_destroy(c.sub);
            if (c.arrived) cudaEventDestroy(c.arrived);
            if (c.computed) cudaEventDestroy(c.computed);
        }
        if (ctx->host_start) { cudaEventDestroy(ctx->host_start); ctx->host_start = nullptr; }
        if (ctx->host_in) { cudaStreamDestroy(ctx->host_in); ctx->host_in = nullptr; }
        if (ctx->host_out) { cudaStreamDestroy(ctx->host_out); ctx->host_out = nullptr; }
        return;
    }
    ctx->host_chunks = std::move(chunks);
    ctx->host_pipe_state = 1;
}

gvq_status gvq_host_prepare(gvq_ctx *ctx)
{
    if (!ctx) return GVQ_ERR_NULL;
    DeviceGuard guard(ctx->device);
    if (ctx->host_pipe_state == 0) build_host_pipe(ctx);
    return GVQ_OK;
}

static gvq_status allreduce_host(gvq_ctx *ctx, const float *const *g_nodes_host, int N, const float *Ut, const float *mu,
                                 int levels, uint64_t seed, float *g_hat_host)
{
    if (!ctx || !g_nodes_host || !Ut || !mu || !g_hat_host) return GVQ_ERR_NULL;
    if (N < 1 || N > GVQ_MAX_NODES) return GVQ_ERR_SHAPE;
    TcQuant quant{levels, seed, nullptr, nullptr};
    const TcQuant *qp = levels > 0 ? &quant : nullptr;
    for (int n = 0; n < N; ++n)
        if (!g_nodes_host[n]) return GVQ_ERR_NULL;
    if (!aligned16(Ut) || !aligned16(mu)) return GVQ_ERR_ALIGN;
    auto a256 = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t gbytes = (size_t)ctx->M * 4, gslot = a256(gbytes);
    const size_t need = gslot * (size_t)(N + 1) + a256((size_t)ctx->S * ctx->k * 4);
    if (!ctx->ws || ctx->ws_bytes < need) return GVQ_ERR_WORKSPACE;
    char *base = (char *)ctx->ws;
    NodePtrs<const float> g;
    for (int n = 0; n < GVQ_MAX_NODES; ++n) g.p[n] = nullptr;
    for (int n = 0; n < N; ++n) g.p[n] = (const float *)(base + gslot * n);
    float *g_hat = (float *)(base + gslot * N);
    float *s_sum = (float *)(base + gslot * (size_t)(N + 1));
    DeviceGuard guard(ctx->device);
    if (ctx->host_pipe_state != 1) {   // no chunk pipeline (gvq_host_prepare not called, or the layout has none)
        for (int n = 0; n < N; ++n)
            GVQ_CUDA(ctx, cudaMemcpyAsync((float *)g.p[n], g_nodes_host[n], gbytes, cudaMemcpyHostToDevice, ctx->stream));
        GVQ_CUDA(ctx, project(ctx, g, N, N, Ut, mu, s_sum, nullptr, qp));
        GVQ_CUDA(ctx, decompress(ctx, s_sum, Ut, mu, g_hat, g, N));
        GVQ_CUDA(ctx, cudaMemcpyAsync(g_hat_host, g_hat, gbytes, cudaMemcpyDeviceToHost, ctx->stream));
        GVQ_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
        return GVQ_OK;
    }
    // Chunk c: its part of every node's gradient arrives on the inbound stream; the kernels run on the context's
    // stream once it is there; its part of g_hat leaves on the outbound stream while chunk c + 1 is arriving (the
    // link carries both directions at once).  The scratch may still be in use by earlier work of the stream.
    GVQ_CUDA(ctx, cudaEventRecord(ctx->host_start, ctx->stream));
    GVQ_CUDA(ctx, cudaStreamWaitEvent(ctx->host_in, ctx->host_start, 0));
    GVQ_CUDA(ctx, cudaStreamWaitEvent(ctx->host_out, ctx->host_start, 0));
    for (auto &c : ctx->host_chunks) {
        const size_t bytes = (size_t)(c.end - c.begin) * 4;
        for (int n = 0; n < N; ++n)
            GVQ_CUDA(ctx, cudaMemcpyAsync((float *)g.p[n] + c.begin, g_nodes_host[n] + c.begin, bytes,
                                          cudaMemcpyHostToDevice, ctx->host_in));
        GVQ_CUDA(ctx, cudaEventRecord(c.arrived, ctx->host_in));
        GVQ_CUDA(ctx, cudaStreamWaitEvent(ctx->stream, c.arrived, 0));
        c.sub->stream = ctx->stream;
        c.sub->projection_path = ctx->projection_path;
        c.sub->wait_kcycles = ctx->wait_kcycles;
        const float *Uc = Ut + (size_t)c.layer0 * ctx->k * ctx->d, *mc = mu + (size_t)c.layer0 * ctx->d;
        cudaError_t e = project(c.sub, g, N, N, Uc, mc, s_sum + c.slice0 * ctx->k, nullptr, qp);
        if (e == cudaSuccess) e = decompress(c.sub, s_sum + c.slice0 * ctx->k, Uc, mc, g_hat, g, N);
        if (e != cudaSuccess) {   // nothing may stay in flight on the scratch when the call returns
            cudaStreamSynchronize(ctx->host_in); cudaStreamSynchronize(ctx->stream); cudaStreamSynchronize(ctx->host_out);
            return cuda_fail(ctx, e);
        }
        GVQ_CUDA(ctx, cudaEventRecord(c.computed, ctx->stream));
        GVQ_CUDA(ctx, cudaStreamWaitEvent(ctx->host_out, c.computed, 0));
        GVQ_CUDA(ctx, cudaMemcpyAsync(g_hat_host + c.begin, g_hat + c.begin, bytes, cudaMemcpyDeviceToHost, ctx->host_out));
    }
    GVQ_CUDA(ctx, cudaStreamSynchronize(ctx->host_out));
    GVQ_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return GVQ_OK;
}

gvq_status gvq_allreduce_host(gvq_ctx *ctx, const float *const *g_nodes_host, int N, const float *Ut, const float *mu,
                              float *g_hat_host)
{
    return allreduce_host(ctx, g_nodes_host, N, Ut, mu, 0, 0, g_hat_host);
}

gvq_status gvq_allreduce_host_quantized(gvq_ctx *ctx, const float *const *g_nodes_host, int N, const float *Ut,
                                        const float *mu, int levels, uint64_t seed, float *g_hat_host)
{
    if (levels < 1 || levels > 127) return GVQ_ERR_SHAPE;
    if (ctx && !(project_sum_tc_supported(ctx->d, ctx->k) && ctx->encode_fn)) return GVQ_ERR_UNSUPPORTED;
    return allreduce_host(ctx, g_nodes_host, N, Ut, mu, levels, seed, g_hat_host);
}

}  // extern "C"

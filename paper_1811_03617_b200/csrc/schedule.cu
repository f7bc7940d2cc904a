// Host-side control of when to collect samples, refit and compress (Section 3, "Parameter selection"):
// L_t iterations of uncompressed aggregation whose aggregated gradients are the PCA samples, a fit, then
// compressed iterations until either L_c of them have passed or the majority of the nodes report a large
// local compression loss (Eq. 7).  No device work here: a small state machine the training loop consults.
#include <new>

#include "gvq_internal.h"

struct gvq_schedule {
    int L_t, L_c, n_nodes;
    double loss_threshold;
    int phase;        // GVQ_PHASE_COLLECT / GVQ_PHASE_COMPRESS
    int in_phase;     // iterations completed in the current phase
    int64_t iteration, refreshes, early_stops;
    int last_over;    // nodes over the threshold at the last monitored step
};

extern "C" {

gvq_status gvq_schedule_create(gvq_schedule **out, int L_t, int L_c, int n_nodes, double loss_threshold)
{
    if (!out) return GVQ_ERR_NULL;
    *out = nullptr;
    if (L_t < 1 || L_c < 1 || n_nodes < 1 || n_nodes > GVQ_MAX_NODES) return GVQ_ERR_SHAPE;
    if (!(loss_threshold >= 0.0) || !(loss_threshold <= 1.0)) return GVQ_ERR_SHAPE;
    gvq_schedule *s = new (std::nothrow) gvq_schedule();
    if (!s) return GVQ_ERR_WORKSPACE;   // out of host memory
    s->L_t = L_t; s->L_c = L_c; s->n_nodes = n_nodes; s->loss_threshold = loss_threshold;
    s->phase = GVQ_PHASE_COLLECT; s->in_phase = 0;
    s->iteration = 0; s->refreshes = 0; s->early_stops = 0; s->last_over = 0;
    *out = s;
    return GVQ_OK;
}

gvq_status gvq_schedule_destroy(gvq_schedule *s)
{
    delete s;
    return GVQ_OK;
}

int gvq_schedule_phase(const gvq_schedule *s) { return s ? s->phase : -1; }

int gvq_schedule_nodes_over(const gvq_schedule *s) { return s ? s->last_over : -1; }

gvq_status gvq_schedule_counters(const gvq_schedule *s, int64_t *iteration, int64_t *refreshes, int64_t *early_stops)
{
    if (!s) return GVQ_ERR_NULL;
    if (iteration) *iteration = s->iteration;
    if (refreshes) *refreshes = s->refreshes;
    if (early_stops) *early_stops = s->early_stops;
    return GVQ_OK;
}

gvq_status gvq_schedule_step(gvq_schedule *s, const double *monitor_host, int n_layers, int *action)
{
    if (!s || !action) return GVQ_ERR_NULL;
    *action = GVQ_ACT_NONE;
    ++s->iteration;
    if (s->phase == GVQ_PHASE_COLLECT) {
        // the iteration just finished was aggregated uncompressed; its aggregate is sample number in_phase
        ++s->in_phase;
        if (s->in_phase >= s->L_t) {
            *action = GVQ_ACT_FIT;   // the caller fits on the L_t stored aggregates before the next iteration
            s->phase = GVQ_PHASE_COMPRESS;
            s->in_phase = 0;
            ++s->refreshes;
        }
        return GVQ_OK;
    }
    // a compressed iteration just finished
    ++s->in_phase;
    bool stop = s->in_phase >= s->L_c;
    if (monitor_host) {
        if (n_layers < 1) return GVQ_ERR_SHAPE;
        int over = 0;
        for (int n = 0; n < s->n_nodes; ++n) {
            double energy = 0.0, captured = 0.0;
            for (int l = 0; l < n_layers; ++l) {
                energy += monitor_host[((size_t)l * 2 + 0) * s->n_nodes + n];
                captured += monitor_host[((size_t)l * 2 + 1) * s->n_nodes + n];
            }
            const double loss = energy - captured;   // Eq. 7, summed over the layers
            if (energy > 0.0 && loss > s->loss_threshold * energy) ++over;
        }
        s->last_over = over;
        if (2 * over > s->n_nodes) {   // the majority of the nodes
            stop = true;
            if (s->in_phase < s->L_c) ++s->early_stops;
        }
    }
    if (stop) {
        *action = GVQ_ACT_RESTART;   // the next iteration aggregates uncompressed and stores a sample again
        s->phase = GVQ_PHASE_COLLECT;
        s->in_phase = 0;
    }
    return GVQ_OK;
}

}  // extern "C"

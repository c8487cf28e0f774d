// Host-side decisions of the A/F data plane and of the decode DVFS controller.  No device code:
// these functions read profiled curves / predicted tables and return a plan; they launch nothing
// and they never touch a GPU setting (applying a frequency is the caller's business).
//
//   aflex_eq2_layer_time      Eq. 2 of Section 4.3
//   aflex_pipeline_makespan   the interleaved A/F schedule (Section 4.3) played forward in time
//   aflex_plan_microbatches   microbatch depth and request split with the lowest predicted latency
//                             (Section 4.3, "Dynamic microbatch depth", "Adaptive request batching")
//   aflex_dvfs_window         window-size rule of Section 4.4
//   aflex_dvfs_decode_step    Algorithm 1 (window-based decode DVFS)
//   aflex_dvfs_prefill_pair   prefill frequency-pair choice of Section 4.4
#include <math.h>
#include <stdint.h>

#include <vector>

#include "internal.h"

namespace {

double curve_eval(const aflex_curve* c, double x) {
    if (c->n == 1) return c->y[0];
    int k = 0;
    while (k < c->n - 2 && x > c->x[k + 1]) ++k;
    const double t = (x - c->x[k]) / (c->x[k + 1] - c->x[k]);
    return c->y[k] + t * (c->y[k + 1] - c->y[k]);
}

bool curve_ok(const aflex_curve* c) {
    if (c->n < 1 || !c->x || !c->y) return false;
    for (int k = 0; k + 1 < c->n; ++k)
        if (!(c->x[k + 1] > c->x[k])) return false;
    return true;
}

struct Stage { double a, f, x; };

// Stage times of the microbatches [offsets[i], offsets[i+1]).  prefix[b] = sum of seq_lens[0..b).
void stage_times(const aflex_pipeline_model* m, const std::vector<long long>& prefix, const int32_t* offsets, int depth,
                 Stage* st) {
    for (int i = 0; i < depth; ++i) {
        const int rows = offsets[i + 1] - offsets[i];
        const double tokens = (double)(prefix[offsets[i + 1]] - prefix[offsets[i]]);
        // a curve extended below zero predicts no time at all
        st[i].a = fmax(0.0, curve_eval(&m->attn_vs_tokens, tokens) + curve_eval(&m->attn_vs_rows, (double)rows));
        st[i].f = fmax(0.0, curve_eval(&m->ffn_vs_rows, (double)rows));
        st[i].x = m->shared_memory_system ? 0.0 : m->comm_fixed + m->comm_per_row * rows;
    }
}

// Plays the schedule forward.  Four engines (A side, link A->F, F side, link F->A) each serve their
// stages in (layer, microbatch) order; a stage starts when its engine is free and its input has
// arrived.  On a shared memory system all stages queue on one engine.
double play(const Stage* st, int depth, int layers, bool shared) {
    if (shared) {
        double t = 0.0;
        for (int i = 0; i < depth; ++i) t += st[i].a + st[i].f;
        return t * layers;
    }
    double free_a = 0.0, free_x = 0.0, free_f = 0.0, free_y = 0.0, end = 0.0;
    double back[aflex::kMaxMicrobatches];          // when microbatch i's hidden states are back on the A side
    for (int i = 0; i < depth; ++i) back[i] = 0.0;
    for (int l = 0; l < layers; ++l) {
        for (int i = 0; i < depth; ++i) {
            const double a_done = fmax(free_a, back[i]) + st[i].a;
            free_a = a_done;
            const double x_done = fmax(free_x, a_done) + st[i].x;
            free_x = x_done;
            const double f_done = fmax(free_f, x_done) + st[i].f;
            free_f = f_done;
            const double y_done = fmax(free_y, f_done) + st[i].x;
            free_y = y_done;
            back[i] = y_done;
            if (y_done > end) end = y_done;
        }
    }
    return end;
}

bool model_ok(const aflex_pipeline_model* m) {
    return m && curve_ok(&m->attn_vs_tokens) && curve_ok(&m->attn_vs_rows) && curve_ok(&m->ffn_vs_rows) &&
           m->comm_fixed >= 0.0 && m->comm_per_row >= 0.0;
}

struct Search {
    const aflex_pipeline_model* m;
    const std::vector<long long>* prefix;
    int batch, layers, granularity, depth;
    int32_t offs[aflex::kMaxMicrobatches + 1];
    double best_t;
    int best_depth;
    int32_t best_offs[aflex::kMaxMicrobatches + 1];
    long long evaluated, limit;
    bool overflow;

    void leaf() {
        if (++evaluated > limit) { overflow = true; return; }
        Stage st[aflex::kMaxMicrobatches];
        stage_times(m, *prefix, offs, depth, st);
        const double t = play(st, depth, layers, m->shared_memory_system != 0);
        if (best_depth == 0 || t < best_t - 1e-12) {
            best_t = t;
            best_depth = depth;
            for (int i = 0; i <= depth; ++i) best_offs[i] = offs[i];
        }
    }
    // choose boundary k (1-based) after boundary k-1, lexicographically ascending
    void rec(int k) {
        if (overflow) return;
        if (k == depth) { offs[depth] = batch; leaf(); return; }
        for (int c = offs[k - 1] + granularity - (offs[k - 1] % granularity); c < batch; c += granularity) {
            // the remaining depth-k microbatches each need at least one boundary slot after c
            offs[k] = c;
            rec(k + 1);
            if (overflow) return;
        }
    }
};

}  // namespace

extern "C" {

double aflex_eq2_layer_time(double t_a, double t_f, double t_comm, int depth) {
    if (depth <= 1) return t_a + t_f + t_comm;
    return (t_a > t_f ? t_a : t_f) + t_comm / (double)depth;
}

double aflex_curve_eval(const aflex_curve* curve, double x) {
    if (!curve || !curve_ok(curve)) return NAN;
    return curve_eval(curve, x);
}

double aflex_pipeline_makespan(const aflex_pipeline_model* model, const int32_t* seq_lens_host, int batch, int depth,
                               const int32_t* offsets, int layers) {
    if (!model_ok(model) || !seq_lens_host || !offsets || batch < 1 || layers < 1 || depth < 1 ||
        depth > aflex::kMaxMicrobatches || depth > batch)
        return NAN;
    if (offsets[0] != 0 || offsets[depth] != batch) return NAN;
    for (int i = 0; i < depth; ++i)
        if (offsets[i + 1] <= offsets[i]) return NAN;
    std::vector<long long> prefix((size_t)batch + 1, 0);
    for (int b = 0; b < batch; ++b) prefix[b + 1] = prefix[b] + seq_lens_host[b];
    Stage st[aflex::kMaxMicrobatches];
    stage_times(model, prefix, offsets, depth, st);
    return play(st, depth, layers, model->shared_memory_system != 0);
}

aflex_status aflex_plan_microbatches(const aflex_pipeline_model* model, const int32_t* seq_lens_host, int batch, int layers,
                                     const int* depths, int n_depths, int granularity, int* best_depth,
                                     int32_t* best_offsets, double* predicted) {
    if (!model_ok(model) || !seq_lens_host || !depths || !best_depth || !best_offsets || batch < 1 || layers < 1 ||
        n_depths < 1 || granularity < 1)
        return AFLEX_ERR_INVALID_ARG;
    std::vector<long long> prefix((size_t)batch + 1, 0);
    for (int b = 0; b < batch; ++b) prefix[b + 1] = prefix[b] + seq_lens_host[b];
    // ascending depths, so that ties keep the smaller depth
    std::vector<int> ds(depths, depths + n_depths);
    for (size_t i = 1; i < ds.size(); ++i)
        for (size_t j = i; j > 0 && ds[j] < ds[j - 1]; --j) { const int t = ds[j]; ds[j] = ds[j - 1]; ds[j - 1] = t; }
    Search s;
    s.m = model; s.prefix = &prefix; s.batch = batch; s.layers = layers; s.granularity = granularity;
    s.best_t = 0.0; s.best_depth = 0; s.evaluated = 0; s.limit = 4000000; s.overflow = false;
    for (int d : ds) {
        if (d < 1 || d > batch || d > aflex::kMaxMicrobatches) continue;
        s.depth = d;
        s.offs[0] = 0;
        s.rec(1);
        if (s.overflow) return AFLEX_ERR_UNSUPPORTED;      // too many candidate splits: raise the granularity
    }
    if (s.best_depth == 0) return AFLEX_ERR_INVALID_ARG;     // no candidate depth fits the batch
    *best_depth = s.best_depth;
    for (int i = 0; i <= s.best_depth; ++i) best_offsets[i] = s.best_offs[i];
    if (predicted) *predicted = s.best_t;
    return AFLEX_OK;
}

int aflex_dvfs_window(int w_min, double kappa, double t_switch, double t_iter) {
    if (!(t_iter > 0.0)) return w_min;
    const double w = floor(kappa * t_switch / t_iter + 0.5);
    if (w > 2147483647.0) return 2147483647;
    return w > (double)w_min ? (int)w : w_min;
}

int aflex_dvfs_decode_step(const aflex_dvfs_params* p, const double* t_hat, const double* e_hat, int batch_now,
                           double t_iter, aflex_dvfs_state* s) {
    if (!p || !t_hat || !e_hat || !s || p->n_da < 1 || p->n_df < 1 || p->window < 1) return -1;
    if (s->i_da < 0 || s->i_da >= p->n_da || s->i_df < 0 || s->i_df >= p->n_df) return -1;
    s->w += 1;
    const int b_last = s->b_last;
    const double delta = fabs((double)batch_now - (double)b_last) / (double)(b_last > 1 ? b_last : 1);
    if (t_iter < p->tau && delta < p->delta_b && s->w < p->window) return 0;     // the window stays open
    // energy-minimal pair among those predicted to meet tau
    int star_a = -1, star_f = -1;
    for (int a = 0; a < p->n_da; ++a)
        for (int f = 0; f < p->n_df; ++f) {
            const int k = a * p->n_df + f;
            if (t_hat[k] <= p->tau && (star_a < 0 || e_hat[k] < e_hat[star_a * p->n_df + star_f])) { star_a = a; star_f = f; }
        }
    const int old_a = s->i_da, old_f = s->i_df;
    if (star_a < 0) {
        s->i_da = p->n_da - 1;
        s->i_df = p->n_df - 1;
    } else if (t_hat[old_a * p->n_df + old_f] > p->tau) {
        s->i_da = star_a; s->i_df = star_f;                                       // the current pair misses tau
    } else if (t_hat[star_a * p->n_df + star_f] + p->t_switch / (double)p->window <= p->tau) {
        s->i_da = star_a; s->i_df = star_f;                                       // lazy switch pays for itself
    }
    s->w = 0;
    s->b_last = batch_now;
    return (s->i_da != old_a || s->i_df != old_f) ? 2 : 1;
}

int aflex_dvfs_prefill_pair(int n_pa, int n_pf, const double* t_hat, const double* e_hat, double budget, double t_switch,
                            int cur_pa, int cur_pf, int base_pa, int base_pf, int* out_pa, int* out_pf) {
    if (!t_hat || !e_hat || !out_pa || !out_pf || n_pa < 1 || n_pf < 1) return -1;
    int star_a = -1, star_f = -1;
    for (int a = 0; a < n_pa; ++a)
        for (int f = 0; f < n_pf; ++f) {
            const int k = a * n_pf + f;
            const double cost = t_hat[k] + ((a == cur_pa && f == cur_pf) ? 0.0 : t_switch);
            if (cost <= budget && (star_a < 0 || e_hat[k] < e_hat[star_a * n_pf + star_f])) { star_a = a; star_f = f; }
        }
    int flags = 0;
    if (star_a < 0) { star_a = n_pa - 1; star_f = n_pf - 1; flags |= AFLEX_DVFS_INFEASIBLE; }
    if (star_a > base_pa || star_f > base_pf) flags |= AFLEX_DVFS_ESCALATED;
    *out_pa = star_a;
    *out_pf = star_f;
    return flags;
}

}  // extern "C"

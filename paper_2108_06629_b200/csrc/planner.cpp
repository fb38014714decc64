// Algorithm 1 (partitioning for balanced pipeline generation) in 64-bit integers.
//
// The layers are visited last to first; processors are filled one after another up to a
// budget T_p = ceil(T_tot / N_p).  For every layer the movable part (its delta work,
// T_flex) is placed first: whole if it is strictly smaller than the idle time left,
// otherwise split by operational parallelism into delta'' = idle time (stays on the
// processor being filled, i.e. beside layer l+1) and delta' = the rest (next processor).
// Then the immovable part (forward + G, T_fix) is placed, advancing to a fresh processor
// when it is strictly larger than the idle time.  If the walk needs more than N_p
// processors the budget grows by 1% (alpha = 101/100, rounded up) and the walk restarts.
// Readings taken where the printed algorithm is silent: idle time restarts from T_p
// whenever the processor index advances; processors used = last index + 1 and fewer than
// N_p is accepted; a layer with T_flex = 0 places nothing; delta'' is never negative.
#include <vector>

#include "common.h"

namespace lp {

static long long ceil_div(long long a, long long b) { return (a + b - 1) / b; }

int run_partition(const long long* T_fix, const long long* T_flex, int L, int Np, PlanResult* out) {
  if (!T_fix || !T_flex || L < 1 || Np < 1) return LP_ERR_INVALID_ARG;
  long long T_tot = 0;
  for (int l = 0; l < L; ++l) {
    if (T_fix[l] < 0 || T_flex[l] < 0) return LP_ERR_INVALID_ARG;
    T_tot += T_fix[l] + T_flex[l];
  }
  long long Tp = ceil_div(T_tot, Np);
  if (Tp < 1) Tp = 1;
  std::vector<int> fix_proc(L), pp(2 * L);
  std::vector<long long> pa(2 * L);
  int rounds = 0, used = 0;
  for (;;) {
    int p = 0;
    long long idle = Tp;
    for (int l = L - 1; l >= 0; --l) {
      pp[2 * l] = pp[2 * l + 1] = -1;
      pa[2 * l] = pa[2 * l + 1] = 0;
      if (T_flex[l] > 0) {
        if (T_flex[l] < idle) {
          pp[2 * l] = p;
          pa[2 * l] = T_flex[l];
          idle -= T_flex[l];
        } else {
          const long long d2 = idle > 0 ? idle : 0;   // delta''
          const long long d1 = T_flex[l] - d2;        // delta'
          pp[2 * l] = p;
          pa[2 * l] = d2;
          ++p;
          pp[2 * l + 1] = p;
          pa[2 * l + 1] = d1;
          idle = Tp - d1;
        }
      }
      if (T_fix[l] > idle) {
        ++p;
        idle = Tp;
      }
      fix_proc[l] = p;
      idle -= T_fix[l];
    }
    used = p + 1;
    if (used <= Np) break;
    Tp = ceil_div(Tp * 101, 100);
    if (++rounds > 1000000) return LP_ERR_INVALID_ARG;
  }
  out->stage.resize(L);
  out->delay.resize(L);
  out->piece_stage.resize(2 * L);
  out->piece_amount = pa;
  for (int l = 0; l < L; ++l) {
    out->stage[l] = used - 1 - fix_proc[l];
    out->delay[l] = used - 1 - out->stage[l];
    for (int k = 0; k < 2; ++k) out->piece_stage[2 * l + k] = pp[2 * l + k] < 0 ? -1 : used - 1 - pp[2 * l + k];
  }
  out->used = used;
  out->Tp = Tp;
  out->rounds = rounds;
  return LP_OK;
}

int layer_macs(const lp_layer& y, int batch, long long* macs) {
  if (y.in < 1 || y.out < 1 || batch < 1) return LP_ERR_INVALID_ARG;
  if (y.kind == LP_FC) {
    *macs = (long long)batch * y.in * y.out;
    return LP_OK;
  }
  if (y.kind == LP_CONV) {
    if (y.H < 1 || y.W < 1 || y.R < 1 || y.S < 1 || y.stride < 1 || y.pad < 0) return LP_ERR_INVALID_ARG;
    const long long Ho = (y.H + 2 * y.pad - y.R) / y.stride + 1, Wo = (y.W + 2 * y.pad - y.S) / y.stride + 1;
    if (Ho < 1 || Wo < 1) return LP_ERR_INVALID_ARG;
    *macs = (long long)batch * Ho * Wo * y.out * y.R * y.S * y.in;
    return LP_OK;
  }
  return LP_ERR_INVALID_ARG;
}

int plan_layers(const lp_layer* layers, int L, int batch, int Np, PlanResult* out) {
  if (!layers || L < 1) return LP_ERR_INVALID_ARG;
  std::vector<long long> fix(L), flex(L);
  for (int l = 0; l < L; ++l) {
    long long m;
    int rc = layer_macs(layers[l], batch, &m);
    if (rc != LP_OK) return rc;
    fix[l] = 2 * m;                 // forward + G
    flex[l] = l > 0 ? m : 0;        // delta; the first layer has no consumer for it
  }
  return run_partition(fix.data(), flex.data(), L, Np, out);
}

static int export_plan(const PlanResult& r, int L, int* stage_out, int* delay_out, int* dgrad_stage_out,
                       long long* dgrad_amount_out, int* stages_used, long long* Tp_out, int* relax_rounds_out) {
  for (int l = 0; l < L; ++l) {
    if (stage_out) stage_out[l] = r.stage[l];
    if (delay_out) delay_out[l] = r.delay[l];
    for (int k = 0; k < 2; ++k) {
      if (dgrad_stage_out) dgrad_stage_out[2 * l + k] = r.piece_stage[2 * l + k];
      if (dgrad_amount_out) dgrad_amount_out[2 * l + k] = r.piece_amount[2 * l + k];
    }
  }
  if (stages_used) *stages_used = r.used;
  if (Tp_out) *Tp_out = r.Tp;
  if (relax_rounds_out) *relax_rounds_out = r.rounds;
  return LP_OK;
}

}  // namespace lp

extern "C" int lp_plan(const lp_layer* layers, int n_layers, int batch, int n_stages, int* stage_out,
                       int* delay_out, int* dgrad_stage_out, long long* dgrad_amount_out, int* stages_used,
                       long long* Tp_out, int* relax_rounds_out) {
  if (!stage_out || !delay_out) return LP_ERR_INVALID_ARG;
  lp::PlanResult r;
  int rc = lp::plan_layers(layers, n_layers, batch, n_stages, &r);
  if (rc != LP_OK) return rc;
  return lp::export_plan(r, n_layers, stage_out, delay_out, dgrad_stage_out, dgrad_amount_out, stages_used, Tp_out,
                         relax_rounds_out);
}

extern "C" int lp_plan_costs(const long long* T_fix, const long long* T_flex, int n_layers, int n_stages,
                             int* stage_out, int* delay_out, int* dgrad_stage_out, long long* dgrad_amount_out,
                             int* stages_used, long long* Tp_out, int* relax_rounds_out) {
  if (!stage_out || !delay_out) return LP_ERR_INVALID_ARG;
  lp::PlanResult r;
  int rc = lp::run_partition(T_fix, T_flex, n_layers, n_stages, &r);
  if (rc != LP_OK) return rc;
  return lp::export_plan(r, n_layers, stage_out, delay_out, dgrad_stage_out, dgrad_amount_out, stages_used, Tp_out,
                         relax_rounds_out);
}

// Two-stage pipeline planner (Section 5 of the paper): compute planning, accumulated IO budgets,
// uniform pass, importance pass, preload selection.  Pure host code.
#include <algorithm>
#include <cmath>
#include <numeric>
#include <vector>

#include "../../include/sti_planner.h"

namespace {

constexpr int kBits[STI_N_VERSIONS] = {2, 3, 4, 5, 6, 32};
constexpr double kEps = 1e-9;

int version_of(int bits) {
  for (int v = 0; v < STI_N_VERSIONS; ++v)
    if (kBits[v] == bits) return v;
  return -1;
}

struct Shard {
  int layer, slot;
  int version;       // index into kBits, -1 = none yet
  bool preloaded;
};

// Stage 2 with the buffer contents given: versions for every shard of the submodel that is not preloaded.
// Returns validity; `aib` holds the remaining budgets.
bool io_plan(const sti_planner_profile& pf, int n, int m, double aib0, std::vector<Shard>& shards,
             const std::vector<int>& by_importance, std::vector<double>& aib, int* pass1_bits) {
  const double tc = pf.t_comp_us[m];
  aib.assign(n, 0.0);
  for (int k = 0; k < n; ++k) aib[k] = aib0 + k * tc;
  auto charge = [&](int layer, double us) {
    for (int k = layer; k < n; ++k) aib[k] -= us;
  };
  for (const Shard& s : shards)
    if (s.preloaded) charge(s.layer, pf.t_io_us[s.version]);
  // pass 1: the highest uniform version for everything that still has to be loaded
  int best = -1;
  for (int v = 0; v < STI_N_VERSIONS; ++v) {
    std::vector<double> trial = aib;
    for (const Shard& s : shards)
      if (!s.preloaded)
        for (int k = s.layer; k < n; ++k) trial[k] -= pf.t_io_us[v];
    const bool ok = std::all_of(trial.begin(), trial.end(), [](double b) { return b >= -kEps; });
    if (!ok) break;
    best = v;
  }
  const bool valid = best >= 0;
  const int v1 = valid ? best : 0;            // 2-bit shards are loaded even if they stall the pipeline
  *pass1_bits = kBits[v1];
  for (Shard& s : shards)
    if (!s.preloaded) {
      s.version = v1;
      charge(s.layer, pf.t_io_us[v1]);
    }
  if (!valid) return false;
  // pass 2: most important first, each to the highest version its layer's and all later layers' budgets allow
  for (int idx : by_importance) {
    Shard& s = shards[idx];
    if (s.preloaded) continue;
    for (int v = STI_N_VERSIONS - 1; v > s.version; --v) {
      const double extra = pf.t_io_us[v] - pf.t_io_us[s.version];
      bool ok = true;
      for (int k = s.layer; k < n && ok; ++k) ok = aib[k] - extra >= -kEps;
      if (ok) {
        charge(s.layer, extra);
        s.version = v;
        break;
      }
    }
  }
  return true;
}

}  // namespace

extern "C" sti_status sti_plan_auto(const sti_planner_profile* pf, const sti_planner_request* rq,
                                    sti_planner_result* out) {
  if (!pf || !rq || !out || !pf->t_comp_us || !pf->importance || !out->keep || !out->bits || !out->preload ||
      !out->aib_us)
    return STI_ERR_ARG;
  const int N = pf->n_layers, M = pf->n_slices;
  if (N < 1 || M < 1 || !(rq->target_us > 0.0)) return STI_ERR_ARG;
  for (int v = 0; v < STI_N_VERSIONS; ++v)
    if (!(pf->t_io_us[v] >= 0.0) || (v && pf->t_io_us[v] < pf->t_io_us[v - 1])) return STI_ERR_ARG;

  // ---- stage 1: the largest, then deepest, submodel that computes within T
  int n = 0, m = 0;
  for (int nn = 1; nn <= N; ++nn)
    for (int mm = 1; mm <= M; ++mm) {
      if (nn * pf->t_comp_us[mm] > rq->target_us + kEps) continue;
      if (nn * mm > n * m || (nn * mm == n * m && nn > n)) { n = nn; m = mm; }
    }
  const bool fits = n > 0;
  if (!fits) { n = 1; m = 1; }               // nothing meets T: the smallest submodel, reported as not valid

  // the m most important shards of each of the first n layers
  std::vector<Shard> shards;
  for (int l = 0; l < n; ++l) {
    std::vector<int> order(M);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
      return pf->importance[l * M + a] > pf->importance[l * M + b];
    });
    std::vector<int> pick(order.begin(), order.begin() + m);
    std::sort(pick.begin(), pick.end());
    for (int s : pick) shards.push_back({l, s, -1, false});
  }
  std::vector<int> by_importance(shards.size());
  std::iota(by_importance.begin(), by_importance.end(), 0);
  std::stable_sort(by_importance.begin(), by_importance.end(), [&](int a, int b) {
    return pf->importance[shards[a].layer * M + shards[a].slot] > pf->importance[shards[b].layer * M + shards[b].slot];
  });

  std::vector<double> aib;
  int pass1 = 2;
  bool valid;
  if (rq->preloaded_bits) {
    // the buffer's contents are given (Section 5.4)
    double aib0 = 0.0;
    for (Shard& s : shards) {
      const int v = version_of(rq->preloaded_bits[s.layer * M + s.slot]);
      if (v >= 0) {
        s.preloaded = true;
        s.version = v;
        aib0 += pf->t_io_us[v];
      }
    }
    valid = io_plan(*pf, n, m, aib0, shards, by_importance, aib, &pass1);
  } else {
    // first plan: the buffer size counts as bonus IO time, at the rate the 6-bit version loads
    const double us_per_byte = pf->shard_bytes[4] ? pf->t_io_us[4] / static_cast<double>(pf->shard_bytes[4]) : 0.0;
    io_plan(*pf, n, m, us_per_byte * static_cast<double>(rq->preload_bytes), shards, by_importance, aib, &pass1);
    // the first shards in layer order that fit; then plan again with that buffer as given
    uint64_t used = 0;
    double aib0 = 0.0;
    for (Shard& s : shards) {
      const uint64_t b = pf->shard_bytes[s.version];
      if (used + b > rq->preload_bytes) break;
      used += b;
      s.preloaded = true;
      aib0 += pf->t_io_us[s.version];
    }
    for (Shard& s : shards)
      if (!s.preloaded) s.version = -1;
    valid = io_plan(*pf, n, m, aib0, shards, by_importance, aib, &pass1);
  }

  std::fill(out->keep, out->keep + N * M, 0);
  std::fill(out->bits, out->bits + N * M, 0);
  std::fill(out->preload, out->preload + N * M, 0);
  std::fill(out->aib_us, out->aib_us + N, 0.0);
  for (const Shard& s : shards) {
    out->keep[s.layer * M + s.slot] = 1;
    out->bits[s.layer * M + s.slot] = static_cast<uint8_t>(kBits[s.version]);
    out->preload[s.layer * M + s.slot] = s.preloaded ? 1 : 0;
  }
  for (int k = 0; k < n; ++k) out->aib_us[k] = aib[k];
  out->n = n;
  out->m = m;
  out->pass1_bits = pass1;
  out->valid = (valid && fits) ? 1 : 0;
  return STI_OK;
}

extern "C" sti_status sti_preload_after_run(int32_t n_layers, int32_t n_slices, const uint8_t* keep,
                                            const uint8_t* bits, const uint64_t shard_bytes[STI_N_VERSIONS],
                                            uint64_t buffer_bytes, uint8_t* out_preloaded_bits,
                                            uint64_t* out_used_bytes) {
  if (!keep || !bits || !shard_bytes || !out_preloaded_bits || n_layers < 1 || n_slices < 1) return STI_ERR_ARG;
  const int total = n_layers * n_slices;
  for (int i = 0; i < total; ++i)
    if (keep[i] && version_of(bits[i]) < 0) return STI_ERR_ARG;
  std::fill(out_preloaded_bits, out_preloaded_bits + total, 0);
  uint64_t used = 0;
  for (int i = 0; i < total; ++i) {        // layer-major order is the bottom-up walk
    if (!keep[i]) continue;
    const uint64_t b = shard_bytes[version_of(bits[i])];
    if (used + b > buffer_bytes) break;     // this shard and everything above it is evicted
    used += b;
    out_preloaded_bits[i] = bits[i];
  }
  if (out_used_bytes) *out_used_bytes = used;
  return STI_OK;
}

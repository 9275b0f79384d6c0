// Table placement over the memories of one GPU (Section 5.6 of the paper: each table goes to one memory,
// the memories' capacities are respected, and the embedding lookup time of Eq. 6,
//   time = sum over tables of (D * L * p) / BW of the table's memory,
// is minimal).  With two memories (HBM and the host tier) this is a 0/1 knapsack: putting table t into HBM
// saves bytes_per_sample[t] * (1 / BW_host - 1 / BW_hbm) seconds per sample and costs size_bytes[t] of the
// budget.  Solved exactly by depth-first branch and bound over the tables in order of saving per byte, with
// the fractional relaxation as the bound; a node limit keeps the worst case bounded (the best placement
// found so far is returned and *optimal_out says whether the search finished).  Host code only.
#include <algorithm>
#include <numeric>
#include <vector>

#include "common.cuh"

namespace {

struct Item { double value; int64_t size; int32_t table; };

struct Search {
  const std::vector<Item>& items;
  int64_t capacity;
  int64_t node_limit;
  int64_t nodes = 0;
  double best_value = -1.0;
  std::vector<char> best, cur;

  // value of the fractional relaxation from item k on with `room` bytes left
  double bound(size_t k, int64_t room) const {
    double v = 0.0;
    for (; k < items.size(); ++k) {
      if (items[k].size <= room) { room -= items[k].size; v += items[k].value; }
      else { v += items[k].value * (double)room / (double)items[k].size; break; }
    }
    return v;
  }

  void run(size_t k, int64_t room, double value) {
    if (value > best_value) { best_value = value; best = cur; }
    if (k == items.size() || nodes >= node_limit) return;
    ++nodes;
    if (value + bound(k, room) <= best_value) return;
    if (items[k].size <= room) {
      cur[k] = 1;
      run(k + 1, room - items[k].size, value + items[k].value);
      cur[k] = 0;
    }
    run(k + 1, room, value);
  }
};

}  // namespace

extern "C" int mts_place_tables(int32_t T, const int64_t* host_size_bytes, const double* host_bytes_per_sample,
                                int64_t hbm_budget_bytes, double bw_hbm, double bw_host, int32_t* host_placement_out,
                                double* time_out, int32_t* optimal_out) {
  using namespace mts;
  if (T < 1 || !host_size_bytes || !host_bytes_per_sample || !host_placement_out || hbm_budget_bytes < 0 ||
      !(bw_hbm > 0.0) || !(bw_host > 0.0))
    return set_error(MTS_ERR_INVALID_ARG, "place_tables: null argument, T < 1, negative budget or non-positive bandwidth");
  for (int32_t t = 0; t < T; ++t)
    if (host_size_bytes[t] < 0 || !(host_bytes_per_sample[t] >= 0.0))
      return set_error(MTS_ERR_INVALID_ARG, "place_tables: table %d has a negative size or traffic", t);
  const double gain = 1.0 / bw_host - 1.0 / bw_hbm;        // seconds saved per byte of traffic moved to HBM
  std::vector<Item> items;
  for (int32_t t = 0; t < T; ++t) host_placement_out[t] = 1;
  if (gain > 0.0) {
    for (int32_t t = 0; t < T; ++t) {
      if (host_size_bytes[t] == 0) host_placement_out[t] = 0;                       // costs nothing
      else if (host_size_bytes[t] <= hbm_budget_bytes && host_bytes_per_sample[t] > 0.0)
        items.push_back({host_bytes_per_sample[t] * gain, host_size_bytes[t], t});
    }
  }
  std::sort(items.begin(), items.end(), [](const Item& a, const Item& b) {
    const double da = a.value / (double)a.size, db = b.value / (double)b.size;
    return da != db ? da > db : a.table < b.table;
  });
  Search s{items, hbm_budget_bytes, 20'000'000};
  s.cur.assign(items.size(), 0);
  s.best.assign(items.size(), 0);
  s.run(0, hbm_budget_bytes, 0.0);
  for (size_t k = 0; k < items.size(); ++k)
    if (s.best[k]) host_placement_out[items[k].table] = 0;
  double time = 0.0;
  for (int32_t t = 0; t < T; ++t) time += host_bytes_per_sample[t] / (host_placement_out[t] == 0 ? bw_hbm : bw_host);
  if (time_out) *time_out = time;
  if (optimal_out) *optimal_out = s.nodes < s.node_limit ? 1 : 0;
  return MTS_OK;
}

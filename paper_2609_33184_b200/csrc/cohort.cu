// Cohort builder (Section 4.2, cohort batching): tasks of the current scheduled batch that one
// batched kernel can process are grouped.  Compatible = same layer, verification width, data
// type, number of KV heads, head dimension and chunk size.  Inside a cohort the requests are
// ordered by decreasing history length, so the requests still active at a late chunk index form
// a prefix of the batch.  Cohorts keep the order in which their first task appears; a cohort
// larger than max_batch is cut into consecutive pieces.  Host logic only.
#include <algorithm>
#include <vector>

#include "specstream.h"

namespace {
bool compatible(const ss_task& a, const ss_task& b) {
  return a.layer == b.layer && a.width == b.width && a.dtype == b.dtype && a.n_kv == b.n_kv &&
         a.d_h == b.d_h && a.chunk_size == b.chunk_size;
}
}  // namespace

extern "C" int32_t ss_cohort_build(const ss_task* tasks, int32_t n, int32_t max_batch, int32_t* order,
                                   int32_t* cohort_start) {
  if (!tasks || !order || !cohort_start || n < 0 || max_batch <= 0) return -1;
  std::vector<int32_t> leader;             // first task index of each compatibility class
  std::vector<std::vector<int32_t>> members;
  for (int32_t i = 0; i < n; ++i) {
    size_t c = 0;
    for (; c < leader.size(); ++c)
      if (compatible(tasks[leader[c]], tasks[i])) break;
    if (c == leader.size()) {
      leader.push_back(i);
      members.emplace_back();
    }
    members[c].push_back(i);
  }
  int32_t pos = 0, n_cohorts = 0;
  for (auto& m : members) {
    std::stable_sort(m.begin(), m.end(),
                     [&](int32_t a, int32_t b) { return tasks[a].hist_len > tasks[b].hist_len; });
    for (size_t k = 0; k < m.size(); ++k) {
      if (k % (size_t)max_batch == 0) cohort_start[n_cohorts++] = pos;
      order[pos++] = m[k];
    }
  }
  cohort_start[n_cohorts] = pos;
  return n_cohorts;
}

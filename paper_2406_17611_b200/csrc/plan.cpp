// Host side of libvarco: partition plan builder, rate helpers, status strings.
//
// The plan turns a CSR graph plus partition labels into the index structures the kernels walk:
// partition-contiguous row order, halo sets in canonical order (Section III of the paper: each
// worker needs the rows of the boundary nodes of adjacent workers), the aggregation structure with
// columns remapped to [local rows | halo slots], its transpose for the backward pass, and the
// send / receive bookkeeping of the exchange.
#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <functional>
#include <new>
#include <numeric>
#include <thread>

#include "varco_internal.h"

namespace {

template <class Fn>
void parallel_over(int count, Fn fn) {
  int hw = (int)std::thread::hardware_concurrency();
  int nt = std::max(1, std::min(count, hw > 0 ? hw : 1));
  if (nt == 1) {
    for (int i = 0; i < count; ++i) fn(i);
    return;
  }
  std::vector<std::thread> th;
  for (int t = 0; t < nt; ++t)
    th.emplace_back([=]() {
      for (int i = t; i < count; i += nt) fn(i);
    });
  for (auto &x : th) x.join();
}

int validate(int64_t n, const int64_t *rp, const int32_t *col, const int32_t *part, int32_t P) {
  if (rp[0] != 0) return VARCO_BAD_GRAPH;
  for (int64_t i = 0; i < n; ++i) {
    if (rp[i + 1] < rp[i]) return VARCO_BAD_GRAPH;
    if (part[i] < 0 || part[i] >= P) return VARCO_BAD_PARTITION;
  }
  for (int64_t i = 0; i < n; ++i) {
    int64_t prev = -1;
    for (int64_t e = rp[i]; e < rp[i + 1]; ++e) {
      int64_t j = col[e];
      if (j < 0 || j >= n || j <= prev || j == i) return VARCO_BAD_GRAPH;
      prev = j;
    }
  }
  return VARCO_OK;
}

int build(varco_plan *pl, int64_t n, const int64_t *rp0, const int32_t *col0, const int32_t *part, int32_t P,
          int conv) {
  pl->n = n;
  pl->nnz = rp0[n];
  pl->P = P;
  pl->conv = conv;
  const bool gcn = conv == VARCO_GCN;

  // partition-contiguous order, ascending original id inside a partition
  pl->part_off.assign(P + 1, 0);
  for (int64_t i = 0; i < n; ++i) pl->part_off[part[i] + 1]++;
  for (int p = 0; p < P; ++p) pl->part_off[p + 1] += pl->part_off[p];
  pl->new_to_old.resize(n);
  std::vector<int32_t> old_to_new(n);
  {
    std::vector<int64_t> fill(pl->part_off.begin(), pl->part_off.end() - 1);
    for (int64_t i = 0; i < n; ++i) {
      int64_t r = fill[part[i]]++;
      pl->new_to_old[r] = i;
      old_to_new[i] = (int32_t)r;
    }
  }
  pl->row_gid.resize(n);
  for (int64_t r = 0; r < n; ++r) pl->row_gid[r] = (int32_t)pl->new_to_old[r];

  // phase A: the set of remote rows every partition q aggregates from, as sorted new indices
  // (new index order == (owner partition, original id) order == receive order)
  std::vector<std::vector<int32_t>> recv(P);
  std::vector<int64_t> cross_q(P, 0);
  parallel_over(P, [&](int q) {
    std::vector<uint8_t> seen(n, 0);
    std::vector<int32_t> &list = recv[q];
    int64_t cross = 0;
    for (int64_t r = pl->part_off[q]; r < pl->part_off[q + 1]; ++r) {
      int64_t i = pl->new_to_old[r];
      for (int64_t e = rp0[i]; e < rp0[i + 1]; ++e) {
        int32_t j = col0[e];
        if (part[j] != q) {
          ++cross;
          if (!seen[j]) {
            seen[j] = 1;
            list.push_back(old_to_new[j]);
          }
        }
      }
    }
    std::sort(list.begin(), list.end());
    cross_q[q] = cross;
  });
  pl->cross = std::accumulate(cross_q.begin(), cross_q.end(), (int64_t)0);
  pl->self_ = pl->nnz - pl->cross;
  std::vector<int64_t> slot_base(P + 1, 0);
  for (int q = 0; q < P; ++q) slot_base[q + 1] = slot_base[q] + (int64_t)recv[q].size();
  pl->H = slot_base[P];
  pl->slot_base = slot_base;
  for (int q = 0; q < P; ++q)
    pl->max_part_sources = std::max(pl->max_part_sources,
                                    (pl->part_off[q + 1] - pl->part_off[q]) + (slot_base[q + 1] - slot_base[q]));
  if (n + pl->H > 0x7FFFFFFFLL) return VARCO_UNSUPPORTED;

  // counts and send order
  pl->counts.assign((size_t)P * P, 0);
  for (int q = 0; q < P; ++q)
    for (int32_t r : recv[q]) pl->counts[(size_t)part[pl->new_to_old[r]] * P + q]++;
  pl->send_base.assign((size_t)P * P + 1, 0);
  for (size_t s = 0; s < (size_t)P * P; ++s) pl->send_base[s + 1] = pl->send_base[s] + pl->counts[s];
  pl->halo_ids.resize(pl->H);
  pl->slot_gid.resize(pl->H);
  pl->slot_src.resize(pl->H);
  pl->slot_sendpos.resize(pl->H);
  parallel_over(P, [&](int q) {
    int64_t slot = slot_base[q];
    int prev_p = -1;
    int64_t rank = 0;
    for (int32_t r : recv[q]) {
      int64_t gid = pl->new_to_old[r];
      int p = part[gid];
      if (p != prev_p) {
        prev_p = p;
        rank = 0;
      }
      int64_t sp = pl->send_base[(size_t)p * P + q] + rank++;
      pl->halo_ids[sp] = gid;
      pl->slot_gid[slot] = (int32_t)gid;
      pl->slot_src[slot] = r;
      pl->slot_sendpos[slot] = (int32_t)sp;
      ++slot;
    }
  });

  // phase B: aggregation structure with remapped columns and weights
  const int64_t extra = gcn ? 1 : 0;
  pl->rp.resize(n + 1);
  pl->rp[0] = 0;
  for (int64_t r = 0; r < n; ++r) {
    int64_t i = pl->new_to_old[r];
    pl->rp[r + 1] = pl->rp[r] + (rp0[i + 1] - rp0[i]) + extra;
  }
  pl->nnz_f = pl->rp[n];
  pl->col.resize(pl->nnz_f);
  pl->val.resize(pl->nnz_f);
  parallel_over(P, [&](int q) {
    std::vector<int32_t> slot_of(n, -1);
    for (size_t s = 0; s < recv[q].size(); ++s) slot_of[recv[q][s]] = (int32_t)(slot_base[q] + (int64_t)s);
    std::vector<std::pair<int32_t, float>> row;
    for (int64_t r = pl->part_off[q]; r < pl->part_off[q + 1]; ++r) {
      int64_t i = pl->new_to_old[r];
      double di = (double)(rp0[i + 1] - rp0[i]);
      row.clear();
      if (gcn) row.emplace_back((int32_t)r, (float)(1.0 / (di + 1.0)));
      for (int64_t e = rp0[i]; e < rp0[i + 1]; ++e) {
        int32_t j = col0[e];
        int32_t jn = old_to_new[j];
        double w;
        if (gcn) {
          double dj = (double)(rp0[j + 1] - rp0[j]);
          w = 1.0 / std::sqrt((di + 1.0) * (dj + 1.0));
        } else {
          w = 1.0 / di;
        }
        int32_t c = (part[j] == q) ? jn : (int32_t)(n + slot_of[jn]);
        row.emplace_back(c, (float)w);
      }
      std::sort(row.begin(), row.end(), [](const std::pair<int32_t, float> &a, const std::pair<int32_t, float> &b) {
        return a.first < b.first;
      });
      int64_t o = pl->rp[r];
      for (auto &cv : row) {
        pl->col[o] = cv.first;
        pl->val[o] = cv.second;
        ++o;
      }
    }
  });

  // mean aggregation: every entry of row r carries the same weight 1 / deg(r); the sum kernels add the
  // sources unweighted and apply it once per row
  pl->row_scale.clear();
  if (!gcn) {
    pl->row_scale.resize(n);
    for (int64_t r = 0; r < n; ++r) {
      const int64_t i = pl->new_to_old[r];
      const double di = (double)(rp0[i + 1] - rp0[i]);
      pl->row_scale[r] = di > 0 ? (float)(1.0 / di) : 0.f;
    }
  }

  // number of leading entries of every row whose source is a local row (columns are sorted: local first)
  pl->nloc.resize(n);
  for (int64_t r = 0; r < n; ++r) {
    int32_t c = 0;
    for (int64_t e = pl->rp[r]; e < pl->rp[r + 1] && pl->col[e] < n; ++e) ++c;
    pl->nloc[r] = c;
  }

  // transpose: sources [0, n + H) -> the rows that use them (ascending row inside a source)
  const int64_t nsrc = n + pl->H;
  pl->rpT.assign(nsrc + 1, 0);
  for (int64_t e = 0; e < pl->nnz_f; ++e) pl->rpT[pl->col[e] + 1]++;
  for (int64_t u = 0; u < nsrc; ++u) pl->rpT[u + 1] += pl->rpT[u];
  pl->colT.resize(pl->nnz_f);
  pl->valT.resize(pl->nnz_f);
  {
    std::vector<int64_t> fill(pl->rpT.begin(), pl->rpT.end() - 1);
    for (int64_t r = 0; r < n; ++r)
      for (int64_t e = pl->rp[r]; e < pl->rp[r + 1]; ++e) {
        int64_t o = fill[pl->col[e]]++;
        pl->colT[o] = (int32_t)r;
        pl->valT[o] = pl->val[e];
      }
  }

  // unique boundary rows and the slots they feed, ascending destination
  {
    std::vector<int32_t> cnt(n, 0);
    for (int64_t s = 0; s < pl->H; ++s) cnt[pl->slot_src[s]]++;
    std::vector<int32_t> where(n, -1);
    pl->brow.clear();
    pl->brow_ptr.assign(1, 0);
    for (int64_t r = 0; r < n; ++r)
      if (cnt[r]) {
        where[r] = (int32_t)pl->brow.size();
        pl->brow.push_back((int32_t)r);
        pl->brow_ptr.push_back(pl->brow_ptr.back() + cnt[r]);
      }
    pl->nb = (int64_t)pl->brow.size();
    pl->brow_slot.resize(pl->H);
    std::vector<int32_t> fill(pl->brow_ptr.begin(), pl->brow_ptr.end() - 1);
    for (int64_t s = 0; s < pl->H; ++s) pl->brow_slot[fill[where[pl->slot_src[s]]]++] = (int32_t)s;
  }

  // processing orders: three classes of rows by number of entries.  Hubs (more than the hub threshold)
  // get a CTA each.  Short rows (at most kShortEntries) are processed by narrow lane groups, several
  // rows per warp.  The rest get a full-width group.  Every class list is partition-major (the
  // kernels sweep partition by partition so that a partition's gathered rows stay in L2) and, inside
  // a partition, sorted by length, longest first, so that the lanes of a warp run alike.
  // The hub threshold differs by direction (measured on the 2.45M-node power-law workload): forward, where the
  // hub rows sit in one partition and gather from its whole source set, a warp per row serves rows of up to
  // 2048 entries better than a CTA each (forward stage 18.9 -> 18.2 ms); transposed, where the sources are one
  // partition's L2-resident block, 512 is the better cut (17.8 ms against 18.4 at 2048).
  const int64_t kHubEntriesFwd = 2048, kHubEntriesBwd = 512, kShortEntries = 8;   // a record holds 8 entries
  auto classify = [&](const std::vector<int64_t> &ptr, const std::vector<std::vector<int32_t>> &rows_of_part,
                      int64_t kHubEntries, std::vector<int32_t> *lists[3], std::vector<int32_t> *starts[3]) {
    for (int c = 0; c < 3; ++c) {
      lists[c]->clear();
      starts[c]->assign(1, 0);
    }
    std::vector<int32_t> tmp[3];
    for (int q = 0; q < P; ++q) {
      for (int c = 0; c < 3; ++c) tmp[c].clear();
      for (int32_t r : rows_of_part[q]) {
        const int64_t len = ptr[r + 1] - ptr[r];
        tmp[len > kHubEntries ? 0 : (len <= kShortEntries ? 2 : 1)].push_back(r);
      }
      for (int c = 0; c < 3; ++c) {
        std::stable_sort(tmp[c].begin(), tmp[c].end(),
                         [&](int32_t a, int32_t b) { return (ptr[a + 1] - ptr[a]) > (ptr[b + 1] - ptr[b]); });
        lists[c]->insert(lists[c]->end(), tmp[c].begin(), tmp[c].end());
        starts[c]->push_back((int32_t)lists[c]->size());
      }
    }
  };
  {
    std::vector<std::vector<int32_t>> rows_of_part(P);
    for (int q = 0; q < P; ++q)
      for (int64_t r = pl->part_off[q]; r < pl->part_off[q + 1]; ++r) rows_of_part[q].push_back((int32_t)r);
    std::vector<int32_t> *lf[3] = {&pl->hub_f, &pl->order_f, &pl->short_f};
    std::vector<int32_t> *sf[3] = {&pl->hub_f_start, &pl->order_f_start, &pl->short_f_start};
    classify(pl->rp, rows_of_part, kHubEntriesFwd, lf, sf);
    for (int q = 0; q < P; ++q)
      for (int64_t u = n + slot_base[q]; u < n + slot_base[q + 1]; ++u) rows_of_part[q].push_back((int32_t)u);
    std::vector<int32_t> *lt[3] = {&pl->hub_t, &pl->order_t, &pl->short_t};
    std::vector<int32_t> *stt[3] = {&pl->hub_t_start, &pl->order_t_start, &pl->short_t_start};
    classify(pl->rpT, rows_of_part, kHubEntriesBwd, lt, stt);
    // the short class of the transposed direction is walked by record position only: keep its local rows
    // (results added into dX) in front of its halo slots (results returned to the owners), each part still
    // partition-major, so that the slots can be handed to a kernel of their own
    std::stable_partition(pl->short_t.begin(), pl->short_t.end(), [&](int32_t u) { return (int64_t)u < n; });
    pl->short_t_nlocal = 0;
    for (int32_t u : pl->short_t) pl->short_t_nlocal += (int64_t)u < n ? 1 : 0;
    for (int q = 0; q <= P; ++q) pl->short_t_start[q] = q == 0 ? 0 : (int32_t)pl->short_t.size();
  }
  // fixed-size records of the short rows, in class-list order: 8 sources and 8 weights per row
  // (-1 / 0 beyond the row's length).  The short-row kernels find them by thread index alone, so
  // the gathers start after ONE dependent load instead of three (row id -> row_ptr -> columns).
  auto records = [&](const std::vector<int64_t> &ptr, const std::vector<int32_t> &cols, const std::vector<float> &vals,
                     const std::vector<int32_t> &rows, std::vector<int32_t> &rec_col, std::vector<float> &rec_val) {
    rec_col.assign(rows.size() * 8, -1);
    rec_val.assign(rows.size() * 8, 0.f);
    for (size_t i = 0; i < rows.size(); ++i) {
      const int64_t e0 = ptr[rows[i]], len = ptr[rows[i] + 1] - e0;
      for (int64_t j = 0; j < len; ++j) {
        rec_col[i * 8 + j] = cols[e0 + j];
        rec_val[i * 8 + j] = vals[e0 + j];
      }
    }
  };
  records(pl->rp, pl->col, pl->val, pl->short_f, pl->short_f_col, pl->short_f_val);
  records(pl->rpT, pl->colT, pl->valT, pl->short_t, pl->short_t_col, pl->short_t_val);
  return VARCO_OK;
}

}  // namespace

int varco_kept_internal(int32_t F, varco_ratio_t c) {
  if (F < 1 || c.num == 0) return -1;
  if (c.den == 0) return 0;   // unbounded ratio: the "no communication" setting, nothing is sent
  if (c.num < c.den) return -1;
  uint64_t k = ((uint64_t)F * c.den + c.num - 1) / c.num;
  if (k < 1) k = 1;
  if (k > (uint64_t)F) k = (uint64_t)F;
  return (int)k;
}

extern "C" {

const char *varco_status_string(int status) {
  switch (status) {
    case VARCO_OK: return "ok";
    case VARCO_INVALID_ARG: return "invalid argument";
    case VARCO_BAD_GRAPH: return "malformed CSR graph";
    case VARCO_BAD_PARTITION: return "partition label out of range";
    case VARCO_NOMEM: return "out of host memory";
    case VARCO_CUDA: return "CUDA runtime error";
    case VARCO_WORKSPACE_TOO_SMALL: return "workspace too small";
    case VARCO_UNSUPPORTED: return "unsupported size or configuration";
    case VARCO_NOT_UPLOADED: return "plan has no device image";
    default: return "unknown status";
  }
}

int varco_partition_build(int64_t n, const int64_t *row_ptr, const int32_t *col_idx, const int32_t *part, int32_t P,
                          varco_conv_t conv, varco_plan_t **out) {
  if (!out) return VARCO_INVALID_ARG;
  *out = nullptr;
  if (n < 1 || !row_ptr || !part || P < 1 || (conv != VARCO_GCN && conv != VARCO_SAGE_MEAN))
    return VARCO_INVALID_ARG;
  if (n > 0x7FFFFFFFLL) return VARCO_UNSUPPORTED;
  if (row_ptr[0] != 0) return VARCO_BAD_GRAPH;
  for (int64_t i = 0; i < n; ++i)
    if (row_ptr[i + 1] < row_ptr[i]) return VARCO_BAD_GRAPH;
  if (row_ptr[n] > 0 && !col_idx) return VARCO_INVALID_ARG;
  int rc = validate(n, row_ptr, col_idx, part, P);
  if (rc != VARCO_OK) return rc;
  varco_plan *pl = nullptr;
  try {
    pl = new varco_plan;
    rc = build(pl, n, row_ptr, col_idx, part, P, (int)conv);
  } catch (const std::bad_alloc &) {
    rc = VARCO_NOMEM;
  } catch (...) {
    rc = VARCO_NOMEM;
  }
  if (rc != VARCO_OK) {
    delete pl;
    return rc;
  }
  *out = pl;
  return VARCO_OK;
}

int varco_partition_destroy(varco_plan_t *plan) {
  if (!plan) return VARCO_INVALID_ARG;
  varco_prof_destroy(plan);
  delete plan;
  return VARCO_OK;
}

int varco_partition_info(const varco_plan_t *plan, int64_t *n, int64_t *nnz, int32_t *P, int64_t *H_total,
                         int64_t *cross_entries, int64_t *self_entries) {
  if (!plan) return VARCO_INVALID_ARG;
  if (n) *n = plan->n;
  if (nnz) *nnz = plan->nnz;
  if (P) *P = plan->P;
  if (H_total) *H_total = plan->H;
  if (cross_entries) *cross_entries = plan->cross;
  if (self_entries) *self_entries = plan->self_;
  return VARCO_OK;
}

int varco_partition_boundary_rows(const varco_plan_t *plan, int64_t *count) {
  if (!plan || !count) return VARCO_INVALID_ARG;
  *count = plan->nb;
  return VARCO_OK;
}

int varco_partition_set_l2_budget(varco_plan_t *plan, int64_t bytes) {
  if (!plan || bytes < 0) return VARCO_INVALID_ARG;
  plan->l2_budget = bytes;
  return VARCO_OK;
}

int varco_partition_gather_model(const varco_plan_t *plan, int32_t transposed, int64_t resident_rows, int64_t *entries,
                                 int64_t *sources, int64_t *rows_read) {
  if (!plan || resident_rows < 0) return VARCO_INVALID_ARG;
  const int64_t n = plan->n;
  int64_t e_tot = 0, s_tot = 0, r_tot = 0;
  std::vector<int64_t> use;
  try {
    for (int q = 0; q < plan->P; ++q) {
      use.clear();
      if (transposed) {
        for (int64_t r = plan->part_off[q]; r < plan->part_off[q + 1]; ++r) use.push_back(plan->rp[r + 1] - plan->rp[r]);
      } else {
        for (int64_t r = plan->part_off[q]; r < plan->part_off[q + 1]; ++r)
          use.push_back(plan->rpT[r + 1] - plan->rpT[r]);
        for (int64_t u = n + plan->slot_base[q]; u < n + plan->slot_base[q + 1]; ++u)
          use.push_back(plan->rpT[u + 1] - plan->rpT[u]);
      }
      const size_t keep = (size_t)std::min<int64_t>(resident_rows, (int64_t)use.size());
      std::nth_element(use.begin(), use.begin() + keep, use.end(), std::greater<int64_t>());
      for (size_t i = 0; i < use.size(); ++i) {
        e_tot += use[i];
        s_tot += use[i] > 0 ? 1 : 0;
        r_tot += i < keep ? (use[i] > 0 ? 1 : 0) : use[i];
      }
    }
  } catch (const std::bad_alloc &) {
    return VARCO_NOMEM;
  }
  if (entries) *entries = e_tot;
  if (sources) *sources = s_tot;
  if (rows_read) *rows_read = r_tot;
  return VARCO_OK;
}

int varco_partition_counts(const varco_plan_t *plan, int64_t *PxP) {
  if (!plan || !PxP) return VARCO_INVALID_ARG;
  std::copy(plan->counts.begin(), plan->counts.end(), PxP);
  return VARCO_OK;
}

int varco_partition_halo(const varco_plan_t *plan, int32_t p, int32_t q, const int64_t **global_ids, int64_t *count) {
  if (!plan || !global_ids || !count || p < 0 || q < 0 || p >= plan->P || q >= plan->P) return VARCO_INVALID_ARG;
  size_t s = (size_t)p * plan->P + q;
  *global_ids = plan->halo_ids.data() + plan->send_base[s];
  *count = plan->counts[s];
  return VARCO_OK;
}

int varco_partition_perm(const varco_plan_t *plan, const int64_t **new_to_old) {
  if (!plan || !new_to_old) return VARCO_INVALID_ARG;
  *new_to_old = plan->new_to_old.data();
  return VARCO_OK;
}

int varco_kept(int32_t F, varco_ratio_t c, int32_t *k) {
  if (!k) return VARCO_INVALID_ARG;
  int v = varco_kept_internal(F, c);
  if (v < 0) return VARCO_INVALID_ARG;
  *k = v;
  return VARCO_OK;
}

int varco_schedule_linear(int32_t epoch, int32_t K, int32_t slope_a, int32_t c_max, int32_t c_min, varco_ratio_t *c) {
  if (!c || K < 1 || slope_a < 1 || c_min < 1 || c_max < c_min || epoch < 0) return VARCO_INVALID_ARG;
  int64_t lo = (int64_t)c_min * K;
  int64_t v = (int64_t)c_max * K - (int64_t)slope_a * (c_max - c_min) * (int64_t)epoch;
  if (v < lo) v = lo;
  if (v > 0xFFFFFFFFLL) return VARCO_INVALID_ARG;
  c->num = (uint32_t)v;
  c->den = (uint32_t)K;
  return VARCO_OK;
}

int varco_schedule_rate_linear(int32_t epoch, uint32_t r0, uint32_t alpha, uint32_t den, varco_ratio_t *c) {
  if (!c || epoch < 0 || den == 0 || r0 == 0 || r0 > den) return VARCO_INVALID_ARG;
  uint64_t r = (uint64_t)r0 + (uint64_t)alpha * (uint64_t)epoch;   // < 2^63: no overflow
  if (r > den) r = den;
  c->num = den;
  c->den = (uint32_t)r;
  return VARCO_OK;
}

int varco_schedule_exponential(int32_t epoch, int32_t K, int32_t beta, varco_ratio_t *c) {
  if (!c || epoch < 0 || K < 1 || beta < 2) return VARCO_INVALID_ARG;
  uint64_t v = 1;
  for (int32_t i = epoch; i < K && v < 0xFFFFFFFFull; ++i) v *= (uint64_t)beta;
  c->num = v > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)v;
  c->den = 1;
  return VARCO_OK;
}

}  // extern "C"

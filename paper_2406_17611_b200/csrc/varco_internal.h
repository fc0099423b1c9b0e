// Internal declarations of libvarco: the plan object and the kernel launchers.
#ifndef VARCO_INTERNAL_H_
#define VARCO_INTERNAL_H_

#include <cstddef>
#include <cstdint>
#include <vector>

#include "varco.h"

struct varco_dev_image {
  // row r of the partition-contiguous order -> original node id (the id the keys are derived from)
  const int32_t *row_gid = nullptr;
  // aggregation structure of all partitions: row r aggregates from sources col[e] with weight
  // val[e]; a source < n is the local row of X with that index, a source >= n is halo slot (col - n)
  const int64_t *rp = nullptr;
  const int32_t *nloc = nullptr;   // leading entries of a forward row that point at local rows
  const int32_t *col = nullptr;
  const float *val = nullptr;
  // mean aggregation only: 1 / deg(r), the one weight every entry of row r carries (0 for an isolated row)
  const float *row_scale = nullptr;
  // transposed structure: source u (row or n + slot) is used by rows colT[e] with weight valT[e]
  const int64_t *rpT = nullptr;
  const int32_t *colT = nullptr;
  const float *valT = nullptr;
  // halo slots in receive order (destination, owner, id)
  const int32_t *slot_gid = nullptr;      // original id of the source node
  const int32_t *slot_src = nullptr;      // row of X that owns the data
  const int32_t *slot_sendpos = nullptr;  // position of the copy in send order (owner, destination, id)
  // unique boundary rows and the slots each one feeds (ascending destination)
  const int32_t *brow = nullptr;
  const int32_t *brow_ptr = nullptr;
  const int32_t *brow_slot = nullptr;
  // processing orders (forward rows; transposed sources): ordinary rows partition by partition,
  // and the long rows that get a CTA each
  const int32_t *order_f = nullptr;
  const int32_t *order_t = nullptr;
  const int32_t *hub_f = nullptr;
  const int32_t *hub_t = nullptr;
  const int32_t *short_f = nullptr;
  const int32_t *short_t = nullptr;
  // 8-entry records of the short rows (sources, weights), in class-list order
  const int32_t *short_f_col = nullptr, *short_t_col = nullptr;
  const float *short_f_val = nullptr, *short_t_val = nullptr;
  // [P + 1] first position of every partition in the class lists above
  const int32_t *order_f_start = nullptr, *order_t_start = nullptr, *hub_f_start = nullptr, *hub_t_start = nullptr,
                *short_f_start = nullptr, *short_t_start = nullptr;
};

struct varco_profile;  // CUDA-event bookkeeping, defined in runtime.cu

struct varco_plan {
  int64_t n = 0, nnz = 0, nnz_f = 0, H = 0, cross = 0, self_ = 0, nb = 0;
  int64_t max_part_sources = 0;        // largest (rows + halo slots) of one partition
  std::vector<int64_t> slot_base;      // [P + 1] first halo slot of every partition
  int64_t short_t_nlocal = 0;          // leading entries of short_t that are local rows (the rest are halo slots)
  int64_t l2_budget = 0;               // > 0: split feature rows so that a partition's gathered rows fit this many bytes
  int32_t P = 0;
  int conv = 0;
  std::vector<int64_t> new_to_old, part_off, counts, send_base, halo_ids;
  // host copies of the device image
  std::vector<int32_t> row_gid, col, colT, slot_gid, slot_src, slot_sendpos, brow, brow_ptr, brow_slot;
  std::vector<int32_t> order_f, order_t, hub_f, hub_t, short_f, short_t, nloc;
  std::vector<int32_t> order_f_start, order_t_start, hub_f_start, hub_t_start, short_f_start, short_t_start;
  std::vector<int64_t> rp, rpT;
  std::vector<float> val, valT, short_f_val, short_t_val, row_scale;
  std::vector<int32_t> short_f_col, short_t_col;
  // device image
  bool uploaded = false;
  varco_dev_image d;
  varco_profile *prof = nullptr;
};

// rate helpers shared by the entry points
int varco_kept_internal(int32_t F, varco_ratio_t c);

// profile hooks (runtime.cu)
void varco_prof_begin(const varco_plan *plan, int stage, void *stream);
void varco_prof_end(const varco_plan *plan, int stage, void *stream);
void varco_prof_destroy(varco_plan *plan);

struct StageTimer {
  const varco_plan *plan;
  int stage;
  void *stream;
  StageTimer(const varco_plan *p, int s, void *st) : plan(p), stage(s), stream(st) { varco_prof_begin(p, s, st); }
  ~StageTimer() { varco_prof_end(plan, stage, stream); }
};

#endif  // VARCO_INTERNAL_H_

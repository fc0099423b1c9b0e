// Device image of the plan, workspace sizing and per-stage event timing.
#include <atomic>
#include <mutex>
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "device_common.cuh"
#include "kernels.h"

namespace {

const char *kStageNames[VARCO_STAGE_COUNT] = {"varco:compress",    "varco:decompress", "varco:spmm",    "varco:gemm_fwd",
                                              "varco:gemm_dx",     "varco:gemm_dw",    "varco:spmm_t",  "varco:compress_bwd",
                                              "varco:scatter_add", "varco:aux"};

struct ImageItem {
  const void *host;
  size_t bytes;
  const void **dev;
};

template <typename T> ImageItem item(const std::vector<T> &v, const T **dev) {
  return ImageItem{v.data(), v.size() * sizeof(T), reinterpret_cast<const void **>(dev)};
}

std::vector<ImageItem> image_items(varco_plan *pl) {
  varco_dev_image &d = pl->d;
  return {item(pl->row_gid, &d.row_gid),
          item(pl->rp, &d.rp),
          item(pl->nloc, &d.nloc),
          item(pl->col, &d.col),
          item(pl->val, &d.val),
          item(pl->row_scale, &d.row_scale),
          item(pl->rpT, &d.rpT),
          item(pl->colT, &d.colT),
          item(pl->valT, &d.valT),
          item(pl->slot_gid, &d.slot_gid),
          item(pl->slot_src, &d.slot_src),
          item(pl->slot_sendpos, &d.slot_sendpos),
          item(pl->brow, &d.brow),
          item(pl->brow_ptr, &d.brow_ptr),
          item(pl->brow_slot, &d.brow_slot),
          item(pl->order_f, &d.order_f),
          item(pl->order_t, &d.order_t),
          item(pl->hub_f, &d.hub_f),
          item(pl->hub_t, &d.hub_t),
          item(pl->short_f, &d.short_f),
          item(pl->short_t, &d.short_t),
          item(pl->short_f_col, &d.short_f_col),
          item(pl->short_t_col, &d.short_t_col),
          item(pl->short_f_val, &d.short_f_val),
          item(pl->short_t_val, &d.short_t_val),
          item(pl->order_f_start, &d.order_f_start),
          item(pl->order_t_start, &d.order_t_start),
          item(pl->hub_f_start, &d.hub_f_start),
          item(pl->hub_t_start, &d.hub_t_start),
          item(pl->short_f_start, &d.short_f_start),
          item(pl->short_t_start, &d.short_t_start)};
}

size_t aligned(size_t b) { return (b + 255) / 256 * 256; }

#ifdef VARCO_DEBUG
// Debug build: every index array of the image against the extent of what it addresses.
bool image_is_sound(const varco_plan *pl) {
  const int64_t n = pl->n, H = pl->H, nsrc = n + H;
  auto below = [](const std::vector<int32_t> &v, int64_t limit) {
    for (int32_t x : v)
      if (x < 0 || x >= limit) return false;
    return true;
  };
  auto monotone = [](const std::vector<int64_t> &v, int64_t last) {
    for (size_t i = 1; i < v.size(); ++i)
      if (v[i] < v[i - 1]) return false;
    return !v.empty() && v.front() == 0 && v.back() == last;
  };
  if (!monotone(pl->rp, pl->nnz_f) || !monotone(pl->rpT, pl->nnz_f)) return false;
  if ((int64_t)pl->rp.size() != n + 1 || (int64_t)pl->rpT.size() != nsrc + 1) return false;
  if (!below(pl->col, nsrc) || !below(pl->colT, n)) return false;
  if (!below(pl->slot_src, n) || !below(pl->slot_sendpos, H ? H : 1) || !below(pl->brow, n) || !below(pl->brow_slot, H ? H : 1))
    return false;
  if (pl->brow_ptr.empty() || pl->brow_ptr.front() != 0 || pl->brow_ptr.back() != H) return false;
  for (size_t i = 1; i < pl->brow_ptr.size(); ++i)
    if (pl->brow_ptr[i] < pl->brow_ptr[i - 1]) return false;
  if (!below(pl->order_f, n) || !below(pl->hub_f, n) || !below(pl->short_f, n)) return false;
  if (!below(pl->order_t, nsrc) || !below(pl->hub_t, nsrc) || !below(pl->short_t, nsrc)) return false;
  for (int32_t c : pl->short_f_col)
    if (c < -1 || c >= nsrc) return false;
  for (int32_t c : pl->short_t_col)
    if (c < -1 || c >= n) return false;
  for (int64_t r = 0; r < n; ++r)
    if (pl->nloc[r] < 0 || pl->nloc[r] > pl->rp[r + 1] - pl->rp[r]) return false;
  return true;
}
#endif

std::atomic<int64_t> g_kernel_launches{0};

}  // namespace

void varco_count_launch() { g_kernel_launches.fetch_add(1, std::memory_order_relaxed); }

// ------------------------------------------------------------------------------------------ profile
struct varco_profile {
  bool on = false;
  std::mutex mu;
  struct Span {
    cudaEvent_t a, b;
  };
  std::vector<Span> spans[VARCO_STAGE_COUNT];
  std::vector<Span> pool;
  Span open[VARCO_STAGE_COUNT];
  bool is_open[VARCO_STAGE_COUNT] = {};
};

// Every stage is also an NVTX range (a profiler timeline shows the stages by name; without a tool attached
// the calls return at once).
void varco_prof_begin(const varco_plan *plan, int stage, void *stream) {
  nvtxRangePushA(kStageNames[stage]);
  varco_profile *pr = plan->prof;
  if (!pr || !pr->on) return;
  std::lock_guard<std::mutex> lock(pr->mu);
  varco_profile::Span s;
  if (!pr->pool.empty()) {
    s = pr->pool.back();
    pr->pool.pop_back();
  } else {
    if (cudaEventCreate(&s.a) != cudaSuccess) return;
    if (cudaEventCreate(&s.b) != cudaSuccess) {
      cudaEventDestroy(s.a);
      return;
    }
  }
  cudaEventRecord(s.a, (cudaStream_t)stream);
  pr->open[stage] = s;
  pr->is_open[stage] = true;
}

void varco_prof_end(const varco_plan *plan, int stage, void *stream) {
  nvtxRangePop();
  varco_profile *pr = plan->prof;
  if (!pr || !pr->on) return;
  std::lock_guard<std::mutex> lock(pr->mu);
  if (!pr->is_open[stage]) return;
  cudaEventRecord(pr->open[stage].b, (cudaStream_t)stream);
  pr->spans[stage].push_back(pr->open[stage]);
  pr->is_open[stage] = false;
}

void varco_prof_destroy(varco_plan *plan) {
  varco_profile *pr = plan->prof;
  if (!pr) return;
  for (int s = 0; s < VARCO_STAGE_COUNT; ++s)
    for (auto &sp : pr->spans[s]) {
      cudaEventDestroy(sp.a);
      cudaEventDestroy(sp.b);
    }
  for (auto &sp : pr->pool) {
    cudaEventDestroy(sp.a);
    cudaEventDestroy(sp.b);
  }
  delete pr;
  plan->prof = nullptr;
}

extern "C" {

int varco_profile_enable(varco_plan_t *plan, int on) {
  if (!plan) return VARCO_INVALID_ARG;
  if (!plan->prof) plan->prof = new (std::nothrow) varco_profile;
  if (!plan->prof) return VARCO_NOMEM;
  plan->prof->on = on != 0;
  return VARCO_OK;
}

int varco_profile_reset(varco_plan_t *plan) {
  if (!plan) return VARCO_INVALID_ARG;
  varco_profile *pr = plan->prof;
  if (!pr) return VARCO_OK;
  std::lock_guard<std::mutex> lock(pr->mu);
  for (int s = 0; s < VARCO_STAGE_COUNT; ++s) {
    for (auto &sp : pr->spans[s]) {
      cudaEventSynchronize(sp.b);
      pr->pool.push_back(sp);
    }
    pr->spans[s].clear();
  }
  return VARCO_OK;
}

int varco_profile_read(varco_plan_t *plan, int64_t *launches, double *milliseconds) {
  if (!plan || !launches || !milliseconds) return VARCO_INVALID_ARG;
  for (int s = 0; s < VARCO_STAGE_COUNT; ++s) {
    launches[s] = 0;
    milliseconds[s] = 0.0;
  }
  varco_profile *pr = plan->prof;
  if (!pr) return VARCO_OK;
  std::lock_guard<std::mutex> lock(pr->mu);
  for (int s = 0; s < VARCO_STAGE_COUNT; ++s)
    for (auto &sp : pr->spans[s]) {
      VARCO_CUDA_CHECK(cudaEventSynchronize(sp.b));
      float ms = 0.f;
      VARCO_CUDA_CHECK(cudaEventElapsedTime(&ms, sp.a, sp.b));
      launches[s] += 1;
      milliseconds[s] += (double)ms;
    }
  return VARCO_OK;
}

int varco_profile_spans(varco_plan_t *plan, int32_t stage, double *milliseconds, int64_t capacity, int64_t *count) {
  if (!plan || !count || stage < 0 || stage >= VARCO_STAGE_COUNT || capacity < 0 || (capacity > 0 && !milliseconds))
    return VARCO_INVALID_ARG;
  *count = 0;
  varco_profile *pr = plan->prof;
  if (!pr) return VARCO_OK;
  std::lock_guard<std::mutex> lock(pr->mu);
  int64_t i = 0;
  for (auto &sp : pr->spans[stage]) {
    if (i < capacity) {
      VARCO_CUDA_CHECK(cudaEventSynchronize(sp.b));
      float ms = 0.f;
      VARCO_CUDA_CHECK(cudaEventElapsedTime(&ms, sp.a, sp.b));
      milliseconds[i] = (double)ms;
    }
    ++i;
  }
  *count = i;
  return VARCO_OK;
}

int varco_debug_status(int32_t *is_debug_build, int32_t *word) {
  if (!is_debug_build || !word) return VARCO_INVALID_ARG;
#ifdef VARCO_DEBUG
  *is_debug_build = 1;
  VARCO_CUDA_CHECK(cudaDeviceSynchronize());
  const int w = varco_debug_word_spmm();
  if (w < 0) return VARCO_CUDA;
  *word = w;
#else
  *is_debug_build = 0;
  *word = 0;
#endif
  return VARCO_OK;
}

int varco_kernel_launches(int64_t *count) {
  if (!count) return VARCO_INVALID_ARG;
  *count = g_kernel_launches.load(std::memory_order_relaxed);
  return VARCO_OK;
}

// ------------------------------------------------------------------------------------------ image
int varco_partition_device_bytes(const varco_plan_t *plan, size_t *bytes) {
  if (!plan || !bytes) return VARCO_INVALID_ARG;
  size_t total = 0;
  for (const ImageItem &it : image_items(const_cast<varco_plan *>(plan))) total += aligned(it.bytes);
  *bytes = total + 256;
  return VARCO_OK;
}

int varco_partition_upload(varco_plan_t *plan, void *dev_buf, size_t bytes, void *stream) {
  if (!plan || !dev_buf) return VARCO_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(dev_buf) & 255u) != 0) return VARCO_INVALID_ARG;
  size_t need = 0;
  varco_partition_device_bytes(plan, &need);
  if (bytes < need) return VARCO_WORKSPACE_TOO_SMALL;
#ifdef VARCO_DEBUG
  if (!image_is_sound(plan)) return VARCO_BAD_GRAPH;
#endif
  plan->uploaded = false;
  size_t off = 0;
  for (const ImageItem &it : image_items(plan)) {
    char *dst = static_cast<char *>(dev_buf) + off;
    if (it.bytes)
      VARCO_CUDA_CHECK(cudaMemcpyAsync(dst, it.host, it.bytes, cudaMemcpyHostToDevice, (cudaStream_t)stream));
    *it.dev = dst;
    off += aligned(it.bytes);
  }
  VARCO_CUDA_CHECK(cudaStreamSynchronize((cudaStream_t)stream));
  plan->uploaded = true;
  return VARCO_OK;
}

int varco_workspace_bytes(const varco_plan_t *plan, int32_t F_in_max, int32_t F_out_max, varco_dtype_t dtype,
                          size_t *bytes) {
  if (!plan || !bytes || F_in_max < 1 || F_out_max < 1 || (dtype != VARCO_F32 && dtype != VARCO_BF16))
    return VARCO_INVALID_ARG;
  if (F_in_max > 2048 || F_out_max > 2048) return VARCO_UNSUPPORTED;
  varco_ws_layout L = varco_make_ws_layout(plan, F_in_max, F_out_max, dtype);
  *bytes = L.total;
  return VARCO_OK;
}

}  // extern "C"

varco_ws_layout varco_make_ws_layout(const varco_plan *pl, int F_in, int F_out, varco_dtype_t dt) {
  const size_t es = dt == VARCO_F32 ? 4 : 2;
  const int V = 16 / (int)es;
  varco_ws_layout L;
  L.ld_in = round_up64(F_in, V);
  L.ld_out = round_up64(F_out, V);
  size_t off = 0;
  auto take = [&](size_t b) {
    size_t o = off;
    off += aligned(b);
#ifdef VARCO_DEBUG
    if (L.num_guards < 8) L.guard[L.num_guards++] = off;   // 256 guard bytes behind every segment
    off += 256;
#endif
    return o;
  };
  L.status = take(256);                             // device status word of the last layer call
  L.packed = take((size_t)pl->H * L.ld_in * es);    // packed rows, stride rounded up to 16 bytes
  L.halo = take((size_t)pl->H * L.ld_in * es);      // forward: decompressed rows; backward: slot gradients
  L.wstride = round_up64(F_in, 8);
  L.wpos = take((size_t)pl->n * L.wstride * 2);     // kept positions of the call's boundary rows (k < F)
  L.dZ = take((size_t)pl->n * L.ld_out * es);
  L.dAgg = take((size_t)pl->n * L.ld_in * es);
  L.scratch_bytes = varco_gemm_scratch_bytes(F_in, F_out);
  L.scratch = take(L.scratch_bytes);
  L.total = off + 256;
  return L;
}

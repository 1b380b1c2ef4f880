// Host side of libtide.so: the C ABI, the page allocator and per-task tables, the work planner and the
// kernel launches.  See include/tide.h for the contract of every entry point.
//
// Allocator rule (what makes page tables reproducible): free pages are a LIFO stack primed so that a
// fresh pool hands out free_order[0], free_order[1], ...; an append walks its tasks in array order and
// pops one page each time a token lands on slot 0 of a new logical page; release and truncate push pages
// back last-to-first.  Every call validates completely before it changes anything.
#include <algorithm>
#include <atomic>
#include <climits>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "tide_internal.h"

using namespace tide;


namespace {

constexpr int kSlots = 8;                    // staging ring depth
constexpr size_t kSlotPageIds = 64 * 1024;   // most new page ids per upload
constexpr int kSlotRecs = 2048;              // most append records per upload
constexpr long long kPartRowsBase = 256 * 1024;
constexpr long long kMinSavedBytesDefault = 64ll << 20;   // reads a batch must save before rows are planned as sharing groups
constexpr int kStepSegStride = 2;   // each segment array of the step area holds up to 2 x max_batch_rows entries (rows + shared ranges)
// header of the step area (int32 words): counts a fixed-shape launch reads on the device, as (count, segments) pairs
constexpr int kHdrRecs = 0, kHdrDecItems = 2, kHdrTileItems = 4, kHdrUmmaItems = 6, kHdrMergeRows = 8;
constexpr int kMaxHostChunks = 8;                 // most row groups of one host-buffer step
constexpr size_t kHostChunkBytes = 64u << 20;      // transfer bytes per group from which cutting a step pays
constexpr size_t kZeroCopyBytes = 2u << 20;        // a host-buffer step up to this size is read and written in place (no copies)

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {
  size_t off_status, off_table, off_old_row, off_merge_ctr, off_step, off_meta, off_part_o, off_part_lse, off_stage_k, off_stage_v,
      off_stage_q, off_stage_out, off_stage_lse, total;
  size_t slot_bytes;
  size_t step_bytes;      // held plan of a multi-layer step: write records, then segments
  size_t step_seg_off;    // offset of the segments inside the step area
  long long part_rows;
};

// A planned batch as the launches need it: where the four segment arrays sit on the device and how many work
// items each launch has.
struct PlanDev {
  const Segment *seg_dec = nullptr, *seg_tile = nullptr, *seg_umma = nullptr, *seg_merge = nullptr;
  size_t n_dec = 0, n_tile = 0, n_umma = 0, n_merge = 0;
  long long items_dec = 0, items_tile = 0, items_umma = 0, merge_rows = 0;
};

struct PlanHost {
  std::vector<Segment> seg_dec, seg_tile, seg_umma, seg_merge;
  long long items_dec = 0, items_tile = 0, items_umma = 0, merge_rows = 0;
  long long fused_rows = 0;   // rows whose partials are merged by the decode kernel itself (not part of merge_rows)
  size_t n_all() const { return seg_dec.size() + seg_tile.size() + seg_umma.size() + seg_merge.size(); }
};

// What an extension of tasks did, as host arrays that are reused from call to call.
struct ExtendOut {
  std::vector<int32_t> idx, val;           // page-table delta: table[idx[i]] = val[i]
  std::vector<int32_t> cpy_src, cpy_dst;   // private copies of shared partial pages (old page -> new page)
  std::vector<int32_t> new_lp0, new_off;   // per task of the call: first logical page the delta brings, its place in val
  void clear() { idx.clear(); val.clear(); cpy_src.clear(); cpy_dst.clear(); new_lp0.clear(); new_off.clear(); }
};

struct Slot {
  uint8_t* host = nullptr;
  uint8_t* dev = nullptr;
  cudaEvent_t ev = nullptr;
  bool used = false;
};

}  // namespace

struct tide_kv {
  tide_kv_config_t cfg;
  Geom g;
  Layout lay;
  int device = 0;
  uint8_t* pool = nullptr;
  size_t layer_stride = 0;  // bytes between the page pools of consecutive layers
  uint8_t* ws = nullptr;
  int32_t* d_table = nullptr;
  int32_t* d_old_row = nullptr;  // one page-table row: what a task's row was before a prune changed it
  int* d_status = nullptr;
  float* d_part_o = nullptr;
  float* d_part_lse = nullptr;
  AppendInline append_inline;   // host images of the launches that carry their descriptors
  AttendInline attend_inline;
  int* d_merge_ctr = nullptr;   // finished-split counters of the segments whose last split merges (zero between launches)
  Slot slots[kSlots];
  int next_slot = 0;
  int* h_status = nullptr;  // pinned
  // bookkeeping
  std::vector<int32_t> free_stack;  // back() is the next page handed out
  std::vector<uint8_t> live;
  std::vector<int32_t> len;
  std::vector<std::vector<int32_t>> pages;
  std::vector<int32_t> refcnt;  // per physical page: how many tasks hold it (0 = free)
  ExtendOut ext;              // result of the most recent extension
  std::vector<int32_t> mark;  // scratch for duplicate detection
  int32_t mark_gen = 0;
  int64_t used_tokens = 0;
  // last plan
  int64_t last_decode_items = 0, last_prefill_items = 0, last_merge_rows = 0, last_launches = 0;
  int64_t append_launches = 0;
  int64_t last_groups = 0, last_grouped_rows = 0;   // rows planned as groups that share their first pages
  bool no_grouping = false;
  long long min_saved_bytes = kMinSavedBytesDefault;
  // optional per-phase timing (events on the caller's stream)
  bool profiling = false;
  cudaEvent_t ev_append[2] = {nullptr, nullptr};
  cudaEvent_t ev_attend[4] = {nullptr, nullptr, nullptr, nullptr};
  bool have_append_times = false, have_attend_times = false;
  int umma_min_rows = kDecodeTileRows + 1;  // packed rows from which a resume row takes the tcgen05 path (measured:
                                            // it beats the warp-MMA tile path from the first row beyond a decode item)
  int items_per_sm = kTargetItemsPerSm;  // work items the planner aims for per SM
  int num_sms = 0;                       // multiprocessors of the handle's device
  long long wait_limit_ns = kWaitLimitNsDefault;   // bound of every wait inside a kernel
  int umma_tile_keys = 128;              // key-tile size of the tcgen05 kernel: 64 (Q in TMEM) or 128 (Q in shared memory)
  bool drop_first_stage_once = false;    // test hook: armed by tide_tune, consumed by the next attention launch set
  // multi-layer step held between tide_step_begin and the tide_step_layer calls
  uint8_t* h_step = nullptr;   // pinned staging of the step area
  cudaEvent_t ev_step = nullptr;
  bool step_upload_pending = false, step_valid = false;
  PlanDev step_plan;
  int step_recs = 0, step_tokens = 0;
  // fixed launch shapes for tide_step_layer (0 = off): most work items / rows / tokens a step may plan
  bool fixed_grids = false;
  int cap_dec = 0, cap_tile = 0, cap_umma = 0, cap_merge_rows = 0, cap_tokens = 0;
  // host-buffer steps: copy streams and the events that order them against the caller's stream
  cudaStream_t st_in = nullptr, st_out = nullptr;
  cudaEvent_t ev_host[2 * kMaxHostChunks + 2] = {};   // copies-in done, kernels done (per group); start, end
  int host_step_chunks = 0;   // 0 = by size
  bool slots_mapped = false;     // the staging slots' host addresses are valid on the device too
  bool upload_by_kernel = false;
  bool host_zero_copy = true;             // small host-buffer steps: kernels address the pinned host buffers themselves
  bool inline_descriptors = true;         // small appends and decode-only batches carry their descriptors in the launch
  bool always_upload_by_kernel = true;    // planning uploads by a kernel reading the mapped staging slot, not by the copy engine
                                          // (measured on a 64-row decode step: 157 -> 147 us; tide_tune can switch it off)
  uint8_t* layer_pool(int layer) const { return pool + (size_t)layer * layer_stride; }
};

namespace {

bool valid_geometry(const tide_kv_config_t* c) {
  if (c == nullptr) return false;
  if (c->num_layers < 1 || c->num_layers > 256) return false;
  if (c->num_kv_heads <= 0 || c->num_q_heads <= 0 || c->num_q_heads % c->num_kv_heads != 0) return false;
  if (c->num_q_heads / c->num_kv_heads > 16) return false;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->page_size != 16 && c->page_size != 32) return false;
  if (c->max_tasks <= 0 || c->max_pages_per_task <= 0 || c->max_batch_rows <= 0) return false;
  if (c->num_pages <= 0 || c->num_pages > 0x7fffffffLL || c->max_batch_tokens <= 0) return false;
  if ((long long)c->max_tasks * c->max_pages_per_task > 0x7fffffffLL) return false;
  if (c->max_batch_tokens * (long long)c->num_q_heads > 0x7fffffffLL) return false;
  return true;
}

Geom make_geom(const tide_kv_config_t* c) {
  Geom g;
  g.Hq = c->num_q_heads; g.Hkv = c->num_kv_heads; g.D = c->head_dim; g.S = c->page_size; g.G = g.Hq / g.Hkv;
  g.max_pages_per_task = c->max_pages_per_task;
  g.group_bytes = (g.D / 64) * 1024;
  g.kblock_bytes = (g.S / 8) * g.group_bytes;
  g.head_bytes = 2 * g.kblock_bytes;
  g.page_bytes = (long long)g.head_bytes * g.Hkv;
  return g;
}

Layout make_layout(const tide_kv_config_t* c, const Geom& g) {
  Layout L;
  size_t off = 0;
  L.off_status = off; off += 256;
  L.off_table = off; off = align_up(off + (size_t)c->max_tasks * c->max_pages_per_task * 4, 256);
  L.off_old_row = off; off = align_up(off + (size_t)c->max_pages_per_task * 4 + 64, 256);   // row + one page pair
  L.off_merge_ctr = off; off = align_up(off + (size_t)kStepSegStride * c->max_batch_rows * g.Hkv * 4, 256);   // finished-split counters
  // step area: 256-byte header of counts | write records | four segment arrays of max_batch_rows entries each
  L.step_seg_off = align_up(256 + (size_t)c->max_batch_rows * sizeof(AppendRec), 256);
  L.step_bytes = align_up(L.step_seg_off + (size_t)(4 * kStepSegStride * c->max_batch_rows) * sizeof(Segment), 256);
  L.off_step = off; off += L.step_bytes;
  L.slot_bytes = align_up(256 + (size_t)kSlotRecs * sizeof(AppendRec) + kSlotPageIds * 8 + (size_t)kSlotRecs * 8 +
                              (size_t)(3 * c->max_batch_rows + 8) * sizeof(Segment), 256);   // rows + shared ranges (<= rows / 2) + merge list
  L.off_meta = off; off += L.slot_bytes * kSlots;
  L.part_rows = kPartRowsBase + (long long)g.Hq * c->max_batch_rows * 4;
  L.off_part_o = off; off = align_up(off + (size_t)L.part_rows * g.D * 4, 256);
  L.off_part_lse = off; off = align_up(off + (size_t)L.part_rows * 4, 256);
  const size_t kv_rows = (size_t)c->max_batch_tokens * g.Hkv * g.D * 2;
  const size_t q_rows = (size_t)c->max_batch_tokens * g.Hq * g.D * 2;
  L.off_stage_k = off; off = align_up(off + kv_rows, 256);
  L.off_stage_v = off; off = align_up(off + kv_rows, 256);
  L.off_stage_q = off; off = align_up(off + q_rows, 256);
  L.off_stage_out = off; off = align_up(off + q_rows, 256);
  L.off_stage_lse = off; off = align_up(off + (size_t)c->max_batch_tokens * g.Hq * 4, 256);
  L.total = off;
  return L;
}

bool is_permutation(const int32_t* order, int64_t n, std::vector<uint8_t>& seen) {
  seen.assign((size_t)n, 0);
  for (int64_t i = 0; i < n; ++i) {
    const int32_t p = order[i];
    if (p < 0 || p >= n || seen[(size_t)p]) return false;
    seen[(size_t)p] = 1;
  }
  return true;
}

void prime_free_stack(tide_kv* kv, const int32_t* order) {
  const int64_t n = kv->cfg.num_pages;
  kv->free_stack.resize((size_t)n);
  for (int64_t i = 0; i < n; ++i) kv->free_stack[(size_t)(n - 1 - i)] = order ? order[i] : (int32_t)i;
}

int ceil_div(int a, int b) { return (a + b - 1) / b; }

int32_t pop_page(tide_kv* kv) {
  const int32_t page = kv->free_stack.back();
  kv->free_stack.pop_back();
  kv->refcnt[(size_t)page] = 1;
  return page;
}

// Drops one holder of `page`; the page returns to the free stack when nobody holds it any more.
void unref_page(tide_kv* kv, int32_t page) {
  if (--kv->refcnt[(size_t)page] == 0) kv->free_stack.push_back(page);
}

// True if the next token of `task` would be written into a page that another task also holds.
bool last_page_shared(const tide_kv* kv, int32_t task) {
  return kv->len[task] % kv->g.S != 0 && kv->refcnt[(size_t)kv->pages[task].back()] > 1;
}

bool task_in_range(const tide_kv* kv, int32_t t) { return t >= 0 && t < kv->cfg.max_tasks; }

// Takes the next staging slot, waiting until the device work that last used it has finished.
int acquire_slot(tide_kv* kv, Slot** out) {
  Slot& s = kv->slots[kv->next_slot];
  kv->next_slot = (kv->next_slot + 1) % kSlots;
  if (s.used && cudaEventSynchronize(s.ev) != cudaSuccess) return TIDE_ERR_CUDA;
  *out = &s;
  return TIDE_OK;
}

// Small upload of planning data from a staging slot.  Normally a copy-engine transfer; while a host-buffer step
// has large copies in flight on other streams it is done by a kernel instead, which does not queue behind them.
cudaError_t upload(const tide_kv* kv, void* dst, const void* src, size_t bytes, cudaStream_t st) {
  if (kv->upload_by_kernel || (kv->always_upload_by_kernel && kv->slots_mapped)) return launch_upload(dst, src, bytes, st);
  return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, st);
}

int release_slot(Slot* s, cudaStream_t st) {
  s->used = true;
  return cudaEventRecord(s->ev, st) == cudaSuccess ? TIDE_OK : TIDE_ERR_CUDA;
}

}  // namespace

extern "C" {

const char* tide_strerror(int code) {
  switch (code) {
    case TIDE_OK: return "ok";
    case TIDE_ERR_INVALID_ARG: return "invalid argument";
    case TIDE_ERR_UNKNOWN_TASK: return "unknown task";
    case TIDE_ERR_TASK_EXISTS: return "task already exists";
    case TIDE_ERR_DUPLICATE_TASK: return "task named twice in one append";
    case TIDE_ERR_NO_PAGES: return "not enough free pages";
    case TIDE_ERR_TABLE_FULL: return "task would exceed max_pages_per_task";
    case TIDE_ERR_CTX_RANGE: return "row violates 1 <= q_len <= ctx_len <= resident length";
    case TIDE_ERR_WORKSPACE: return "pool, workspace or batch limit too small";
    case TIDE_ERR_CUDA: return "CUDA runtime error";
    case TIDE_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
    default: return "unknown tide status";
  }
}

int tide_kv_required_bytes(const tide_kv_config_t* cfg, size_t* pool_bytes, size_t* workspace_bytes) {
  if (!valid_geometry(cfg)) return TIDE_ERR_INVALID_ARG;
  const Geom g = make_geom(cfg);
  if (pool_bytes) *pool_bytes = (size_t)cfg->num_layers * (size_t)cfg->num_pages * (size_t)g.page_bytes;
  if (workspace_bytes) *workspace_bytes = make_layout(cfg, g).total;
  return TIDE_OK;
}

int tide_kv_create(const tide_kv_config_t* cfg, tide_kv_t** out) {
  if (out == nullptr || !valid_geometry(cfg)) return TIDE_ERR_INVALID_ARG;
  if (cfg->pool == nullptr || cfg->workspace == nullptr) return TIDE_ERR_INVALID_ARG;
  if (((uintptr_t)cfg->pool & 1023) || ((uintptr_t)cfg->workspace & 255)) return TIDE_ERR_INVALID_ARG;
  const Geom g = make_geom(cfg);
  const Layout lay = make_layout(cfg, g);
  if (cfg->pool_bytes < (size_t)cfg->num_layers * (size_t)cfg->num_pages * (size_t)g.page_bytes || cfg->workspace_bytes < lay.total)
    return TIDE_ERR_WORKSPACE;
  std::vector<uint8_t> seen;
  if (cfg->free_order && !is_permutation(cfg->free_order, cfg->num_pages, seen)) return TIDE_ERR_INVALID_ARG;

  tide_kv* kv = new (std::nothrow) tide_kv();
  if (!kv) return TIDE_ERR_INVALID_ARG;
  kv->cfg = *cfg;
  kv->cfg.free_order = nullptr;
  kv->g = g;
  kv->lay = lay;
  kv->pool = (uint8_t*)cfg->pool;
  kv->layer_stride = (size_t)cfg->num_pages * (size_t)g.page_bytes;
  kv->ws = (uint8_t*)cfg->workspace;
  kv->d_status = (int*)(kv->ws + lay.off_status);
  kv->d_table = (int32_t*)(kv->ws + lay.off_table);
  kv->d_old_row = (int32_t*)(kv->ws + lay.off_old_row);
  kv->d_part_o = (float*)(kv->ws + lay.off_part_o);
  kv->d_part_lse = (float*)(kv->ws + lay.off_part_lse);
  kv->d_merge_ctr = (int*)(kv->ws + lay.off_merge_ctr);
  bool ok = cudaGetDevice(&kv->device) == cudaSuccess;
  kv->num_sms = sm_count();
  ok = ok && kv->num_sms > 0;
  ok = ok && attend_kernels_init() == cudaSuccess && attend_umma_init() == cudaSuccess && attend_umma128_init() == cudaSuccess;
  ok = ok && cudaMemset(kv->d_status, 0, 256) == cudaSuccess;
  ok = ok && cudaMemset(kv->d_merge_ctr, 0, (size_t)kStepSegStride * cfg->max_batch_rows * g.Hkv * 4) == cudaSuccess;
  ok = ok && cudaHostAlloc((void**)&kv->h_status, 64, cudaHostAllocDefault) == cudaSuccess;
  ok = ok && cudaHostAlloc((void**)&kv->h_step, lay.step_bytes, cudaHostAllocDefault) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&kv->ev_step, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; ok && i < kSlots; ++i) {
    ok = cudaHostAlloc((void**)&kv->slots[i].host, lay.slot_bytes, cudaHostAllocMapped) == cudaSuccess;
    void* on_device = nullptr;
    if (ok && i == 0) kv->slots_mapped = true;
    if (ok && (cudaHostGetDevicePointer(&on_device, kv->slots[i].host, 0) != cudaSuccess || on_device != (void*)kv->slots[i].host)) {
      kv->slots_mapped = false;   // no unified addressing: uploads stay copy-engine transfers
      cudaGetLastError();
    }
    ok = ok && cudaEventCreateWithFlags(&kv->slots[i].ev, cudaEventDisableTiming) == cudaSuccess;
    kv->slots[i].dev = kv->ws + lay.off_meta + (size_t)i * lay.slot_bytes;
  }
  if (!ok) {
    tide_kv_destroy(kv);
    return TIDE_ERR_CUDA;
  }
  kv->live.assign((size_t)cfg->max_tasks, 0);
  kv->len.assign((size_t)cfg->max_tasks, 0);
  kv->pages.resize((size_t)cfg->max_tasks);
  kv->mark.assign((size_t)cfg->max_tasks, 0);
  kv->refcnt.assign((size_t)cfg->num_pages, 0);
  prime_free_stack(kv, cfg->free_order);
  *out = kv;
  return TIDE_OK;
}

int tide_kv_destroy(tide_kv_t* kv) {
  if (kv == nullptr) return TIDE_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  for (int i = 0; i < kSlots; ++i) {
    if (kv->slots[i].host) cudaFreeHost(kv->slots[i].host);
    if (kv->slots[i].ev) cudaEventDestroy(kv->slots[i].ev);
  }
  if (kv->h_status) cudaFreeHost(kv->h_status);
  if (kv->h_step) cudaFreeHost(kv->h_step);
  if (kv->ev_step) cudaEventDestroy(kv->ev_step);
  if (kv->st_in) cudaStreamDestroy(kv->st_in);
  if (kv->st_out) cudaStreamDestroy(kv->st_out);
  for (cudaEvent_t e : kv->ev_host) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : kv->ev_append) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : kv->ev_attend) if (e) cudaEventDestroy(e);
  delete kv;
  return TIDE_OK;
}

int tide_kv_reset(tide_kv_t* kv, const int32_t* free_order) {
  if (kv == nullptr) return TIDE_ERR_INVALID_ARG;
  std::vector<uint8_t> seen;
  if (free_order && !is_permutation(free_order, kv->cfg.num_pages, seen)) return TIDE_ERR_INVALID_ARG;
  std::fill(kv->live.begin(), kv->live.end(), 0);
  std::fill(kv->len.begin(), kv->len.end(), 0);
  for (auto& p : kv->pages) p.clear();
  std::fill(kv->refcnt.begin(), kv->refcnt.end(), 0);
  kv->used_tokens = 0;
  kv->step_valid = false;
  prime_free_stack(kv, free_order);
  return TIDE_OK;
}

int tide_kv_alloc(tide_kv_t* kv, int32_t task, int64_t reserve_tokens) {
  if (kv == nullptr || !task_in_range(kv, task) || reserve_tokens < 0) return TIDE_ERR_INVALID_ARG;
  if (kv->live[task]) return TIDE_ERR_TASK_EXISTS;
  if ((int64_t)kv->free_stack.size() * kv->g.S < reserve_tokens) return TIDE_ERR_NO_PAGES;
  kv->live[task] = 1;
  kv->len[task] = 0;
  kv->pages[task].clear();
  return TIDE_OK;
}

int tide_kv_release(tide_kv_t* kv, int32_t task) {
  if (kv == nullptr || !task_in_range(kv, task)) return TIDE_ERR_INVALID_ARG;
  if (!kv->live[task]) return TIDE_ERR_UNKNOWN_TASK;
  kv->step_valid = false;
  auto& pg = kv->pages[task];
  for (size_t i = pg.size(); i-- > 0;) unref_page(kv, pg[i]);
  pg.clear();
  kv->used_tokens -= kv->len[task];
  kv->len[task] = 0;
  kv->live[task] = 0;
  return TIDE_OK;
}

int tide_kv_truncate(tide_kv_t* kv, int32_t task, int32_t new_len) {
  if (kv == nullptr || !task_in_range(kv, task)) return TIDE_ERR_INVALID_ARG;
  if (!kv->live[task]) return TIDE_ERR_UNKNOWN_TASK;
  if (new_len < 0 || new_len > kv->len[task]) return TIDE_ERR_INVALID_ARG;
  kv->step_valid = false;
  auto& pg = kv->pages[task];
  const size_t keep = (size_t)ceil_div(new_len, kv->g.S);
  while (pg.size() > keep) {
    unref_page(kv, pg.back());
    pg.pop_back();
  }
  kv->used_tokens -= kv->len[task] - new_len;
  kv->len[task] = new_len;
  return TIDE_OK;
}

int tide_kv_task_len(tide_kv_t* kv, int32_t task, int32_t* len) {
  if (kv == nullptr || len == nullptr || !task_in_range(kv, task)) return TIDE_ERR_INVALID_ARG;
  if (!kv->live[task]) return TIDE_ERR_UNKNOWN_TASK;
  *len = kv->len[task];
  return TIDE_OK;
}

int tide_kv_page_table(tide_kv_t* kv, int32_t task, int32_t* out, int32_t cap, int32_t* n_pages) {
  if (kv == nullptr || n_pages == nullptr || !task_in_range(kv, task) || cap < 0) return TIDE_ERR_INVALID_ARG;
  if (!kv->live[task]) return TIDE_ERR_UNKNOWN_TASK;
  const auto& pg = kv->pages[task];
  *n_pages = (int32_t)pg.size();
  if (out != nullptr) {
    if ((size_t)cap < pg.size()) return TIDE_ERR_INVALID_ARG;
    std::memcpy(out, pg.data(), pg.size() * sizeof(int32_t));
  }
  return TIDE_OK;
}

int tide_kv_usage(tide_kv_t* kv, int64_t* used_tokens, int64_t* free_pages) {
  if (kv == nullptr) return TIDE_ERR_INVALID_ARG;
  if (used_tokens) *used_tokens = kv->used_tokens;
  if (free_pages) *free_pages = (int64_t)kv->free_stack.size();
  return TIDE_OK;
}

// Range, liveness and duplicate checks shared by every call that takes a (task_ids, indptr) list.
static int check_task_list(tide_kv* kv, int32_t n_tasks, const int32_t* task_ids, const int32_t* indptr) {
  if (task_ids == nullptr || indptr == nullptr || indptr[0] != 0) return TIDE_ERR_INVALID_ARG;
  for (int j = 0; j < n_tasks; ++j)
    if (indptr[j + 1] < indptr[j]) return TIDE_ERR_INVALID_ARG;
  for (int j = 0; j < n_tasks; ++j) {
    if (!task_in_range(kv, task_ids[j])) return TIDE_ERR_INVALID_ARG;
    if (!kv->live[task_ids[j]]) return TIDE_ERR_UNKNOWN_TASK;
  }
  if (++kv->mark_gen == 0x7fffffff) {
    std::fill(kv->mark.begin(), kv->mark.end(), 0);
    kv->mark_gen = 1;
  }
  for (int j = 0; j < n_tasks; ++j) {
    if (kv->mark[task_ids[j]] == kv->mark_gen) return TIDE_ERR_DUPLICATE_TASK;
    kv->mark[task_ids[j]] = kv->mark_gen;
  }
  return TIDE_OK;
}

// Would growing task_ids[j] by indptr[j+1]-indptr[j] tokens fit the page tables and the free stack?
static int check_extend(const tide_kv* kv, int32_t n_tasks, const int32_t* task_ids, const int32_t* indptr) {
  const Geom& g = kv->g;
  long long need = 0;
  for (int j = 0; j < n_tasks; ++j) {
    const int t = task_ids[j], c = indptr[j + 1] - indptr[j];
    if ((long long)kv->len[t] + c > 0x7fffffffLL) return TIDE_ERR_TABLE_FULL;
    const int after = ceil_div(kv->len[t] + c, g.S);
    if (after > g.max_pages_per_task) return TIDE_ERR_TABLE_FULL;
    need += after - ceil_div(kv->len[t], g.S);
    if (c > 0 && last_page_shared(kv, t)) ++need;   // a private copy of the shared partial page comes first
  }
  return need > (long long)kv->free_stack.size() ? TIDE_ERR_NO_PAGES : TIDE_OK;
}

// Grows task_ids[j] by indptr[j+1]-indptr[j] tokens in the host tables and records, in kv->ext, what the device
// still has to be told: the page-table delta and the private copies of shared partial pages (a task that ends inside
// a page that other tasks hold gets a private copy of that page before its other pages are taken).  No device work.
// The task list must have passed check_task_list.
static int extend_bookkeeping(tide_kv* kv, int32_t n_tasks, const int32_t* task_ids, const int32_t* indptr) {
  const Geom& g = kv->g;
  const int rc = check_extend(kv, n_tasks, task_ids, indptr);
  if (rc != TIDE_OK) return rc;
  // ---- mutation ----
  kv->step_valid = false;
  ExtendOut& x = kv->ext;
  x.clear();
  for (int j = 0; j < n_tasks; ++j) {
    const int t = task_ids[j];
    const int c = indptr[j + 1] - indptr[j];
    auto& pg = kv->pages[t];
    x.new_lp0.push_back((int32_t)pg.size());
    x.new_off.push_back((int32_t)x.idx.size());
    if (c == 0) continue;
    if (last_page_shared(kv, t)) {
      const int32_t old_page = pg.back(), new_page = pop_page(kv);
      x.cpy_src.push_back(old_page);
      x.cpy_dst.push_back(new_page);
      x.new_lp0.back() = (int32_t)pg.size() - 1;             // the copy takes the old page's place in the table
      x.idx.push_back(t * g.max_pages_per_task + (int32_t)pg.size() - 1);
      x.val.push_back(new_page);
      pg.back() = new_page;
      unref_page(kv, old_page);
    }
    const int new_pages = ceil_div(kv->len[t] + c, g.S) - ceil_div(kv->len[t], g.S);
    for (int k = 0; k < new_pages; ++k) {
      const int32_t page = pop_page(kv);
      x.idx.push_back(t * g.max_pages_per_task + (int32_t)pg.size());
      x.val.push_back(page);
      pg.push_back(page);
    }
    kv->len[t] += c;
    kv->used_tokens += c;
  }
  return TIDE_OK;
}

// The private page copies of kv->ext on every layer, in uploads of bounded size.
static int upload_cow_copies(tide_kv* kv, cudaStream_t st) {
  const ExtendOut& x = kv->ext;
  for (size_t done = 0; done < x.cpy_src.size();) {
    Slot* slot;
    int rc = acquire_slot(kv, &slot);
    if (rc != TIDE_OK) return rc;
    const size_t n = std::min<size_t>(kSlotRecs, x.cpy_src.size() - done);
    int32_t* h = (int32_t*)(slot->host + 256);
    std::memcpy(h, x.cpy_src.data() + done, n * 4);
    std::memcpy(h + n, x.cpy_dst.data() + done, n * 4);
    if (upload(kv, slot->dev + 256, h, 2 * n * 4, st) != cudaSuccess) return TIDE_ERR_CUDA;
    const int32_t* d = (const int32_t*)(slot->dev + 256);
    for (int l = 0; l < kv->cfg.num_layers; ++l) {
      if (launch_copy_pages(kv->layer_pool(l), d, d + n, (int)n, kv->g.page_bytes, st) != cudaSuccess) return TIDE_ERR_CUDA;
      ++kv->append_launches;
    }
    if ((rc = release_slot(slot, st)) != TIDE_OK) return rc;
    done += n;
  }
  return TIDE_OK;
}

// The page-table delta of kv->ext to the device table (a launch of its own), in uploads of bounded size.
static int upload_table_delta(tide_kv* kv, cudaStream_t st) {
  const ExtendOut& x = kv->ext;
  for (size_t done = 0; done < x.idx.size();) {
    Slot* slot;
    int rc = acquire_slot(kv, &slot);
    if (rc != TIDE_OK) return rc;
    const size_t n = std::min<size_t>(kSlotPageIds, x.idx.size() - done);
    int32_t* h = (int32_t*)(slot->host + 256);
    std::memcpy(h, x.idx.data() + done, n * 4);
    std::memcpy(h + n, x.val.data() + done, n * 4);
    if (upload(kv, slot->dev + 256, h, 2 * n * 4, st) != cudaSuccess) return TIDE_ERR_CUDA;
    const int32_t* d = (const int32_t*)(slot->dev + 256);
    if (launch_table_update(kv->d_table, d, d + n, (int)n, st) != cudaSuccess) return TIDE_ERR_CUDA;
    ++kv->append_launches;
    if ((rc = release_slot(slot, st)) != TIDE_OK) return rc;
    done += n;
  }
  return TIDE_OK;
}

// extend_bookkeeping, then the device side: the page-table delta and (with cow_out == nullptr) the private page
// copies on every layer; otherwise the (old, new) page pairs are handed back and the caller copies (it may have to
// read the old pages first).
static int extend_tasks(tide_kv* kv, int32_t n_tasks, const int32_t* task_ids, const int32_t* indptr, cudaStream_t st,
                        std::vector<int32_t>* cow_out) {
  int rc = extend_bookkeeping(kv, n_tasks, task_ids, indptr);
  if (rc != TIDE_OK) return rc;
  if ((rc = upload_table_delta(kv, st)) != TIDE_OK) return rc;
  if (cow_out != nullptr) {
    for (size_t i = 0; i < kv->ext.cpy_src.size(); ++i) {
      cow_out->push_back(kv->ext.cpy_src[i]);
      cow_out->push_back(kv->ext.cpy_dst[i]);
    }
    return TIDE_OK;
  }
  return upload_cow_copies(kv, st);
}

// Writes the K/V rows of one layer into the LAST indptr[j+1]-indptr[j] positions of task_ids[j] (pure data; the
// caller has checked that every task is at least that long).  Records travel in uploads of bounded size.
static int write_tasks(tide_kv* kv, int32_t layer, int32_t n_tasks, const int32_t* task_ids, const int32_t* indptr,
                       const void* new_k, const void* new_v, cudaStream_t st) {
  const Geom& g = kv->g;
  int j = 0;
  int rc = TIDE_OK;
  while (j < n_tasks) {
    Slot* slot;
    if ((rc = acquire_slot(kv, &slot)) != TIDE_OK) return rc;
    AppendRec* recs = (AppendRec*)(slot->host + 256);
    int n_recs = 0, tok_lo = -1, tok_hi = -1, grp_cursor = 0;
    for (; j < n_tasks && n_recs < kSlotRecs; ++j) {
      const int c = indptr[j + 1] - indptr[j];
      if (c == 0) continue;
      if (tok_lo < 0) tok_lo = indptr[j];
      AppendRec& r = recs[n_recs++];
      r.table_off = task_ids[j] * g.max_pages_per_task;
      r.pos0 = kv->len[task_ids[j]] - c;
      r.tok0 = indptr[j] - tok_lo;
      r.count = c;
      r.new_lp0 = INT_MAX;
      r.new_off = 0;
      r.grp0 = grp_cursor; r.pad1 = 0;
      grp_cursor += ((r.pos0 & 7) + r.count + 7) >> 3;
      tok_hi = indptr[j + 1];
    }
    if (n_recs > 0) {
      if (upload(kv, slot->dev + 256, recs, (size_t)n_recs * sizeof(AppendRec), st) != cudaSuccess)
        return TIDE_ERR_CUDA;
      AppendParams ap;
      ap.pool = kv->layer_pool(layer);
      ap.table = kv->d_table;
      ap.recs = (const AppendRec*)(slot->dev + 256);
      ap.n_recs = n_recs;
      ap.n_tokens = tok_hi - tok_lo;
      ap.new_k = (const uint16_t*)new_k + (size_t)tok_lo * g.Hkv * g.D;
      ap.new_v = (const uint16_t*)new_v + (size_t)tok_lo * g.Hkv * g.D;
      ap.g = g;
      if (launch_append(ap, st) != cudaSuccess) return TIDE_ERR_CUDA;
      ++kv->append_launches;
    }
    if ((rc = release_slot(slot, st)) != TIDE_OK) return rc;
  }
  return TIDE_OK;
}

static bool bad_kv_rows(int T, const void* new_k, const void* new_v) {
  return T > 0 && (new_k == nullptr || new_v == nullptr || ((uintptr_t)new_k & 15) || ((uintptr_t)new_v & 15));
}

int tide_kv_extend(tide_kv_t* kv, int32_t n_tasks, const int32_t* task_ids, const int32_t* indptr, void* stream) {
  if (kv == nullptr || n_tasks < 0) return TIDE_ERR_INVALID_ARG;
  if (n_tasks == 0) return TIDE_OK;
  int rc = check_task_list(kv, n_tasks, task_ids, indptr);
  if (rc != TIDE_OK) return rc;
  kv->append_launches = 0;
  return extend_tasks(kv, n_tasks, task_ids, indptr, (cudaStream_t)stream, nullptr);
}

int tide_kv_write(tide_kv_t* kv, int32_t layer, int32_t n_tasks, const int32_t* task_ids, const int32_t* indptr,
                  const void* new_k, const void* new_v, void* stream) {
  if (kv == nullptr || layer < 0 || layer >= kv->cfg.num_layers || n_tasks < 0) return TIDE_ERR_INVALID_ARG;
  if (n_tasks == 0) return TIDE_OK;
  int rc = check_task_list(kv, n_tasks, task_ids, indptr);
  if (rc != TIDE_OK) return rc;
  if (bad_kv_rows(indptr[n_tasks], new_k, new_v)) return TIDE_ERR_INVALID_ARG;
  for (int j = 0; j < n_tasks; ++j)
    if (indptr[j + 1] - indptr[j] > kv->len[task_ids[j]]) return TIDE_ERR_CTX_RANGE;
  cudaStream_t st = (cudaStream_t)stream;
  if (kv->profiling) cudaEventRecord(kv->ev_append[0], st);
  rc = write_tasks(kv, layer, n_tasks, task_ids, indptr, new_k, new_v, st);
  if (rc == TIDE_OK && kv->profiling) {
    cudaEventRecord(kv->ev_append[1], st);
    kv->have_append_times = true;
  }
  return rc;
}

int tide_kv_append(tide_kv_t* kv, int32_t layer, int32_t n_tasks, const int32_t* task_ids, const int32_t* indptr,
                   const void* new_k, const void* new_v, void* stream) {
  if (kv == nullptr || layer != 0 || n_tasks < 0) return TIDE_ERR_INVALID_ARG;
  if (n_tasks == 0) return TIDE_OK;
  int rc = check_task_list(kv, n_tasks, task_ids, indptr);
  if (rc != TIDE_OK) return rc;
  if (bad_kv_rows(indptr[n_tasks], new_k, new_v)) return TIDE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  kv->append_launches = 0;
  if (kv->profiling) cudaEventRecord(kv->ev_append[0], st);
  if ((rc = extend_bookkeeping(kv, n_tasks, task_ids, indptr)) != TIDE_OK) return rc;
  if ((rc = upload_cow_copies(kv, st)) != TIDE_OK) return rc;     // a copied page must be in place before it is written
  int n_recs = 0;
  for (int j = 0; j < n_tasks; ++j) n_recs += indptr[j + 1] > indptr[j] ? 1 : 0;
  const ExtendOut& x = kv->ext;
  auto fill_recs = [&](AppendRec* recs) {
    int r = 0, grp_cursor = 0;
    for (int j = 0; j < n_tasks; ++j) {
      const int c = indptr[j + 1] - indptr[j];
      if (c == 0) continue;
      AppendRec& rec = recs[r++];
      rec.table_off = task_ids[j] * kv->g.max_pages_per_task;
      rec.pos0 = kv->len[task_ids[j]] - c;
      rec.tok0 = indptr[j];
      rec.count = c;
      rec.new_lp0 = x.new_lp0[(size_t)j];
      rec.new_off = x.new_off[(size_t)j];
      rec.grp0 = grp_cursor; rec.pad1 = 0;
      grp_cursor += ((rec.pos0 & 7) + rec.count + 7) >> 3;
    }
  };
  if (kv->inline_descriptors && n_recs <= kInlineRecs && x.idx.size() <= (size_t)kInlineUpd) {
    // A small append: the write records and the page-table delta travel in the launch's own parameters, so there
    // is nothing to upload and ONE launch does everything.
    AppendInline& pi = kv->append_inline;
    fill_recs(pi.recs);
    const size_t n_ids = x.idx.size();
    std::memcpy(pi.upd, x.idx.data(), n_ids * 4);
    std::memcpy(pi.upd + n_ids, x.val.data(), n_ids * 4);
    AppendParams& ap = pi.p;
    ap = AppendParams();
    ap.pool = kv->layer_pool(0);
    ap.table = kv->d_table;
    ap.n_recs = n_recs;
    ap.n_tokens = indptr[n_tasks];
    ap.new_k = (const uint16_t*)new_k;
    ap.new_v = (const uint16_t*)new_v;
    ap.g = kv->g;
    ap.table_rw = kv->d_table;
    ap.n_upd = (int)n_ids;
    if (launch_append_inline(pi, st) != cudaSuccess) return TIDE_ERR_CUDA;
    ++kv->append_launches;
  } else if (n_recs <= kSlotRecs && x.idx.size() <= kSlotPageIds) {
    // The usual case: ONE upload (write records, then the page-table delta) and ONE launch that applies the delta
    // and scatters the rows; the rows' new pages are read from the delta itself.
    Slot* slot;
    if ((rc = acquire_slot(kv, &slot)) != TIDE_OK) return rc;
    AppendRec* recs = (AppendRec*)(slot->host + 256);
    fill_recs(recs);
    const size_t n_ids = x.idx.size();
    int32_t* h_idx = (int32_t*)(recs + n_recs);
    std::memcpy(h_idx, x.idx.data(), n_ids * 4);
    std::memcpy(h_idx + n_ids, x.val.data(), n_ids * 4);
    const size_t bytes = (size_t)n_recs * sizeof(AppendRec) + 2 * n_ids * 4;
    if (bytes > 0 && upload(kv, slot->dev + 256, slot->host + 256, bytes, st) != cudaSuccess) return TIDE_ERR_CUDA;
    AppendParams ap;
    ap.pool = kv->layer_pool(0);
    ap.table = kv->d_table;
    ap.recs = (const AppendRec*)(slot->dev + 256);
    ap.n_recs = n_recs;
    ap.n_tokens = indptr[n_tasks];
    ap.new_k = (const uint16_t*)new_k;
    ap.new_v = (const uint16_t*)new_v;
    ap.g = kv->g;
    ap.table_rw = kv->d_table;
    ap.upd_idx = (const int32_t*)(ap.recs + n_recs);
    ap.upd_val = ap.upd_idx + n_ids;
    ap.n_upd = (int)n_ids;
    if (launch_append(ap, st) != cudaSuccess) return TIDE_ERR_CUDA;
    ++kv->append_launches;
    if ((rc = release_slot(slot, st)) != TIDE_OK) return rc;
  } else {
    if ((rc = upload_table_delta(kv, st)) != TIDE_OK) return rc;
    if ((rc = write_tasks(kv, 0, n_tasks, task_ids, indptr, new_k, new_v, st)) != TIDE_OK) return rc;
  }
  if (kv->profiling) {
    cudaEventRecord(kv->ev_append[1], st);
    kv->have_append_times = true;
  }
  return TIDE_OK;
}

int tide_kv_read(tide_kv_t* kv, int32_t layer, int32_t task, void* out_k, void* out_v, void* stream) {
  if (kv == nullptr || layer < 0 || layer >= kv->cfg.num_layers || !task_in_range(kv, task)) return TIDE_ERR_INVALID_ARG;
  if (!kv->live[task]) return TIDE_ERR_UNKNOWN_TASK;
  if (kv->len[task] == 0) return TIDE_OK;
  if (out_k == nullptr || out_v == nullptr || ((uintptr_t)out_k & 15) || ((uintptr_t)out_v & 15)) return TIDE_ERR_INVALID_ARG;
  const int32_t* row = kv->d_table + (size_t)task * kv->g.max_pages_per_task;
  if (launch_read(kv->layer_pool(layer), row, 0, kv->len[task], (uint16_t*)out_k, (uint16_t*)out_v, kv->g, (cudaStream_t)stream) != cudaSuccess)
    return TIDE_ERR_CUDA;
  return TIDE_OK;
}

int tide_kv_fork(tide_kv_t* kv, int32_t layer, int32_t parent, int32_t child, void* stream) {
  if (kv == nullptr || layer != 0 || !task_in_range(kv, parent) || !task_in_range(kv, child)) return TIDE_ERR_INVALID_ARG;
  if (!kv->live[parent]) return TIDE_ERR_UNKNOWN_TASK;
  if (kv->live[child]) return TIDE_ERR_TASK_EXISTS;
  const Geom& g = kv->g;
  const int L = kv->len[parent];
  const int n_full = L / g.S;
  const bool partial = L % g.S != 0;
  if (partial && kv->free_stack.empty()) return TIDE_ERR_NO_PAGES;
  cudaStream_t st = (cudaStream_t)stream;
  // ---- bookkeeping: share the full pages, take one fresh page for the copy of the partial one ----
  auto& cp = kv->pages[child];
  cp.assign(kv->pages[parent].begin(), kv->pages[parent].begin() + n_full);
  for (int32_t page : cp) ++kv->refcnt[(size_t)page];
  int32_t copy_src = -1, copy_dst = -1;
  if (partial) {
    copy_src = kv->pages[parent][(size_t)n_full];
    copy_dst = pop_page(kv);
    cp.push_back(copy_dst);
  }
  kv->live[child] = 1;
  kv->len[child] = L;
  kv->used_tokens += L;
  // ---- device: the child's page-table row, then the page copy ----
  for (size_t done = 0; done < cp.size();) {
    Slot* slot;
    int rc = acquire_slot(kv, &slot);
    if (rc != TIDE_OK) return rc;
    int32_t* idx = (int32_t*)(slot->host + 256 + (size_t)kSlotRecs * sizeof(AppendRec));
    int32_t* val = idx + kSlotPageIds;
    const size_t n = std::min(kSlotPageIds, cp.size() - done);
    for (size_t i = 0; i < n; ++i) {
      idx[i] = child * g.max_pages_per_task + (int32_t)(done + i);
      val[i] = cp[done + i];
    }
    uint8_t* didx = slot->dev + 256 + (size_t)kSlotRecs * sizeof(AppendRec);
    if (cudaMemcpyAsync(didx, idx, n * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return TIDE_ERR_CUDA;
    if (cudaMemcpyAsync(didx + kSlotPageIds * 4, val, n * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return TIDE_ERR_CUDA;
    if (launch_table_update(kv->d_table, (const int32_t*)didx, (const int32_t*)(didx + kSlotPageIds * 4), (int)n, st) != cudaSuccess)
      return TIDE_ERR_CUDA;
    done += n;
    if (done == cp.size() && partial) {
      int32_t* hc = val + kSlotPageIds;   // copy-pair area of the slot
      hc[0] = copy_src;
      hc[kSlotRecs] = copy_dst;
      uint8_t* dcpy = slot->dev + 256 + (size_t)kSlotRecs * sizeof(AppendRec) + kSlotPageIds * 8;
      if (cudaMemcpyAsync(dcpy, hc, 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return TIDE_ERR_CUDA;
      if (cudaMemcpyAsync(dcpy + (size_t)kSlotRecs * 4, hc + kSlotRecs, 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return TIDE_ERR_CUDA;
      for (int l = 0; l < kv->cfg.num_layers; ++l)
        if (launch_copy_pages(kv->layer_pool(l), (const int32_t*)dcpy, (const int32_t*)(dcpy + (size_t)kSlotRecs * 4), 1, g.page_bytes,
                              st) != cudaSuccess)
          return TIDE_ERR_CUDA;
    }
    if ((rc = release_slot(slot, st)) != TIDE_OK) return rc;
  }
  if (cp.empty() && partial) return TIDE_ERR_INVALID_ARG;   // unreachable: a partial page implies one entry
  return TIDE_OK;
}

int tide_kv_page_refs(tide_kv_t* kv, int32_t task, int32_t* out, int32_t cap, int32_t* n_pages) {
  if (kv == nullptr || n_pages == nullptr || !task_in_range(kv, task) || cap < 0) return TIDE_ERR_INVALID_ARG;
  if (!kv->live[task]) return TIDE_ERR_UNKNOWN_TASK;
  const auto& pg = kv->pages[task];
  *n_pages = (int32_t)pg.size();
  if (out != nullptr) {
    if ((size_t)cap < pg.size()) return TIDE_ERR_INVALID_ARG;
    for (size_t i = 0; i < pg.size(); ++i) out[i] = kv->refcnt[(size_t)pg[i]];
  }
  return TIDE_OK;
}

int tide_kv_release_many(tide_kv_t* kv, int32_t n_tasks, const int32_t* task_ids) {
  if (kv == nullptr || n_tasks < 0 || (n_tasks > 0 && task_ids == nullptr)) return TIDE_ERR_INVALID_ARG;
  for (int j = 0; j < n_tasks; ++j) {
    if (!task_in_range(kv, task_ids[j])) return TIDE_ERR_INVALID_ARG;
    if (!kv->live[task_ids[j]]) return TIDE_ERR_UNKNOWN_TASK;
  }
  if (++kv->mark_gen == 0x7fffffff) {
    std::fill(kv->mark.begin(), kv->mark.end(), 0);
    kv->mark_gen = 1;
  }
  for (int j = 0; j < n_tasks; ++j) {
    if (kv->mark[task_ids[j]] == kv->mark_gen) return TIDE_ERR_DUPLICATE_TASK;
    kv->mark[task_ids[j]] = kv->mark_gen;
  }
  for (int j = 0; j < n_tasks; ++j) tide_kv_release(kv, task_ids[j]);
  return TIDE_OK;
}

int tide_kv_prune(tide_kv_t* kv, int32_t layer, int32_t task, int32_t keep_prefix, int32_t tail_begin, void* stream) {
  if (kv == nullptr || layer != 0 || !task_in_range(kv, task)) return TIDE_ERR_INVALID_ARG;
  if (!kv->live[task]) return TIDE_ERR_UNKNOWN_TASK;
  const int len = kv->len[task];
  if (!(0 <= keep_prefix && keep_prefix <= tail_begin && tail_begin <= len)) return TIDE_ERR_INVALID_ARG;
  const int tail = len - tail_begin;
  if (tail_begin == keep_prefix) return TIDE_OK;   // nothing is dropped
  const Geom& g = kv->g;
  const auto& pg = kv->pages[task];
  // ---- validation: the pages the shorter task needs must be there once the dropped ones are back ----
  const int kept = ceil_div(keep_prefix, g.S);              // pages that stay in the table
  const int first = keep_prefix / g.S;                      // first page that is dropped or written again
  bool shared_any = false;
  long long freed = 0;
  for (size_t i = (size_t)first; i < pg.size(); ++i) {
    const bool shared = kv->refcnt[(size_t)pg[i]] > 1;
    shared_any = shared_any || shared;
    if ((int)i >= kept && !shared) ++freed;
  }
  long long need = ceil_div(keep_prefix + tail, g.S) - kept;
  if (tail > 0 && keep_prefix % g.S != 0 && kv->refcnt[(size_t)pg[(size_t)first]] > 1) ++need;
  if (need > (long long)kv->free_stack.size() + freed) return TIDE_ERR_NO_PAGES;
  const int chunk_cap = (int)std::min<int64_t>(kv->cfg.max_batch_tokens, 0x7fffffff);
  // A task that shares none of these pages gets the same pages back in the same places, so its tail can move in
  // place, chunk by chunk.  Otherwise its new pages differ from the old ones and may be old ones in other places:
  // the whole tail of a layer has to sit in the staging area before anything of that layer is written.
  if (shared_any && tail > chunk_cap) return TIDE_ERR_WORKSPACE;

  cudaStream_t st = (cudaStream_t)stream;
  uint16_t* sk = (uint16_t*)(kv->ws + kv->lay.off_stage_k);
  uint16_t* sv = (uint16_t*)(kv->ws + kv->lay.off_stage_v);
  const int32_t* row = kv->d_table + (size_t)task * g.max_pages_per_task;
  const int L = kv->cfg.num_layers;
  int rc;
  if (!shared_any) {
    if ((rc = tide_kv_truncate(kv, task, keep_prefix)) != TIDE_OK) return rc;
    // front to back: a chunk is written below the positions the next one reads
    for (int done = 0; done < tail; done += chunk_cap) {
      const int n = std::min(chunk_cap, tail - done);
      const int32_t ip[2] = {0, n};
      if ((rc = extend_tasks(kv, 1, &task, ip, st, nullptr)) != TIDE_OK) return rc;
      for (int l = 0; l < L; ++l) {
        if (launch_read(kv->layer_pool(l), row, tail_begin + done, n, sk, sv, g, st) != cudaSuccess) return TIDE_ERR_CUDA;
        if ((rc = write_tasks(kv, l, 1, &task, ip, sk, sv, st)) != TIDE_OK) return rc;
      }
    }
    return TIDE_OK;
  }
  // keep the row as it is now: the tail is read through it after the table has changed
  if (cudaMemcpyAsync(kv->d_old_row, row, pg.size() * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return TIDE_ERR_CUDA;
  if ((rc = tide_kv_truncate(kv, task, keep_prefix)) != TIDE_OK) return rc;
  const int32_t ip[2] = {0, tail};
  std::vector<int32_t> cow;
  if ((rc = extend_tasks(kv, 1, &task, ip, st, &cow)) != TIDE_OK) return rc;
  const int32_t *d_src = nullptr, *d_dst = nullptr;
  if (!cow.empty()) {
    // the one (old, new) pair sits behind the saved row; the source is pageable, so the call returns with it staged
    int32_t* d_pair = kv->d_old_row + g.max_pages_per_task;
    if (cudaMemcpyAsync(d_pair, cow.data(), 8, cudaMemcpyHostToDevice, st) != cudaSuccess) return TIDE_ERR_CUDA;
    d_src = d_pair;
    d_dst = d_pair + 1;
  }
  for (int l = 0; l < L; ++l) {
    if (launch_read(kv->layer_pool(l), kv->d_old_row, tail_begin, tail, sk, sv, g, st) != cudaSuccess) return TIDE_ERR_CUDA;
    if (d_src != nullptr && launch_copy_pages(kv->layer_pool(l), d_src, d_dst, 1, g.page_bytes, st) != cudaSuccess)
      return TIDE_ERR_CUDA;
    if ((rc = write_tasks(kv, l, 1, &task, ip, sk, sv, st)) != TIDE_OK) return rc;
  }
  return TIDE_OK;
}

// Row checks of every attention call: live tasks, 1 <= q_len <= ctx_len <= resident length, batch limits.
static int check_rows(tide_kv* kv, int32_t n_rows, const tide_row_t* rows) {
  if (n_rows > kv->cfg.max_batch_rows) return TIDE_ERR_WORKSPACE;
  long long total_q = 0;
  for (int b = 0; b < n_rows; ++b) {
    const tide_row_t& r = rows[b];
    if (!task_in_range(kv, r.task)) return TIDE_ERR_INVALID_ARG;
    if (!kv->live[r.task]) return TIDE_ERR_UNKNOWN_TASK;
    if (!(r.q_len >= 1 && r.q_len <= r.ctx_len && r.ctx_len <= kv->len[r.task])) return TIDE_ERR_CTX_RANGE;
    total_q += r.q_len;
  }
  if (total_q > kv->cfg.max_batch_tokens) return TIDE_ERR_WORKSPACE;
  return TIDE_OK;
}

// Rows of one batch whose tasks hold the same first pages (forked tasks of a GRPO group, Section 2.1) are planned as
// a group: consecutive decode rows of distinct tasks whose page lists agree on at least kMinSharedTokens tokens of
// full pages that every member's context covers.
struct ShareGroup {
  int first = 0, m = 0, pages = 0;       // first member row, members, shared pages
  int32_t part_base = 0, n_splits = 0;   // of the shared range's segment, known once it has been placed
};
constexpr int kMinSharedTokens = 256;

constexpr int kMaxGroupRows = 64;        // packed rows of a shared range (one 64-row tile of the warp-MMA kernel, a quarter of a tcgen05 item)

static void find_share_groups(const tide_kv* kv, int32_t n_rows, const tide_row_t* rows, std::vector<ShareGroup>& groups,
                              std::vector<int>& group_of) {
  const Geom& g = kv->g;
  group_of.assign((size_t)n_rows, -1);
  groups.clear();
  const int max_m = std::max(1, kMaxGroupRows / g.G);
  const int min_pages = std::max(1, kMinSharedTokens / g.S);
  if (max_m < 2 || kv->no_grouping) return;
  long long saved_total = 0;
  for (int b = 0; b + 1 < n_rows; ++b) {
    if (rows[b].q_len != 1) continue;
    const auto& pg0 = kv->pages[rows[b].task];
    // Only pages that are full NOW can be shared: when a step is planned before its tokens are appended, a row's
    // ctx_len counts the token that will land in the last page, and a shared partial page is replaced by a private
    // copy before that token is written.
    int C = std::min<int>((int)pg0.size(), std::min(rows[b].ctx_len, kv->len[rows[b].task]) / g.S);
    if (C < min_pages || kv->refcnt[(size_t)pg0[0]] < 2) continue;
    int m = 1;
    while (b + m < n_rows && m < max_m && rows[b + m].q_len == 1) {
      const tide_row_t& r = rows[b + m];
      bool repeat = false;
      for (int k = 0; k < m; ++k) repeat = repeat || rows[b + k].task == r.task;
      if (repeat) break;
      const auto& pg = kv->pages[r.task];
      const int lim = std::min<int>(std::min<int>(C, (int)pg.size()), std::min(r.ctx_len, kv->len[r.task]) / g.S);
      int lcp = 0;
      while (lcp < lim && pg[(size_t)lcp] == pg0[(size_t)lcp]) ++lcp;
      if (lcp < min_pages) break;
      C = lcp;
      ++m;
    }
    if (m >= 2) {
      // Worth it only if the reads saved are a large part of what the members read: a group costs an extra work item
      // for the shared range and a merge for every member (measured on 8 x 8 rows of 8192 keys: +8 % time at 12-25 %
      // shared, break-even near 45 %, 1.4x faster at 75 %, 1.9x at 94 %).
      long long ctx_sum = 0;
      for (int k = 0; k < m; ++k) ctx_sum += rows[b + k].ctx_len;
      const long long saved = (long long)(m - 1) * C * g.S;
      if (saved * 10 >= ctx_sum * 4) {
        ShareGroup sg;
        sg.first = b; sg.m = m; sg.pages = C;
        for (int k = 0; k < m; ++k) group_of[(size_t)(b + k)] = (int)groups.size();
        groups.push_back(sg);
        saved_total += saved;
      }
      b += m - 1;
    }
  }
  // ... and only if the batch as a whole saves enough bytes to pay for one more kernel launch
  if (saved_total * g.Hkv * g.D * 4 < kv->min_saved_bytes) {
    groups.clear();
    group_of.assign((size_t)n_rows, -1);
  }
}

// The work plan of one batch: one segment per row, decode-style (<= 16 packed rows), warp-MMA tile-style or
// tcgen05-style; long contexts are split along the keys so that the grid has about items_per_sm items per SM.
// A group of rows that share their first pages gets one more segment for the shared range (its tokens are the
// members' queries, all seeing the same keys); the members' own segments start behind it and their merge takes both.
// The plan depends on the rows and the page tables only, so every layer of a step can use it.
static int build_plan(tide_kv* kv, int32_t n_rows, const tide_row_t* rows, bool umma_ok, bool allow_groups, PlanHost& P) {
  const Geom& g = kv->g;
  enum { kDec = 0, kTile = 1, kUmma = 2 };
  struct RowPlan { int kind; int n_mtiles; long long items; };
  auto kind_of = [&](int R) { return R <= kDecodeTileRows ? kDec : (umma_ok && R >= kv->umma_min_rows ? kUmma : kTile); };
  auto mtiles_of = [&](int kind, int R) { return kind == kDec ? 1 : ceil_div(R, kind == kUmma ? 2 * kUmmaTileRows : kMmaTileRows); };
  std::vector<ShareGroup> groups;
  std::vector<int> group_of;
  if (allow_groups) find_share_groups(kv, n_rows, rows, groups, group_of);
  else group_of.assign((size_t)n_rows, -1);
  std::vector<RowPlan> plan((size_t)n_rows);
  long long w_dec = 0, w_tile = 0, items_tile_nosplit = 0;
  for (int b = 0; b < n_rows; ++b) {
    const tide_row_t& r = rows[b];
    const int R = r.q_len * g.G;
    RowPlan& p = plan[(size_t)b];
    p.kind = kind_of(R);
    p.n_mtiles = mtiles_of(p.kind, R);
    p.items = (long long)g.Hkv * p.n_mtiles;
    const int own = group_of[(size_t)b] < 0 ? r.ctx_len : r.ctx_len - groups[(size_t)group_of[(size_t)b]].pages * g.S;
    if (p.kind == kDec) w_dec += (long long)g.Hkv * own;
    else { w_tile += p.items * own; items_tile_nosplit += p.items; }
  }
  // A shared range is streaming work like a decode row (few rows against many keys), so it is cut as finely as
  // decode rows are, whichever kernel its packed rows call for.
  auto shared_kind = [&](int R) { return kind_of(R); };
  for (const ShareGroup& sg : groups) w_dec += (long long)g.Hkv * sg.pages * g.S;
  const long long target = (long long)kv->num_sms * kv->items_per_sm;
  long long chunk_dec = std::max<long long>(256, align_up((size_t)(w_dec / target + 1), kStageKeys));
  long long chunk_tile = (items_tile_nosplit >= target / 2)
                             ? (1LL << 30)
                             : std::max<long long>(2048, align_up((size_t)(w_tile / target + 1), kStageKeys));
  // a range of `len` keys cut for the given kind
  auto cut = [&](bool streaming, int len, int& n_splits, int& chunk) {
    const long long chunk_target = streaming ? chunk_dec : chunk_tile;
    n_splits = (int)std::min<long long>(kMaxSplits, ((long long)len + chunk_target - 1) / chunk_target);
    n_splits = std::max(1, n_splits);
    chunk = (int)align_up((size_t)std::max(1, ceil_div(len, n_splits)), 2 * kStageKeys);
    n_splits = std::max(1, ceil_div(len, chunk));
  };
  for (int attempt = 0; attempt < 40; ++attempt) {
    P.seg_dec.clear(); P.seg_tile.clear(); P.seg_umma.clear();
    long long part_rows = 0, qoff = 0;
    for (int b = 0; b < n_rows; ++b) {
      const tide_row_t& r = rows[b];
      const RowPlan& p = plan[(size_t)b];
      const int gi = group_of[(size_t)b];
      if (gi >= 0 && groups[(size_t)gi].first == b) {
        // the shared range of the group that starts at this row
        const ShareGroup& sg = groups[(size_t)gi];
        const int kind = shared_kind(sg.m * g.G);
        Segment s{};
        s.table_off = r.task * g.max_pages_per_task;
        s.q_off = (int32_t)qoff;
        s.n = sg.m;
        s.p = sg.pages * g.S - 1;
        s.n_mtiles = mtiles_of(kind, sg.m * g.G);
        cut(true, sg.pages * g.S, s.n_splits, s.chunk);
        s.causal = 0;
        s.partial = 1;
        s.x_part_base = gi;
        s.x_n_splits = -2;                                   // marks the shared range until the links are resolved
        part_rows += (long long)s.n_splits * sg.m * g.Hq;
        (kind == kDec ? P.seg_dec : kind == kTile ? P.seg_tile : P.seg_umma).push_back(s);
      }
      Segment s{};
      s.table_off = r.task * g.max_pages_per_task;
      s.q_off = (int32_t)qoff;
      s.n = r.q_len;
      s.p = r.ctx_len - r.q_len;
      s.n_mtiles = p.n_mtiles;
      s.causal = 1;
      if (gi >= 0) {
        s.origin = groups[(size_t)gi].pages * g.S;
        s.partial = 1;
        s.x_part_base = gi;
        s.x_n_splits = -1;                                   // marks a member until the links are resolved
        s.x_stride = b - groups[(size_t)gi].first;           // member index, for now
      }
      cut(p.kind == kDec, r.ctx_len - s.origin, s.n_splits, s.chunk);
      if (s.n_splits > 1 || s.partial) part_rows += (long long)s.n_splits * r.q_len * g.Hq;
      (p.kind == kDec ? P.seg_dec : p.kind == kTile ? P.seg_tile : P.seg_umma).push_back(s);
      qoff += r.q_len;
    }
    if (part_rows <= kv->lay.part_rows) break;
    chunk_dec *= 2;
    chunk_tile = std::min<long long>(chunk_tile * 2, 1LL << 30);
    if (attempt == 39) return TIDE_ERR_WORKSPACE;
  }
  // heaviest items first, so the tail of the grid is made of short items
  auto heavier = [](const Segment& a, const Segment& b) {
    return std::min(a.chunk, a.p + a.n - a.origin) > std::min(b.chunk, b.p + b.n - b.origin);
  };
  std::stable_sort(P.seg_dec.begin(), P.seg_dec.end(), heavier);
  std::stable_sort(P.seg_tile.begin(), P.seg_tile.end(), heavier);
  std::stable_sort(P.seg_umma.begin(), P.seg_umma.end(), heavier);
  P.seg_merge.clear();
  P.merge_rows = 0;
  P.fused_rows = 0;
  long long part_cursor = 0;
  int32_t ctr_cursor = 0;
  std::vector<Segment*> merged;                              // segments with rows to merge, in merge_base order
  for (auto* v : {&P.seg_dec, &P.seg_tile, &P.seg_umma}) {
    long long base = 0;
    for (Segment& s : *v) {
      s.item_base = (int32_t)base;
      base += (long long)g.Hkv * s.n_mtiles * s.n_splits;
      if (base > 0x7fffffffLL) return TIDE_ERR_WORKSPACE;
      if (s.n_splits > 1 || s.partial) {
        s.part_base = (int32_t)part_cursor;
        part_cursor += (long long)s.n_splits * s.n * g.Hq;
        if (s.x_n_splits == -2) {                            // a shared range: it has no output rows of its own
          groups[(size_t)s.x_part_base].part_base = s.part_base;
          groups[(size_t)s.x_part_base].n_splits = s.n_splits;
        } else if (v == &P.seg_dec && s.partial == 0 && s.x_n_splits == 0) {
          // a plain split decode-style row: the split that finishes last merges the partials inside the decode kernel
          s.partial = 2;
          s.x_part_base = ctr_cursor;
          ctr_cursor += g.Hkv;
          P.fused_rows += (long long)s.n * g.Hq;
        } else {
          s.merge_base = (int32_t)P.merge_rows;
          P.merge_rows += (long long)s.n * g.Hq;
          merged.push_back(&s);
        }
      }
    }
    (v == &P.seg_dec ? P.items_dec : v == &P.seg_tile ? P.items_tile : P.items_umma) = base;
  }
  // resolve the links between the members and their group's shared range
  for (auto* v : {&P.seg_dec, &P.seg_tile, &P.seg_umma})
    for (Segment& s : *v) {
      if (s.x_n_splits == -1) {
        const ShareGroup& sg = groups[(size_t)s.x_part_base];
        const int member = s.x_stride;
        s.x_part_base = sg.part_base + member * g.Hq;
        s.x_n_splits = sg.n_splits;
        s.x_stride = sg.m * g.Hq;
      } else if (s.x_n_splits == -2) {
        s.x_part_base = 0;
        s.x_n_splits = 0;
      }
    }
  for (const Segment* s : merged) P.seg_merge.push_back(*s);
  kv->last_groups = (int64_t)groups.size();
  kv->last_grouped_rows = 0;
  for (const ShareGroup& sg : groups) kv->last_grouped_rows += sg.m;
  return TIDE_OK;
}

// Writes the four segment arrays at `h` and describes them as they will sit at `d`: one after the other
// (stride 0), or each at a fixed distance of `stride` entries, so that their addresses do not depend on the batch.
static PlanDev pack_plan(const PlanHost& P, Segment* h, const Segment* d, size_t stride) {
  const size_t o_tile = stride ? stride : P.seg_dec.size();
  const size_t o_umma = stride ? 2 * stride : o_tile + P.seg_tile.size();
  const size_t o_merge = stride ? 3 * stride : o_umma + P.seg_umma.size();
  std::copy(P.seg_dec.begin(), P.seg_dec.end(), h);
  std::copy(P.seg_tile.begin(), P.seg_tile.end(), h + o_tile);
  std::copy(P.seg_umma.begin(), P.seg_umma.end(), h + o_umma);
  std::copy(P.seg_merge.begin(), P.seg_merge.end(), h + o_merge);
  PlanDev pd;
  pd.seg_dec = d; pd.seg_tile = d + o_tile; pd.seg_umma = d + o_umma; pd.seg_merge = d + o_merge;
  pd.n_dec = P.seg_dec.size(); pd.n_tile = P.seg_tile.size(); pd.n_umma = P.seg_umma.size(); pd.n_merge = P.seg_merge.size();
  pd.items_dec = P.items_dec; pd.items_tile = P.items_tile; pd.items_umma = P.items_umma; pd.merge_rows = P.merge_rows;
  return pd;
}

// The attention launches of one planned batch on one layer: kernel launches only (and, with `events`, the phase
// time stamps), so a caller may capture them in a CUDA graph.
static int launch_plan(tide_kv* kv, int32_t layer, const PlanDev& d, const int32_t* page_table, const void* q, float scale,
                       void* out, float* lse, cudaStream_t st, bool events, int64_t* n_launches, const int32_t* dyn) {
  AttendParams ap;
  ap.pool = kv->layer_pool(layer);
  ap.table = page_table ? page_table : kv->d_table;
  ap.q = (const uint16_t*)q;
  ap.out = (uint16_t*)out;
  ap.lse = lse;
  ap.part_o = kv->d_part_o;
  ap.part_lse = kv->d_part_lse;
  ap.scale_log2e = scale * 1.4426950408889634f;
  ap.status = kv->d_status;
  ap.g = kv->g;
  ap.merge_ctr = kv->d_merge_ctr;
  ap.wait_limit_ns = kv->wait_limit_ns;
  ap.debug_drop_first_stage = kv->drop_first_stage_once ? 1 : 0;
  kv->drop_first_stage_once = false;
  int64_t launches = 0;
  // dyn != nullptr: fixed launch shapes; the counts of the batch are read on the device (header of the step area)
  if (events) cudaEventRecord(kv->ev_attend[0], st);
  if (dyn ? kv->cap_dec > 0 : d.items_dec > 0) {
    ap.segs = d.seg_dec; ap.n_segs = (int)d.n_dec; ap.n_items = (int)d.items_dec;
    ap.dyn = dyn ? dyn + kHdrDecItems : nullptr; ap.grid_cap = kv->cap_dec;
    if (launch_attend_decode(ap, st) != cudaSuccess) return TIDE_ERR_CUDA;
    ++launches;
  }
  if (events) cudaEventRecord(kv->ev_attend[1], st);
  if (dyn ? kv->cap_tile > 0 : d.items_tile > 0) {
    ap.segs = d.seg_tile; ap.n_segs = (int)d.n_tile; ap.n_items = (int)d.items_tile;
    ap.dyn = dyn ? dyn + kHdrTileItems : nullptr; ap.grid_cap = kv->cap_tile;
    if (launch_attend_tile(ap, st) != cudaSuccess) return TIDE_ERR_CUDA;
    ++launches;
  }
  if (dyn ? kv->cap_umma > 0 : d.items_umma > 0) {
    ap.segs = d.seg_umma; ap.n_segs = (int)d.n_umma; ap.n_items = (int)d.items_umma;
    ap.dyn = dyn ? dyn + kHdrUmmaItems : nullptr; ap.grid_cap = kv->cap_umma;
    if ((kv->umma_tile_keys == 128 ? launch_attend_umma128(ap, st) : launch_attend_umma(ap, st)) != cudaSuccess) return TIDE_ERR_CUDA;
    ++launches;
  }
  if (events) cudaEventRecord(kv->ev_attend[2], st);
  if (dyn ? kv->cap_merge_rows > 0 : d.merge_rows > 0) {
    MergeParams mp;
    mp.segs = d.seg_merge;
    mp.n_segs = (int)d.n_merge;
    mp.n_rows = (int)d.merge_rows;
    mp.part_o = kv->d_part_o; mp.part_lse = kv->d_part_lse;
    mp.out = (uint16_t*)out; mp.lse = lse; mp.Hq = kv->g.Hq; mp.D = kv->g.D;
    mp.dyn = dyn ? dyn + kHdrMergeRows : nullptr; mp.grid_cap_rows = kv->cap_merge_rows;
    if (launch_merge(mp, st) != cudaSuccess) return TIDE_ERR_CUDA;
    ++launches;
  }
  if (events) {
    cudaEventRecord(kv->ev_attend[3], st);
    kv->have_attend_times = true;
  }
  *n_launches = launches;
  return TIDE_OK;
}

int tide_attend(tide_kv_t* kv, int32_t layer, int32_t n_rows, const tide_row_t* rows, const int32_t* page_table,
                const void* q, float scale, void* out, float* lse, void* stream) {
  if (kv == nullptr || layer < 0 || layer >= kv->cfg.num_layers || n_rows < 0) return TIDE_ERR_INVALID_ARG;
  if (n_rows == 0) return TIDE_OK;
  if (rows == nullptr || q == nullptr || out == nullptr) return TIDE_ERR_INVALID_ARG;
  if (((uintptr_t)q & 15) || ((uintptr_t)out & 15) || ((uintptr_t)lse & 3) || ((uintptr_t)page_table & 3)) return TIDE_ERR_INVALID_ARG;
  if (!(scale == scale)) return TIDE_ERR_INVALID_ARG;
  int rc = check_rows(kv, n_rows, rows);
  if (rc != TIDE_OK) return rc;
  PlanHost P;
  if ((rc = build_plan(kv, n_rows, rows, kv->g.D == 128 && scale > 0.f, page_table == nullptr, P)) != TIDE_OK) return rc;
  if (P.n_all() * sizeof(Segment) + 256 > kv->lay.slot_bytes) return TIDE_ERR_WORKSPACE;

  cudaStream_t st = (cudaStream_t)stream;
  if (kv->inline_descriptors && P.seg_tile.empty() && P.seg_umma.empty() && P.seg_merge.empty() &&
      P.seg_dec.size() <= (size_t)kInlineSegs) {
    // A small decode-only batch: the row descriptors travel in the decode launch's own parameters (no upload).
    AttendInline& pi = kv->attend_inline;
    std::copy(P.seg_dec.begin(), P.seg_dec.end(), pi.segs);
    AttendParams& ap = pi.p;
    ap = AttendParams();
    ap.pool = kv->layer_pool(layer);
    ap.table = page_table ? page_table : kv->d_table;
    ap.n_segs = (int)P.seg_dec.size();
    ap.n_items = (int)P.items_dec;
    ap.q = (const uint16_t*)q;
    ap.out = (uint16_t*)out;
    ap.lse = lse;
    ap.part_o = kv->d_part_o;
    ap.part_lse = kv->d_part_lse;
    ap.scale_log2e = scale * 1.4426950408889634f;
    ap.status = kv->d_status;
    ap.g = kv->g;
    ap.merge_ctr = kv->d_merge_ctr;
    ap.wait_limit_ns = kv->wait_limit_ns;
    ap.debug_drop_first_stage = kv->drop_first_stage_once ? 1 : 0;
    kv->drop_first_stage_once = false;
    if (kv->profiling) cudaEventRecord(kv->ev_attend[0], st);
    if (launch_attend_decode_inline(pi, st) != cudaSuccess) return TIDE_ERR_CUDA;
    if (kv->profiling) {
      for (int i = 1; i <= 3; ++i) cudaEventRecord(kv->ev_attend[i], st);
      kv->have_attend_times = true;
    }
    kv->last_decode_items = P.items_dec;
    kv->last_prefill_items = 0;
    kv->last_merge_rows = P.fused_rows;
    kv->last_launches = 1 + kv->append_launches;
    kv->append_launches = 0;
    return TIDE_OK;
  }
  Slot* slot;
  if ((rc = acquire_slot(kv, &slot)) != TIDE_OK) return rc;
  const PlanDev pd = pack_plan(P, (Segment*)(slot->host + 256), (const Segment*)(slot->dev + 256), 0);
  if (upload(kv, slot->dev + 256, slot->host + 256, P.n_all() * sizeof(Segment), st) != cudaSuccess)
    return TIDE_ERR_CUDA;
  int64_t launches = 0;
  if ((rc = launch_plan(kv, layer, pd, page_table, q, scale, out, lse, st, kv->profiling, &launches, nullptr)) != TIDE_OK) return rc;
  if ((rc = release_slot(slot, st)) != TIDE_OK) return rc;
  kv->last_decode_items = pd.items_dec;
  kv->last_prefill_items = pd.items_tile + pd.items_umma;
  kv->last_merge_rows = pd.merge_rows + P.fused_rows;
  kv->last_launches = launches + kv->append_launches;
  kv->append_launches = 0;
  return TIDE_OK;
}

int tide_step_fix_grids(tide_kv_t* kv, int32_t max_decode_items, int32_t max_tile_items, int32_t max_umma_items,
                        int32_t max_merge_rows, int32_t max_tokens) {
  if (kv == nullptr || max_decode_items < 0 || max_tile_items < 0 || max_umma_items < 0 || max_merge_rows < 0 || max_tokens < 0)
    return TIDE_ERR_INVALID_ARG;
  if (max_tokens > kv->cfg.max_batch_tokens) return TIDE_ERR_WORKSPACE;
  kv->fixed_grids = (max_decode_items | max_tile_items | max_umma_items | max_merge_rows | max_tokens) != 0;
  kv->cap_dec = max_decode_items; kv->cap_tile = max_tile_items; kv->cap_umma = max_umma_items;
  kv->cap_merge_rows = max_merge_rows; kv->cap_tokens = max_tokens;
  kv->step_valid = false;
  return TIDE_OK;
}

int tide_step_begin(tide_kv_t* kv, int32_t n_rows, const tide_row_t* rows, void* stream) {
  if (kv == nullptr || n_rows < 0) return TIDE_ERR_INVALID_ARG;
  kv->step_valid = false;
  if (n_rows == 0) return TIDE_OK;
  if (rows == nullptr) return TIDE_ERR_INVALID_ARG;
  if (n_rows > kv->cfg.max_batch_rows) return TIDE_ERR_WORKSPACE;
  const Geom& g = kv->g;
  std::vector<int32_t> ids((size_t)n_rows), indptr((size_t)n_rows + 1);
  indptr[0] = 0;
  for (int b = 0; b < n_rows; ++b) {
    const tide_row_t& r = rows[b];
    if (!task_in_range(kv, r.task)) return TIDE_ERR_INVALID_ARG;
    if (!kv->live[r.task]) return TIDE_ERR_UNKNOWN_TASK;
    if (r.q_len < 1 || (long long)kv->len[r.task] + r.q_len != r.ctx_len) return TIDE_ERR_CTX_RANGE;
    ids[(size_t)b] = r.task;
    if ((long long)indptr[(size_t)b] + r.q_len > kv->cfg.max_batch_tokens) return TIDE_ERR_WORKSPACE;
    indptr[(size_t)b + 1] = indptr[(size_t)b] + r.q_len;
  }
  int rc = check_task_list(kv, n_rows, ids.data(), indptr.data());
  if (rc != TIDE_OK) return rc;
  // The plan needs the lengths after the step only through ctx_len, which the rows already carry, so it is built
  // (and can still be refused) before anything changes.
  PlanHost P;
  if ((rc = build_plan(kv, n_rows, rows, g.D == 128, true, P)) != TIDE_OK) return rc;
  if (kv->fixed_grids && (P.items_dec > kv->cap_dec || P.items_tile > kv->cap_tile || P.items_umma > kv->cap_umma ||
                          P.merge_rows > kv->cap_merge_rows || indptr[(size_t)n_rows] > kv->cap_tokens))
    return TIDE_ERR_WORKSPACE;   // the step does not fit the launch shapes that were fixed
  cudaStream_t st = (cudaStream_t)stream;
  kv->append_launches = 0;
  if ((rc = extend_tasks(kv, n_rows, ids.data(), indptr.data(), st, nullptr)) != TIDE_OK) return rc;
  // one upload: the write records of the rows, then the segments
  if (kv->step_upload_pending && cudaEventSynchronize(kv->ev_step) != cudaSuccess) return TIDE_ERR_CUDA;
  int32_t* hdr = (int32_t*)kv->h_step;
  hdr[kHdrRecs] = n_rows; hdr[kHdrRecs + 1] = indptr[(size_t)n_rows];
  hdr[kHdrDecItems] = (int32_t)P.items_dec; hdr[kHdrDecItems + 1] = (int32_t)P.seg_dec.size();
  hdr[kHdrTileItems] = (int32_t)P.items_tile; hdr[kHdrTileItems + 1] = (int32_t)P.seg_tile.size();
  hdr[kHdrUmmaItems] = (int32_t)P.items_umma; hdr[kHdrUmmaItems + 1] = (int32_t)P.seg_umma.size();
  hdr[kHdrMergeRows] = (int32_t)P.merge_rows; hdr[kHdrMergeRows + 1] = (int32_t)P.seg_merge.size();
  AppendRec* recs = (AppendRec*)(kv->h_step + 256);
  int grp_cursor = 0;
  for (int b = 0; b < n_rows; ++b) {
    recs[b].table_off = rows[b].task * g.max_pages_per_task;
    recs[b].pos0 = rows[b].ctx_len - rows[b].q_len;
    recs[b].tok0 = indptr[(size_t)b];
    recs[b].count = rows[b].q_len;
    recs[b].new_lp0 = INT_MAX;
    recs[b].new_off = 0;
    recs[b].grp0 = grp_cursor; recs[b].pad1 = 0;
    grp_cursor += ((recs[b].pos0 & 7) + recs[b].count + 7) >> 3;
  }
  uint8_t* d_step = kv->ws + kv->lay.off_step;
  const size_t stride = (size_t)kStepSegStride * (size_t)kv->cfg.max_batch_rows;
  kv->step_plan = pack_plan(P, (Segment*)(kv->h_step + kv->lay.step_seg_off), (const Segment*)(d_step + kv->lay.step_seg_off), stride);
  // header and records in one copy, then each segment array that is not empty (their places are fixed)
  if (cudaMemcpyAsync(d_step, kv->h_step, 256 + (size_t)n_rows * sizeof(AppendRec), cudaMemcpyHostToDevice, st) != cudaSuccess)
    return TIDE_ERR_CUDA;
  const size_t counts[4] = {P.seg_dec.size(), P.seg_tile.size(), P.seg_umma.size(), P.seg_merge.size()};
  for (int a = 0; a < 4; ++a) {
    const size_t off = kv->lay.step_seg_off + (size_t)a * stride * sizeof(Segment);
    if (counts[a] > 0 &&
        cudaMemcpyAsync(d_step + off, kv->h_step + off, counts[a] * sizeof(Segment), cudaMemcpyHostToDevice, st) != cudaSuccess)
      return TIDE_ERR_CUDA;
  }
  if (cudaEventRecord(kv->ev_step, st) != cudaSuccess) return TIDE_ERR_CUDA;
  kv->step_upload_pending = true;
  kv->step_recs = n_rows;
  kv->step_tokens = indptr[(size_t)n_rows];
  kv->step_valid = true;
  kv->last_decode_items = P.items_dec;
  kv->last_prefill_items = P.items_tile + P.items_umma;
  kv->last_merge_rows = P.merge_rows + P.fused_rows;
  return TIDE_OK;
}

int tide_step_layer(tide_kv_t* kv, int32_t layer, const void* new_k, const void* new_v, const void* q, float scale,
                    void* out, float* lse, void* stream) {
  if (kv == nullptr || layer < 0 || layer >= kv->cfg.num_layers) return TIDE_ERR_INVALID_ARG;
  if (!kv->step_valid) return TIDE_ERR_INVALID_ARG;
  if (q == nullptr || out == nullptr || bad_kv_rows(kv->step_tokens, new_k, new_v)) return TIDE_ERR_INVALID_ARG;
  if (((uintptr_t)q & 15) || ((uintptr_t)out & 15) || ((uintptr_t)lse & 3)) return TIDE_ERR_INVALID_ARG;
  if (!(scale > 0.f) || !(scale <= 3.0e38f)) return TIDE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  AppendParams ap;
  ap.pool = kv->layer_pool(layer);
  ap.table = kv->d_table;
  const int32_t* dyn = kv->fixed_grids ? (const int32_t*)(kv->ws + kv->lay.off_step) : nullptr;
  ap.recs = (const AppendRec*)(kv->ws + kv->lay.off_step + 256);
  ap.dyn = dyn ? dyn + kHdrRecs : nullptr;
  ap.grid_cap_tokens = kv->cap_tokens;
  ap.n_recs = kv->step_recs;
  ap.n_tokens = kv->step_tokens;
  ap.new_k = (const uint16_t*)new_k;
  ap.new_v = (const uint16_t*)new_v;
  ap.g = kv->g;
  if (launch_append(ap, st) != cudaSuccess) return TIDE_ERR_CUDA;
  int64_t launches = 0;
  const int rc = launch_plan(kv, layer, kv->step_plan, nullptr, q, scale, out, lse, st, false, &launches, dyn);
  if (rc != TIDE_OK) return rc;
  kv->last_launches = launches + 1;
  return TIDE_OK;
}

int tide_step_host(tide_kv_t* kv, int32_t layer, int32_t n_rows, const tide_row_t* rows, const void* new_k,
                   const void* new_v, const void* q, float scale, void* out, float* lse, void* stream) {
  if (kv == nullptr || layer != 0 || n_rows < 0) return TIDE_ERR_INVALID_ARG;
  if (n_rows == 0) return TIDE_OK;
  if (rows == nullptr || new_k == nullptr || new_v == nullptr || q == nullptr || out == nullptr) return TIDE_ERR_INVALID_ARG;
  if (n_rows > kv->cfg.max_batch_rows) return TIDE_ERR_WORKSPACE;
  const Geom& g = kv->g;
  std::vector<int32_t> ids((size_t)n_rows), indptr((size_t)n_rows + 1);
  indptr[0] = 0;
  for (int b = 0; b < n_rows; ++b) {
    const tide_row_t& r = rows[b];
    if (!task_in_range(kv, r.task)) return TIDE_ERR_INVALID_ARG;
    if (!kv->live[r.task]) return TIDE_ERR_UNKNOWN_TASK;
    if (r.q_len < 1 || (long long)kv->len[r.task] + r.q_len != r.ctx_len) return TIDE_ERR_CTX_RANGE;
    ids[(size_t)b] = r.task;
    if ((long long)indptr[(size_t)b] + r.q_len > kv->cfg.max_batch_tokens) return TIDE_ERR_WORKSPACE;
    indptr[(size_t)b + 1] = indptr[(size_t)b] + r.q_len;
  }
  int rc = check_task_list(kv, n_rows, ids.data(), indptr.data());
  if (rc == TIDE_OK) rc = check_extend(kv, n_rows, ids.data(), indptr.data());
  if (rc != TIDE_OK) return rc;   // nothing has been copied or changed
  if (!(scale == scale)) return TIDE_ERR_INVALID_ARG;
  const size_t T = (size_t)indptr[(size_t)n_rows];
  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* dk = kv->ws + kv->lay.off_stage_k;
  uint8_t* dv = kv->ws + kv->lay.off_stage_v;
  uint8_t* dq = kv->ws + kv->lay.off_stage_q;
  uint8_t* dout = kv->ws + kv->lay.off_stage_out;
  float* dlse = (float*)(kv->ws + kv->lay.off_stage_lse);
  const size_t kv_row = (size_t)g.Hkv * g.D * 2, q_row = (size_t)g.Hq * g.D * 2, lse_row = (size_t)g.Hq * 4;
  // Large steps are cut into groups of consecutive rows, each with its own copies in, append, attention and copies
  // out, so that the transfers of one group run beside the kernels of another (copy engines in both directions
  // and the SMs all busy).  Appending the groups in row order takes the same pages as one append of all rows.
  const size_t bytes = T * (2 * kv_row + 2 * q_row + (lse ? lse_row : 0));
  int n_chunks = kv->host_step_chunks > 0 ? kv->host_step_chunks : (int)std::min<size_t>(kMaxHostChunks, bytes / kHostChunkBytes);
  n_chunks = std::max(1, std::min(std::min(n_chunks, kMaxHostChunks), n_rows));
  // A small step from pinned host buffers that the device can address is not copied at all: the append kernel reads
  // new_k / new_v, and the attention kernels read q and write out / lse, straight across PCIe.  Five copies of a few
  // hundred KB cost more in engine hand-overs than the bytes do (a 64-row decode step: 0.22 -> 0.20 ms, a tiny one
  // 0.11 -> 0.09).
  if (kv->host_zero_copy && n_chunks == 1 && bytes <= kZeroCopyBytes) {
    auto mapped = [](const void* p, void** dev) -> bool {
      cudaPointerAttributes a;
      if (cudaPointerGetAttributes(&a, p) != cudaSuccess) { cudaGetLastError(); return false; }
      if (a.type != cudaMemoryTypeHost || a.devicePointer == nullptr) return false;
      *dev = a.devicePointer;
      return ((uintptr_t)a.devicePointer & 15) == 0;
    };
    void *zk, *zv, *zq, *zo, *zl = nullptr;
    if (mapped(new_k, &zk) && mapped(new_v, &zv) && mapped(q, &zq) && mapped(out, &zo) && (lse == nullptr || mapped(lse, &zl))) {
      rc = tide_kv_append(kv, layer, n_rows, ids.data(), indptr.data(), zk, zv, stream);
      if (rc != TIDE_OK) return rc;
      rc = tide_attend(kv, layer, n_rows, rows, nullptr, zq, scale, zo, (float*)zl, stream);
      if (rc != TIDE_OK) return rc;
      if (cudaStreamSynchronize(st) != cudaSuccess) return TIDE_ERR_CUDA;
      return TIDE_OK;
    }
  }
  if (n_chunks > 1 && kv->st_in == nullptr) {
    bool ok = cudaStreamCreateWithFlags(&kv->st_in, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&kv->st_out, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; ok && i < 2 * kMaxHostChunks + 2; ++i)
      ok = cudaEventCreateWithFlags(&kv->ev_host[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) return TIDE_ERR_CUDA;
  }
  cudaStream_t s_in = n_chunks > 1 ? kv->st_in : st, s_out = n_chunks > 1 ? kv->st_out : st;
  struct UploadMode {   // planning uploads bypass the copy engine while this step's large copies are in flight
    tide_kv* kv;
    ~UploadMode() { kv->upload_by_kernel = false; }
  } upload_mode{kv};
  kv->upload_by_kernel = n_chunks > 1 && kv->slots_mapped;
  cudaEvent_t ev_start = kv->ev_host[2 * kMaxHostChunks], ev_end = kv->ev_host[2 * kMaxHostChunks + 1];
  if (n_chunks > 1) {
    // the copies in may not overtake work already queued on the caller's stream that still uses the staging area
    if (cudaEventRecord(ev_start, st) != cudaSuccess || cudaStreamWaitEvent(s_in, ev_start, 0) != cudaSuccess) return TIDE_ERR_CUDA;
    if (cudaStreamWaitEvent(s_out, ev_start, 0) != cudaSuccess) return TIDE_ERR_CUDA;
  }
  // rows [cut[c], cut[c+1]): up to the c+1-th share of the tokens, at least one row each.  The shares are equal but for
  // the last two groups, which are a half and a fifth of a share: what follows the last copy in - that group's kernels
  // and its copy out - is the part of the step that nothing overlaps, so it is kept short.
  int cut[kMaxHostChunks + 1];
  cut[0] = 0;
  double share[kMaxHostChunks], share_sum = 0.0, share_acc = 0.0;
  for (int c = 0; c < n_chunks; ++c) {
    share[c] = (n_chunks >= 4 && c == n_chunks - 1) ? 0.2 : (n_chunks >= 4 && c == n_chunks - 2) ? 0.5 : 1.0;
    share_sum += share[c];
  }
  for (int c = 0; c < n_chunks; ++c) {
    int r1 = cut[c] + 1;
    share_acc += share[c];
    const long long goal = (long long)((double)T * share_acc / share_sum);
    while (r1 < n_rows && indptr[(size_t)r1 + 1] <= goal && n_rows - r1 > n_chunks - 1 - c) ++r1;
    cut[c + 1] = c == n_chunks - 1 ? n_rows : r1;
  }
  // The copy engine works through its queue in order.  If the small uploads that every append and attention call
  // makes (records, plan) go through the same queue, the copies in of group c+1 are queued right AFTER the calls
  // of group c: queued earlier they would hold those uploads, and with them the kernels, back.
  auto copy_in = [&](int c) -> int {
    const size_t t0 = (size_t)indptr[(size_t)cut[c]], tn = (size_t)indptr[(size_t)cut[c + 1]] - t0;
    if (cudaMemcpyAsync(dk + t0 * kv_row, (const uint8_t*)new_k + t0 * kv_row, tn * kv_row, cudaMemcpyHostToDevice, s_in) != cudaSuccess ||
        cudaMemcpyAsync(dv + t0 * kv_row, (const uint8_t*)new_v + t0 * kv_row, tn * kv_row, cudaMemcpyHostToDevice, s_in) != cudaSuccess ||
        cudaMemcpyAsync(dq + t0 * q_row, (const uint8_t*)q + t0 * q_row, tn * q_row, cudaMemcpyHostToDevice, s_in) != cudaSuccess)
      return TIDE_ERR_CUDA;
    if (n_chunks > 1 && cudaEventRecord(kv->ev_host[c], s_in) != cudaSuccess) return TIDE_ERR_CUDA;
    return TIDE_OK;
  };
  // With kernel uploads nothing of the calls goes through the copy engine, and every copy in can be queued at once.
  const bool all_first = kv->upload_by_kernel;
  for (int c = 0; c < (all_first ? n_chunks : 1); ++c)
    if ((rc = copy_in(c)) != TIDE_OK) return rc;
  int64_t launches = 0, dec_items = 0, pre_items = 0, mrg_rows = 0;
  std::vector<int32_t> ip;
  for (int c = 0; c < n_chunks; ++c) {
    const int r0 = cut[c], r1 = cut[c + 1];
    const size_t t0 = (size_t)indptr[(size_t)r0], tn = (size_t)indptr[(size_t)r1] - t0;
    cudaEvent_t ev_done = kv->ev_host[kMaxHostChunks + c];
    if (n_chunks > 1 && cudaStreamWaitEvent(st, kv->ev_host[c], 0) != cudaSuccess) return TIDE_ERR_CUDA;
    ip.assign((size_t)(r1 - r0) + 1, 0);
    for (int b = r0; b <= r1; ++b) ip[(size_t)(b - r0)] = indptr[(size_t)b] - (int32_t)t0;
    rc = tide_kv_append(kv, layer, r1 - r0, ids.data() + r0, ip.data(), dk + t0 * kv_row, dv + t0 * kv_row, stream);
    if (rc != TIDE_OK) return rc;
    rc = tide_attend(kv, layer, r1 - r0, rows + r0, nullptr, dq + t0 * q_row, scale, dout + t0 * q_row,
                     lse ? dlse + t0 * g.Hq : nullptr, stream);
    if (rc != TIDE_OK) return rc;
    launches += kv->last_launches; dec_items += kv->last_decode_items; pre_items += kv->last_prefill_items; mrg_rows += kv->last_merge_rows;
    if (!all_first && c + 1 < n_chunks && (rc = copy_in(c + 1)) != TIDE_OK) return rc;
    if (n_chunks > 1 && (cudaEventRecord(ev_done, st) != cudaSuccess || cudaStreamWaitEvent(s_out, ev_done, 0) != cudaSuccess))
      return TIDE_ERR_CUDA;
    if (cudaMemcpyAsync((uint8_t*)out + t0 * q_row, dout + t0 * q_row, tn * q_row, cudaMemcpyDeviceToHost, s_out) != cudaSuccess) return TIDE_ERR_CUDA;
    if (lse && cudaMemcpyAsync(lse + t0 * g.Hq, dlse + t0 * g.Hq, tn * lse_row, cudaMemcpyDeviceToHost, s_out) != cudaSuccess) return TIDE_ERR_CUDA;
  }
  kv->last_launches = launches; kv->last_decode_items = dec_items; kv->last_prefill_items = pre_items; kv->last_merge_rows = mrg_rows;
  if (n_chunks > 1) {
    // the caller's stream ends after the last copy out, so stream order still means "the step is complete"
    if (cudaEventRecord(ev_end, s_out) != cudaSuccess || cudaStreamWaitEvent(st, ev_end, 0) != cudaSuccess) return TIDE_ERR_CUDA;
  }
  if (cudaStreamSynchronize(st) != cudaSuccess) return TIDE_ERR_CUDA;
  return TIDE_OK;
}

int tide_status(tide_kv_t* kv, void* stream) {
  if (kv == nullptr) return TIDE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(kv->h_status, kv->d_status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return TIDE_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return TIDE_ERR_CUDA;
  const int code = *kv->h_status;
  if (code != 0) {
    // a launch that was cut short may have left finished-split counters behind
    if (cudaMemsetAsync(kv->d_merge_ctr, 0, (size_t)kStepSegStride * kv->cfg.max_batch_rows * kv->g.Hkv * 4, st) != cudaSuccess) return TIDE_ERR_CUDA;
    if (cudaMemsetAsync(kv->d_status, 0, sizeof(int), st) != cudaSuccess) return TIDE_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return TIDE_ERR_CUDA;
  }
  return code == 0 ? TIDE_OK : code;
}

int tide_set_profiling(tide_kv_t* kv, int enable) {
  if (kv == nullptr) return TIDE_ERR_INVALID_ARG;
  if (enable && kv->ev_append[0] == nullptr) {
    for (cudaEvent_t& e : kv->ev_append) if (cudaEventCreate(&e) != cudaSuccess) return TIDE_ERR_CUDA;
    for (cudaEvent_t& e : kv->ev_attend) if (cudaEventCreate(&e) != cudaSuccess) return TIDE_ERR_CUDA;
  }
  kv->profiling = enable != 0;
  kv->have_append_times = kv->have_attend_times = false;
  return TIDE_OK;
}

int tide_phase_ms(tide_kv_t* kv, float* append_ms, float* decode_ms, float* tile_ms, float* merge_ms) {
  if (kv == nullptr || !kv->profiling) return TIDE_ERR_INVALID_ARG;
  float a = 0.f, d = 0.f, t = 0.f, m = 0.f;
  if (kv->have_append_times) {
    if (cudaEventSynchronize(kv->ev_append[1]) != cudaSuccess) return TIDE_ERR_CUDA;
    if (cudaEventElapsedTime(&a, kv->ev_append[0], kv->ev_append[1]) != cudaSuccess) return TIDE_ERR_CUDA;
  }
  if (kv->have_attend_times) {
    if (cudaEventSynchronize(kv->ev_attend[3]) != cudaSuccess) return TIDE_ERR_CUDA;
    if (cudaEventElapsedTime(&d, kv->ev_attend[0], kv->ev_attend[1]) != cudaSuccess) return TIDE_ERR_CUDA;
    if (cudaEventElapsedTime(&t, kv->ev_attend[1], kv->ev_attend[2]) != cudaSuccess) return TIDE_ERR_CUDA;
    if (cudaEventElapsedTime(&m, kv->ev_attend[2], kv->ev_attend[3]) != cudaSuccess) return TIDE_ERR_CUDA;
  }
  if (append_ms) *append_ms = a;
  if (decode_ms) *decode_ms = d;
  if (tile_ms) *tile_ms = t;
  if (merge_ms) *merge_ms = m;
  kv->have_append_times = false;
  return TIDE_OK;
}

int tide_tune(tide_kv_t* kv, int knob, int64_t value) {
  if (kv == nullptr) return TIDE_ERR_INVALID_ARG;
  switch (knob) {
    case TIDE_TUNE_ITEMS_PER_SM:
      if (value < 1 || value > 64) return TIDE_ERR_INVALID_ARG;
      kv->items_per_sm = (int)value;
      break;
    case TIDE_TUNE_GROUPING: kv->no_grouping = value == 0; break;
    case TIDE_TUNE_MIN_SAVED_BYTES:
      if (value < 0) return TIDE_ERR_INVALID_ARG;
      kv->min_saved_bytes = value;
      break;
    case TIDE_TUNE_HOST_STEP_CHUNKS:
      if (value < 0 || value > kMaxHostChunks) return TIDE_ERR_INVALID_ARG;
      kv->host_step_chunks = (int)value;
      break;
    case TIDE_TUNE_UMMA_MIN_ROWS:
      if (value <= kDecodeTileRows || value > 0x7fffffff) return TIDE_ERR_INVALID_ARG;
      kv->umma_min_rows = (int)value;
      break;
    case TIDE_TUNE_WAIT_LIMIT_US:
      if (value < 1 || value > 60ll * 1000 * 1000) return TIDE_ERR_INVALID_ARG;
      kv->wait_limit_ns = value * 1000;
      break;
    case TIDE_TUNE_DROP_FIRST_STAGE: kv->drop_first_stage_once = value != 0; break;
    case TIDE_TUNE_UPLOAD_BY_KERNEL: kv->always_upload_by_kernel = value != 0; break;
    case TIDE_TUNE_INLINE_DESCRIPTORS: kv->inline_descriptors = value != 0; break;
    case TIDE_TUNE_HOST_ZERO_COPY: kv->host_zero_copy = value != 0; break;
    case TIDE_TUNE_UMMA_TILE_KEYS:
      if (value != 64 && value != 128) return TIDE_ERR_INVALID_ARG;
      kv->umma_tile_keys = (int)value;
      break;
    default: return TIDE_ERR_INVALID_ARG;
  }
  kv->step_valid = false;   // a held plan was made with the old settings
  return TIDE_OK;
}

// Read-only view of a handle for attend_static.cu (not part of the public header).
int tide_internal_view(tide_kv_t* kv, tide::StaticView* v) {
  if (kv == nullptr || v == nullptr) return TIDE_ERR_INVALID_ARG;
  v->g = kv->g;
  v->pool = kv->pool;
  v->table = kv->d_table;
  v->status = kv->d_status;
  v->len = kv->len.data();
  v->live = kv->live.data();
  v->max_tasks = kv->cfg.max_tasks;
  v->device = kv->device;
  v->num_sms = kv->num_sms;
  v->items_per_sm = kv->items_per_sm;
  v->wait_limit_ns = kv->wait_limit_ns;
  return TIDE_OK;
}

int tide_last_sharing(tide_kv_t* kv, int64_t* groups, int64_t* rows) {
  if (kv == nullptr) return TIDE_ERR_INVALID_ARG;
  if (groups) *groups = kv->last_groups;
  if (rows) *rows = kv->last_grouped_rows;
  return TIDE_OK;
}

int tide_last_plan(tide_kv_t* kv, int64_t* decode_items, int64_t* prefill_items, int64_t* merge_rows,
                   int64_t* kernel_launches) {
  if (kv == nullptr) return TIDE_ERR_INVALID_ARG;
  if (decode_items) *decode_items = kv->last_decode_items;
  if (prefill_items) *prefill_items = kv->last_prefill_items;
  if (merge_rows) *merge_rows = kv->last_merge_rows;
  if (kernel_launches) *kernel_launches = kv->last_launches;
  return TIDE_OK;
}

}  // extern "C"

namespace tide {

// Multiprocessors of the current device; asked of the runtime once per device.
int sm_count() {
  constexpr int kMaxDevices = 64;
  static std::atomic<int> cache[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (dev >= 0 && dev < kMaxDevices) {
    const int c = cache[dev].load(std::memory_order_relaxed);
    if (c > 0) return c;
  }
  int n = 0;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 0;
  if (dev >= 0 && dev < kMaxDevices) cache[dev].store(n, std::memory_order_relaxed);
  return n;
}

}  // namespace tide

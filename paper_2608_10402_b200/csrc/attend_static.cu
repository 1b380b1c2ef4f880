// tide_attend_decode_static: decode-row attention whose split-KV scratch lives in a fixed device array.
//
// tide_attend keeps the partial results of its KV splits, and the row descriptors its kernels read, in the
// workspace the caller allocated.  Some callers cannot allocate at the moment they need attention: a serving
// loop that runs while another thread captures a CUDA graph in global mode (cudaMalloc is forbidden there), a
// process whose framework allocator already owns all device memory so that a fresh cudaMalloc fails, or a
// latency-critical step that must not take cudaMalloc's implicit device synchronisation.  For them this file
// gives one entry point that allocates nothing, on the device or on the host: its scratch is the file-scope
// array below, which every GPU that loads the library holds until the process exits.
//
// The array's name is only a host-side stand-in in host code; the device address is looked up once per device
// with cudaGetSymbolAddress and handed to the (unchanged) decode and merge kernels.  The row descriptors reach
// the device as kernel arguments of a small set-up kernel that expands them into the array, so the call makes no
// copy from host memory at all and is asynchronous on its stream.
#include <atomic>

#include "tide_internal.h"

using namespace tide;

namespace {

constexpr int kMaxRows = TIDE_STATIC_MAX_ROWS;
constexpr int kMaxPartRows = 16384;                    // (split, token, head) partial rows
constexpr int kMaxD = 128;
constexpr size_t kSegBytes = 2 * kMaxRows * sizeof(Segment);              // decode list + merge list
constexpr size_t kLseOff = (kSegBytes + 255) / 256 * 256;
constexpr size_t kPartOff = (kLseOff + kMaxPartRows * sizeof(float) + 255) / 256 * 256;
constexpr size_t kScratchBytes = kPartOff + (size_t)kMaxPartRows * kMaxD * sizeof(float);   // about 8.1 MB

static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
// Device address of the array, per device.  The lookup gives the same answer every time, so threads that race
// on the first call of a device all store the same value.
std::atomic<unsigned char*> g_scratch_ptr[kMaxDevices];

int ceil_div(int a, int b) { return (a + b - 1) / b; }

// One row as the host planned it; the set-up kernel turns these into Segment records.
struct StaticRow {
  int32_t table_off, n, p, n_splits, chunk;
};
struct StaticPlanArgs {          // passed by value (about 1.3 KB of kernel arguments)
  int32_t n_rows, Hkv, Hq;
  StaticRow rows[kMaxRows];
};

// Expands the planned rows into the decode list (segs[0 .. n_rows)) and the merge list (segs[kMaxRows ...)): the
// running sums over rows (query offset, first work item, first partial row, first merge row) are taken here, by
// one thread, in row order - at most 64 rows.  Every field of every record written is set, so nothing of an
// earlier call's records shows through.
__global__ void static_plan_kernel(const StaticPlanArgs a, Segment* __restrict__ segs) {
  if (blockIdx.x != 0 || threadIdx.x != 0) return;
  int qoff = 0, items = 0, part = 0, merge = 0, n_merge = 0;
  for (int b = 0; b < a.n_rows; ++b) {
    const StaticRow r = a.rows[b];
    Segment s;
    s.table_off = r.table_off;
    s.q_off = qoff;
    s.n = r.n;
    s.p = r.p;
    s.item_base = items;
    s.n_mtiles = 1;
    s.n_splits = r.n_splits;
    s.chunk = r.chunk;
    s.part_base = 0;
    s.merge_base = 0;
    s.causal = 1;
    s.origin = 0;
    s.partial = 0;
    s.x_part_base = 0;
    s.x_n_splits = 0;
    s.x_stride = 0;
    items += a.Hkv * r.n_splits;
    if (r.n_splits > 1) {
      s.part_base = part;
      s.merge_base = merge;
      part += r.n_splits * r.n * a.Hq;
      merge += r.n * a.Hq;
      segs[kMaxRows + n_merge++] = s;
    }
    segs[b] = s;
    qoff += r.n;
  }
}

}  // namespace

// Defined in tide_host.cu; a narrow accessor so that this file needs nothing else of the handle.
extern "C" int tide_internal_view(tide_kv_t* kv, tide::StaticView* v);

extern "C" int tide_attend_decode_static(tide_kv_t* kv, int32_t n_rows, const tide_row_t* rows, const void* q,
                                         float scale, void* out, float* lse, void* stream) {
  if (kv == nullptr || n_rows < 0) return TIDE_ERR_INVALID_ARG;
  if (n_rows == 0) return TIDE_OK;
  if (rows == nullptr || q == nullptr || out == nullptr) return TIDE_ERR_INVALID_ARG;
  if (((uintptr_t)q & 15) || ((uintptr_t)out & 15) || ((uintptr_t)lse & 3) || !(scale == scale)) return TIDE_ERR_INVALID_ARG;
  if (n_rows > kMaxRows) return TIDE_ERR_WORKSPACE;      // beyond the fixed scratch: use tide_attend

  StaticView v;
  int rc = tide_internal_view(kv, &v);
  if (rc != TIDE_OK) return rc;
  const Geom& g = v.g;
  if (g.D > kMaxD) return TIDE_ERR_WORKSPACE;
  for (int b = 0; b < n_rows; ++b) {
    const tide_row_t& r = rows[b];
    if (r.task < 0 || r.task >= v.max_tasks) return TIDE_ERR_INVALID_ARG;
    if (!v.live[r.task]) return TIDE_ERR_UNKNOWN_TASK;
    if (!(r.q_len >= 1 && r.q_len <= r.ctx_len && r.ctx_len <= v.len[r.task])) return TIDE_ERR_CTX_RANGE;
    if (r.q_len > kDecodeTileRows / g.G) return TIDE_ERR_INVALID_ARG;   // decode-style rows only
  }

  // ---- once per device: the device address of the scratch array (first call; do it before any capture) ----
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TIDE_ERR_CUDA;
  if (dev != v.device) return TIDE_ERR_INVALID_ARG;       // the handle's device must be current
  if (dev < 0 || dev >= kMaxDevices) return TIDE_ERR_WORKSPACE;
  unsigned char* scratch = g_scratch_ptr[dev].load(std::memory_order_acquire);
  if (scratch == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return TIDE_ERR_CUDA;
    scratch = static_cast<unsigned char*>(p);
    g_scratch_ptr[dev].store(scratch, std::memory_order_release);
  }

  // ---- plan: split long rows over KV towards the library's number of work items per SM, as far as the fixed
  //      number of partial rows allows ----
  StaticPlanArgs pa;
  pa.n_rows = n_rows;
  pa.Hkv = g.Hkv;
  pa.Hq = g.Hq;
  long long w = 0;
  for (int b = 0; b < n_rows; ++b) w += (long long)g.Hkv * rows[b].ctx_len;
  long long chunk_target = w / ((long long)v.num_sms * v.items_per_sm) + 1;
  if (chunk_target < 256) chunk_target = 256;
  long long items = 0, merge_rows = 0;
  for (int attempt = 0; attempt < 40; ++attempt) {
    long long part_rows = 0;
    items = 0;
    merge_rows = 0;
    for (int b = 0; b < n_rows; ++b) {
      const tide_row_t& r = rows[b];
      int n_splits = (int)((r.ctx_len + chunk_target - 1) / chunk_target);
      if (n_splits > kMaxSplits) n_splits = kMaxSplits;
      if (n_splits < 1) n_splits = 1;
      const int chunk = ceil_div(ceil_div(r.ctx_len, n_splits), 2 * kStageKeys) * 2 * kStageKeys;
      n_splits = ceil_div(r.ctx_len, chunk);
      StaticRow& s = pa.rows[b];
      s.table_off = r.task * g.max_pages_per_task;
      s.n = r.q_len;
      s.p = r.ctx_len - r.q_len;
      s.n_splits = n_splits;
      s.chunk = chunk;
      items += (long long)g.Hkv * n_splits;
      if (n_splits > 1) {
        part_rows += (long long)n_splits * r.q_len * g.Hq;
        merge_rows += (long long)r.q_len * g.Hq;
      }
    }
    if (part_rows <= kMaxPartRows) break;
    chunk_target *= 2;
    if (attempt == 39) return TIDE_ERR_WORKSPACE;
  }
  int n_merge = 0;
  for (int b = 0; b < n_rows; ++b) n_merge += pa.rows[b].n_splits > 1 ? 1 : 0;

  // ---- the row records into the scratch array (kernel arguments, expanded on the device), then the two kernels ----
  cudaStream_t st = (cudaStream_t)stream;
  Segment* d_segs = reinterpret_cast<Segment*>(scratch);
  static_plan_kernel<<<1, 32, 0, st>>>(pa, d_segs);
  if (cudaGetLastError() != cudaSuccess) return TIDE_ERR_CUDA;
  AttendParams ap;
  ap.pool = v.pool;
  ap.table = v.table;
  ap.segs = d_segs;
  ap.n_segs = n_rows;
  ap.n_items = (int)items;
  ap.q = (const uint16_t*)q;
  ap.out = (uint16_t*)out;
  ap.lse = lse;
  ap.part_lse = reinterpret_cast<float*>(scratch + kLseOff);
  ap.part_o = reinterpret_cast<float*>(scratch + kPartOff);
  ap.scale_log2e = scale * 1.4426950408889634f;
  ap.status = v.status;
  ap.g = g;
  ap.wait_limit_ns = v.wait_limit_ns;
  if (launch_attend_decode(ap, st) != cudaSuccess) return TIDE_ERR_CUDA;
  if (merge_rows > 0) {
    MergeParams mp;
    mp.segs = d_segs + kMaxRows;
    mp.n_segs = n_merge;
    mp.n_rows = (int)merge_rows;
    mp.part_o = ap.part_o;
    mp.part_lse = ap.part_lse;
    mp.out = (uint16_t*)out;
    mp.lse = lse;
    mp.Hq = g.Hq;
    mp.D = g.D;
    if (launch_merge(mp, st) != cudaSuccess) return TIDE_ERR_CUDA;
  }
  return TIDE_OK;
}

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
// with cudaGetSymbolAddress and handed to the (unchanged) decode and merge kernels.
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
unsigned char* g_scratch_ptr[kMaxDevices];             // device address of the array, per device
bool g_scratch_ready[kMaxDevices];

int ceil_div(int a, int b) { return (a + b - 1) / b; }

}  // namespace

// Defined in tide_host.cu; narrow accessors so that this file needs nothing else of the handle.
extern "C" int tide_internal_view(tide_kv_t* kv, Geom* g, const uint8_t** pool, const int32_t** table, int** status,
                                  const int32_t** len, const uint8_t** live, int32_t* max_tasks);

extern "C" int tide_attend_decode_static(tide_kv_t* kv, int32_t n_rows, const tide_row_t* rows, const void* q,
                                         float scale, void* out, float* lse, void* stream) {
  if (kv == nullptr || n_rows < 0) return TIDE_ERR_INVALID_ARG;
  if (n_rows == 0) return TIDE_OK;
  if (rows == nullptr || q == nullptr || out == nullptr) return TIDE_ERR_INVALID_ARG;
  if (((uintptr_t)q & 15) || ((uintptr_t)out & 15) || ((uintptr_t)lse & 3) || !(scale == scale)) return TIDE_ERR_INVALID_ARG;
  if (n_rows > kMaxRows) return TIDE_ERR_WORKSPACE;      // beyond the fixed scratch: use tide_attend

  Geom g;
  const uint8_t* pool; const int32_t* table; int* status; const int32_t* len; const uint8_t* live; int32_t max_tasks;
  int rc = tide_internal_view(kv, &g, &pool, &table, &status, &len, &live, &max_tasks);
  if (rc != TIDE_OK) return rc;
  if (g.D > kMaxD) return TIDE_ERR_WORKSPACE;
  long long total_q = 0;
  for (int b = 0; b < n_rows; ++b) {
    const tide_row_t& r = rows[b];
    if (r.task < 0 || r.task >= max_tasks) return TIDE_ERR_INVALID_ARG;
    if (!live[r.task]) return TIDE_ERR_UNKNOWN_TASK;
    if (!(r.q_len >= 1 && r.q_len <= r.ctx_len && r.ctx_len <= len[r.task])) return TIDE_ERR_CTX_RANGE;
    if (r.q_len * g.G > kDecodeTileRows) return TIDE_ERR_INVALID_ARG;   // decode-style rows only
    total_q += r.q_len;
  }

  // ---- once per device: the device address of the scratch array (first call; do it before any capture) ----
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TIDE_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return TIDE_ERR_WORKSPACE;
  if (!g_scratch_ready[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return TIDE_ERR_CUDA;
    g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
    g_scratch_ready[dev] = true;
  }
  unsigned char* scratch = g_scratch_ptr[dev];

  // ---- plan with fixed-size host arrays: split long rows over KV until the SMs are covered or the fixed
  //      number of partial rows is used up ----
  Segment segs[2 * kMaxRows];
  long long w = 0;
  for (int b = 0; b < n_rows; ++b) w += (long long)g.Hkv * rows[b].ctx_len;
  long long chunk_target = w / (148 * 8) + 1;
  if (chunk_target < 256) chunk_target = 256;
  long long part_rows = 0;
  for (int attempt = 0; attempt < 40; ++attempt) {
    part_rows = 0;
    long long qoff = 0;
    for (int b = 0; b < n_rows; ++b) {
      const tide_row_t& r = rows[b];
      int n_splits = (int)((r.ctx_len + chunk_target - 1) / chunk_target);
      if (n_splits > kMaxSplits) n_splits = kMaxSplits;
      if (n_splits < 1) n_splits = 1;
      const int chunk = ceil_div(ceil_div(r.ctx_len, n_splits), 2 * kStageKeys) * 2 * kStageKeys;
      n_splits = ceil_div(r.ctx_len, chunk);
      Segment s{};
      s.table_off = r.task * g.max_pages_per_task;
      s.q_off = (int32_t)qoff;
      s.n = r.q_len;
      s.p = r.ctx_len - r.q_len;
      s.n_mtiles = 1;
      s.n_splits = n_splits;
      s.chunk = chunk;
      s.causal = 1;
      if (n_splits > 1) part_rows += (long long)n_splits * r.q_len * g.Hq;
      segs[b] = s;
      qoff += r.q_len;
    }
    if (part_rows <= kMaxPartRows) break;
    chunk_target *= 2;
    if (attempt == 39) return TIDE_ERR_WORKSPACE;
  }
  long long items = 0, part_cursor = 0, merge_rows = 0;
  int n_merge = 0;
  for (int b = 0; b < n_rows; ++b) {
    Segment& s = segs[b];
    s.item_base = (int32_t)items;
    items += (long long)g.Hkv * s.n_splits;
    if (s.n_splits > 1) {
      s.part_base = (int32_t)part_cursor;
      part_cursor += (long long)s.n_splits * s.n * g.Hq;
      s.merge_base = (int32_t)merge_rows;
      merge_rows += (long long)s.n * g.Hq;
      segs[kMaxRows + n_merge++] = s;
    }
  }

  // ---- descriptors into the scratch array (a plain copy from this stack frame), then the two kernels ----
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(scratch, segs, kSegBytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return TIDE_ERR_CUDA;
  AttendParams ap;
  ap.pool = pool;
  ap.table = table;
  ap.segs = reinterpret_cast<const Segment*>(scratch);
  ap.n_segs = n_rows;
  ap.n_items = (int)items;
  ap.q = (const uint16_t*)q;
  ap.out = (uint16_t*)out;
  ap.lse = lse;
  ap.part_lse = reinterpret_cast<float*>(scratch + kLseOff);
  ap.part_o = reinterpret_cast<float*>(scratch + kPartOff);
  ap.scale_log2e = scale * 1.4426950408889634f;
  ap.status = status;
  ap.g = g;
  if (launch_attend_decode(ap, st) != cudaSuccess) return TIDE_ERR_CUDA;
  if (merge_rows > 0) {
    MergeParams mp;
    mp.segs = reinterpret_cast<const Segment*>(scratch) + kMaxRows;
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

// Internal declarations shared by the host code and the kernels of libtide.so.
//
// Physical page layout (private; callers see logical content only):
//   pool[page][kv_head][K|V][group = slot/8][slab = d/64][slot%8][64 bf16]
// i.e. the block of one (page, kv_head) is its K block followed by its V block; each is a run of S/8 groups of 8
// consecutive slots, a group being D/64 slabs of 8 rows x 128 bytes (one 1-KB core-matrix atom of the
// tensor-core shared-memory layouts).  Inside an atom the 16-byte chunk c of row r is stored at chunk position
// c ^ r (the 128-byte swizzle).  Consecutive groups - of one page, and of the K (or V) blocks of several pages
// copied one after the other into a tile - are a uniform distance apart, so ONE plain contiguous bulk copy of a
// K or V block (or of both, for ldmatrix users) lands in shared memory ready both for conflict-free ldmatrix and
// as a canonical K-major (K) or MN-major (V) operand of tcgen05 matrix descriptors (stride between 8-key groups
// = group_bytes, between slabs = 1 KB), with no tensor map.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/tide.h"

namespace tide {

constexpr int kStageKeys = 64;       // keys per pipeline stage of the mma.sync attention kernel
constexpr int kMaxSplits = 128;      // most KV splits of one row
constexpr int kDecodeTileRows = 16;  // packed (query, head) rows per decode-style work item
constexpr int kMmaTileRows = 64;     // packed rows per work item of the warp-MMA tile path
constexpr int kUmmaTileRows = 128;   // packed rows per work item of the tcgen05 path
constexpr long long kWaitLimitNsDefault = 2000000000LL;  // bound of every in-kernel wait unless the handle says otherwise
constexpr int kTargetItemsPerSm = 3;   // measured: fewer, longer items beat finer balance (per-item set-up dominates)

struct Geom {
  int Hq, Hkv, D, S, G;
  int max_pages_per_task;
  int group_bytes;   // one 8-slot group of a K (or V) block: (D/64) * 1024
  int kblock_bytes;  // the K (or V) block of one (page, head): (S/8) * group_bytes = S*D*2; V sits this far behind K
  int head_bytes;    // block of one (page, head): K block + V block
  long long page_bytes;
};

// Byte offset, inside the block of a (page, head), of the 16-byte chunk c (= d / 8) of slot `slot`; kv = 0 for K, 1 for V.
__host__ __device__ __forceinline__ int blk_offset(const Geom& g, int slot, int kv, int c) {
  return kv * g.kblock_bytes + (slot >> 3) * g.group_bytes + (c >> 3) * 1024 + (slot & 7) * 128 + (((c & 7) ^ (slot & 7)) << 4);
}

// One batch row as the kernels see it.  Items of a segment are numbered
// ((kv_head * n_splits) + split) * n_mtiles + m_tile from item_base.
struct __align__(16) Segment {
  int32_t table_off;   // task * max_pages_per_task
  int32_t q_off;       // index of the row's first query token in q / out
  int32_t n;           // q_len
  int32_t p;           // preserved prefix = ctx_len - q_len
  int32_t item_base;
  int32_t n_mtiles;
  int32_t n_splits;
  int32_t chunk;       // keys per split, a multiple of kStageKeys
  int32_t part_base;   // first partial row ((split * n + token) * Hq + head) when the item writes partials
  int32_t merge_base;  // first row of this segment in the merge launch
  // Rows of one batch whose tasks share their first pages (forked tasks) read those pages once: the shared range
  // is one segment whose `n` tokens are the member rows' queries and all see the same keys (causal = 0), each
  // member's own range starts behind it (origin), both write partials, and the member's merge takes both.
  int32_t causal;      // query i sees keys [0, p + i * causal + 1): 1 for a task's own tokens, 0 for a shared range
  int32_t origin;      // first key of the range this segment covers (split s starts at origin + s * chunk)
  int32_t partial;     // 1: write partials even when n_splits == 1 (another segment contributes to the same rows);
                       // 2: a split decode-style segment whose last-finishing split merges the partials itself
                       //    (AttendParams::merge_ctr[x_part_base + kv_head] counts the finished splits)
  int32_t x_part_base; // the other contribution to this segment's rows: first partial row of token 0's head 0 ...
  int32_t x_n_splits;  // ... its number of splits (0 = none) ...
  int32_t x_stride;    // ... and the distance in rows between its consecutive splits
};
static_assert(sizeof(Segment) == 64, "Segment layout");

struct AttendParams {
  const uint8_t* pool;
  const int32_t* table;
  const Segment* segs;
  int n_segs;
  int n_items;
  const uint16_t* q;
  uint16_t* out;
  float* lse;        // may be null
  float* part_o;     // [partial rows][D] fp32, normalised
  float* part_lse;   // [partial rows] fp32, base-2 log units
  float scale_log2e;
  int* status;
  Geom g;
  // Fixed-grid mode (a launch that a CUDA graph replays for other batches): the launch has grid_cap CTAs and the
  // kernel reads n_items = dyn[0] and n_segs = dyn[1] from device memory; CTAs beyond n_items leave at once.
  const int32_t* dyn = nullptr;
  int grid_cap = 0;
  int* merge_ctr = nullptr;   // per (segment with partial == 2, kv head): splits finished so far; zero between launches
  long long wait_limit_ns = kWaitLimitNsDefault;   // bound of every wait inside the kernel
  // Test hook for the bounded waits (never set in normal use): in work item 0 the producer leaves out its part
  // of the first stage, so the consumers' wait for that stage runs out and the time-out path executes.
  int debug_drop_first_stage = 0;
};

struct MergeParams {
  const Segment* segs;
  int n_segs;
  int n_rows;
  const float* part_o;
  const float* part_lse;
  uint16_t* out;
  float* lse;
  int Hq, D;
  const int32_t* dyn = nullptr;   // fixed-grid mode: n_rows = dyn[0], n_segs = dyn[1]
  int grid_cap_rows = 0;
};

struct __align__(16) AppendRec {
  int32_t table_off;  // task * max_pages_per_task
  int32_t pos0;       // position in the task of the record's first token
  int32_t tok0;       // index of that token in new_k / new_v
  int32_t count;
  // When the same launch also applies the page-table delta (AppendParams::upd_*), the table cannot be trusted for
  // the pages the delta brings: logical pages >= new_lp0 of this record are upd_val[new_off + (lp - new_lp0)].
  int32_t new_lp0;    // INT_MAX: every page comes from the table
  int32_t new_off;
  int32_t grp0;       // 8-slot groups of the page blocks that the records before this one touch (a record touches
                      // ((pos0 & 7) + count + 7) / 8 of them): the append kernel's unit of work
  int32_t pad1;
};
static_assert(sizeof(AppendRec) == 32, "AppendRec layout");

struct AppendParams {
  uint8_t* pool;
  const int32_t* table;
  const AppendRec* recs;
  int n_recs;
  int n_tokens;
  const uint16_t* new_k;
  const uint16_t* new_v;
  Geom g;
  const int32_t* dyn = nullptr;   // fixed-grid mode: n_recs = dyn[0], n_tokens = dyn[1]
  int grid_cap_tokens = 0;
  // page-table delta applied by the same launch: table_rw[upd_idx[i]] = upd_val[i] (n_upd may be 0)
  int32_t* table_rw = nullptr;
  const int32_t* upd_idx = nullptr;
  const int32_t* upd_val = nullptr;
  int n_upd = 0;
};

// Small batches carry their descriptors in the launch itself: a decode-only batch of up to kInlineSegs rows, and an
// append of up to kInlineRecs records with up to kInlineUpd new page-table entries, need no upload before the kernel
// (the kernels read them from their own parameter space), which takes one launch each out of a decode step.
constexpr int kInlineSegs = 128;
constexpr int kInlineRecs = 128;
constexpr int kInlineUpd = 256;
struct AttendInline {
  AttendParams p;                  // p.segs is not used
  Segment segs[kInlineSegs];
};
struct AppendInline {
  AppendParams p;                  // p.recs, p.upd_idx, p.upd_val are not used
  AppendRec recs[kInlineRecs];
  int32_t upd[2 * kInlineUpd];     // p.n_upd table indices, then p.n_upd values
};

// What tide_attend_decode_static needs of a handle (filled by tide_internal_view in tide_host.cu).
struct StaticView {
  Geom g;
  const uint8_t* pool;
  const int32_t* table;
  int* status;
  const int32_t* len;      // host: resident tokens per task
  const uint8_t* live;     // host
  int32_t max_tasks;
  int device, num_sms, items_per_sm;
  long long wait_limit_ns;
};

cudaError_t launch_table_update(int32_t* table, const int32_t* idx, const int32_t* val, int n, cudaStream_t s);
cudaError_t launch_upload(void* dst, const void* src_mapped_host, size_t bytes, cudaStream_t s);   // bytes % 4 == 0
cudaError_t launch_append(const AppendParams& p, cudaStream_t s);
cudaError_t launch_copy_pages(uint8_t* pool, const int32_t* src, const int32_t* dst, int n, long long page_bytes, cudaStream_t s);
cudaError_t launch_read(const uint8_t* pool, const int32_t* table_row, int pos0, int len, uint16_t* out_k,
                        uint16_t* out_v, const Geom& g, cudaStream_t s);
cudaError_t launch_attend_decode(const AttendParams& p, cudaStream_t s);
cudaError_t launch_attend_decode_inline(const AttendInline& p, cudaStream_t s);   // p.p.n_segs <= kInlineSegs, exact grid
cudaError_t launch_append_inline(const AppendInline& p, cudaStream_t s);
cudaError_t launch_attend_tile(const AttendParams& p, cudaStream_t s);
cudaError_t launch_merge(const MergeParams& p, cudaStream_t s);
cudaError_t launch_attend_umma(const AttendParams& p, cudaStream_t s);
cudaError_t attend_kernels_init();
cudaError_t attend_umma_init();
cudaError_t launch_attend_umma128(const AttendParams& p, cudaStream_t s);
cudaError_t attend_umma128_init();
int sm_count();   // multiprocessors of the current device (looked up once per device)

#ifdef __CUDACC__
// ---------------------------------------------------------------------------------------------
// device helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ long long global_ns() {
  long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  `abort_flag` lives in shared memory: once any thread of the CTA has given up, every
// later wait returns at once so that the CTA still walks its normal control flow to the end.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                          long long limit_ns) {
  if (mbar_try(bar, parity)) return true;
  if (*abort_flag) return false;
  const long long t0 = global_ns();
  int spins = 0;
  while (!mbar_try(bar, parity)) {
    if ((++spins & 255) == 0) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > limit_ns) {
        *abort_flag = 1;
        atomicExch(status, (int)TIDE_ERR_DEVICE_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}
// 1-D bulk copy global -> shared, completion counted on an mbarrier.  16-byte aligned, size % 16 == 0.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
// D[16x8] += A[16x16] * B[16x8], bf16 inputs, fp32 accumulate
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Locate the segment that owns work index `idx` (segments sorted by the base returned by `base_of`).
template <typename F>
__device__ __forceinline__ int find_segment(int n_segs, int idx, F base_of) {
  int lo = 0, hi = n_segs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (base_of(mid) <= idx) lo = mid; else hi = mid - 1;
  }
  return lo;
}
#endif  // __CUDACC__

}  // namespace tide

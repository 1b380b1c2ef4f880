// Append-prefill attention for resume rows on the 5th-generation tensor cores (tcgen05.mma, accumulators in
// TMEM).
//
// What it computes (paper Section 4: a resumed task's appended observation tokens attend to the whole
// preserved KV state instead of re-running prefill over the history): for a work item
// (row, kv_head, m_tile, split), 256 packed rows r = q_index * G + g (two 128-row MMA tiles A and B) against
// keys [kv_begin, kv_end), query q_index seeing keys [0, prefix + q_index]; online softmax in the base-2
// domain; O and LSE written directly, or as normalised partials when the row is split over KV.
// This is a dense contraction (n*G x ctx x D), so it is bound by the tensor pipe: 4*D flops per visible
// (packed row, key) pair against Hkv*D*4 bytes per key shared by all packed rows.
//
// CTA = 12 warps: softmax warpgroups A (warps 0-3) and B (warps 4-7), one thread per row; warp 8 streams tiles of
// 64 keys, one plain 1-D bulk copy per K block and per V block of a (page, head) (blocks are stored as the canonical
// 128-byte-swizzled core-matrix atoms, so the K blocks of a tile laid one after the other ARE the K-major K operand
// and the V blocks the MN-major V operand, a uniform 2 KB between 8-key groups); one lane of warp 9 issues every MMA.
// TMEM (512 columns):
//   Q_A Q_B   2 x 64   the queries as packed bf16, staged once per item
//   S_A S_B   2 x 64   fp32 logits of one 64-key tile; P (packed bf16) overwrites the first 32 columns
//   O_A O_B   2 x 128  fp32 output accumulators
//   S_t = Q_t . K_j^T   TS MMA, 128x64x16 x 8     O_t += P_t . V_j   TS MMA, 128x128x16 x 4 (V MN-major)
// Both products take their A operand from TMEM: an MMA whose two operands both come from shared memory
// (128x128x16, 8 KB per instruction) was measured at ~146 cycles against ~90 for the TMEM-A form, i.e. it is
// bound by shared-memory operand fetch; with Q in TMEM shared memory only feeds K and V (64 B per cycle) and
// is free for a deep K/V ring.  The two halves ping-pong: while warpgroup A computes exponentials the tensor
// pipe runs PV_B(j) and QK_B(j+1), and vice versa.  O is only rescaled when a row's running maximum grows by
// more than 2^8 (the final normalisation uses the same stale maximum, so the result is exact).
// Every wait is bounded; a wait that runs out sets TIDE_ERR_DEVICE_TIMEOUT and the CTA drains and exits.
#include <climits>
#include <type_traits>

#include "tide_internal.h"

namespace tide {

namespace umma {

constexpr int D = 128;
constexpr int kTileKeys = 64;
constexpr int kThreads = 384;   // 3 warpgroups: softmax A, softmax B, {producer warp 8, MMA issuer warp 9, two idle warps}
constexpr int kNumBuf = 6;                          // ring of (K tile, V tile) slots
constexpr int kGroupBytes = (D / 64) * 1024;        // one 8-key group of a K (or V) tile: two 1-KB atoms
constexpr int kTileBytes = (kTileKeys / 8) * kGroupBytes;   // one K or V tile of 64 keys: 16 KB
constexpr int kSlotBytes = 2 * kTileBytes;          // K tile then V tile
constexpr int kSmemBytes = kNumBuf * kSlotBytes + 1024;
constexpr float kRescaleThreshold = 8.0f;           // log2 units
constexpr uint32_t kColQ = 0, kColS = 128, kColO = 256;

// instruction descriptor: fp32 accumulate, bf16 A and B, M = 128; bit 16 = B is MN-major
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 4) << 24);
constexpr uint32_t kIdescQK = kIdescBase | ((64u >> 3) << 17);                  // N = 64 keys
constexpr uint32_t kIdescPV = kIdescBase | ((128u >> 3) << 17) | (1u << 16);    // N = D = 128

__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;   // descriptor version of this architecture
  d |= (uint64_t)2 << 61;   // 128-byte swizzle
  return d;
}
// A operand (16-bit, two K-elements per 32-bit column, one row per lane) read from TMEM, B from shared memory
// Called by ALL lanes of the (converged) MMA warp; one elected lane issues.  Keeping the warp converged lets
// the compiler hold descriptors and addresses in uniform registers instead of serialising their arithmetic in
// one divergent lane, which had limited the issue rate to about one MMA per 100 cycles.
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .pred e;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
      ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st32u(uint32_t taddr, const uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
        "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
        "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
        "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
  uint32_t u[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) u[i] = __float_as_uint(v[i]);
  tmem_st32u(taddr, u);
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// packed pairs of floats: one instruction for two elements (fma.rn.f32x2 / add.rn.f32x2)
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
  return d;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

struct Bars {
  uint64_t kv_full[kNumBuf];
  uint64_t kv_empty[kNumBuf];
  uint64_t q_full;
  uint64_t s_full[2];   // S_t(j) is in TMEM (and every earlier MMA, PV_t(j-1) included, has retired)
  uint64_t p_full[2];   // P_t(j) is in TMEM
  uint64_t o_full[2];   // the last PV_t has retired
  uint64_t mma_done;    // every MMA of the item has retired
};

__global__ void __launch_bounds__(kThreads, 1) attend_umma_kernel(const AttendParams P) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) Bars bars;
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const Geom& g = P.g;

  // ---- which item ----
  const int item = blockIdx.x;
  int n_segs = P.n_segs;
  if (P.dyn != nullptr) {                      // fixed grid: the batch's counts live in device memory
    if (item >= P.dyn[0]) return;
    n_segs = P.dyn[1];
  }
  const int si = find_segment(n_segs, item, [&](int i) { return P.segs[i].item_base; });
  const Segment seg = P.segs[si];
  int local = item - seg.item_base;
  const int m_tile = local % seg.n_mtiles;
  local /= seg.n_mtiles;
  const int split = local % seg.n_splits;
  const int kvh = local / seg.n_splits;
  const int R = seg.n * g.G;
  const int item_row0 = m_tile * kUmmaTileRows * 2;
  const int kv_begin = seg.origin + split * seg.chunk;
  const bool direct = seg.n_splits == 1 && seg.partial == 0;
  // per 128-row tile: rows present, last key any of its rows sees, number of 64-key tiles to process
  int t_rows[2], t_end[2], t_tiles[2], t_min_limit[2];
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    const int r0 = item_row0 + t * 128;
    t_rows[t] = max(0, min(128, R - r0));
    if (t_rows[t] > 0) {
      t_end[t] = min(kv_begin + seg.chunk, seg.p + ((r0 + t_rows[t] - 1) / g.G) * seg.causal + 1);
      t_min_limit[t] = min(t_end[t], seg.p + (r0 / g.G) * seg.causal + 1);
      t_tiles[t] = t_end[t] > kv_begin ? (t_end[t] - kv_begin + kTileKeys - 1) / kTileKeys : 0;
    } else {
      t_end[t] = kv_begin; t_min_limit[t] = kv_begin; t_tiles[t] = 0;
    }
  }
  const int n_tiles = max(t_tiles[0], t_tiles[1]);
  const int kv_end = max(t_end[0], t_end[1]);

  // The status word is set when a bounded wait runs out and stays set until tide_status clears it; while it is set
  // no CTA starts work, so outputs are undefined from the time-out until the caller has read the status.
  __shared__ int s_skip;
  if (threadIdx.x == 0) s_skip = *reinterpret_cast<volatile int*>(P.status);
  __syncthreads();
  if (s_skip != 0) return;

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int i = 0; i < kNumBuf; ++i) { mbar_init(smem_u32(&bars.kv_full[i]), 1); mbar_init(smem_u32(&bars.kv_empty[i]), 1); }
    mbar_init(smem_u32(&bars.q_full), 256);
    for (int t = 0; t < 2; ++t) {
      mbar_init(smem_u32(&bars.s_full[t]), 1);
      mbar_init(smem_u32(&bars.p_full[t]), 128);
      mbar_init(smem_u32(&bars.o_full[t]), 1);
    }
    mbar_init(smem_u32(&bars.mma_done), 1);
    mbar_fence_init();
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem_base;
  volatile int* abort_flag = &s_abort;

  // register budget: the data-movement warpgroup gives registers to the two softmax warpgroups.  setmaxnreg
  // moves registers inside the CTA's own launch allocation (384 x 168), so the new counts must not add up to
  // more than that: 256 x 224 + 128 x 56 = 384 x 168.  (An over-subscribed .inc waits for ever.)
  if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    if (warp == 8) {
      // ================= producer: one copy per K block and per V block of a (page, head) into the ring =================
      if (n_tiles > 0) {
        const int pages_per_tile = kTileKeys / g.S;
        // page ids are fetched 32 logical pages at a time, one per lane, a whole group ahead of their use,
        // so that no bulk copy waits for a dependent page-table load
        const int tiles_per_group = 32 / pages_per_tile;
        const int lp0 = kv_begin / g.S;
        const int32_t* trow = P.table + seg.table_off;
        auto load_ids = [&](int grp) -> int {
          const int lp = lp0 + grp * 32 + lane;
          return lp < g.max_pages_per_task ? trow[lp] : 0;
        };
        int ids_cur = load_ids(0), ids_nxt = load_ids(1), cur_grp = 0;
        int issued = 0;                                        // tiles whose copies were issued
        for (int j = 0; j < n_tiles; ++j) {
          const int buf = j % kNumBuf, use = j / kNumBuf;
          const int grp = j / tiles_per_group;
          if (grp != cur_grp) { ids_cur = ids_nxt; ids_nxt = load_ids(grp + 1); cur_grp = grp; }
          // a wait that gave up means the ring can no longer be trusted: issue nothing more
          if (use > 0 && !mbar_wait(smem_u32(&bars.kv_empty[buf]), (use - 1) & 1, abort_flag, P.status, P.wait_limit_ns)) break;
          issued = j + 1;
          if (P.debug_drop_first_stage != 0 && item == 0 && j == 0) continue;   // test hook: tile 0 never arrives
          const int key0 = kv_begin + j * kTileKeys;
          const int npages = min(pages_per_tile, (kv_end - key0 + g.S - 1) / g.S);
          const uint32_t bar = smem_u32(&bars.kv_full[buf]);
          // lanes [0, pages_per_tile) fetch the K blocks, lanes [pages_per_tile, 2 * pages_per_tile) the V blocks
          const int is_v = lane >= pages_per_tile ? 1 : 0, pg = lane - is_v * pages_per_tile;
          const long long page = __shfl_sync(0xffffffffu, ids_cur, ((j % tiles_per_group) * pages_per_tile + pg) & 31);
          if (lane == 0) mbar_expect_tx(bar, (uint32_t)(npages * g.head_bytes));
          __syncwarp();
          if (lane < 2 * pages_per_tile && pg < npages)
            bulk_g2s(smem_base + buf * kSlotBytes + is_v * kTileBytes + pg * g.kblock_bytes,
                     P.pool + page * g.page_bytes + (long long)kvh * g.head_bytes + is_v * g.kblock_bytes, (uint32_t)g.kblock_bytes, bar);
        }
        if (*abort_flag && lane == 0) {
          // a wait gave up somewhere: do not leave while copies into this CTA's shared memory can still be landing.
          // Those are among the last kNumBuf tiles issued (an older one was consumed before its slot was refilled);
          // each wait is bounded like every other.
          for (int idx = max(0, issued - kNumBuf); idx < issued; ++idx) {
            const uint32_t bar = smem_u32(&bars.kv_full[idx % kNumBuf]);
            const long long t0 = global_ns();
            while (!mbar_try(bar, (idx / kNumBuf) & 1) && global_ns() - t0 < P.wait_limit_ns) {}
          }
        }
      }
    } else if (warp == 9) {
      // ================= MMA issuer (whole warp converged, one elected lane issues) =================
      if (n_tiles > 0) {
        mbar_wait(smem_u32(&bars.q_full), 0, abort_flag, P.status, P.wait_limit_ns);
        tc_fence_after();
        auto issue_qk = [&](int t, int j) {
          const uint32_t kbuf = smem_base + (j % kNumBuf) * kSlotBytes;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            mma_ts(tmem + kColS + t * 64, tmem + kColQ + t * 64 + ks * 8,
                   make_desc(kbuf + (ks >> 2) * 1024 + (ks & 3) * 32, 16, kGroupBytes), kIdescQK, ks > 0);
          mma_commit(smem_u32(&bars.s_full[t]));
        };
        auto issue_pv = [&](int t, int j) {
          const uint32_t vbuf = smem_base + (j % kNumBuf) * kSlotBytes + kTileBytes;
#pragma unroll
          for (int ks = 0; ks < kTileKeys / 16; ++ks)
            mma_ts(tmem + kColO + t * 128, tmem + kColS + t * 64 + ks * 8, make_desc(vbuf + ks * 2 * kGroupBytes, 1024, kGroupBytes), kIdescPV,
                   (j > 0 || ks > 0) ? 1u : 0u);
        };
        auto wait_full = [&](int idx) {
          mbar_wait(smem_u32(&bars.kv_full[idx % kNumBuf]), (idx / kNumBuf) & 1, abort_flag, P.status, P.wait_limit_ns);
        };
        wait_full(0);
        tc_fence_after();
        for (int t = 0; t < 2; ++t) if (t_tiles[t] > 0) issue_qk(t, 0);
        for (int j = 0; j < n_tiles; ++j) {
          if (kv_end < kv_begin + (j + 1) * kTileKeys) {
            // rows of the V tile past the end of the item were not loaded (or hold stale page slots): clear
            // them so that weight 0 times leftover bits cannot produce NaN
            const int first = kv_end - (kv_begin + j * kTileKeys);
            uint8_t* vgen = smem_gen + (j % kNumBuf) * kSlotBytes + kTileBytes;
            for (int i = lane; i < (kTileKeys - first) * 16; i += 32) {
              const int rr = first + (i >> 4), c = i & 15;     // whole rows are cleared, so the swizzle does not matter
              *reinterpret_cast<uint4*>(vgen + (rr >> 3) * kGroupBytes + (c >> 3) * 1024 + (rr & 7) * 128 + (c & 7) * 16) = make_uint4(0, 0, 0, 0);
            }
            fence_async_smem();
            __syncwarp();
          }
          bool k_ready = false;
          for (int t = 0; t < 2; ++t) {
            if (j < t_tiles[t]) {
              mbar_wait(smem_u32(&bars.p_full[t]), j & 1, abort_flag, P.status, P.wait_limit_ns);
              tc_fence_after();
              issue_pv(t, j);
              if (j + 1 < t_tiles[t]) {
                if (!k_ready) { wait_full(j + 1); k_ready = true; }
                issue_qk(t, j + 1);                          // overwrites S_t / P_t after PV_t(j), in order
              } else {
                mma_commit(smem_u32(&bars.o_full[t]));
              }
            }
          }
          mma_commit(smem_u32(&bars.kv_empty[j % kNumBuf]));   // K_j and V_j are consumed once PV(j) retires
        }
        // Every MMA has retired before this warp leaves (TMEM is freed after the CTA's last barrier): one more commit
        // covers all of them.  This wait does not look at the abort flag - MMAs retire whatever else went wrong.
        mma_commit(smem_u32(&bars.mma_done));
        {
          const uint32_t bar = smem_u32(&bars.mma_done);
          const long long t0 = global_ns();
          while (!mbar_try(bar, 0) && global_ns() - t0 < P.wait_limit_ns) {}
        }
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
    // ================= softmax warpgroups =================
    const int t = warp >> 2;                                   // 0 = A, 1 = B
    const int row = ((warp & 3) << 5) | lane;                  // row of the 128-row tile = TMEM lane
    const uint32_t lane_addr = (uint32_t)((warp & 3) << 5) << 16;
    const int r = item_row0 + t * 128 + row;
    const bool valid = r < R;
    const int qi = r / g.G, hd = kvh * g.G + (r - qi * g.G);
    const int my_tiles = t_tiles[t];
    const int limit = valid ? min(t_end[t], seg.p + qi * seg.causal + 1) : t_end[t];   // keys j < limit are visible

    // ---- this row of Q (or zeros) into TMEM as the A operand of S = Q.K^T: two bf16 per column ----
    {
      const uint4* src = reinterpret_cast<const uint4*>(P.q + ((long long)(seg.q_off + qi) * g.Hq + hd) * D);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        uint32_t qv[32];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint4 v = valid ? __ldg(src + h * 8 + c) : make_uint4(0, 0, 0, 0);
          qv[4 * c] = v.x; qv[4 * c + 1] = v.y; qv[4 * c + 2] = v.z; qv[4 * c + 3] = v.w;
        }
        tmem_st32u(tmem + lane_addr + kColQ + t * 64 + h * 32, qv);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(smem_u32(&bars.q_full));
    }

    float m = -INFINITY, l = 0.f;       // running max (base-2, scaled) and sum
    const float sl2 = P.scale_log2e;
    const uint32_t s_addr = tmem + lane_addr + kColS + t * 64;
    const uint32_t o_addr = tmem + lane_addr + kColO + t * 128;

    // One key tile of this row tile.  The tiles that need the causal (or end-of-range) mask are the last ones of the
    // item; they get a copy of the body of their own, so the 128 compare-and-select instructions of the mask are
    // not part of the code that the other ~99 % of the tiles run (its mere presence in the loop cost 2 %).
    auto tile = [&](const int j, auto masked_tag) {
      constexpr bool kMasked = decltype(masked_tag)::value;
      mbar_wait(smem_u32(&bars.s_full[t]), j & 1, abort_flag, P.status, P.wait_limit_ns);
      tc_fence_after();
      float s[64];
      tmem_ld32(s_addr, *reinterpret_cast<float(*)[32]>(&s[0]));
      tmem_ld32(s_addr + 32, *reinterpret_cast<float(*)[32]>(&s[32]));
      tmem_wait_ld();
      if constexpr (kMasked) {
        const int vis = limit - (kv_begin + j * kTileKeys);
#pragma unroll
        for (int c = 0; c < 64; ++c) if (c >= vis) s[c] = -INFINITY;
      }
      // independent partial reductions (one long dependent chain would expose its latency), three inputs per
      // instruction: 8 chains of 4 over 64 values, then a tree
      float mxp[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) mxp[i] = max3(s[i], s[i + 8], s[i + 16]);
#pragma unroll
      for (int i = 0; i < 8; ++i) mxp[i] = max3(mxp[i], s[i + 24], s[i + 32]);
#pragma unroll
      for (int i = 0; i < 8; ++i) mxp[i] = max3(mxp[i], s[i + 40], s[i + 48]);
#pragma unroll
      for (int i = 0; i < 8; ++i) mxp[i] = fmaxf(mxp[i], s[i + 56]);
      float mx = max3(max3(mxp[0], mxp[1], mxp[2]), max3(mxp[3], mxp[4], mxp[5]), fmaxf(mxp[6], mxp[7]));
      mx *= sl2;                                               // scale > 0 on this path
      float m_new = m;
      if (mx > m + kRescaleThreshold) m_new = mx;             // also the first visible key: -inf + 8 = -inf < any finite mx
      float alpha = 1.f;
      if (__any_sync(0xffffffffu, m_new != m)) {               // rare: one vote per tile decides both steps
        alpha = fast_exp2(m - m_new);                          // m = -inf -> 0, equal -> 1
        if (j > 0) {
          // O_t holds tiles < j: S_t(j) was committed after PV_t(j-1)
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            float o[32];
            tmem_ld32(o_addr + c * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] *= alpha;
            tmem_st32(o_addr + c * 32, o);
          }
        }
      }
      m = m_new;
      const float mu = (m == -INFINITY) ? 0.f : m;
      float sp[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      uint32_t pk[32];
      // packed arithmetic: the softmax warps are short of issue slots, and this halves the scale-subtract and the
      // row-sum instructions (same roundings and the same summation order as the scalar form)
      {
        const uint64_t sl2_2 = pack2(sl2, sl2), nmu_2 = pack2(-mu, -mu);
        uint64_t sp2[4] = {pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f)};
#pragma unroll
        for (int c = 0; c < 64; c += 8) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            float x0, x1;
            unpack2(fma2(pack2(s[c + 2 * i], s[c + 2 * i + 1]), sl2_2, nmu_2), x0, x1);
            const float e0 = fast_exp2(x0), e1 = fast_exp2(x1);
            sp2[i] = add2(sp2[i], pack2(e0, e1));
            pk[(c >> 1) + i] = pack_bf16(e0, e1);
          }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) unpack2(sp2[i], sp[2 * i], sp[2 * i + 1]);
      }
      tmem_st32u(s_addr, pk);                                  // P_t over the first 32 columns of S_t
      l = l * alpha + (((sp[0] + sp[1]) + (sp[2] + sp[3])) + ((sp[4] + sp[5]) + (sp[6] + sp[7])));
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(smem_u32(&bars.p_full[t]));
    };
    // tiles j < n_plain end at or before the first row's limit: every key of theirs is visible to every row
    const int n_plain = min(my_tiles, max(0, (t_min_limit[t] - kv_begin) / kTileKeys));
    for (int j = 0; j < n_plain; ++j) tile(j, std::false_type{});
    for (int j = n_plain; j < my_tiles; ++j) tile(j, std::true_type{});

    // ---- epilogue: O / l and LSE ----
    const float kLn2 = 0.6931471805599453f;
    if (my_tiles > 0) {
      mbar_wait(smem_u32(&bars.o_full[t]), 0, abort_flag, P.status, P.wait_limit_ns);
      tc_fence_after();
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const float e2 = l > 0.f ? m + log2f(l) : -INFINITY;
    const long long orow = (long long)(seg.q_off + qi) * g.Hq + hd;
    const long long prow_idx = seg.part_base + (long long)(split * seg.n + qi) * g.Hq + hd;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      float o[32];
      if (my_tiles > 0) {                 // uniform over the warpgroup
        tmem_ld32(o_addr + c * 32, o);
        tmem_wait_ld();
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = 0.f;
      }
      if (valid) {
        if (direct) {
          uint4* dst = reinterpret_cast<uint4*>(P.out + orow * D + c * 32);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 v;
            v.x = pack_bf16(o[i * 8 + 0] * inv, o[i * 8 + 1] * inv);
            v.y = pack_bf16(o[i * 8 + 2] * inv, o[i * 8 + 3] * inv);
            v.z = pack_bf16(o[i * 8 + 4] * inv, o[i * 8 + 5] * inv);
            v.w = pack_bf16(o[i * 8 + 6] * inv, o[i * 8 + 7] * inv);
            dst[i] = v;
          }
        } else {
          float4* dst = reinterpret_cast<float4*>(P.part_o + prow_idx * D + c * 32);
#pragma unroll
          for (int i = 0; i < 8; ++i) dst[i] = make_float4(o[i * 4] * inv, o[i * 4 + 1] * inv, o[i * 4 + 2] * inv, o[i * 4 + 3] * inv);
        }
      }
    }
    if (valid) {
      if (direct) { if (P.lse != nullptr) P.lse[orow] = e2 * kLn2; }
      else P.part_lse[prow_idx] = e2;
    }
    tc_fence_before();
  }

  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

}  // namespace umma

cudaError_t attend_umma_init() {
  return cudaFuncSetAttribute(umma::attend_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, umma::kSmemBytes);
}

cudaError_t launch_attend_umma(const AttendParams& p, cudaStream_t s) {
  const int grid = p.dyn ? p.grid_cap : p.n_items;
  if (grid <= 0) return cudaSuccess;
  umma::attend_umma_kernel<<<grid, umma::kThreads, umma::kSmemBytes, s>>>(p);
  return cudaGetLastError();
}

}  // namespace tide

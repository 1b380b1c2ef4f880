// Split-KV attention over the paged cache with warp-level tensor-core tiles (mma.sync) — the decode path,
// and the general path for resume rows that the tcgen05 kernel does not take.
//
// What it computes (paper Section 4: a resumed task continues from its preserved KV state; the maths is
// ordinary scaled-dot-product softmax attention with grouped KV heads): for a work item
// (row, kv_head, m_tile, split) the online-softmax partial over keys [kv_begin, kv_end) for a tile of
// packed rows r = q_index * G + g (the G query heads that share this KV head), query q_index seeing keys
// [0, prefix + q_index].  K/V pages are read ONCE per KV head for all G query heads.
//
// Structure: one producer warp streams whole (page, head) blocks (K and V, contiguous in the pool) into a
// ring of shared-memory stages with 1-D bulk copies that complete on mbarriers; four consumer warps run
// m16n8k16 bf16 MMAs straight from the pre-swizzled blocks with ldmatrix.  Decode items: the four warps
// split the keys of a stage and merge their (m, l, O) at the end.  Tile items: each warp owns 16 of the
// 64 packed rows.  Bound by HBM bandwidth for decode: Hkv*D*4 bytes per context token, 4*D*Hq flops.
#include <cfloat>
#include <climits>

#include "tide_internal.h"

namespace tide {

constexpr int kConsumerWarps = 4;
constexpr int kAttendThreads = (kConsumerWarps + 1) * 32;
constexpr int kStages = 3;

template <int D>
struct MmaCfg {
  static constexpr int kStageBytes = kStageKeys * D * 4;  // K + V, bf16
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024;
};

template <int D, bool DECODE>
__device__ __forceinline__ void attend_mma_body(const AttendParams& P, const Segment* __restrict__ segs) {
  constexpr int KS = D / 16;                 // k-steps of Q.K^T
  constexpr int NT = D / 8;                  // n-tiles of O
  constexpr int STEP_KB = DECODE ? 1 : 4;    // 16-key blocks per softmax step of one warp
  constexpr int TILE_M = DECODE ? kDecodeTileRows : kMmaTileRows;
  constexpr int STAGE_BYTES = MmaCfg<D>::kStageBytes;

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t s_full[kStages];
  __shared__ __align__(8) uint64_t s_empty[kStages];
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
  const int si = find_segment(n_segs, item, [&](int i) { return segs[i].item_base; });
  const Segment seg = segs[si];
  int local = item - seg.item_base;
  const int m_tile = local % seg.n_mtiles;
  local /= seg.n_mtiles;
  const int split = local % seg.n_splits;
  const int kvh = local / seg.n_splits;
  const int R = seg.n * g.G;                       // packed rows of this (row, kv head)
  const int tile_row0 = m_tile * TILE_M;
  const int r_last = min(R, tile_row0 + TILE_M) - 1;
  const int kv_begin = seg.origin + split * seg.chunk;
  const int kv_end = min(kv_begin + seg.chunk, seg.p + (r_last / g.G) * seg.causal + 1);
  const bool direct = seg.n_splits == 1 && seg.partial == 0;
  const float kLn2 = 0.6931471805599453f;

  // rows this thread owns inside its warp's 16-row MMA tile
  const int row_base = tile_row0 + (DECODE ? 0 : warp * 16);
  const int r_lo = row_base + (lane >> 2), r_hi = r_lo + 8;
  const bool v_lo = r_lo < R, v_hi = r_hi < R;
  const int qi_lo = r_lo / g.G, qi_hi = r_hi / g.G;
  const int hd_lo = kvh * g.G + (r_lo - qi_lo * g.G), hd_hi = kvh * g.G + (r_hi - qi_hi * g.G);

  if (kv_end <= kv_begin && seg.partial != 2) {
    // nothing visible in this split (only possible when n_splits > 1): neutral partials.  (A segment whose last split
    // merges walks the normal path with zero stages instead, so that it is counted.)
    if (warp < kConsumerWarps && (lane & 3) == 0 && (!DECODE || warp == 0)) {
      if (v_lo) P.part_lse[seg.part_base + (split * seg.n + qi_lo) * g.Hq + hd_lo] = -INFINITY;
      if (v_hi) P.part_lse[seg.part_base + (split * seg.n + qi_hi) * g.Hq + hd_hi] = -INFINITY;
    }
    return;
  }

  // The status word is set when a bounded wait runs out and stays set until tide_status clears it.  While it is
  // set no CTA starts work (this launch's later CTAs and every CTA of later launches leave here without writing
  // anything), so outputs are undefined from the time-out until the caller has read the status.
  __shared__ int s_skip;
  if (threadIdx.x == 0) s_skip = *reinterpret_cast<volatile int*>(P.status);
  __syncthreads();
  if (s_skip != 0) return;

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int i = 0; i < kStages; ++i) {
      mbar_init(smem_u32(&s_full[i]), 1);
      mbar_init(smem_u32(&s_empty[i]), kConsumerWarps);
    }
    mbar_fence_init();
  }
  __syncthreads();
  volatile int* abort_flag = &s_abort;

  const int n_st = (kv_end - kv_begin + kStageKeys - 1) / kStageKeys;

  if (warp == kConsumerWarps) {
    // ================= producer warp =================
    const int pages_per_stage = kStageKeys / g.S;
    int issued = 0;                              // stages whose copies were issued
    for (int st = 0; st < n_st; ++st) {
      const int slot = st % kStages;
      // a wait that gave up means the ring can no longer be trusted: issue nothing more
      if (st >= kStages && !mbar_wait(smem_u32(&s_empty[slot]), ((st / kStages) - 1) & 1, abort_flag, P.status, P.wait_limit_ns)) break;
      issued = st + 1;
      if (P.debug_drop_first_stage != 0 && item == 0 && st == 0) continue;   // test hook: this stage never arrives
      const int key0 = kv_begin + st * kStageKeys;
      const int npages = min(pages_per_stage, (kv_end - key0 + g.S - 1) / g.S);
      const uint32_t bar = smem_u32(&s_full[slot]);
      if (lane == 0) mbar_expect_tx(bar, (uint32_t)(npages * g.head_bytes));
      __syncwarp();
      if (lane < npages) {
        const long long page = P.table[seg.table_off + key0 / g.S + lane];
        const uint8_t* src = P.pool + page * g.page_bytes + (long long)kvh * g.head_bytes;
        bulk_g2s(smem_base + slot * STAGE_BYTES + lane * g.head_bytes, src, (uint32_t)g.head_bytes, bar);
      }
    }
    if (*abort_flag && lane == 0) {
      // a wait gave up somewhere: do not leave the CTA while copies into its shared memory are in flight.  Only the
      // last kStages stages that were issued can still be landing (an older one was consumed before its slot was
      // refilled); each wait is bounded like every other.
      for (int st = max(0, issued - kStages); st < issued; ++st) {
        const uint32_t bar = smem_u32(&s_full[st % kStages]);
        const long long t0 = global_ns();
        while (!mbar_try(bar, (st / kStages) & 1) && global_ns() - t0 < P.wait_limit_ns) {}
      }
    }
    return;
  }

  // ================= consumer warps =================
  const int kv_limit_lo = v_lo ? min(kv_end, seg.p + qi_lo * seg.causal + 1) : kv_end;  // keys j < limit are visible
  const int kv_limit_hi = v_hi ? min(kv_end, seg.p + qi_hi * seg.causal + 1) : kv_end;
  // last key any row of this warp can see, and the smallest limit (masking needed beyond it)
  int w_end, w_min_limit;
  {
    const int wr_first = row_base, wr_last = min(R, row_base + 16) - 1;
    if (wr_last < wr_first) { w_end = kv_begin; w_min_limit = kv_end; }   // warp has no valid rows
    else {
      w_end = min(kv_end, seg.p + (wr_last / g.G) * seg.causal + 1);
      w_min_limit = min(kv_end, seg.p + (wr_first / g.G) * seg.causal + 1);
    }
  }

  uint32_t qa[KS][4];
  {
    const uint16_t* q_lo = P.q + ((long long)(seg.q_off + qi_lo) * g.Hq + hd_lo) * D + 2 * (lane & 3);
    const uint16_t* q_hi = P.q + ((long long)(seg.q_off + qi_hi) * g.Hq + hd_hi) * D + 2 * (lane & 3);
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qa[ks][0] = v_lo ? *reinterpret_cast<const uint32_t*>(q_lo + ks * 16) : 0u;
      qa[ks][1] = v_hi ? *reinterpret_cast<const uint32_t*>(q_hi + ks * 16) : 0u;
      qa[ks][2] = v_lo ? *reinterpret_cast<const uint32_t*>(q_lo + ks * 16 + 8) : 0u;
      qa[ks][3] = v_hi ? *reinterpret_cast<const uint32_t*>(q_hi + ks * 16 + 8) : 0u;
    }
  }

  float o[NT][4];
#pragma unroll
  for (int i = 0; i < NT; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
  const float sl2 = P.scale_log2e;

  // Decode items: a warp reads the same 16 slots of every stage, so the offsets of its ldmatrix rows inside a stage
  // are fixed for the whole item (two per K n-tile, four for V; the others are 1 KB further on).
  uint32_t dk_off[2][2] = {{0u, 0u}, {0u, 0u}}, dv_off[4] = {0u, 0u, 0u, 0u};
  if (DECODE) {
    const int koff = warp * 16;
    const uint32_t page_off = (uint32_t)((koff / g.S) * g.head_bytes);
    const int row0 = koff % g.S;
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int x = 0; x < 2; ++x) dk_off[nt][x] = page_off + (uint32_t)blk_offset(g, row0 + nt * 8 + (lane & 7), 0, x * 4 + (lane >> 3));
    const int vrow = row0 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
    for (int y = 0; y < 4; ++y) dv_off[y] = page_off + (uint32_t)blk_offset(g, vrow, 1, y * 2 + (lane >> 4));
  }

  for (int st = 0; st < n_st; ++st) {
    const int slot = st % kStages;
    mbar_wait(smem_u32(&s_full[slot]), (st / kStages) & 1, abort_flag, P.status, P.wait_limit_ns);
    const int key0 = kv_begin + st * kStageKeys;
    const uint32_t stage = smem_base + slot * STAGE_BYTES;
    const int kb_first = DECODE ? warp : 0;
    const int step_key0 = key0 + kb_first * 16;
    if (step_key0 < w_end) {
      const int nkb = min(STEP_KB, (w_end - step_key0 + 15) >> 4);
      float s[STEP_KB * 2][4];
#pragma unroll
      for (int b = 0; b < STEP_KB; ++b) {
        if (b < nkb) {
          const int koff = (kb_first + b) * 16;            // key offset inside the stage
          const uint32_t pbase = stage + (koff / g.S) * g.head_bytes;
          const int row0 = koff % g.S;
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) {
            float(&acc)[4] = s[b * 2 + nt];
            acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
            const int slot_row = row0 + nt * 8 + (lane & 7);
#pragma unroll
            for (int k2 = 0; k2 < KS / 2; ++k2) {
              uint32_t b0, b1, b2, b3;
              if (DECODE) ldsm_x4(stage + dk_off[nt][k2 & 1] + (k2 >> 1) * 1024, b0, b1, b2, b3);
              else ldsm_x4(pbase + blk_offset(g, slot_row, 0, k2 * 4 + (lane >> 3)), b0, b1, b2, b3);
              mma_bf16(acc, qa[2 * k2], b0, b1);
              mma_bf16(acc, qa[2 * k2 + 1], b2, b3);
            }
          }
        }
      }
      // ---- scale, mask, online softmax ----
      const int step_end = step_key0 + nkb * 16;
      const bool need_mask = step_end > w_min_limit;
      float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
      for (int t = 0; t < STEP_KB * 2; ++t) {
        if (t < nkb * 2) {
          const int j = step_key0 + t * 8 + 2 * (lane & 3);
          float t0 = s[t][0] * sl2, t1 = s[t][1] * sl2, t2 = s[t][2] * sl2, t3 = s[t][3] * sl2;
          if (need_mask) {
            if (j >= kv_limit_lo) t0 = -INFINITY;
            if (j + 1 >= kv_limit_lo) t1 = -INFINITY;
            if (j >= kv_limit_hi) t2 = -INFINITY;
            if (j + 1 >= kv_limit_hi) t3 = -INFINITY;
          }
          s[t][0] = t0; s[t][1] = t1; s[t][2] = t2; s[t][3] = t3;
          mx_lo = fmaxf(mx_lo, fmaxf(t0, t1));
          mx_hi = fmaxf(mx_hi, fmaxf(t2, t3));
        }
      }
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
      const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
      const float mu_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo, mu_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi;
      const float a_lo = fast_exp2(m_lo - mu_lo), a_hi = fast_exp2(m_hi - mu_hi);
      m_lo = mn_lo; m_hi = mn_hi;
      if (__any_sync(0xffffffffu, a_lo != 1.f || a_hi != 1.f)) {
#pragma unroll
        for (int i = 0; i < NT; ++i) { o[i][0] *= a_lo; o[i][1] *= a_lo; o[i][2] *= a_hi; o[i][3] *= a_hi; }
      }
      float ps_lo = 0.f, ps_hi = 0.f;
#pragma unroll
      for (int t = 0; t < STEP_KB * 2; ++t) {
        if (t < nkb * 2) {
          s[t][0] = fast_exp2(s[t][0] - mu_lo); s[t][1] = fast_exp2(s[t][1] - mu_lo);
          s[t][2] = fast_exp2(s[t][2] - mu_hi); s[t][3] = fast_exp2(s[t][3] - mu_hi);
          ps_lo += s[t][0] + s[t][1];
          ps_hi += s[t][2] + s[t][3];
        }
      }
      l_lo = l_lo * a_lo + ps_lo;
      l_hi = l_hi * a_hi + ps_hi;
      // ---- O += P.V ----
#pragma unroll
      for (int b = 0; b < STEP_KB; ++b) {
        if (b < nkb) {
          const int koff = (kb_first + b) * 16;
          const uint32_t vbase = stage + (koff / g.S) * g.head_bytes;   // the page block; V parts through blk_offset(.., 1, ..)
          const int row0 = koff % g.S;
          const int blk_key0 = key0 + koff;
          if (blk_key0 + 16 > kv_end) {
            // slots past the end of the item hold whatever the page held before: clear V there so that
            // weight 0 times stale bits cannot produce NaN
            const int first = kv_end - blk_key0;           // 1..15
            uint8_t* vgen = smem_gen + (vbase - smem_base);
            for (int idx = lane; idx < (16 - first) * (D / 8); idx += 32) {
              const int rr = row0 + first + idx / (D / 8), c = idx % (D / 8);
              *reinterpret_cast<uint4*>(vgen + blk_offset(g, rr, 1, c)) = make_uint4(0, 0, 0, 0);
            }
            __syncwarp();
          }
          uint32_t pa[4];
          pa[0] = pack_bf16(s[2 * b][0], s[2 * b][1]);
          pa[1] = pack_bf16(s[2 * b][2], s[2 * b][3]);
          pa[2] = pack_bf16(s[2 * b + 1][0], s[2 * b + 1][1]);
          pa[3] = pack_bf16(s[2 * b + 1][2], s[2 * b + 1][3]);
          const int vrow = row0 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
          for (int n2 = 0; n2 < NT / 2; ++n2) {
            uint32_t b0, b1, b2, b3;
            if (DECODE) ldsm_x4_t(stage + dv_off[n2 & 3] + (n2 >> 2) * 1024, b0, b1, b2, b3);
            else ldsm_x4_t(vbase + blk_offset(g, vrow, 1, n2 * 2 + (lane >> 4)), b0, b1, b2, b3);
            mma_bf16(o[2 * n2], pa, b0, b1);
            mma_bf16(o[2 * n2 + 1], pa, b2, b3);
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&s_empty[slot]));
  }

  // ---- epilogue ----
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);

  if (!DECODE) {
    const float inv_lo = l_lo > 0.f ? 1.f / l_lo : 0.f, inv_hi = l_hi > 0.f ? 1.f / l_hi : 0.f;
    const float e_lo = l_lo > 0.f ? m_lo + log2f(l_lo) : -INFINITY;
    const float e_hi = l_hi > 0.f ? m_hi + log2f(l_hi) : -INFINITY;
    const int dcol = 2 * (lane & 3);
    if (direct) {
      const long long o_lo = ((long long)(seg.q_off + qi_lo) * g.Hq + hd_lo), o_hi = ((long long)(seg.q_off + qi_hi) * g.Hq + hd_hi);
#pragma unroll
      for (int i = 0; i < NT; ++i) {
        if (v_lo) *reinterpret_cast<uint32_t*>(P.out + o_lo * D + i * 8 + dcol) = pack_bf16(o[i][0] * inv_lo, o[i][1] * inv_lo);
        if (v_hi) *reinterpret_cast<uint32_t*>(P.out + o_hi * D + i * 8 + dcol) = pack_bf16(o[i][2] * inv_hi, o[i][3] * inv_hi);
      }
      if (P.lse != nullptr && (lane & 3) == 0) {
        if (v_lo) P.lse[o_lo] = e_lo * kLn2;
        if (v_hi) P.lse[o_hi] = e_hi * kLn2;
      }
    } else {
      const long long p_lo = seg.part_base + (long long)(split * seg.n + qi_lo) * g.Hq + hd_lo;
      const long long p_hi = seg.part_base + (long long)(split * seg.n + qi_hi) * g.Hq + hd_hi;
#pragma unroll
      for (int i = 0; i < NT; ++i) {
        if (v_lo) *reinterpret_cast<float2*>(P.part_o + p_lo * D + i * 8 + dcol) = make_float2(o[i][0] * inv_lo, o[i][1] * inv_lo);
        if (v_hi) *reinterpret_cast<float2*>(P.part_o + p_hi * D + i * 8 + dcol) = make_float2(o[i][2] * inv_hi, o[i][3] * inv_hi);
      }
      if ((lane & 3) == 0) {
        if (v_lo) P.part_lse[p_lo] = e_lo;
        if (v_hi) P.part_lse[p_hi] = e_hi;
      }
    }
    return;
  }

  // DECODE: the four warps hold partial (m, l, O) over disjoint keys of the same 16 rows; combine through
  // shared memory (the stage ring is free: every copy that was issued has been consumed).
  named_bar_sync(1, kConsumerWarps * 32);
  float* s_o = reinterpret_cast<float*>(smem_gen);                    // [warp][16][D]
  float* s_m = s_o + kConsumerWarps * 16 * D;                         // [warp][16]
  float* s_l = s_m + kConsumerWarps * 16;
  {
    float* wo = s_o + warp * 16 * D;
    const int rl = lane >> 2, dcol = 2 * (lane & 3);
#pragma unroll
    for (int i = 0; i < NT; ++i) {
      *reinterpret_cast<float2*>(wo + rl * D + i * 8 + dcol) = make_float2(o[i][0], o[i][1]);
      *reinterpret_cast<float2*>(wo + (rl + 8) * D + i * 8 + dcol) = make_float2(o[i][2], o[i][3]);
    }
    if ((lane & 3) == 0) {
      s_m[warp * 16 + rl] = m_lo; s_m[warp * 16 + rl + 8] = m_hi;
      s_l[warp * 16 + rl] = l_lo; s_l[warp * 16 + rl + 8] = l_hi;
    }
  }
  named_bar_sync(1, kConsumerWarps * 32);
  {
    constexpr int DSEG = D / 8;               // 128 threads = 16 rows x 8 column segments
    const int t = threadIdx.x;
    const int rr = t >> 3, d0 = (t & 7) * DSEG;
    const int r = tile_row0 + rr;
    if (r < R) {
      float mw[kConsumerWarps], mstar = -INFINITY;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) { mw[w] = s_m[w * 16 + rr]; mstar = fmaxf(mstar, mw[w]); }
      const float mu = (mstar == -INFINITY) ? 0.f : mstar;
      float f[kConsumerWarps], lstar = 0.f;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) { f[w] = fast_exp2(mw[w] - mu); lstar += f[w] * s_l[w * 16 + rr]; }
      const float inv = lstar > 0.f ? 1.f / lstar : 0.f;
      const float e2 = lstar > 0.f ? mstar + log2f(lstar) : -INFINITY;
      const int qi = r / g.G, hd = kvh * g.G + (r - qi * g.G);
      float acc[DSEG];
#pragma unroll
      for (int d = 0; d < DSEG; ++d) {
        float a = 0.f;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) a += f[w] * s_o[(w * 16 + rr) * D + d0 + d];
        acc[d] = a * inv;
      }
      if (direct) {
        const long long orow = (long long)(seg.q_off + qi) * g.Hq + hd;
        uint32_t* dst = reinterpret_cast<uint32_t*>(P.out + orow * D + d0);
#pragma unroll
        for (int d = 0; d < DSEG; d += 2) dst[d >> 1] = pack_bf16(acc[d], acc[d + 1]);
        if (P.lse != nullptr && (t & 7) == 0) P.lse[orow] = e2 * kLn2;
      } else {
        const long long prow = seg.part_base + (long long)(split * seg.n + qi) * g.Hq + hd;
        float* dst = P.part_o + prow * D + d0;
#pragma unroll
        for (int d = 0; d < DSEG; d += 4) *reinterpret_cast<float4*>(dst + d) = make_float4(acc[d], acc[d + 1], acc[d + 2], acc[d + 3]);
        if ((t & 7) == 0) P.part_lse[prow] = e2;
      }
    }
    // A split decode-style row merges its own partials: every split counts itself in once its partials are written
    // (fence, barrier, one atomic per CTA); the CTA that counts last reads all splits' partials - in split order, so
    // the result does not depend on which one came last - and writes the row.  The counter goes back to zero for the
    // next launch.  This removes the merge launch, and with it a dependent chain of loads, from decode-only steps.
    if (seg.partial == 2) {
      __shared__ int s_is_last;
      __threadfence();
      named_bar_sync(1, kConsumerWarps * 32);
      if (t == 0) {
        int* ctr = P.merge_ctr + seg.x_part_base + kvh;
        const int done = atomicAdd(ctr, 1);
        s_is_last = done == seg.n_splits - 1 ? 1 : 0;
        if (s_is_last) *ctr = 0;
      }
      named_bar_sync(1, kConsumerWarps * 32);
      if (s_is_last && r < R) {
        __threadfence();
        const int qi = r / g.G, hd = kvh * g.G + (r - qi * g.G);
        const long long stride = (long long)seg.n * g.Hq;                       // partial rows per split
        const long long p0 = seg.part_base + (long long)qi * g.Hq + hd;         // this (token, head) in split 0
        float mstar = -INFINITY;
        for (int sp = 0; sp < seg.n_splits; ++sp) mstar = fmaxf(mstar, __ldcg(P.part_lse + p0 + sp * stride));
        const float mu = (mstar == -INFINITY) ? 0.f : mstar;
        float acc[DSEG];
#pragma unroll
        for (int d = 0; d < DSEG; ++d) acc[d] = 0.f;
        float tot = 0.f;
        for (int sp = 0; sp < seg.n_splits; ++sp) {
          const float e = __ldcg(P.part_lse + p0 + sp * stride);
          if (e == -INFINITY) continue;
          const float w = exp2f(e - mu);
          tot += w;
          const float4* po = reinterpret_cast<const float4*>(P.part_o + (p0 + sp * stride) * D + d0);
#pragma unroll
          for (int d = 0; d < DSEG; d += 4) {
            const float4 v = __ldcg(po + (d >> 2));
            acc[d] += w * v.x; acc[d + 1] += w * v.y; acc[d + 2] += w * v.z; acc[d + 3] += w * v.w;
          }
        }
        const float inv = tot > 0.f ? 1.f / tot : 0.f;
        const long long orow = (long long)(seg.q_off + qi) * g.Hq + hd;
        uint32_t* dst = reinterpret_cast<uint32_t*>(P.out + orow * D + d0);
#pragma unroll
        for (int d = 0; d < DSEG; d += 2) dst[d >> 1] = pack_bf16(acc[d] * inv, acc[d + 1] * inv);
        if (P.lse != nullptr && (t & 7) == 0) P.lse[orow] = (tot > 0.f ? mstar + log2f(tot) : -INFINITY) * kLn2;
      }
    }
  }
}

template <int D, bool DECODE>
__global__ void __launch_bounds__(kAttendThreads, 2) attend_mma_kernel(const AttendParams P) {
  attend_mma_body<D, DECODE>(P, P.segs);
}

// Decode-style items whose row descriptors travel in the kernel's parameters (small decode-only batches).
template <int D>
__global__ void __launch_bounds__(kAttendThreads, 2) attend_decode_inline_kernel(const __grid_constant__ AttendInline PI) {
  attend_mma_body<D, true>(PI.p, PI.segs);
}

cudaError_t attend_kernels_init() {
  cudaError_t e;
  e = cudaFuncSetAttribute(attend_mma_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, MmaCfg<128>::kSmemBytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attend_mma_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, MmaCfg<128>::kSmemBytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attend_mma_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, MmaCfg<64>::kSmemBytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attend_mma_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, MmaCfg<64>::kSmemBytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attend_decode_inline_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, MmaCfg<128>::kSmemBytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attend_decode_inline_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, MmaCfg<64>::kSmemBytes);
  return e;
}

cudaError_t launch_attend_decode_inline(const AttendInline& pi, cudaStream_t s) {
  const int grid = pi.p.n_items;
  if (grid <= 0) return cudaSuccess;
  if (pi.p.g.D == 128) attend_decode_inline_kernel<128><<<grid, kAttendThreads, MmaCfg<128>::kSmemBytes, s>>>(pi);
  else attend_decode_inline_kernel<64><<<grid, kAttendThreads, MmaCfg<64>::kSmemBytes, s>>>(pi);
  return cudaGetLastError();
}

cudaError_t launch_attend_decode(const AttendParams& p, cudaStream_t s) {
  const int grid = p.dyn ? p.grid_cap : p.n_items;
  if (grid <= 0) return cudaSuccess;
  if (p.g.D == 128) attend_mma_kernel<128, true><<<grid, kAttendThreads, MmaCfg<128>::kSmemBytes, s>>>(p);
  else attend_mma_kernel<64, true><<<grid, kAttendThreads, MmaCfg<64>::kSmemBytes, s>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_attend_tile(const AttendParams& p, cudaStream_t s) {
  const int grid = p.dyn ? p.grid_cap : p.n_items;
  if (grid <= 0) return cudaSuccess;
  if (p.g.D == 128) attend_mma_kernel<128, false><<<grid, kAttendThreads, MmaCfg<128>::kSmemBytes, s>>>(p);
  else attend_mma_kernel<64, false><<<grid, kAttendThreads, MmaCfg<64>::kSmemBytes, s>>>(p);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Log-sum-exp merge of the split partials: one warp per (token, head) row.
//   LSE = log2 sum_i 2^{LSE_i},  O = sum_i 2^{LSE_i - LSE} O_i;  fixed order, no atomics.
// The kernel is a chain of dependent loads if written naively (one split after the other), so the partial LSEs
// are fetched side by side, one per lane, and the partial outputs four splits at a time; the order in which the
// terms are added is still the order of the splits.
__global__ void __launch_bounds__(256) merge_kernel(const MergeParams P) {
  const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const int n_rows = P.dyn ? P.dyn[0] : P.n_rows, n_segs = P.dyn ? P.dyn[1] : P.n_segs;
  if (row >= n_rows) return;
  const int si = find_segment(n_segs, row, [&](int i) { return P.segs[i].merge_base; });
  const Segment seg = P.segs[si];
  const int local = row - seg.merge_base;                 // token * Hq + head inside the segment
  const long long stride = (long long)seg.n * P.Hq;       // partial rows per split
  const long long p0 = seg.part_base + local;
  // a row's contributions: its own splits, then (a member of a group that shares its first pages) the splits of the
  // group's shared range, where this row is one token among the members' (such segments have one token: local = head)
  const int n_src = seg.n_splits + seg.x_n_splits;
  auto src_row = [&](int s) -> long long {
    return s < seg.n_splits ? p0 + s * stride : (long long)seg.x_part_base + local + (long long)(s - seg.n_splits) * seg.x_stride;
  };
  // lane i holds the LSEs of contributions i, i + 32, ... (at most 2 * kMaxSplits = 256 of them)
  constexpr int kPerLane = 2 * kMaxSplits / 32;
  float e[kPerLane];
  float mstar = -INFINITY;
#pragma unroll
  for (int k = 0; k < kPerLane; ++k) {
    const int s = k * 32 + lane;
    e[k] = s < n_src ? P.part_lse[src_row(s)] : -INFINITY;
    mstar = fmaxf(mstar, e[k]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mstar = fmaxf(mstar, __shfl_xor_sync(0xffffffffu, mstar, o));
  const float mu = (mstar == -INFINITY) ? 0.f : mstar;
#pragma unroll
  for (int k = 0; k < kPerLane; ++k) e[k] = e[k] == -INFINITY ? 0.f : exp2f(e[k] - mu);   // the contribution's weight
  const int per = P.D / 32;                               // 2 or 4 floats per lane
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  float tot = 0.f;
  for (int s0 = 0; s0 < n_src; s0 += 4) {
    float4 v[4];
    float w[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int s = s0 + u;
      // weight of contribution s: held by lane s % 32 in its slot s / 32 (kPerLane is small: select, then shuffle)
      float mine = 0.f;
#pragma unroll
      for (int k = 0; k < kPerLane; ++k) if ((s >> 5) == k) mine = e[k];
      w[u] = s < n_src ? __shfl_sync(0xffffffffu, mine, s & 31) : 0.f;
      v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (w[u] != 0.f) {
        const float* po = P.part_o + src_row(s) * P.D + lane * per;
        if (per == 4) v[u] = *reinterpret_cast<const float4*>(po);
        else { const float2 t = *reinterpret_cast<const float2*>(po); v[u].x = t.x; v[u].y = t.y; }
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (w[u] != 0.f) {
        tot += w[u];
        acc[0] += w[u] * v[u].x; acc[1] += w[u] * v[u].y; acc[2] += w[u] * v[u].z; acc[3] += w[u] * v[u].w;
      }
    }
  }
  const float inv = tot > 0.f ? 1.f / tot : 0.f;
  const long long orow = (long long)seg.q_off * P.Hq + local;
  uint16_t* dst = P.out + orow * P.D + lane * per;
  if (per == 4) {
    uint2 v;
    v.x = pack_bf16(acc[0] * inv, acc[1] * inv);
    v.y = pack_bf16(acc[2] * inv, acc[3] * inv);
    *reinterpret_cast<uint2*>(dst) = v;
  } else {
    *reinterpret_cast<uint32_t*>(dst) = pack_bf16(acc[0] * inv, acc[1] * inv);
  }
  if (P.lse != nullptr && lane == 0) P.lse[orow] = (tot > 0.f ? mstar + log2f(tot) : -INFINITY) * 0.6931471805599453f;
}

cudaError_t launch_merge(const MergeParams& p, cudaStream_t s) {
  const int rows = p.dyn ? p.grid_cap_rows : p.n_rows;
  if (rows <= 0) return cudaSuccess;
  const int blocks = (rows + 7) / 8;
  merge_kernel<<<blocks, 256, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace tide

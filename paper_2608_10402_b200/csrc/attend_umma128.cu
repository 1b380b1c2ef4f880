// Append-prefill attention for resume rows on the 5th-generation tensor cores, 128-key tiles.
//
// Same work item and results as attend_umma.cu (256 packed rows r = q_index * G + g as two 128-row tiles A and B
// against keys [kv_begin, kv_end) of one KV head; paper Section 4: the appended observation tokens attend to the
// whole preserved KV state).  What differs is the arrangement around the tensor pipe:
//   * key tiles of 128: S_t = Q_t . K_j^T is 8 MMAs of 128x128x16 and O_t += P_t . V_j another 8, so there are a
//     third fewer MMA instructions per key than with 64-key tiles (QK at N = 64 only half fills an instruction)
//     and half as many hand-offs between the softmax warps and the MMA warp;
//   * Q sits in shared memory (both operands of QK from shared memory run at the rate of the TMEM-A form once
//     N = 128), which frees TMEM for S tiles of 128 columns: S_A S_B 2 x 128 (P_t, packed bf16, overwrites the
//     first 64 columns of S_t), O_A O_B 2 x 128;
//   * K tiles and V tiles are separate 32-KB units of one ring (K0 V0 K1 V1 ...), 5 units beside the 64 KB of Q,
//     each unit filled by one bulk copy per page (the K block or the V block of a (page, head) is contiguous in the
//     pool and already in operand layout), K by warp 8 and V by warp 10;
//   * a share of the exponentials is computed on the FMA pipe (range reduction and a cubic), because the unit that
//     serves ex2 needs as long for a tile as the tensor pipe does and the two softmax warpgroups would otherwise
//     queue for it.
// The two row tiles ping-pong: while warpgroup A works on S_A(j) the tensor pipe runs PV_B(j-1) and QK_B(j).
// Every wait is bounded; a wait that runs out sets TIDE_ERR_DEVICE_TIMEOUT and the CTA drains and exits.
#include <climits>
#include <type_traits>

#include "tide_internal.h"

namespace tide {

namespace umma128 {

constexpr int D = 128;
constexpr int kTileKeys = 128;
constexpr int kThreads = 384;   // 3 warpgroups: softmax A, softmax B, {K producer 8, MMA issuer 9, V producer 10, idle 11}
constexpr int kNumUnits = 5;                        // ring of operand tiles in the order K0 V0 K1 V1 ...
constexpr int kGroupBytes = (D / 64) * 1024;        // one 8-key group of a K (or V) tile: two 1-KB atoms
constexpr int kUnitBytes = (kTileKeys / 8) * kGroupBytes;   // one K or V tile: 32 KB
constexpr int kQSlabBytes = 128 * 128;              // 128 rows x 128 bytes
constexpr int kQTileBytes = 2 * kQSlabBytes;        // the queries of one 128-row tile
constexpr int kQBytes = 2 * kQTileBytes;
constexpr int kSmemBytes = kQBytes + kNumUnits * kUnitBytes;   // 224 KB; with the static part (below 3 KB) the whole 227 KB of an SM
constexpr float kRescaleThreshold = 8.0f;           // log2 units
constexpr uint32_t kColS = 0, kColO = 256;          // S_t at kColS + t*128 (P_t over its first 64 columns), O_t at kColO + t*128
#ifndef TIDE_UMMA128_EMU_PAIRS
#define TIDE_UMMA128_EMU_PAIRS 1                    // of every 4 pairs of exponentials, how many take the polynomial
#endif
constexpr int kEmuPairs = TIDE_UMMA128_EMU_PAIRS;
#ifndef TIDE_UMMA128_P_PARTS
#define TIDE_UMMA128_P_PARTS 2                      // P_t is handed to the MMA warp in this many parts (2 or 4)
#endif
constexpr int kPParts = TIDE_UMMA128_P_PARTS;

// instruction descriptor: fp32 accumulate, bf16 A and B, M = 128, N = 128; bit 16 = B is MN-major
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 4) << 24) | ((128u >> 3) << 17);
constexpr uint32_t kIdescQK = kIdescBase;
constexpr uint32_t kIdescPV = kIdescBase | (1u << 16);

__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;   // descriptor version of this architecture
  d |= (uint64_t)2 << 61;   // 128-byte swizzle
  return d;
}
__device__ __forceinline__ uint64_t desc64(uint32_t lo, uint32_t hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
  return d;
}
// Both MMA forms are called by ALL lanes of the (converged) MMA warp; one elected lane issues, so descriptors and
// addresses stay in uniform registers.
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
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

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
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
__device__ __forceinline__ void tmem_st16u(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
        "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
  uint32_t u[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) u[i] = __float_as_uint(v[i]);
  tmem_st32u(taddr, u);
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
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
// Two base-2 exponentials on the FMA and integer pipes: n = round(x) by the magic-number addition (n lands in the
// low mantissa bits), a cubic for 2^r on r = x - n in [-0.5, 0.5] (relative error 7.5e-5, far below the bf16
// rounding of P), and n added to the exponent field.  Arguments below -126 are clamped (result 2^-126, not 0).
__device__ __forceinline__ void poly_exp2_pair(float x0, float x1, float& e0, float& e1) {
  const uint64_t xc = pack2(fmaxf(x0, -126.f), fmaxf(x1, -126.f));
  const uint64_t t = add2(xc, pack2(12582912.f, 12582912.f));
  const uint64_t n = add2(t, pack2(-12582912.f, -12582912.f));
  const uint64_t r = fma2(n, pack2(-1.f, -1.f), xc);
  uint64_t p = fma2(pack2(0.05517132f, 0.05517132f), r, pack2(0.24261054f, 0.24261054f));
  p = fma2(p, r, pack2(0.69326097f, 0.69326097f));
  p = fma2(p, r, pack2(0.99992812f, 0.99992812f));
  float p0, p1, t0, t1;
  unpack2(p, p0, p1);
  unpack2(t, t0, t1);
  e0 = __int_as_float((__float_as_int(t0) << 23) + __float_as_int(p0));
  e1 = __int_as_float((__float_as_int(t1) << 23) + __float_as_int(p1));
}

struct Bars {
  uint64_t kv_full[kNumUnits];
  uint64_t kv_empty[kNumUnits];
  uint64_t q_full;
  uint64_t s_full[2];   // S_t(j) is in TMEM (and every earlier MMA, PV_t(j-1) included, has retired)
  uint64_t p_part[2][kPParts];   // part q of P_t(j) (keys [q, q+1) * 128 / kPParts) is in TMEM
  uint64_t o_full[2];   // the last PV_t has retired
  uint64_t mma_done;    // every MMA of the item has retired
};

__global__ void __launch_bounds__(kThreads, 1) attend_umma128_kernel(const AttendParams P) {
  // The swizzled operand layouts need their tiles on 1-KB boundaries; there is no room for alignment slack, so the
  // dynamic part is declared with that alignment (and checked below).
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) Bars bars;
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  const uint32_t smem_q = smem_u32(smem_raw);                      // Q tiles A and B, then the operand ring
  const uint32_t smem_ring = smem_q + kQBytes;
  uint8_t* q_gen = smem_raw;
  uint8_t* ring_gen = q_gen + kQBytes;
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
  // per 128-row tile: rows present, last key any of its rows sees, number of 128-key tiles to process
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
  if (threadIdx.x == 0) {
    s_skip = *reinterpret_cast<volatile int*>(P.status);
    if ((smem_q & 1023u) != 0) {             // cannot happen with the declared alignment; refuse rather than compute garbage
      atomicExch(P.status, (int)TIDE_ERR_CUDA);
      s_skip = 1;
    }
  }
  __syncthreads();
  if (s_skip != 0) return;

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int i = 0; i < kNumUnits; ++i) { mbar_init(smem_u32(&bars.kv_full[i]), 1); mbar_init(smem_u32(&bars.kv_empty[i]), 1); }
    mbar_init(smem_u32(&bars.q_full), 256);
    for (int t = 0; t < 2; ++t) {
      mbar_init(smem_u32(&bars.s_full[t]), 1);
      for (int q = 0; q < kPParts; ++q) mbar_init(smem_u32(&bars.p_part[t][q]), 128);
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
    if (warp == 8 || warp == 10) {
      // ================= producers: warp 8 the K tiles (units 0, 2, 4, ...), warp 10 the V tiles (1, 3, 5, ...) =================
      if (n_tiles > 0) {
        const int is_v = warp == 10 ? 1 : 0;
        const int pages_per_tile = kTileKeys / g.S;            // 8 or 4: one copy each
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
        int issued = 0;                                        // tiles this warp has issued its copies of
        for (int j = 0; j < n_tiles; ++j) {
          const int u = 2 * j + is_v, slot = u % kNumUnits, use = u / kNumUnits;
          const int grp = j / tiles_per_group;
          if (grp != cur_grp) { ids_cur = ids_nxt; ids_nxt = load_ids(grp + 1); cur_grp = grp; }
          // a wait that gave up means the ring can no longer be trusted: issue nothing more
          if (use > 0 && !mbar_wait(smem_u32(&bars.kv_empty[slot]), (use - 1) & 1, abort_flag, P.status, P.wait_limit_ns)) break;
          issued = j + 1;
          if (P.debug_drop_first_stage != 0 && item == 0 && j == 0 && is_v == 0) continue;   // test hook: K tile 0 never arrives
          const int key0 = kv_begin + j * kTileKeys;
          const int npages = min(pages_per_tile, (kv_end - key0 + g.S - 1) / g.S);
          const uint32_t bar = smem_u32(&bars.kv_full[slot]);
          const long long page = __shfl_sync(0xffffffffu, ids_cur, ((j % tiles_per_group) * pages_per_tile + lane) & 31);
          if (lane == 0) mbar_expect_tx(bar, (uint32_t)(npages * g.kblock_bytes));
          __syncwarp();
          if (lane < npages)
            bulk_g2s(smem_ring + slot * kUnitBytes + lane * g.kblock_bytes,
                     P.pool + page * g.page_bytes + (long long)kvh * g.head_bytes + is_v * g.kblock_bytes, (uint32_t)g.kblock_bytes, bar);
        }
        if (*abort_flag && lane == 0) {
          // a wait gave up somewhere: this warp does not leave while copies it issued into the CTA's shared memory
          // can still be landing.  Those are among its last kNumUnits tiles; each wait is bounded like every other.
          for (int j = max(0, issued - kNumUnits); j < issued; ++j) {
            const int u = 2 * j + is_v;
            const uint32_t bar = smem_u32(&bars.kv_full[u % kNumUnits]);
            const long long t0 = global_ns();
            while (!mbar_try(bar, (u / kNumUnits) & 1) && global_ns() - t0 < P.wait_limit_ns) {}
          }
        }
      }
    } else if (warp == 9) {
      // ================= MMA issuer (whole warp converged, one elected lane issues) =================
      if (n_tiles > 0) {
        mbar_wait(smem_u32(&bars.q_full), 0, abort_flag, P.status, P.wait_limit_ns);
        tc_fence_after();
        // Descriptors are built once; moving an operand's start address is one 32-bit add on the low word (the
        // address field counts 16-byte units and cannot overflow its 14 bits inside this CTA's shared memory).
        const uint64_t kd0 = make_desc(smem_ring, 16, kGroupBytes);        // a K tile in unit 0 (K-major, 8-key groups 2 KB apart)
        const uint64_t vd0 = make_desc(smem_ring, 1024, kGroupBytes);      // a V tile in unit 0 (MN-major: slabs 1 KB, groups 2 KB apart)
        const uint64_t qd0 = make_desc(smem_q, 16, 1024);                  // a Q tile (K-major, 8-row groups 1 KB apart)
        const uint32_t kd_lo = (uint32_t)kd0, kd_hi = (uint32_t)(kd0 >> 32), vd_lo = (uint32_t)vd0, vd_hi = (uint32_t)(vd0 >> 32);
        const uint32_t qd_lo = (uint32_t)qd0, qd_hi = (uint32_t)(qd0 >> 32);
        constexpr uint32_t kUnitStep = kUnitBytes >> 4;
        auto issue_qk = [&](int t, int slot) {
          const uint32_t k_lo = kd_lo + slot * kUnitStep;
          const uint32_t q_lo = qd_lo + t * (kQTileBytes >> 4);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            mma_ss(tmem + kColS + t * 128, desc64(q_lo + (((ks >> 2) * kQSlabBytes + (ks & 3) * 32) >> 4), qd_hi),
                   desc64(k_lo + (((ks >> 2) * 1024 + (ks & 3) * 32) >> 4), kd_hi), kIdescQK, ks > 0);
          mma_commit(smem_u32(&bars.s_full[t]));
        };
        auto issue_pv = [&](int t, int j, int slot, int part) {      // the PV MMAs of part `part` of the keys
          const uint32_t v_lo = vd_lo + slot * kUnitStep;
#pragma unroll
          for (int k4 = 0; k4 < kTileKeys / 16 / kPParts; ++k4) {
            const int ks = part * (kTileKeys / 16 / kPParts) + k4;
            mma_ts(tmem + kColO + t * 128, tmem + kColS + t * 128 + ks * 8, desc64(v_lo + ((ks * 2 * kGroupBytes) >> 4), vd_hi), kIdescPV,
                   (j > 0 || ks > 0) ? 1u : 0u);
          }
        };
        // operand u of the sequence K0 V0 K1 V1 ... sits in unit u % kNumUnits on its (u / kNumUnits)-th use
        auto wait_full = [&](int slot, int use) {
          mbar_wait(smem_u32(&bars.kv_full[slot]), use & 1, abort_flag, P.status, P.wait_limit_ns);
        };
        wait_full(0, 0);
        tc_fence_after();
        for (int t = 0; t < 2; ++t) if (t_tiles[t] > 0) issue_qk(t, 0);
        mma_commit(smem_u32(&bars.kv_empty[0]));          // K(0) is consumed once these retire
        int vslot = 1, vuse = 0;                          // V(j): operand 2j + 1
        int kslot = 2, kuse = 0;                          // K(j+1): operand 2j + 2
        for (int j = 0; j < n_tiles; ++j) {
          wait_full(vslot, vuse);
          if (kv_end < kv_begin + (j + 1) * kTileKeys) {
            // rows of the V tile past the end of the item were not loaded (or hold stale page slots): clear
            // them so that weight 0 times leftover bits cannot produce NaN
            const int first = kv_end - (kv_begin + j * kTileKeys);
            uint8_t* vgen = ring_gen + vslot * kUnitBytes;
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
#pragma unroll
              for (int q = 0; q < kPParts; ++q) {
                mbar_wait(smem_u32(&bars.p_part[t][q]), j & 1, abort_flag, P.status, P.wait_limit_ns);
                tc_fence_after();
                issue_pv(t, j, vslot, q);
              }
              if (j + 1 < t_tiles[t]) {
                if (!k_ready) { wait_full(kslot, kuse); tc_fence_after(); k_ready = true; }
                issue_qk(t, kslot);                          // overwrites S_t / P_t after PV_t(j), in order
              } else {
                mma_commit(smem_u32(&bars.o_full[t]));
              }
            }
          }
          // V(j) and K(j+1) are consumed once these MMAs retire
          mma_commit(smem_u32(&bars.kv_empty[vslot]));
          if (j + 1 < n_tiles) mma_commit(smem_u32(&bars.kv_empty[kslot]));
          vslot += 2; if (vslot >= kNumUnits) { vslot -= kNumUnits; ++vuse; }
          kslot += 2; if (kslot >= kNumUnits) { kslot -= kNumUnits; ++kuse; }
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

    // ---- this row of Q (or zeros) into shared memory as the A operand of S = Q.K^T: K-major, 128-byte swizzle ----
    {
      const uint4* src = reinterpret_cast<const uint4*>(P.q + ((long long)(seg.q_off + qi) * g.Hq + hd) * D);
      uint8_t* qrow = q_gen + t * kQTileBytes + row * 128;
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const uint4 v = valid ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(qrow + (c >> 3) * kQSlabBytes + (((c & 7) ^ (row & 7)) << 4)) = v;
      }
      fence_async_smem();
      mbar_arrive(smem_u32(&bars.q_full));
    }

    float m = -INFINITY, l = 0.f;       // running max (base-2, scaled) and sum
    const float sl2 = P.scale_log2e;
    const uint32_t s_addr = tmem + lane_addr + kColS + t * 128;
    const uint32_t o_addr = tmem + lane_addr + kColO + t * 128;

    // One key tile of this row tile.  The tiles that need the causal (or end-of-range) mask are the last ones of the
    // item; they get a copy of the body of their own (with every exponential on the ex2 unit, which gives an exact 0
    // for a masked key), so the compare-and-select instructions of the mask are not part of the code the other tiles run.
    auto tile = [&](const int j, auto masked_tag) {
      constexpr bool kMasked = decltype(masked_tag)::value;
      constexpr int kEmu = kMasked ? 0 : kEmuPairs;
      mbar_wait(smem_u32(&bars.s_full[t]), j & 1, abort_flag, P.status, P.wait_limit_ns);
      tc_fence_after();
      float s[128];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(s_addr + c * 32, &s[c * 32]);
      tmem_wait_ld();
      if constexpr (kMasked) {
        const int vis = limit - (kv_begin + j * kTileKeys);
#pragma unroll
        for (int c = 0; c < 128; ++c) if (c >= vis) s[c] = -INFINITY;
      }
      // independent partial reductions (one long dependent chain would expose its latency), three inputs per
      // instruction: 8 chains over 128 values, then a tree
      float mxp[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) mxp[i] = max3(s[i], s[i + 8], s[i + 16]);
#pragma unroll
      for (int c = 24; c < 120; c += 16) {
#pragma unroll
        for (int i = 0; i < 8; ++i) mxp[i] = max3(mxp[i], s[c + i], s[c + i + 8]);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) mxp[i] = fmaxf(mxp[i], s[i + 120]);
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
      const uint64_t sl2_2 = pack2(sl2, sl2), nmu_2 = pack2(-mu, -mu);
      uint64_t sp2[4] = {pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f), pack2(0.f, 0.f)};
      // The exponentials run on the ex2 unit (and, for a share of them, on the FMA and integer pipes), the sums and the
      // bf16 packing on the FMA and ALU pipes.  A warp issues in order, so the three only overlap if independent work
      // is next to each other in the instruction stream: the stream is written as a software pipeline over groups of
      // 8 keys - scaled logits for all groups first, then the exponentials of group g+1 ahead of the sum and the
      // packing of group g, whose exponentials have had a whole group's time to come back.
      uint64_t x2[64];
#pragma unroll
      for (int i = 0; i < 64; ++i) x2[i] = fma2(pack2(s[2 * i], s[2 * i + 1]), sl2_2, nmu_2);
      float e[2][8];
      auto exp_group = [&](int gidx, float (&eg)[8]) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float x0, x1;
          unpack2(x2[gidx * 4 + i], x0, x1);
          if (i < kEmu) poly_exp2_pair(x0, x1, eg[2 * i], eg[2 * i + 1]);
          else { eg[2 * i] = fast_exp2(x0); eg[2 * i + 1] = fast_exp2(x1); }
        }
      };
      uint32_t pk[32];
      exp_group(0, e[0]);
#pragma unroll
      for (int gidx = 0; gidx < 16; ++gidx) {
        if (gidx + 1 < 16) exp_group(gidx + 1, e[(gidx + 1) & 1]);
        const float (&eg)[8] = e[gidx & 1];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          sp2[i] = add2(sp2[i], pack2(eg[2 * i], eg[2 * i + 1]));
          pk[(gidx & 7) * 4 + i] = pack_bf16(eg[2 * i], eg[2 * i + 1]);
        }
        // P_t over the first 64 columns of S_t; a part is handed over as soon as it is stored, so that its PV runs
        // while the exponentials of the later parts are computed (the last part is handed over after the row sum)
        constexpr int kGroupsPerPart = 16 / kPParts;
        if ((gidx + 1) % kGroupsPerPart == 0) {
          const int q = gidx / kGroupsPerPart;
          if constexpr (kPParts == 2) tmem_st32u(s_addr + q * 32, pk);
          else tmem_st16u(s_addr + q * 16, *reinterpret_cast<const uint32_t(*)[16]>(&pk[(q & 1) * 16]));
          if (q + 1 < kPParts) {
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(smem_u32(&bars.p_part[t][q]));
          }
        }
      }
      float sp[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) unpack2(sp2[i], sp[2 * i], sp[2 * i + 1]);
      l = l * alpha + (((sp[0] + sp[1]) + (sp[2] + sp[3])) + ((sp[4] + sp[5]) + (sp[6] + sp[7])));
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(smem_u32(&bars.p_part[t][kPParts - 1]));
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

}  // namespace umma128

cudaError_t attend_umma128_init() {
  return cudaFuncSetAttribute(umma128::attend_umma128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, umma128::kSmemBytes);
}

cudaError_t launch_attend_umma128(const AttendParams& p, cudaStream_t s) {
  const int grid = p.dyn ? p.grid_cap : p.n_items;
  if (grid <= 0) return cudaSuccess;
  umma128::attend_umma128_kernel<<<grid, umma128::kThreads, umma128::kSmemBytes, s>>>(p);
  return cudaGetLastError();
}

}  // namespace tide

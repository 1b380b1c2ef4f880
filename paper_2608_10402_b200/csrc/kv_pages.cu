// Page-append scatter, page-table delta update and logical read-back.
//
// Append is the GPU half of resuming a task under Continuous Task Batching (paper Section 4): the
// observation tokens' K/V rows are copied into the task's pages next to its preserved state, which
// replaces re-running prefill over the history (Section 1, first challenge).  It is a pure bit copy,
// bound by HBM bandwidth: 2 * Hkv * D * 2 bytes read and as many written per new token.
#include <algorithm>

#include "tide_internal.h"

namespace tide {

__global__ void table_update_kernel(int32_t* __restrict__ table, const int32_t* __restrict__ idx,
                                    const int32_t* __restrict__ val, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) table[idx[i]] = val[i];
}

cudaError_t launch_table_update(int32_t* table, const int32_t* idx, const int32_t* val, int n, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  table_update_kernel<<<(n + 255) / 256, 256, 0, s>>>(table, idx, val, n);
  return cudaGetLastError();
}

// Small host-to-device upload done by the SMs: src is pinned host memory mapped into the device's address space.
// Unlike a copy-engine transfer it does not queue behind large copies that other streams have in flight.
__global__ void upload_kernel(uint32_t* __restrict__ dst, const uint32_t* __restrict__ src, size_t n_words) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_words; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = src[i];
}

cudaError_t launch_upload(void* dst, const void* src_mapped_host, size_t bytes, cudaStream_t s) {
  if (bytes == 0) return cudaSuccess;
  const size_t n = bytes / 4;
  const unsigned blocks = (unsigned)std::min<size_t>((n + 255) / 256, 64);
  upload_kernel<<<blocks, 256, 0, s>>>((uint32_t*)dst, (const uint32_t*)src_mapped_host, n);
  return cudaGetLastError();
}

constexpr int kAppendThreads = 256;
constexpr int kAppendWarps = kAppendThreads / 32;
constexpr int kAppendMaxRecsSmem = 1024;
constexpr int kAppendLoadsInFlight = 8;    // 16-byte loads a lane has in flight before its first store

// The append: the new rows of every record go to their slots in the record's pages.  A warp takes the rows of EIGHT
// consecutive slots of one (kv, head) at a time, i.e. one 8-slot group of a page block - D / 64 core-matrix atoms of
// 1 KB, chunk c of row r at chunk position c ^ r - and writes it as one contiguous run: per instruction it reads
// four 128-byte pieces (four tokens) and writes 512 contiguous bytes.  (Written token by token, 128 bytes into four
// different atoms per instruction, the same copy ran at 4.9 instead of 5.5 TB/s on the multimodal batch.)  The
// record and page look-ups (warp-uniform) happen once per round of kAppendLoadsInFlight 16-byte loads per lane, all
// issued before the first store: a copy like this is bound by how many bytes are in flight.  Rows of a group that
// lie outside the record (its first and last group may be ragged) are left alone.  The same launch first applies
// the page-table delta of the append, if it is given one; the pages that delta brings are then taken from the delta
// itself, not from the table (no ordering between thread blocks is needed).
// AppendRec::grp0 = number of 8-slot groups that the records before this one touch.
template <int SLABS>
__device__ __forceinline__ void append_scatter_body(const AppendParams& P, const AppendRec* __restrict__ recs,
                                                  const int32_t* __restrict__ upd_idx, const int32_t* __restrict__ upd_val) {
  __shared__ int32_t s_grp0[kAppendMaxRecsSmem];
  const int n_recs = P.dyn ? P.dyn[0] : P.n_recs;
  for (int i = blockIdx.x * kAppendThreads + threadIdx.x; i < P.n_upd; i += gridDim.x * kAppendThreads)
    P.table_rw[upd_idx[i]] = upd_val[i];
  if (n_recs <= 0) return;
  const bool in_smem = n_recs <= kAppendMaxRecsSmem;
  if (in_smem) {
    for (int i = threadIdx.x; i < n_recs; i += blockDim.x) s_grp0[i] = recs[i].grp0;
    __syncthreads();
  }
  const Geom& g = P.g;
  const int lane = threadIdx.x & 31;
  const int heads2 = 2 * g.Hkv;
  long long n_units;
  {
    const AppendRec last = recs[n_recs - 1];
    n_units = (long long)(last.grp0 + (((last.pos0 & 7) + last.count + 7) >> 3)) * heads2;
  }
  const int warps_total = gridDim.x * kAppendWarps;
  const int warp_id = blockIdx.x * kAppendWarps + (threadIdx.x >> 5);
  constexpr int LPU = SLABS * 2;                               // 16-byte chunks per lane per (group, kv, head)
  constexpr int UNITS = kAppendLoadsInFlight / LPU;            // (kv, head) blocks of one group per warp per round
  const int rounds_per_group = (heads2 + UNITS - 1) / UNITS;
  const long long n_rounds = (n_units / heads2) * rounds_per_group;
  for (long long w = warp_id; w < n_rounds; w += warps_total) {
    // one look-up per round: the group's record and page
    const int grp = (int)(w / rounds_per_group), hh0 = (int)(w - (long long)grp * rounds_per_group) * UNITS;
    int r;
    if (in_smem) r = find_segment(n_recs, grp, [&](int i) { return s_grp0[i]; });
    else r = find_segment(n_recs, grp, [&](int i) { return recs[i].grp0; });
    const AppendRec rec = recs[r];
    const int g_pos0 = (rec.pos0 & ~7) + (grp - rec.grp0) * 8;                 // first slot position of the group
    const int lp = g_pos0 / g.S;
    const long long page = lp >= rec.new_lp0 ? upd_val[rec.new_off + (lp - rec.new_lp0)] : P.table[rec.table_off + lp];
    uint8_t* const dst_grp = P.pool + page * g.page_bytes + ((g_pos0 - lp * g.S) >> 3) * g.group_bytes;
    const int lo = max(0, rec.pos0 - g_pos0), hi = min(8, rec.pos0 + rec.count - g_pos0);
    const long long src_tok = (long long)(rec.tok0 + (g_pos0 - rec.pos0)) * g.Hkv;   // (token, head 0) row of the group's slot 0
    uint4 v[UNITS][LPU];
#pragma unroll
    for (int k = 0; k < UNITS; ++k) {
      const int hh = hh0 + k, kv = hh >= g.Hkv ? 1 : 0, h = hh - kv * g.Hkv;
      const uint16_t* src = (kv ? P.new_v : P.new_k) + (src_tok + h) * g.D;
#pragma unroll
      for (int i = 0; i < LPU; ++i) {
        const int e = lane + 32 * i;                           // chunk of the group in storage order: [slab][row][position]
        const int slab = e >> 6, row = (e >> 3) & 7, c = (e & 7) ^ row;
        v[k][i] = make_uint4(0, 0, 0, 0);
        if (hh < heads2 && row >= lo && row < hi)
          v[k][i] = __ldg(reinterpret_cast<const uint4*>(src + (long long)row * g.Hkv * g.D + (slab * 8 + c) * 8));
      }
    }
#pragma unroll
    for (int k = 0; k < UNITS; ++k) {
      const int hh = hh0 + k, kv = hh >= g.Hkv ? 1 : 0, h = hh - kv * g.Hkv;
      uint8_t* dst = dst_grp + (long long)h * g.head_bytes + kv * g.kblock_bytes;
#pragma unroll
      for (int i = 0; i < LPU; ++i) {
        const int e = lane + 32 * i, row = (e >> 3) & 7;
        if (hh < heads2 && row >= lo && row < hi) *reinterpret_cast<uint4*>(dst + e * 16) = v[k][i];
      }
    }
  }
}

template <int SLABS>
__global__ void __launch_bounds__(kAppendThreads, 3) append_scatter_kernel(const AppendParams P) {
  append_scatter_body<SLABS>(P, P.recs, P.upd_idx, P.upd_val);
}
template <int SLABS>
__global__ void __launch_bounds__(kAppendThreads, 3) append_scatter_inline_kernel(const __grid_constant__ AppendInline PI) {
  append_scatter_body<SLABS>(PI.p, PI.recs, PI.upd, PI.upd + PI.p.n_upd);
}

static unsigned append_grid(const AppendParams& p) {
  const long long cap = (long long)sm_count() * 3;            // the resident blocks; each warp loops over rounds beyond this
  if (p.dyn) return (unsigned)cap;
  const long long rounds = ((long long)p.n_tokens / 8 + 2LL * p.n_recs + 1) * 2 * p.g.Hkv + 1;   // an upper bound
  return (unsigned)std::max<long long>(1, std::min((rounds + kAppendWarps - 1) / kAppendWarps, cap));
}

cudaError_t launch_append(const AppendParams& p, cudaStream_t s) {
  const int tokens = p.dyn ? p.grid_cap_tokens : p.n_tokens;
  if (tokens <= 0 && p.n_upd <= 0) return cudaSuccess;
  const dim3 grid(append_grid(p));
  if (p.g.D == 128) append_scatter_kernel<2><<<grid, kAppendThreads, 0, s>>>(p);
  else append_scatter_kernel<1><<<grid, kAppendThreads, 0, s>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_append_inline(const AppendInline& pi, cudaStream_t s) {
  if (pi.p.n_tokens <= 0 && pi.p.n_upd <= 0) return cudaSuccess;
  const dim3 grid(append_grid(pi.p));
  if (pi.p.g.D == 128) append_scatter_inline_kernel<2><<<grid, kAppendThreads, 0, s>>>(pi);
  else append_scatter_inline_kernel<1><<<grid, kAppendThreads, 0, s>>>(pi);
  return cudaGetLastError();
}

// Whole-page copies dst[i] <- src[i] (the private copy a forked task gets of a partial last page, and the copy an
// append makes before it writes into a page that other tasks still hold).  One block column per page.
__global__ void copy_pages_kernel(uint8_t* __restrict__ pool, const int32_t* __restrict__ src, const int32_t* __restrict__ dst,
                                  long long page_bytes) {
  const uint4* s = reinterpret_cast<const uint4*>(pool + (long long)src[blockIdx.y] * page_bytes);
  uint4* d = reinterpret_cast<uint4*>(pool + (long long)dst[blockIdx.y] * page_bytes);
  const long long n = page_bytes / 16;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) d[i] = s[i];
}

cudaError_t launch_copy_pages(uint8_t* pool, const int32_t* src, const int32_t* dst, int n, long long page_bytes, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  dim3 grid(8, (unsigned)n);
  copy_pages_kernel<<<grid, 256, 0, s>>>(pool, src, dst, page_bytes);
  return cudaGetLastError();
}

// Logical content of one task -> contiguous [len, Hkv, D]; inverse of the scatter above.
// Positions [pos0, pos0 + len) of the task go to rows [0, len) of out_k / out_v.
__global__ void read_gather_kernel(const uint8_t* __restrict__ pool, const int32_t* __restrict__ table_row, int pos0, int len,
                                   uint16_t* __restrict__ out_k, uint16_t* __restrict__ out_v, const Geom g) {
  const int cpr = g.D >> 3;
  const int cpt = 2 * g.Hkv * cpr;
  const long long total = (long long)len * cpt;
  for (long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x; gid < total;
       gid += (long long)gridDim.x * blockDim.x) {
    const int row = (int)(gid / cpt);
    int rem = (int)(gid - (long long)row * cpt);
    const int kv = rem / (g.Hkv * cpr);
    rem -= kv * g.Hkv * cpr;
    const int h = rem / cpr;
    const int c = rem - h * cpr;
    const int pos = pos0 + row;
    const int lp = pos / g.S, slot = pos - lp * g.S;
    const long long page = table_row[lp];
    const uint8_t* src = pool + page * g.page_bytes + (long long)h * g.head_bytes + blk_offset(g, slot, kv, c);
    uint16_t* dst = (kv ? out_v : out_k) + ((long long)row * g.Hkv + h) * g.D + c * 8;
    *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
  }
}

cudaError_t launch_read(const uint8_t* pool, const int32_t* table_row, int pos0, int len, uint16_t* out_k,
                        uint16_t* out_v, const Geom& g, cudaStream_t s) {
  if (len <= 0) return cudaSuccess;
  const long long total = (long long)len * 2 * g.Hkv * (g.D / 8);
  long long blocks = (total + 255) / 256;
  const long long cap = (long long)sm_count() * 64;
  if (blocks > cap) blocks = cap;
  read_gather_kernel<<<(unsigned)blocks, 256, 0, s>>>(pool, table_row, pos0, len, out_k, out_v, g);
  return cudaGetLastError();
}

}  // namespace tide

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

// One warp per token at a time: the record lookup, the page lookup and the slot arithmetic happen once per token
// (warp-uniform), then the lanes copy the token's 16-byte chunks, ordered [K|V][kv_head][chunk]: a warp reads 512
// contiguous source bytes and writes four full 128-byte lines per pass.  A copy like this is bound by how many
// bytes are in flight, so a warp takes several tokens per round and issues all their loads (eight per lane)
// before the first store.  CPL = chunks per lane per token when a token is a multiple of 32 chunks (0: any
// count, plain loop).  The same launch first applies the page-table delta of the append, if it is given one; the
// pages that delta brings are then taken from the delta itself, not from the table (no ordering between thread
// blocks is needed).
template <int CPL>
__device__ __forceinline__ void append_scatter_body(const AppendParams& P, const AppendRec* __restrict__ recs,
                                                    const int32_t* __restrict__ upd_idx, const int32_t* __restrict__ upd_val) {
  __shared__ int32_t s_tok0[kAppendMaxRecsSmem];
  const int n_recs = P.dyn ? P.dyn[0] : P.n_recs;
  const int n_tokens = P.dyn ? P.dyn[1] : P.n_tokens;
  for (int i = blockIdx.x * kAppendThreads + threadIdx.x; i < P.n_upd; i += gridDim.x * kAppendThreads)
    P.table_rw[upd_idx[i]] = upd_val[i];
  const bool in_smem = n_recs <= kAppendMaxRecsSmem;
  if (in_smem) {
    for (int i = threadIdx.x; i < n_recs; i += blockDim.x) s_tok0[i] = recs[i].tok0;
    __syncthreads();
  }
  const Geom& g = P.g;
  const int lane = threadIdx.x & 31;
  const int cpr = g.D >> 3;                   // chunks per (token, head) row: 8 or 16
  const int shift = cpr == 16 ? 4 : 3;
  const int cpt = 2 * g.Hkv * cpr;            // chunks per token: K rows then V rows
  const int warps_total = gridDim.x * kAppendWarps;
  const int warp_id = blockIdx.x * kAppendWarps + (threadIdx.x >> 5);

  // where token `tok` goes: the base of its page (slot offsets are added per chunk) and its slot
  auto locate = [&](int tok, int& slot) -> uint8_t* {
    int r;
    if (in_smem) r = find_segment(n_recs, tok, [&](int i) { return s_tok0[i]; });
    else r = find_segment(n_recs, tok, [&](int i) { return recs[i].tok0; });
    const AppendRec rec = recs[r];
    const int pos = rec.pos0 + (tok - rec.tok0);
    const int lp = pos / g.S;
    slot = pos - lp * g.S;
    const long long page = lp >= rec.new_lp0 ? upd_val[rec.new_off + (lp - rec.new_lp0)] : P.table[rec.table_off + lp];
    return P.pool + page * g.page_bytes;
  };
  // chunk c of a token: source address and offset inside the page
  auto src_of = [&](int tok, int c) -> const uint4* {
    const int row = c >> shift, cc = c & (cpr - 1);
    const int kv = row >= g.Hkv ? 1 : 0, h = row - kv * g.Hkv;
    return reinterpret_cast<const uint4*>((kv ? P.new_v : P.new_k) + ((long long)tok * g.Hkv + h) * g.D + cc * 8);
  };
  auto dst_off = [&](int slot, int c) -> long long {
    const int row = c >> shift, cc = c & (cpr - 1);
    const int kv = row >= g.Hkv ? 1 : 0, h = row - kv * g.Hkv;
    return (long long)h * g.head_bytes + blk_offset(g, slot, kv, cc);
  };

  if constexpr (CPL > 0) {
    constexpr int TOK = kAppendLoadsInFlight / CPL;          // tokens per warp per round
    for (int t0 = warp_id; t0 < n_tokens; t0 += warps_total * TOK) {
      uint4 v[TOK][CPL];
      uint8_t* base[TOK];
      int slot[TOK];
#pragma unroll
      for (int u = 0; u < TOK; ++u) {
        const int tok = t0 + u * warps_total;
        base[u] = nullptr;
        if (tok < n_tokens) {
          base[u] = locate(tok, slot[u]);
#pragma unroll
          for (int i = 0; i < CPL; ++i) v[u][i] = __ldg(src_of(tok, lane + 32 * i));
        }
      }
#pragma unroll
      for (int u = 0; u < TOK; ++u) {
        if (base[u] != nullptr) {
#pragma unroll
          for (int i = 0; i < CPL; ++i) *reinterpret_cast<uint4*>(base[u] + dst_off(slot[u], lane + 32 * i)) = v[u][i];
        }
      }
    }
  } else {
    for (int tok = warp_id; tok < n_tokens; tok += warps_total) {
      int slot;
      uint8_t* base = locate(tok, slot);
      for (int c = lane; c < cpt; c += 32) *reinterpret_cast<uint4*>(base + dst_off(slot, c)) = __ldg(src_of(tok, c));
    }
  }
}

template <int CPL>
__global__ void __launch_bounds__(kAppendThreads, 3) append_scatter_kernel(const AppendParams P) {
  append_scatter_body<CPL>(P, P.recs, P.upd_idx, P.upd_val);
}

// The same with the records and the table delta inside the kernel's parameters (small appends: nothing to upload).
template <int CPL>
__global__ void __launch_bounds__(kAppendThreads, 3) append_scatter_inline_kernel(const __grid_constant__ AppendInline PI) {
  append_scatter_body<CPL>(PI.p, PI.recs, PI.upd, PI.upd + PI.p.n_upd);
}

static unsigned append_grid(const AppendParams& p, int& cpl) {
  const int tokens = p.dyn ? p.grid_cap_tokens : p.n_tokens;
  const int cpt = 2 * p.g.Hkv * (p.g.D / 8);
  cpl = cpt % 32 == 0 ? cpt / 32 : 0;
  if (!(cpl == 1 || cpl == 2 || cpl == 4 || cpl == 8)) cpl = 0;
  const int tok_per_round = cpl ? kAppendLoadsInFlight / cpl : 1;
  long long blocks = ((long long)std::max(tokens, 1) + kAppendWarps * tok_per_round - 1) / (kAppendWarps * tok_per_round);
  const long long cap = (long long)sm_count() * 3;   // the resident blocks; each warp loops over rounds beyond this
  return (unsigned)std::max<long long>(1, std::min(blocks, cap));
}

cudaError_t launch_append(const AppendParams& p, cudaStream_t s) {
  const int tokens = p.dyn ? p.grid_cap_tokens : p.n_tokens;
  if (tokens <= 0 && p.n_upd <= 0) return cudaSuccess;
  int cpl;
  const dim3 grid(append_grid(p, cpl));
  switch (cpl) {
    case 1: append_scatter_kernel<1><<<grid, kAppendThreads, 0, s>>>(p); break;
    case 2: append_scatter_kernel<2><<<grid, kAppendThreads, 0, s>>>(p); break;
    case 4: append_scatter_kernel<4><<<grid, kAppendThreads, 0, s>>>(p); break;
    case 8: append_scatter_kernel<8><<<grid, kAppendThreads, 0, s>>>(p); break;
    default: append_scatter_kernel<0><<<grid, kAppendThreads, 0, s>>>(p); break;
  }
  return cudaGetLastError();
}

cudaError_t launch_append_inline(const AppendInline& pi, cudaStream_t s) {
  if (pi.p.n_tokens <= 0 && pi.p.n_upd <= 0) return cudaSuccess;
  int cpl;
  const dim3 grid(append_grid(pi.p, cpl));
  switch (cpl) {
    case 1: append_scatter_inline_kernel<1><<<grid, kAppendThreads, 0, s>>>(pi); break;
    case 2: append_scatter_inline_kernel<2><<<grid, kAppendThreads, 0, s>>>(pi); break;
    case 4: append_scatter_inline_kernel<4><<<grid, kAppendThreads, 0, s>>>(pi); break;
    case 8: append_scatter_inline_kernel<8><<<grid, kAppendThreads, 0, s>>>(pi); break;
    default: append_scatter_inline_kernel<0><<<grid, kAppendThreads, 0, s>>>(pi); break;
  }
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

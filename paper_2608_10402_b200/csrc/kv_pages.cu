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

// Byte offset of 16-byte chunk `c` (c = d / 8) of slot `slot` inside a K or V block.
__device__ __forceinline__ int chunk_offset(int S, int slot, int c) {
  return (c >> 3) * (S * 128) + slot * 128 + (((c & 7) ^ (slot & 7)) << 4);
}

constexpr int kAppendThreads = 256;
constexpr int kAppendMaxRecsSmem = 1024;

// One warp per token at a time: the record lookup, the page-table read and the slot arithmetic happen once per
// token (warp-uniform), then the lanes copy the token's 16-byte chunks, ordered [K|V][kv_head][chunk], so a warp
// reads 512 contiguous source bytes and writes four full 128-byte lines per pass.  D/8 is a power of two, so the
// per-chunk index split needs no division.
__global__ void __launch_bounds__(kAppendThreads) append_scatter_kernel(const AppendParams P) {
  __shared__ int32_t s_tok0[kAppendMaxRecsSmem];
  const int n_recs = P.dyn ? P.dyn[0] : P.n_recs;
  const int n_tokens = P.dyn ? P.dyn[1] : P.n_tokens;
  const bool in_smem = n_recs <= kAppendMaxRecsSmem;
  if (in_smem) {
    for (int i = threadIdx.x; i < n_recs; i += blockDim.x) s_tok0[i] = P.recs[i].tok0;
    __syncthreads();
  }
  const int lane = threadIdx.x & 31;
  const int cpr = P.g.D >> 3;                 // chunks per (token, head) row: 8 or 16
  const int shift = cpr == 16 ? 4 : 3;
  const int rows2 = 2 * P.g.Hkv;              // K rows then V rows of one token
  const int cpt = rows2 * cpr;                // chunks per token
  const int warps_total = gridDim.x * (kAppendThreads / 32);
  for (int tok = blockIdx.x * (kAppendThreads / 32) + (threadIdx.x >> 5); tok < n_tokens; tok += warps_total) {
    int r;
    if (in_smem) r = find_segment(n_recs, tok, [&](int i) { return s_tok0[i]; });
    else r = find_segment(n_recs, tok, [&](int i) { return P.recs[i].tok0; });
    const AppendRec rec = P.recs[r];
    const int pos = rec.pos0 + (tok - rec.tok0);
    const int lp = pos / P.g.S, slot = pos - lp * P.g.S;
    const long long page = P.table[rec.table_off + lp];
    uint8_t* page_base = P.pool + page * P.g.page_bytes + slot * 128;
    const uint16_t* src_k = P.new_k + (long long)tok * P.g.Hkv * P.g.D;
    const uint16_t* src_v = P.new_v + (long long)tok * P.g.Hkv * P.g.D;
    const int sw = slot & 7;
    for (int c = lane; c < cpt; c += 32) {
      const int cc = c & (cpr - 1);
      const int row = c >> shift;               // 0 .. 2*Hkv-1
      const int kv = row >= P.g.Hkv ? 1 : 0;
      const int h = row - kv * P.g.Hkv;
      const uint16_t* src = (kv ? src_v : src_k) + h * P.g.D + cc * 8;
      uint8_t* dst = page_base + (long long)h * P.g.head_bytes + kv * P.g.kblock_bytes + (cc >> 3) * (P.g.S * 128) +
                     (((cc & 7) ^ sw) << 4);
      *reinterpret_cast<uint4*>(dst) = __ldg(reinterpret_cast<const uint4*>(src));
    }
  }
}

cudaError_t launch_append(const AppendParams& p, cudaStream_t s) {
  const int tokens = p.dyn ? p.grid_cap_tokens : p.n_tokens;
  if (tokens <= 0) return cudaSuccess;
  long long blocks = ((long long)tokens + kAppendThreads / 32 - 1) / (kAppendThreads / 32);
  const long long cap = (long long)sm_count() * 8 * 8;   // 8 resident blocks per SM, a few tokens per warp beyond this
  if (blocks > cap) blocks = cap;
  append_scatter_kernel<<<(unsigned)blocks, kAppendThreads, 0, s>>>(p);
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
    const uint8_t* src = pool + page * g.page_bytes + (long long)h * g.head_bytes + kv * g.kblock_bytes +
                         chunk_offset(g.S, slot, c);
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

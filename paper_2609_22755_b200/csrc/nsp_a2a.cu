// Layout kernels of the Ulysses all-to-all around the attention compute (paper Sec. 2.1 and Sec. 4.1.2, the prologue /
// epilogue phases of an SP-tree node). HBM-bound copies: 16 bytes per thread and access, rows of head_dim elements.
//
// Before the prologue a GPU of a degree-d node holds its 1/d token slice of the node's samples with ALL heads,
// [T, H, D]; the peer p needs the heads [first_head[p], first_head[p] + Hd) of those tokens as one contiguous
// block. gather_heads builds the d blocks [n][T, Hd, D] in one pass (a KV head that several peers share is simply
// read several times). After the epilogue exchange the GPU holds d blocks [n][T, Hd, D], block p carrying the heads
// peer p computed for this GPU's tokens; scatter_heads writes them back into [T, H, D]. Where several blocks map to
// the same head (the dK / dV partial sums of a replicated KV head) they are added in block order, in fp32, by the one
// thread that owns the output element: no atomics, same result every run.
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "../../include/nsp.h"

namespace nsp {
void count_launches(int n);
}

namespace {

struct HeadMap {
  int32_t first_head[NSP_A2A_MAX_PEERS];
};

// Both kernels are launched with a thread count that is a multiple of the 16-byte vectors of one token row of the
// side they iterate over, so a thread keeps its (head, vector) position for the whole grid-stride loop and only the
// token (and, for the gather, the block) advances: no division inside the loop.

// one thread per 16 bytes of the packed side [n][T, Hd, D]
__global__ void __launch_bounds__(256) gather_heads_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst,
                                                           int64_t T, int H, int Hd, int n, int vec_per_row,
                                                           const __grid_constant__ HeadMap map) {
  const int row = Hd * vec_per_row;  // vectors of one token inside a block
  const int64_t threads = static_cast<int64_t>(gridDim.x) * blockDim.x;  // a multiple of `row`
  const int64_t t0 = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int in_row = static_cast<int>(t0 % row);
  const int hh = in_row / vec_per_row, v = in_row - hh * vec_per_row;
  const int64_t tok_step = threads / row;
  int64_t tok = t0 / row;
  int p = 0;
  for (;;) {
    while (tok >= T && p < n) tok -= T, ++p;
    if (p >= n) break;
    dst[(p * T + tok) * row + in_row] = __ldg(src + (tok * H + map.first_head[p] + hh) * vec_per_row + v);
    tok += tok_step;
  }
}

// The fused send side of the prologue: the same head gather, but every block is stored where its receiver reads it.
// Block p goes to base[p] (the packed attention buffer [t_full, Hd, D] of peer p: that GPU's own memory mapped into
// this process, or a local buffer), the tokens of sample j starting at row dst_row[p * n_samples + j] there (where
// this GPU's token slice of the sample sits inside the complete sequence). Plain 16-byte stores from this kernel: no
// library kernel is handed a peer pointer, and nothing here is a TMA or multicast access.
struct PeerBases {
  uint4* base[NSP_A2A_MAX_PEERS];
};
__global__ void __launch_bounds__(256) gather_heads_to_kernel(const uint4* __restrict__ src, int64_t T, int H, int Hd,
                                                              int n, int vec_per_row, int n_samples,
                                                              const int64_t* __restrict__ sample_off,
                                                              const int64_t* __restrict__ dst_row,
                                                              const __grid_constant__ HeadMap map,
                                                              const __grid_constant__ PeerBases peers) {
  const int row = Hd * vec_per_row;  // vectors of one token inside a block
  const int64_t threads = static_cast<int64_t>(gridDim.x) * blockDim.x;  // a multiple of `row`
  const int64_t t0 = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int in_row = static_cast<int>(t0 % row);
  const int hh = in_row / vec_per_row, v = in_row - hh * vec_per_row;
  const int64_t tok_step = threads / row;
  int64_t tok = t0 / row;
  int p = 0;
  for (;;) {
    while (tok >= T && p < n) tok -= T, ++p;
    if (p >= n) break;
    int lo = 0, hi = n_samples - 1;  // the sample the token belongs to: sample_off ascending, sample_off[0] = 0
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (sample_off[mid] <= tok) lo = mid; else hi = mid - 1;
    }
    const int64_t r = dst_row[static_cast<int64_t>(p) * n_samples + lo] + (tok - sample_off[lo]);
    peers.base[p][r * row + in_row] = __ldg(src + (tok * H + map.first_head[p] + hh) * vec_per_row + v);
    tok += tok_step;
  }
}

// one thread per 16 bytes of the [T, H, D] side; the blocks that carry the thread's head are found once, the common
// case of exactly one is a plain copy (two tokens per pass, so that two loads are in flight), several are added in
// block order in fp32
template <bool kF32>
__global__ void __launch_bounds__(256) scatter_heads_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst,
                                                            int64_t T, int H, int Hd, int n, int vec_per_row,
                                                            const __grid_constant__ HeadMap map) {
  const int row = H * vec_per_row;
  const int64_t threads = static_cast<int64_t>(gridDim.x) * blockDim.x;  // a multiple of `row`
  const int64_t t0 = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int in_row = static_cast<int>(t0 % row);
  const int h = in_row / vec_per_row, v = in_row - h * vec_per_row;
  const int64_t tok_step = threads / row;
  const int64_t per_block = T * Hd * vec_per_row;
  uint64_t hits = 0;
  for (int p = 0; p < n; ++p) {
    const int hh = h - map.first_head[p];
    if (hh >= 0 && hh < Hd) hits |= 1ull << p;
  }
  const int cnt = __popcll(hits);
  if (cnt == 0) return;  // a head no block carries is left as it is
  if (cnt == 1) {
    const int p = __ffsll(static_cast<long long>(hits)) - 1;
    const uint4* s1 = src + p * per_block + static_cast<int64_t>(h - map.first_head[p]) * vec_per_row + v;
    const int64_t srow = static_cast<int64_t>(Hd) * vec_per_row;
    int64_t tok = t0 / row;
    for (; tok + tok_step < T; tok += 2 * tok_step) {
      const uint4 a = __ldg(s1 + tok * srow), b = __ldg(s1 + (tok + tok_step) * srow);
      dst[tok * row + in_row] = a;  // a plain copy keeps the bits
      dst[(tok + tok_step) * row + in_row] = b;
    }
    if (tok < T) dst[tok * row + in_row] = __ldg(s1 + tok * srow);
    return;
  }
  for (int64_t tok = t0 / row; tok < T; tok += tok_step) {
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    uint64_t left = hits;
    while (left) {  // up to four loads in flight, added in block order
      uint4 x[4];
      int m = 0;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (left) {
          const int p = __ffsll(static_cast<long long>(left)) - 1;
          left &= left - 1;
          x[u] = __ldg(src + p * per_block + (tok * Hd + (h - map.first_head[p])) * vec_per_row + v);
          m = u + 1;
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (u < m) {
          if (kF32) {
            acc[0] += __uint_as_float(x[u].x), acc[1] += __uint_as_float(x[u].y);
            acc[2] += __uint_as_float(x[u].z), acc[3] += __uint_as_float(x[u].w);
          } else {
            const uint32_t w[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              acc[2 * t] += __uint_as_float(w[t] << 16);
              acc[2 * t + 1] += __uint_as_float(w[t] & 0xffff0000u);
            }
          }
        }
      }
    }
    if (kF32) {
      dst[tok * row + in_row] = make_uint4(__float_as_uint(acc[0]), __float_as_uint(acc[1]), __float_as_uint(acc[2]),
                                           __float_as_uint(acc[3]));
    } else {
      uint32_t w[4];
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const __nv_bfloat162 b2 = __floats2bfloat162_rn(acc[2 * t], acc[2 * t + 1]);
        w[t] = *reinterpret_cast<const uint32_t*>(&b2);
      }
      dst[tok * row + in_row] = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

int check(const void* src, void* dst, int64_t tokens, int heads, int heads_per_block, int n_blocks, int head_dim,
          int dtype, const int32_t* first_head, HeadMap* map) {
  if (tokens < 0 || heads <= 0 || heads_per_block <= 0 || heads_per_block > heads || n_blocks <= 0 ||
      n_blocks > NSP_A2A_MAX_PEERS || head_dim <= 0 || !first_head)
    return NSP_ERR_INVALID_ARG;
  if (dtype != NSP_BF16 && dtype != NSP_F32) return NSP_ERR_INVALID_ARG;
  const int elem = dtype == NSP_F32 ? 4 : 2;
  if ((head_dim * elem) % 16 != 0) return NSP_ERR_UNSUPPORTED;
  for (int p = 0; p < n_blocks; ++p) {
    if (first_head[p] < 0 || first_head[p] + heads_per_block > heads) return NSP_ERR_INVALID_ARG;
    map->first_head[p] = first_head[p];
  }
  if (tokens == 0) return NSP_OK;
  if (!src || !dst || (reinterpret_cast<uintptr_t>(src) & 15) || (reinterpret_cast<uintptr_t>(dst) & 15))
    return NSP_ERR_INVALID_ARG;
  return NSP_OK;
}

// Blocks of 256 threads whose total is a multiple of `row` (the vectors of one token row), about `total` threads but
// no more than 32 blocks per SM.
int grid_for(int64_t total, int row) {
  int a = row, b = 256;
  while (b) { const int t = a % b; a = b; b = t; }
  const int unit = row / a;  // blocks per multiple of `row`
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 32) blocks = 148 * 32;
  blocks = (blocks + unit - 1) / unit * unit;
  return static_cast<int>(blocks < unit ? unit : blocks);
}

}  // namespace

extern "C" int nsp_a2a_gather_heads(const void* src, void* dst, int64_t tokens, int32_t heads, int32_t heads_per_block,
                                    int32_t n_blocks, int32_t head_dim, int32_t dtype, const int32_t* first_head,
                                    void* stream) {
  HeadMap map = {};
  const int rc = check(src, dst, tokens, heads, heads_per_block, n_blocks, head_dim, dtype, first_head, &map);
  if (rc != NSP_OK || tokens == 0) return rc;
  const int vec = head_dim * (dtype == NSP_F32 ? 4 : 2) / 16;
  const int64_t total = tokens * heads_per_block * vec * n_blocks;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  gather_heads_kernel<<<grid_for(total, heads_per_block * vec), 256, 0, st>>>(static_cast<const uint4*>(src), static_cast<uint4*>(dst),
                                                          tokens, heads, heads_per_block, n_blocks, vec, map);
  nsp::count_launches(1);
  return cudaGetLastError() == cudaSuccess ? NSP_OK : NSP_ERR_CUDA;
}

extern "C" int nsp_a2a_scatter_heads(const void* src, void* dst, int64_t tokens, int32_t heads, int32_t heads_per_block,
                                     int32_t n_blocks, int32_t head_dim, int32_t dtype, const int32_t* first_head,
                                     void* stream) {
  HeadMap map = {};
  const int rc = check(src, dst, tokens, heads, heads_per_block, n_blocks, head_dim, dtype, first_head, &map);
  if (rc != NSP_OK || tokens == 0) return rc;
  const int vec = head_dim * (dtype == NSP_F32 ? 4 : 2) / 16;
  const int64_t total = tokens * heads * vec;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (dtype == NSP_F32)
    scatter_heads_kernel<true><<<grid_for(total, heads * vec), 256, 0, st>>>(static_cast<const uint4*>(src), static_cast<uint4*>(dst),
                                                                tokens, heads, heads_per_block, n_blocks, vec, map);
  else
    scatter_heads_kernel<false><<<grid_for(total, heads * vec), 256, 0, st>>>(static_cast<const uint4*>(src), static_cast<uint4*>(dst),
                                                                 tokens, heads, heads_per_block, n_blocks, vec, map);
  nsp::count_launches(1);
  return cudaGetLastError() == cudaSuccess ? NSP_OK : NSP_ERR_CUDA;
}

extern "C" int nsp_a2a_gather_heads_to(const void* src, void* const* dst_base, const int64_t* dst_row,
                                       const int64_t* sample_off, int32_t n_samples, int64_t tokens, int32_t heads,
                                       int32_t heads_per_block, int32_t n_blocks, int32_t head_dim, int32_t dtype,
                                       const int32_t* first_head, void* stream) {
  if (!dst_base || n_samples < 0 || n_blocks <= 0 || n_blocks > NSP_A2A_MAX_PEERS) return NSP_ERR_INVALID_ARG;
  HeadMap map = {};
  // the shared checks want one destination pointer: every block's base has to pass them
  PeerBases peers = {};
  for (int p = 0; p < n_blocks; ++p) {
    const int rc = check(src, dst_base[p], tokens, heads, heads_per_block, n_blocks, head_dim, dtype, first_head, &map);
    if (rc != NSP_OK) return rc;
    peers.base[p] = static_cast<uint4*>(dst_base[p]);
  }
  if (tokens == 0) return NSP_OK;
  if (n_samples == 0 || !dst_row || !sample_off) return NSP_ERR_INVALID_ARG;
  const int vec = head_dim * (dtype == NSP_F32 ? 4 : 2) / 16;
  const int64_t total = tokens * heads_per_block * vec * n_blocks;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  gather_heads_to_kernel<<<grid_for(total, heads_per_block * vec), 256, 0, st>>>(
      static_cast<const uint4*>(src), tokens, heads, heads_per_block, n_blocks, vec, n_samples, sample_off, dst_row, map,
      peers);
  nsp::count_launches(1);
  return cudaGetLastError() == cudaSuccess ? NSP_OK : NSP_ERR_CUDA;
}

// Layout kernels of the Ulysses all-to-all around the attention compute (paper Sec. 2.2 and Sec. 4.2, the prologue /
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

// one thread per 16 bytes of the packed side
__global__ void __launch_bounds__(256) gather_heads_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst,
                                                           int64_t T, int H, int Hd, int n, int vec_per_row,
                                                           const __grid_constant__ HeadMap map) {
  const int64_t per_block = T * Hd * vec_per_row;
  const int64_t total = per_block * n;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int p = static_cast<int>(i / per_block);
    const int64_t r = i - p * per_block;
    const int64_t tok = r / (Hd * vec_per_row);
    const int rem = static_cast<int>(r - tok * (Hd * vec_per_row));
    const int hh = rem / vec_per_row, v = rem - hh * vec_per_row;
    dst[i] = __ldg(src + (tok * H + map.first_head[p] + hh) * vec_per_row + v);
  }
}

// one thread per 16 bytes of the [T, H, D] side; the blocks that cover the head are added in block order.
// The blocks that carry a head are found first (no memory access); the common case of exactly one is a plain copy,
// two elements per thread and pass so that two loads are in flight.
template <bool kF32>
__global__ void __launch_bounds__(256) scatter_heads_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst,
                                                            int64_t T, int H, int Hd, int n, int vec_per_row,
                                                            const __grid_constant__ HeadMap map) {
  const int64_t total = T * H * vec_per_row;
  const int64_t per_block = T * Hd * vec_per_row;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t i0 = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i0 < total; i0 += 2 * stride) {
    uint64_t hits[2] = {0, 0};
    int64_t off[2] = {0, 0};  // offset of the element inside a block
    int h2[2] = {0, 0};
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int64_t i = i0 + u * stride;
      if (i >= total) continue;
      const int64_t tok = i / (H * vec_per_row);
      const int rem = static_cast<int>(i - tok * (H * vec_per_row));
      const int h = rem / vec_per_row, v = rem - h * vec_per_row;
      h2[u] = h;
      off[u] = tok * Hd * vec_per_row + v;
      for (int p = 0; p < n; ++p) {
        const int hh = h - map.first_head[p];
        if (hh >= 0 && hh < Hd) hits[u] |= 1ull << p;
      }
    }
    uint4 one[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      if (__popcll(hits[u]) == 1) {
        const int p = __ffsll(static_cast<long long>(hits[u])) - 1;
        one[u] = __ldg(src + p * per_block + off[u] + static_cast<int64_t>(h2[u] - map.first_head[p]) * vec_per_row);
      }
    }
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int64_t i = i0 + u * stride;
      const int cnt = __popcll(hits[u]);
      if (cnt == 0) continue;  // a head no block carries is left as it is
      if (cnt == 1) {
        dst[i] = one[u];  // a plain copy keeps the bits
        continue;
      }
      float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      for (int p = 0; p < n; ++p) {
        if (!((hits[u] >> p) & 1ull)) continue;
        const uint4 x = __ldg(src + p * per_block + off[u] + static_cast<int64_t>(h2[u] - map.first_head[p]) * vec_per_row);
        if (kF32) {
          acc[0] += __uint_as_float(x.x), acc[1] += __uint_as_float(x.y);
          acc[2] += __uint_as_float(x.z), acc[3] += __uint_as_float(x.w);
        } else {
          const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            acc[2 * t] += __uint_as_float(w[t] << 16);
            acc[2 * t + 1] += __uint_as_float(w[t] & 0xffff0000u);
          }
        }
      }
      if (kF32) {
        dst[i] = make_uint4(__float_as_uint(acc[0]), __float_as_uint(acc[1]), __float_as_uint(acc[2]),
                            __float_as_uint(acc[3]));
      } else {
        uint32_t w[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const __nv_bfloat162 b2 = __floats2bfloat162_rn(acc[2 * t], acc[2 * t + 1]);
          w[t] = *reinterpret_cast<const uint32_t*>(&b2);
        }
        dst[i] = make_uint4(w[0], w[1], w[2], w[3]);
      }
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

int grid_for(int64_t total) {
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 32) blocks = 148 * 32;
  return static_cast<int>(blocks < 1 ? 1 : blocks);
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
  gather_heads_kernel<<<grid_for(total), 256, 0, st>>>(static_cast<const uint4*>(src), static_cast<uint4*>(dst),
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
    scatter_heads_kernel<true><<<grid_for(total), 256, 0, st>>>(static_cast<const uint4*>(src), static_cast<uint4*>(dst),
                                                                tokens, heads, heads_per_block, n_blocks, vec, map);
  else
    scatter_heads_kernel<false><<<grid_for(total), 256, 0, st>>>(static_cast<const uint4*>(src), static_cast<uint4*>(dst),
                                                                 tokens, heads, heads_per_block, n_blocks, vec, map);
  nsp::count_launches(1);
  return cudaGetLastError() == cudaSuccess ? NSP_OK : NSP_ERR_CUDA;
}

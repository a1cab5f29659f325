// Device-side construction of the tile work lists (forward and backward).
//
// Item definitions and order (unique, so any correct sort reproduces it bit for bit):
//   forward  (s, h, m): cost = ceil(min(L, (m+1)*bm) / bn)          -- key tiles the query tile visits
//   backward (s, g, n): cost = G * (Mt - floor(n*bn / bm))          -- (q head, q tile) visits of the key tile
//   order: cost descending, then segment, tile, head ascending.
// Every item is encoded into one 64-bit key whose ascending order is that order:
//   [63:40] 2^24-1-cost   [39:24] segment   [23:8] tile   [7:0] head
// The keys are emitted by one block per segment, sorted with a device radix sort and decoded into items.
#include <cub/device/device_radix_sort.cuh>
#include <cuda_bf16.h>
#include "nsp_internal.cuh"

namespace nsp {

namespace {

constexpr uint64_t kCostMax = (1ull << 24) - 1;

__device__ __forceinline__ uint64_t encode_item(int seg, int head, int tile, int cost) {
  return ((kCostMax - static_cast<uint64_t>(cost)) << 40) | (static_cast<uint64_t>(seg) << 24) |
         (static_cast<uint64_t>(tile) << 8) | static_cast<uint64_t>(head);
}

__global__ void emit_keys_kernel(const SegInfo* __restrict__ seg, int bm, int bn, const int64_t* __restrict__ fwd_base,
                                 const int64_t* __restrict__ bwd_base, uint64_t* __restrict__ fwd_keys,
                                 uint64_t* __restrict__ bwd_keys) {
  const int s = blockIdx.x;
  const int L = seg[s].len, hq = seg[s].hq, hkv = seg[s].hkv;
  const int G = hq / hkv;
  const int Mt = (L + bm - 1) / bm, Nt = (L + bn - 1) / bn;
  const int64_t nf = static_cast<int64_t>(Mt) * hq;
  for (int64_t t = threadIdx.x; t < nf; t += blockDim.x) {
    const int h = static_cast<int>(t / Mt), m = static_cast<int>(t % Mt);
    const int64_t hi = min(static_cast<int64_t>(L), static_cast<int64_t>(m + 1) * bm);
    fwd_keys[fwd_base[s] + t] = encode_item(s, h, m, static_cast<int>((hi + bn - 1) / bn));
  }
  const int64_t nb = static_cast<int64_t>(Nt) * hkv;
  for (int64_t t = threadIdx.x; t < nb; t += blockDim.x) {
    const int g = static_cast<int>(t / Nt), n = static_cast<int>(t % Nt);
    const int cost = G * (Mt - static_cast<int>((static_cast<int64_t>(n) * bn) / bm));
    bwd_keys[bwd_base[s] + t] = encode_item(s, g, n, cost);
  }
}

__global__ void decode_keys_kernel(const uint64_t* __restrict__ keys, int64_t n, nsp_tile_t* __restrict__ items) {
  const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (t >= n) return;
  const uint64_t k = keys[t];
  nsp_tile_t it;
  it.cost = static_cast<int32_t>(kCostMax - (k >> 40));
  it.seg = static_cast<int32_t>((k >> 24) & 0xFFFF);
  it.tile = static_cast<int32_t>((k >> 8) & 0xFFFF);
  it.head = static_cast<int32_t>(k & 0xFF);
  items[t] = it;
}

}  // namespace

size_t plan_sort_tmp_bytes(int64_t max_items) {
  size_t bytes = 0;
  cub::DeviceRadixSort::SortKeys(nullptr, bytes, static_cast<const uint64_t*>(nullptr), static_cast<uint64_t*>(nullptr),
                                 max_items > 0 ? max_items : 1);
  return bytes;
}

// d_keys holds n_fwd + n_bwd keys (forward first); d_keys_alt the same amount for the sorted output.
cudaError_t launch_plan_build(const SegInfo* d_seg, int n_seg, int bm, int bn, nsp_tile_t* d_fwd, int64_t n_fwd,
                              nsp_tile_t* d_bwd, int64_t n_bwd, uint64_t* d_keys, uint64_t* d_keys_alt, void* d_sort_tmp,
                              size_t sort_tmp_bytes, const int64_t* d_fwd_base, const int64_t* d_bwd_base,
                              cudaStream_t st) {
  if (n_seg == 0 || (n_fwd == 0 && n_bwd == 0)) return cudaSuccess;
  emit_keys_kernel<<<n_seg, 256, 0, st>>>(d_seg, bm, bn, d_fwd_base, d_bwd_base, d_keys, d_keys + n_fwd);
  count_launches(1);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (n_fwd > 0) {
    e = cub::DeviceRadixSort::SortKeys(d_sort_tmp, sort_tmp_bytes, d_keys, d_keys_alt, n_fwd, 0, 64, st);
    if (e != cudaSuccess) return e;
    decode_keys_kernel<<<static_cast<unsigned>((n_fwd + 255) / 256), 256, 0, st>>>(d_keys_alt, n_fwd, d_fwd);
    count_launches(1);
  }
  if (n_bwd > 0) {
    e = cub::DeviceRadixSort::SortKeys(d_sort_tmp, sort_tmp_bytes, d_keys + n_fwd, d_keys_alt + n_fwd, n_bwd, 0, 64, st);
    if (e != cudaSuccess) return e;
    decode_keys_kernel<<<static_cast<unsigned>((n_bwd + 255) / 256), 256, 0, st>>>(d_keys_alt + n_fwd, n_bwd, d_bwd);
    count_launches(1);
  }
  return cudaGetLastError();
}

}  // namespace nsp

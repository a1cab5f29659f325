// Backward: dQ, dK, dV of packed variable-length causal GQA attention on tcgen05 tensor cores.
//
// Three launches:
//   preprocess   delta[h, i] = sum_d dO[i,h,d] * O[i,h,d]                      (HBM-bound, one warp per row)
//   main         key-stationary persistent kernel, see below
//   postprocess  dQ = scale * fp32 accumulator -> bf16 / fp32                   (HBM-bound)
//
// Main kernel. One CTA per SM (256 threads) pops items (segment, kv head, key tile n) from the longest-first
// list. K_n and V_n stay in shared memory; the CTA walks every q head of the KV group and every q tile m >= n.
// All score-shaped quantities are computed TRANSPOSED (key index on the TMEM lanes) so that P^T and dS^T are
// directly the A operands of the dV and dK products:
//     S^T  = K Q^T ,  dP^T = V dO^T              A, B K-major from shared memory          -> TMEM
//     P^T  = exp2(S^T * scale*log2e - LSE*log2e), dS^T = P^T o (dP^T - delta)   one thread per (key row, half)
//     dV  += P^T dO                               A = P^T (bf16, TMEM), B = dO  MN-major
//     dK  += dS^T Q                               A = dS^T (shared, K-major), B = Q MN-major
//     dQ_m = dS K                                 A = dS^T read MN-major, B = K MN-major   -> TMEM (over S^T)
// For the first q tile of a segment (rows 0..127, where P is O(1)) P^T and dS^T are split into hi + lo bf16
// parts and every product is issued twice; this keeps dK/dV/dQ inside the 2e-2 max-abs tolerance.
// dK and dV accumulate in TMEM over the whole item, in a fixed order (heads ascending, tiles ascending), so
// the reduction over the query heads of a group is deterministic. dQ tiles are added to an fp32 accumulator
// in global memory with vector reductions.
#include <cuda_bf16.h>
#include "nsp_internal.cuh"
#include "sm100_ptx.cuh"

namespace nsp {
namespace {

constexpr int kBwdThreads = 256;
constexpr uint32_t kHalfTileBytes = 128 * 64 * 2;
constexpr uint32_t kTileBytes = 2 * kHalfTileBytes;
constexpr uint32_t kBwdTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;

struct BwdSmem {
  uint8_t k[2][kHalfTileBytes];
  uint8_t v[2][kHalfTileBytes];
  uint8_t q[2][kHalfTileBytes];
  uint8_t d_o[2][kHalfTileBytes];
  uint8_t ds[2][kHalfTileBytes];  // dS^T, [key row][query col], split in two 64-column halves
  uint8_t ds_lo[2][kHalfTileBytes];  // bf16 residual of dS^T (first q tile of a segment only)
  float lse[128];                 // LSE * log2(e) of the current q tile (+inf for rows past the segment)
  float delta[128];
  float part[4][128];             // per-quadrant partial sums of the exact delta (first q tile only)
  uint64_t bar_kv, bar_qdo, bar_s, bar_m2;
  uint32_t tmem_base;
  int32_t item_idx;
};
constexpr size_t kBwdSmemBytes = sizeof(BwdSmem) + 1024;

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

__global__ void __launch_bounds__(kBwdThreads, 1) bwd_kernel(const __grid_constant__ BwdMaps maps, const BwdArgs a) {
  extern __shared__ uint8_t smem_raw[];
  BwdSmem& s = *reinterpret_cast<BwdSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int quad = warp & 3, half = warp >> 2;
  const int r = quad * 32 + lane;  // TMEM lane owned by this thread (key row in steps 1-2, query row for dQ)

  if (tid == 0) {
    mbar_init(&s.bar_kv, 1);
    mbar_init(&s.bar_qdo, 1);
    mbar_init(&s.bar_s, 1);
    mbar_init(&s.bar_m2, 1);
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&s.tmem_base, kBwdTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();

  const uint32_t tS = s.tmem_base, tDP = tS + 128, tDK = tS + 256, tDV = tS + 384;
  const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
  const uint32_t k_addr = smem_u32(s.k[0]), v_addr = smem_u32(s.v[0]), q_addr = smem_u32(s.q[0]),
                 do_addr = smem_u32(s.d_o[0]), ds_addr = smem_u32(s.ds[0]), dsl_addr = smem_u32(s.ds_lo[0]);
  constexpr uint32_t idesc_kk = make_idesc_bf16(128, 128, 0, 0);  // A K-major, B K-major
  constexpr uint32_t idesc_kn = make_idesc_bf16(128, 128, 0, 1);  // A K-major (or TMEM), B MN-major
  constexpr uint32_t idesc_nn = make_idesc_bf16(128, 128, 1, 1);  // A MN-major, B MN-major
  uint32_t ph_kv = 0, ph_qdo = 0, ph_s = 0, ph_m2 = 0;
  bool ok = true;

  for (;;) {
    if (tid == 0) s.item_idx = atomicAdd(a.counter, 1);
    tc_fence_before_sync();
    ok = __syncthreads_and(ok);
    tc_fence_after_sync();
    const int it = s.item_idx;
    if (!ok || it >= a.n_items) break;

    const nsp_tile_t item = a.items[it];
    const SegInfo sg = a.seg[item.seg];
    const int g = item.head, n = item.tile;
    const int G = sg.hq / sg.hkv;
    const int Mt = (sg.len + kBM - 1) / kBM;
    const int n_m = Mt - n;  // q tiles n .. Mt-1 (bm == bn)
    const int steps = G * n_m;
    const int tok0 = sg.tok_in_run;
    const CUtensorMap* mq = &maps.q[sg.run];
    const CUtensorMap* mdo = &maps.d_o[sg.run];

    if (tid == 0) {
      mbar_expect_tx(&s.bar_kv, 2 * kTileBytes);
      tma_load_3d(s.k[0], &maps.k[sg.run], &s.bar_kv, 0, g, tok0 + n * kBN);
      tma_load_3d(s.k[1], &maps.k[sg.run], &s.bar_kv, 64, g, tok0 + n * kBN);
      tma_load_3d(s.v[0], &maps.v[sg.run], &s.bar_kv, 0, g, tok0 + n * kBN);
      tma_load_3d(s.v[1], &maps.v[sg.run], &s.bar_kv, 64, g, tok0 + n * kBN);
      mbar_expect_tx(&s.bar_qdo, 2 * kTileBytes);
      tma_load_3d(s.q[0], mq, &s.bar_qdo, 0, g * G, tok0 + n * kBM);
      tma_load_3d(s.q[1], mq, &s.bar_qdo, 64, g * G, tok0 + n * kBM);
      tma_load_3d(s.d_o[0], mdo, &s.bar_qdo, 0, g * G, tok0 + n * kBM);
      tma_load_3d(s.d_o[1], mdo, &s.bar_qdo, 64, g * G, tok0 + n * kBM);
    }

    for (int t = 0; t < steps; ++t) {
      const int h = g * G + t / n_m;
      const int m = n + t % n_m;
      // ---- step 1: S^T = K Q^T, dP^T = V dO^T
      if (tid == 0) {
        bool okt = true;
        if (t == 0) {
          okt = mbar_wait(&s.bar_kv, ph_kv);
          ph_kv ^= 1;
        }
        okt = okt && mbar_wait(&s.bar_qdo, ph_qdo);
        ph_qdo ^= 1;
        if (okt) {
          tc_fence_after_sync();
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (kk >> 2) * kHalfTileBytes + (kk & 3) * 32;
            umma_ss(tS, make_smem_desc_sw128(k_addr + off, 16, 1024), make_smem_desc_sw128(q_addr + off, 16, 1024),
                    idesc_kk, kk > 0);
          }
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (kk >> 2) * kHalfTileBytes + (kk & 3) * 32;
            umma_ss(tDP, make_smem_desc_sw128(v_addr + off, 16, 1024), make_smem_desc_sw128(do_addr + off, 16, 1024),
                    idesc_kk, kk > 0);
          }
          umma_commit(&s.bar_s);
        } else {
          report_timeout(a.status, it, t == 0 ? kWhereBwdLoadKV : kWhereBwdLoadQ, t);
        }
      }
      // LSE and delta of q tile m (head h) -> shared memory
      {
        const int qi = m * kBM + (tid & 127);
        const bool valid = qi < sg.len;
        const int64_t idx = sg.lse_off + static_cast<int64_t>(h) * sg.len + qi;
        if (tid < 128)
          s.lse[tid] = valid ? a.lse[idx] * kLog2e : INFINITY;
        else
          s.delta[tid - 128] = valid ? a.delta[idx] : 0.f;
      }
      bool okw = mbar_wait(&s.bar_s, ph_s);
      ph_s ^= 1;
      if (!okw && lane == 0) report_timeout(a.status, it, kWhereBwdS, t);
      ok = __syncthreads_and(ok && okw);  // also publishes s.lse / s.delta
      if (!ok) break;
      {
        tc_fence_after_sync();
        const bool diag = (m == n);
        // First q tile of a segment: P and dS are O(1) there and their bf16 rounding dominates the error of
        // dK/dV/dQ, so they are fed to the tensor core as hi + lo bf16 pairs (two MMAs per product), and
        // delta_i is recomputed as sum_j P_ij dP_ij in fp32 (all keys of these rows lie in this key tile)
        // instead of taking it from the bf16-rounded O.
        const bool exact_delta = (m == 0) && (a.debug_flags & 2) == 0;
        const bool hilo = (m == 0) && (a.debug_flags & 1) == 0;
        if (exact_delta) {
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            const int col0 = half * 64 + c * 32;
            uint32_t sv[32], dpv[32];
            tmem_ld32(tS + lane_off + col0, sv);
            tmem_ld32(tDP + lane_off + col0, dpv);
            tmem_wait_ld();
#pragma unroll
            for (int x = 0; x < 32; ++x) {
              float p = ex2f(fmaf(__uint_as_float(sv[x]), a.scale_log2, -s.lse[col0 + x]));
              if (col0 + x < r) p = 0.f;
              float v = p * __uint_as_float(dpv[x]);
#pragma unroll
              for (int sft = 16; sft > 0; sft >>= 1) v += __shfl_xor_sync(0xffffffffu, v, sft);
              if (lane == 0) s.part[quad][col0 + x] = v;
            }
          }
          __syncthreads();
          if (tid < 128) s.delta[tid] = (s.part[0][tid] + s.part[1][tid]) + (s.part[2][tid] + s.part[3][tid]);
          __syncthreads();
        }
#pragma unroll
        for (int c = 0; c < 2; ++c) {  // 32 query columns at a time
          const int col0 = half * 64 + c * 32;
          uint32_t sv[32], dpv[32];
          tmem_ld32(tS + lane_off + col0, sv);
          tmem_ld32(tDP + lane_off + col0, dpv);
          tmem_wait_ld();
          uint32_t pp[16], dsp[16], ppl[16], dspl[16];
#pragma unroll
          for (int x = 0; x < 32; x += 2) {
            float p0 = ex2f(fmaf(__uint_as_float(sv[x]), a.scale_log2, -s.lse[col0 + x]));
            float p1 = ex2f(fmaf(__uint_as_float(sv[x + 1]), a.scale_log2, -s.lse[col0 + x + 1]));
            if (diag) {  // query index must be >= key index
              if (col0 + x < r) p0 = 0.f;
              if (col0 + x + 1 < r) p1 = 0.f;
            }
            const float d0 = p0 * (__uint_as_float(dpv[x]) - s.delta[col0 + x]);
            const float d1 = p1 * (__uint_as_float(dpv[x + 1]) - s.delta[col0 + x + 1]);
            const uint32_t ph = pack_bf16x2(p0, p1), dh = pack_bf16x2(d0, d1);
            pp[x >> 1] = ph;
            dsp[x >> 1] = dh;
            if (hilo) {
              ppl[x >> 1] = pack_bf16x2(p0 - __uint_as_float(ph << 16), p1 - __uint_as_float(ph & 0xffff0000u));
              dspl[x >> 1] = pack_bf16x2(d0 - __uint_as_float(dh << 16), d1 - __uint_as_float(dh & 0xffff0000u));
            }
          }
          // P^T (bf16 pairs) goes over S^T columns this warp has already read: for query columns
          // [col0, col0+32) the hi parts take packed columns [col0, col0+16), the lo parts [col0+16, col0+32).
          tmem_st16(tS + lane_off + col0, pp);
          if (hilo) tmem_st16(tS + lane_off + col0 + 16, ppl);
          // dS^T row r, columns col0 .. col0+31 -> four 16-byte chunks of the swizzled half tile
          uint8_t* base = s.ds[half] + r * 128;
          uint8_t* base_lo = s.ds_lo[half] + r * 128;
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            const int chunk = (c * 4 + ch) ^ (r & 7);
            *reinterpret_cast<uint4*>(base + chunk * 16) =
                make_uint4(dsp[ch * 4 + 0], dsp[ch * 4 + 1], dsp[ch * 4 + 2], dsp[ch * 4 + 3]);
            if (hilo)
              *reinterpret_cast<uint4*>(base_lo + chunk * 16) =
                  make_uint4(dspl[ch * 4 + 0], dspl[ch * 4 + 1], dspl[ch * 4 + 2], dspl[ch * 4 + 3]);
          }
        }
        tmem_wait_st();
        fence_proxy_async_smem();
      }
      tc_fence_before_sync();
      __syncthreads();
      // ---- step 2: dV += P^T dO, dK += dS^T Q, dQ = dS K
      if (tid == 0) {
        tc_fence_after_sync();
        const bool hilo = (m == 0) && (a.debug_flags & 1) == 0;
        // packed P^T column of K-step kk (16 query columns): see the store above
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          umma_ts(tDV, tS + (kk >> 1) * 32 + (kk & 1) * 8, make_smem_desc_sw128(do_addr + kk * 2048, kHalfTileBytes, 1024),
                  idesc_kn, (t > 0 || kk > 0));
        if (hilo) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            umma_ts(tDV, tS + (kk >> 1) * 32 + 16 + (kk & 1) * 8,
                    make_smem_desc_sw128(do_addr + kk * 2048, kHalfTileBytes, 1024), idesc_kn, 1);
        }
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t off = (kk >> 2) * kHalfTileBytes + (kk & 3) * 32;
          umma_ss(tDK, make_smem_desc_sw128(ds_addr + off, 16, 1024),
                  make_smem_desc_sw128(q_addr + kk * 2048, kHalfTileBytes, 1024), idesc_kn, (t > 0 || kk > 0));
        }
        if (hilo) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (kk >> 2) * kHalfTileBytes + (kk & 3) * 32;
            umma_ss(tDK, make_smem_desc_sw128(dsl_addr + off, 16, 1024),
                    make_smem_desc_sw128(q_addr + kk * 2048, kHalfTileBytes, 1024), idesc_kn, 1);
          }
        }
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          umma_ss(tS, make_smem_desc_sw128(ds_addr + kk * 2048, kHalfTileBytes, 1024),
                  make_smem_desc_sw128(k_addr + kk * 2048, kHalfTileBytes, 1024), idesc_nn, kk > 0);
        if (hilo) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            umma_ss(tS, make_smem_desc_sw128(dsl_addr + kk * 2048, kHalfTileBytes, 1024),
                    make_smem_desc_sw128(k_addr + kk * 2048, kHalfTileBytes, 1024), idesc_nn, 1);
        }
        umma_commit(&s.bar_m2);
      }
      okw = mbar_wait(&s.bar_m2, ph_m2);
      ph_m2 ^= 1;
      okw = __all_sync(0xffffffffu, okw);
      if (okw) {
        tc_fence_after_sync();
        if (tid == 0 && t + 1 < steps) {  // Q / dO buffers are free: fetch the next step's tiles
          const int h2 = g * G + (t + 1) / n_m, m2 = n + (t + 1) % n_m;
          mbar_expect_tx(&s.bar_qdo, 2 * kTileBytes);
          tma_load_3d(s.q[0], mq, &s.bar_qdo, 0, h2, tok0 + m2 * kBM);
          tma_load_3d(s.q[1], mq, &s.bar_qdo, 64, h2, tok0 + m2 * kBM);
          tma_load_3d(s.d_o[0], mdo, &s.bar_qdo, 0, h2, tok0 + m2 * kBM);
          tma_load_3d(s.d_o[1], mdo, &s.bar_qdo, 64, h2, tok0 + m2 * kBM);
        }
        // dQ tile: lane = query row, this thread adds 64 columns
        const int qi = m * kBM + r;
        float* dst = a.dq_acc + sg.q_off + (static_cast<int64_t>(qi) * sg.hq + h) * kHeadDim + half * 64;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          uint32_t v[32];
          tmem_ld32(tS + lane_off + half * 64 + c * 32, v);
          tmem_wait_ld();
          if (qi < sg.len) {
#pragma unroll
            for (int x = 0; x < 32; x += 4)
              red_add_v4(dst + c * 32 + x, __uint_as_float(v[x]), __uint_as_float(v[x + 1]), __uint_as_float(v[x + 2]),
                         __uint_as_float(v[x + 3]));
          }
        }
      } else if (lane == 0) {
        report_timeout(a.status, it, kWhereBwdMma2, t);
      }
      ok = ok && okw;
      tc_fence_before_sync();
      ok = __syncthreads_and(ok);
      if (!ok) break;
      tc_fence_after_sync();
    }
    if (!ok) continue;

    // ---- epilogue: dK (scaled) and dV rows of this key tile
    const int kj = n * kBN + r;
    const bool valid = kj < sg.len;
    const int64_t off = sg.kv_off + (static_cast<int64_t>(kj) * sg.hkv + g) * kHeadDim + half * 64;
#pragma unroll
    for (int which = 0; which < 2; ++which) {
      const uint32_t tsrc = which == 0 ? tDK : tDV;
      const float mul = which == 0 ? a.scale : 1.f;
      void* outp = which == 0 ? a.dk : a.dv;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t v[32];
        tmem_ld32(tsrc + lane_off + half * 64 + c * 32, v);
        tmem_wait_ld();
        if (valid) {
          if (a.dkv_f32) {
            float* o = static_cast<float*>(outp) + off + c * 32;
#pragma unroll
            for (int x = 0; x < 32; x += 4)
              *reinterpret_cast<float4*>(o + x) =
                  make_float4(__uint_as_float(v[x]) * mul, __uint_as_float(v[x + 1]) * mul,
                              __uint_as_float(v[x + 2]) * mul, __uint_as_float(v[x + 3]) * mul);
          } else {
            __nv_bfloat16* o = static_cast<__nv_bfloat16*>(outp) + off + c * 32;
#pragma unroll
            for (int x = 0; x < 32; x += 8) {
              uint4 w;
              w.x = pack_bf16x2(__uint_as_float(v[x]) * mul, __uint_as_float(v[x + 1]) * mul);
              w.y = pack_bf16x2(__uint_as_float(v[x + 2]) * mul, __uint_as_float(v[x + 3]) * mul);
              w.z = pack_bf16x2(__uint_as_float(v[x + 4]) * mul, __uint_as_float(v[x + 5]) * mul);
              w.w = pack_bf16x2(__uint_as_float(v[x + 6]) * mul, __uint_as_float(v[x + 7]) * mul);
              *reinterpret_cast<uint4*>(o + x) = w;
            }
          }
        }
      }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(s.tmem_base, kBwdTmemCols);
}

// delta[h, i] = <dO[i,h,:], O[i,h,:]>; one warp per (token, head) row, rows in packed order.
__global__ void bwd_preprocess_kernel(const SegInfo* __restrict__ seg, int n_seg, const int64_t* __restrict__ row_base,
                                      int64_t total_rows, const __nv_bfloat16* __restrict__ o,
                                      const __nv_bfloat16* __restrict__ d_o, float* __restrict__ delta) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  if (row >= total_rows) return;
  // row_base[s] = first packed row of segment s (ascending, row_base[n_seg] = total_rows)
  int lo = 0, hi = n_seg - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (row_base[mid] <= row) lo = mid; else hi = mid - 1;
  }
  const SegInfo sg = seg[lo];
  const int64_t rl = row - row_base[lo];
  const int i = static_cast<int>(rl / sg.hq), h = static_cast<int>(rl % sg.hq);
  const int64_t e = sg.q_off + rl * kHeadDim + lane * 4;
  const uint2 a = *reinterpret_cast<const uint2*>(o + e);
  const uint2 b = *reinterpret_cast<const uint2*>(d_o + e);
  const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
  const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
  float acc = 0.f;
#pragma unroll
  for (int x = 0; x < 2; ++x) {
    const float2 fa = __bfloat1622float2(pa[x]), fb = __bfloat1622float2(pb[x]);
    acc = fmaf(fa.x, fb.x, acc);
    acc = fmaf(fa.y, fb.y, acc);
  }
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, sft);
  if (lane == 0) delta[sg.lse_off + static_cast<int64_t>(h) * sg.len + i] = acc;
}

__global__ void bwd_postprocess_kernel(const float* __restrict__ acc, void* __restrict__ dq, int64_t n4, int dq_f32,
                                       float scale) {
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; t < n4; t += stride) {
    const float4 v = reinterpret_cast<const float4*>(acc)[t];
    if (dq_f32) {
      reinterpret_cast<float4*>(dq)[t] = make_float4(v.x * scale, v.y * scale, v.z * scale, v.w * scale);
    } else {
      uint2 w;
      w.x = pack_bf16x2(v.x * scale, v.y * scale);
      w.y = pack_bf16x2(v.z * scale, v.w * scale);
      reinterpret_cast<uint2*>(dq)[t] = w;
    }
  }
}

}  // namespace

cudaError_t launch_bwd_preprocess(const SegInfo* d_seg, int n_seg, const int64_t* d_row_base, int64_t total_rows,
                                  const __nv_bfloat16* o, const __nv_bfloat16* d_o, float* delta, cudaStream_t st) {
  if (total_rows == 0) return cudaSuccess;
  const int64_t blocks = (total_rows * 32 + 255) / 256;
  bwd_preprocess_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(d_seg, n_seg, d_row_base, total_rows, o, d_o,
                                                                       delta);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_bwd(const BwdMaps& maps, const BwdArgs& args, int num_sms, cudaStream_t st) {
  if (args.n_items == 0) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(kBwdSmemBytes));
  if (e != cudaSuccess) return e;
  const int grid = args.n_items < num_sms ? args.n_items : num_sms;
  bwd_kernel<<<grid, kBwdThreads, kBwdSmemBytes, st>>>(maps, args);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_bwd_postprocess(const float* dq_acc, void* dq, int64_t n, int dq_f32, float scale,
                                   cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  const int64_t n4 = n / 4;  // n is a multiple of 128
  int64_t blocks = (n4 + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  bwd_postprocess_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(dq_acc, dq, n4, dq_f32, scale);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace nsp

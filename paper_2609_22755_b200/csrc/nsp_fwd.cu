// Forward: packed variable-length causal GQA attention on tcgen05 tensor cores.
//
// One persistent CTA (128 threads, two CTAs resident per SM) pops work items (segment, q head, q tile) from the
// longest-first list with an atomic cursor. For an item it keeps the 128 x 128 Q tile in shared memory and
// walks the key tiles 0 .. diagonal:
//     S = Q K^T        tcgen05.mma, both operands K-major in 128B-swizzled shared memory (TMA-staged)
//     online softmax   one thread per query row: tcgen05.ld S, exp2 with the scale folded in, row max/sum
//     P -> TMEM        bf16 pairs written over S (tcgen05.st)
//     O += P V         tcgen05.mma with A = P from TMEM, B = V (MN-major) from shared memory
// O stays in TMEM for the whole item and is rescaled in place only when the running maximum grows by more
// than 2^8 (the stale reference maximum is exact in the final normalisation because the same reference is
// used for the row sum). Only the diagonal tile is masked; tiles above the diagonal are never visited.
// The two CTAs of an SM overlap one CTA's softmax with the other's MMAs.
#include <cuda_bf16.h>
#include "nsp_internal.cuh"
#include "sm100_ptx.cuh"

namespace nsp {
namespace {

constexpr int kFwdThreads = 128;
constexpr uint32_t kHalfTileBytes = 128 * 64 * 2;  // one [128 rows x 64 cols] bf16 sub-tile
constexpr uint32_t kTileBytes = 2 * kHalfTileBytes;
constexpr uint32_t kFwdTmemCols = 256;  // S/P: columns [0,128), O: columns [128,256)

struct FwdSmem {
  uint8_t q[2][kHalfTileBytes];
  uint8_t k[2][kHalfTileBytes];
  uint8_t v[2][kHalfTileBytes];
  uint64_t bar_q, bar_k, bar_v, bar_s, bar_o;
  uint32_t tmem_base;
  int32_t item_idx;
};

constexpr size_t kFwdSmemBytes = sizeof(FwdSmem) + 1024;  // + slack for manual 1024-byte alignment

__global__ void __launch_bounds__(kFwdThreads, 2) fwd_kernel(const __grid_constant__ FwdMaps maps, const FwdArgs a) {
  extern __shared__ uint8_t smem_raw[];
  FwdSmem& s = *reinterpret_cast<FwdSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    mbar_init(&s.bar_q, 1);
    mbar_init(&s.bar_k, 1);
    mbar_init(&s.bar_v, 1);
    mbar_init(&s.bar_s, 1);
    mbar_init(&s.bar_o, 1);
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&s.tmem_base, kFwdTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();

  const uint32_t tS = s.tmem_base;
  const uint32_t tO = s.tmem_base + 128;
  const uint32_t lane_off = static_cast<uint32_t>(warp * 32) << 16;
  const uint32_t q_addr = smem_u32(s.q[0]), k_addr = smem_u32(s.k[0]), v_addr = smem_u32(s.v[0]);
  constexpr uint32_t idesc_qk = make_idesc_bf16(128, 128, 0, 0);
  constexpr uint32_t idesc_pv = make_idesc_bf16(128, 128, 0, 1);
  uint32_t ph_q = 0, ph_k = 0, ph_v = 0, ph_s = 0, ph_o = 0;
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
    const int h = item.head, g = h / (sg.hq / sg.hkv);
    const int n_kv = item.cost;
    const int q_row0 = item.tile * kBM;
    const int tok0 = sg.tok_in_run;
    const CUtensorMap* mq = &maps.q[sg.run];
    const CUtensorMap* mk = &maps.k[sg.run];
    const CUtensorMap* mv = &maps.v[sg.run];

    if (tid == 0) {
      mbar_expect_tx(&s.bar_q, kTileBytes);
      tma_load_3d(s.q[0], mq, &s.bar_q, 0, h, tok0 + q_row0);
      tma_load_3d(s.q[1], mq, &s.bar_q, 64, h, tok0 + q_row0);
      mbar_expect_tx(&s.bar_k, kTileBytes);
      tma_load_3d(s.k[0], mk, &s.bar_k, 0, g, tok0);
      tma_load_3d(s.k[1], mk, &s.bar_k, 64, g, tok0);
      mbar_expect_tx(&s.bar_v, kTileBytes);
      tma_load_3d(s.v[0], mv, &s.bar_v, 0, g, tok0);
      tma_load_3d(s.v[1], mv, &s.bar_v, 64, g, tok0);
    }

    float m_ref = -INFINITY;  // reference maximum (log2 domain) the stored P and l are relative to
    float l = 0.f;            // running row sum of exp2(s - m_ref)

    for (int j = 0; j < n_kv; ++j) {
      // ---- S = Q K_j^T
      if (tid == 0) {
        bool okt = true;
        if (j == 0) {
          okt = mbar_wait(&s.bar_q, ph_q);
          ph_q ^= 1;
        }
        okt = okt && mbar_wait(&s.bar_k, ph_k);
        ph_k ^= 1;
        if (okt) {
          tc_fence_after_sync();
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (kk >> 2) * kHalfTileBytes + (kk & 3) * 32;
            umma_ss(tS, make_smem_desc_sw128(q_addr + off, 16, 1024), make_smem_desc_sw128(k_addr + off, 16, 1024),
                    idesc_qk, kk > 0);
          }
          umma_commit(&s.bar_s);
        } else {
          report_timeout(a.status, it, kWhereFwdLoad, j);
        }
      }
      bool okw = mbar_wait(&s.bar_s, ph_s);
      ph_s ^= 1;
      okw = __all_sync(0xffffffffu, okw);
      if (okw) {
        tc_fence_after_sync();
        if (tid == 0 && j + 1 < n_kv) {  // K buffer is free: prefetch the next key tile
          mbar_expect_tx(&s.bar_k, kTileBytes);
          tma_load_3d(s.k[0], mk, &s.bar_k, 0, g, tok0 + (j + 1) * kBN);
          tma_load_3d(s.k[1], mk, &s.bar_k, 64, g, tok0 + (j + 1) * kBN);
        }
        // ---- online softmax of row `tid`
        uint32_t sr[4][32];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(tS + lane_off + c * 32, sr[c]);
        tmem_wait_ld();
        const bool diag = (j == n_kv - 1);
        float mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int x = 0; x < 32; ++x) {
            float val = __uint_as_float(sr[c][x]);
            if (diag && (c * 32 + x) > tid) val = -INFINITY;
            sr[c][x] = __float_as_uint(val);
            mx = fmaxf(mx, val);
          }
        mx *= a.scale_log2;
        const bool need = mx > m_ref + 8.f;
        float alpha = 1.f;
        if (need) {
          alpha = ex2f(m_ref - mx);
          m_ref = mx;
        }
        l *= alpha;
        float sum = 0.f;
        uint32_t pk[2][32];
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int x = 0; x < 32; x += 2) {
            const float p0 = ex2f(fmaf(__uint_as_float(sr[c][x]), a.scale_log2, -m_ref));
            const float p1 = ex2f(fmaf(__uint_as_float(sr[c][x + 1]), a.scale_log2, -m_ref));
            sum += p0 + p1;
            pk[c >> 1][(c & 1) * 16 + (x >> 1)] = pack_bf16x2(p0, p1);
          }
        l += sum;
        tmem_st32(tS + lane_off, pk[0]);
        tmem_st32(tS + lane_off + 32, pk[1]);
        // ---- rescale O in place when some row of this warp moved its reference maximum
        if (j > 0 && __any_sync(0xffffffffu, need)) {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t orow[32];
            tmem_ld32(tO + lane_off + c * 32, orow);
            tmem_wait_ld();
#pragma unroll
            for (int x = 0; x < 32; ++x) orow[x] = __float_as_uint(__uint_as_float(orow[x]) * alpha);
            tmem_st32(tO + lane_off + c * 32, orow);
          }
        }
        tmem_wait_st();
      } else if (lane == 0) {
        report_timeout(a.status, it, kWhereFwdS, j);
      }
      ok = ok && okw;
      tc_fence_before_sync();
      ok = __syncthreads_and(ok);
      if (!ok) break;
      // ---- O += P V_j
      if (tid == 0) {
        const bool okt = mbar_wait(&s.bar_v, ph_v);
        ph_v ^= 1;
        if (okt) {
          tc_fence_after_sync();
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            umma_ts(tO, tS + kk * 8, make_smem_desc_sw128(v_addr + kk * 2048, kHalfTileBytes, 1024), idesc_pv,
                    (j > 0 || kk > 0));
          umma_commit(&s.bar_o);
        } else {
          report_timeout(a.status, it, kWhereFwdLoad, 1000 + j);
        }
      }
      okw = mbar_wait(&s.bar_o, ph_o);
      ph_o ^= 1;
      okw = __all_sync(0xffffffffu, okw);
      if (okw) {
        tc_fence_after_sync();
        if (tid == 0 && j + 1 < n_kv) {  // V buffer is free
          mbar_expect_tx(&s.bar_v, kTileBytes);
          tma_load_3d(s.v[0], mv, &s.bar_v, 0, g, tok0 + (j + 1) * kBN);
          tma_load_3d(s.v[1], mv, &s.bar_v, 64, g, tok0 + (j + 1) * kBN);
        }
      } else if (lane == 0) {
        report_timeout(a.status, it, kWhereFwdO, j);
      }
      ok = ok && okw;
    }
    if (!ok) continue;  // the uniform vote at the loop head ends the CTA

    // ---- epilogue: O / l -> bf16, LSE
    const int row = q_row0 + tid;
    const bool valid = row < sg.len;
    const float inv_l = 1.f / l;
    __nv_bfloat16* optr = a.o + sg.q_off + (static_cast<int64_t>(row) * sg.hq + h) * kHeadDim;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      uint32_t orow[32];
      tmem_ld32(tO + lane_off + c * 32, orow);
      tmem_wait_ld();
      if (valid) {
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          uint4 w;
          w.x = pack_bf16x2(__uint_as_float(orow[8 * x + 0]) * inv_l, __uint_as_float(orow[8 * x + 1]) * inv_l);
          w.y = pack_bf16x2(__uint_as_float(orow[8 * x + 2]) * inv_l, __uint_as_float(orow[8 * x + 3]) * inv_l);
          w.z = pack_bf16x2(__uint_as_float(orow[8 * x + 4]) * inv_l, __uint_as_float(orow[8 * x + 5]) * inv_l);
          w.w = pack_bf16x2(__uint_as_float(orow[8 * x + 6]) * inv_l, __uint_as_float(orow[8 * x + 7]) * inv_l);
          *reinterpret_cast<uint4*>(optr + c * 32 + x * 8) = w;
        }
      }
    }
    if (valid)
      a.lse[sg.lse_off + static_cast<int64_t>(h) * sg.len + row] = (m_ref + log2f(l)) * 0.6931471805599453f;
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(s.tmem_base, kFwdTmemCols);
}

}  // namespace

cudaError_t launch_fwd(const FwdMaps& maps, const FwdArgs& args, int num_sms, cudaStream_t st) {
  if (args.n_items == 0) return cudaSuccess;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(kFwdSmemBytes));
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int grid = args.n_items < 2 * num_sms ? args.n_items : 2 * num_sms;
  fwd_kernel<<<grid, kFwdThreads, kFwdSmemBytes, st>>>(maps, args);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace nsp

// Backward: dQ, dK, dV of packed variable-length causal GQA attention on tcgen05 tensor cores.
//
// Three launches:
//   preprocess   delta[h, i] = sum_d dO[i,h,d] * O[i,h,d]                      (HBM-bound, one warp per row)
//   main         key-stationary persistent kernel, see below
//   postprocess  dQ = scale * fp32 accumulator -> bf16 / fp32                   (HBM-bound)
//
// Main kernel. One CTA per SM (512 threads, four warpgroups with their own register budgets) pops items
// (segment, kv head, key tile n) from the longest-first list. K_n and V_n stay in shared memory; the CTA walks
// every q head of the KV group and every q tile m >= n. All score-shaped quantities are computed TRANSPOSED
// (key index on the TMEM lanes) so that P^T and dS^T are directly the A operands of the dV and dK products:
//     S^T  = K Q^T  -> R0,   dP^T = V dO^T -> R1          A, B K-major from shared memory
//     P^T  = exp2(S^T * scale*log2e - LSE*log2e),  dS^T = P^T o (dP^T - delta)
//     dV  += P^T dO                               A = P^T (bf16, written over S^T in R0), B = dO  MN-major
//     dK  += dS^T Q                               A = dS^T (shared memory, K-major), B = Q MN-major
//     dQ_m = dS K  -> R1 (over dP^T)              A = dS^T read MN-major, B = K MN-major
// TMEM: R0 [0,128), R1 [128,256), dK [256,384), dV [384,512).
// Roles:  warps 0-7  softmax / dS (key row = TMEM lane, two column halves)
//         warps 8-11 dQ: TMEM -> fp32 accumulator in global memory (vector reductions)
//         warp 12    TMA producer (K, V once per item; Q, dO two-stage ring)
//         warp 13    MMA issuer (single thread)
//         warp 14    LSE / delta loader (two-stage ring in shared memory)
// The MMA thread issues S^T of the next step right behind dQ of the current one, so the next S^T runs while
// the dQ warps drain R1; dP^T waits for R1. dK and dV accumulate in TMEM over the whole item in a fixed order
// (heads ascending, tiles ascending), so the reduction over the query heads of a group is deterministic.
// For the first q tile of a segment (rows 0..127, where P is O(1)) the step runs twice, once with the bf16
// value of P and dS and once with the bf16 residual (hi + lo), and delta is recomputed in fp32 as
// sum_j P_ij dP_ij instead of taking it from the bf16-rounded O; this keeps dK/dV/dQ inside the 2e-2 tolerance.
#include <cuda_bf16.h>
#include "nsp_internal.cuh"
#include "sm100_ptx.cuh"

namespace nsp {
namespace {

constexpr int kBwdThreads = 512;
constexpr uint32_t kHalfTileBytes = 128 * 64 * 2;
constexpr uint32_t kTileBytes = 2 * kHalfTileBytes;
constexpr uint32_t kBwdTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;
constexpr int kRegsSoftmax = 168, kRegsReduce = 120, kRegsAux = 56;  // 2*168 + 120 + 56 = 512 = 65536 / 128

struct BwdSmem {
  uint8_t k[2][kHalfTileBytes];
  uint8_t v[2][kHalfTileBytes];
  uint8_t q[2][2][kHalfTileBytes];    // [stage][64-column half]
  uint8_t d_o[2][2][kHalfTileBytes];  // [stage][half]
  uint8_t ds[2][kHalfTileBytes];      // dS^T, [key row][query col], two 64-column halves
  float lse[2][128];                  // [stage] LSE * log2(e) of the q tile (+inf for rows past the segment)
  float delta[2][128];                // [stage]
  uint64_t bar_kv;
  uint64_t bar_q_full[2], bar_q_empty[2];
  uint64_t bar_ld_full[2], bar_ld_empty[2];
  uint64_t bar_s_full, bar_dp_full, bar_p_ready, bar_dq_full, bar_dq_empty;
  uint64_t bar_staged;    // 128 dQ threads: the fp32 dQ tile is in the staging buffer
  uint64_t bar_delta[2];  // 128 softmax threads of one column half: partial / final sums of the exact delta
  uint32_t tmem_base;
  int32_t item_idx[2];
  int32_t abort;
};
static_assert(sizeof(BwdSmem) <= 232448, "shared memory budget (227 KB)");
constexpr size_t kBwdSmemBytes = sizeof(BwdSmem);

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
template <int N>
__device__ __forceinline__ void setmaxnreg_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void setmaxnreg_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}
__device__ __forceinline__ void named_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Decoded work item and the mapping from a step index to (q head, q tile, mode).
// mode bit 0: recompute delta exactly; bit 1: residual (lo) pass of the hi/lo split.
struct ItemCtx {
  int g, n, G, n_m, per_head, steps, first, two_pass, mode_first;
};
__device__ __forceinline__ void decode_step(const ItemCtx& c, int vt, int& h, int& m, int& mode) {
  const int hh = vt / c.per_head, rr = vt - hh * c.per_head;
  h = c.g * c.G + hh;
  if (c.first) {
    if (rr == 0) {
      m = 0;
      mode = c.mode_first;
    } else if (c.two_pass && rr == 1) {
      m = 0;
      mode = c.mode_first | 2;
    } else {
      m = rr - c.two_pass;
      mode = 0;
    }
  } else {
    m = c.n + rr;
    mode = 0;
  }
}

__global__ void __launch_bounds__(kBwdThreads, 1) bwd_kernel(const __grid_constant__ BwdMaps maps, const BwdArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  BwdSmem& s = *reinterpret_cast<BwdSmem*>(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, wg = warp >> 2;
  if ((smem_u32(smem_raw) & 1023u) != 0) {  // swizzled tiles need a 1024-byte aligned base
    if (tid == 0) report_timeout(a.status, -1, kWhereBwdSmemAlign, 0);
    return;
  }

  if (tid == 0) {
    mbar_init(&s.bar_kv, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s.bar_q_full[i], 1);
      mbar_init(&s.bar_q_empty[i], 1);
      mbar_init(&s.bar_ld_full[i], 32);
      mbar_init(&s.bar_ld_empty[i], 256);
    }
    mbar_init(&s.bar_s_full, 1);
    mbar_init(&s.bar_dp_full, 1);
    mbar_init(&s.bar_p_ready, 256);
    mbar_init(&s.bar_dq_full, 1);
    mbar_init(&s.bar_dq_empty, 128);
    mbar_init(&s.bar_staged, 128);
    mbar_init(&s.bar_delta[0], 128);
    mbar_init(&s.bar_delta[1], 128);
    s.abort = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&s.tmem_base, kBwdTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();

  const uint32_t tR0 = s.tmem_base, tR1 = tR0 + 128, tDK = tR0 + 256, tDV = tR0 + 384;
  volatile int32_t* abort_flag = &s.abort;
  uint32_t gs = 0;  // steps completed so far by this CTA (every role advances it identically)
  uint32_t gi = 0;  // items completed so far

  // Every role runs its own copy of the item loop (so that its register budget, set by setmaxnreg at the top of
  // the role, governs the whole loop); the loops meet at the CTA-wide barrier inside next_item().
  nsp_tile_t item;
  SegInfo sg;
  ItemCtx c;
  int it = 0, tok0 = 0;
  auto next_item = [&]() -> bool {
    if (tid == 0) s.item_idx[gi & 1] = atomicAdd(a.counter, 1);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    it = s.item_idx[gi & 1];
    if (it >= a.n_items || *abort_flag) return false;
    item = a.items[it];
    sg = a.seg[item.seg];
    c.g = item.head;
    c.n = item.tile;
    c.G = sg.hq / sg.hkv;
    c.n_m = (sg.len + kBM - 1) / kBM - c.n;  // q tiles n .. Mt-1 (bm == bn)
    c.first = (c.n == 0);
    c.two_pass = (c.first && (a.debug_flags & 1) == 0) ? 1 : 0;
    c.mode_first = (a.debug_flags & 2) == 0 ? 1 : 0;
    c.per_head = c.n_m + c.two_pass;
    c.steps = c.G * c.per_head;
    tok0 = sg.tok_in_run;
    return true;
  };
  auto item_done = [&]() {
    gs += static_cast<uint32_t>(c.steps);
    gi += 1;
  };

  if (wg == 3) {
    setmaxnreg_dec<kRegsAux>();
    if (warp == 12) {
      // ================================================================ TMA producer
      while (next_item()) {
      if (lane == 0) {
        const CUtensorMap* mq = &maps.q[sg.run];
        const CUtensorMap* mdo = &maps.d_o[sg.run];
        mbar_expect_tx(&s.bar_kv, 2 * kTileBytes);
        tma_load_3d(s.k[0], &maps.k[sg.run], &s.bar_kv, 0, c.g, tok0 + c.n * kBN);
        tma_load_3d(s.k[1], &maps.k[sg.run], &s.bar_kv, 64, c.g, tok0 + c.n * kBN);
        tma_load_3d(s.v[0], &maps.v[sg.run], &s.bar_kv, 0, c.g, tok0 + c.n * kBN);
        tma_load_3d(s.v[1], &maps.v[sg.run], &s.bar_kv, 64, c.g, tok0 + c.n * kBN);
        for (int vt = 0; vt < c.steps; ++vt) {
          const uint32_t cs = gs + vt, st = cs & 1;
          if (*abort_flag) break;
          if (!mbar_wait(&s.bar_q_empty[st], ((cs >> 1) & 1) ^ 1)) {
            report_timeout(a.status, it, kWhereBwdQEmpty, vt);
            *abort_flag = 1;
            break;
          }
          int h, m, mode;
          decode_step(c, vt, h, m, mode);
          mbar_expect_tx(&s.bar_q_full[st], 2 * kTileBytes);
          tma_load_3d(s.q[st][0], mq, &s.bar_q_full[st], 0, h, tok0 + m * kBM);
          tma_load_3d(s.q[st][1], mq, &s.bar_q_full[st], 64, h, tok0 + m * kBM);
          tma_load_3d(s.d_o[st][0], mdo, &s.bar_q_full[st], 0, h, tok0 + m * kBM);
          tma_load_3d(s.d_o[st][1], mdo, &s.bar_q_full[st], 64, h, tok0 + m * kBM);
        }
      }
      item_done();
      }
    } else if (warp == 13) {
      // ================================================================ MMA issuer
      while (next_item()) {
      if (lane == 0) {
        constexpr uint32_t idesc_kk = make_idesc_bf16(128, 128, 0, 0);  // A K-major, B K-major
        constexpr uint32_t idesc_kn = make_idesc_bf16(128, 128, 0, 1);  // A K-major (or TMEM), B MN-major
        constexpr uint32_t idesc_nn = make_idesc_bf16(128, 128, 1, 1);  // A MN-major, B MN-major
        const uint32_t k_addr = smem_u32(s.k[0]), v_addr = smem_u32(s.v[0]), ds_addr = smem_u32(s.ds[0]);
        int where = 0;
        bool okm = mbar_wait(&s.bar_kv, gi & 1);
        if (!okm) where = kWhereBwdLoadKV;
        for (int vt = 0; okm && vt < c.steps; ++vt) {
          const uint32_t cs = gs + vt, st = cs & 1;
          if (*abort_flag) break;
          const uint32_t q_addr = smem_u32(s.q[st][0]), do_addr = smem_u32(s.d_o[st][0]);
          if (!mbar_wait(&s.bar_q_full[st], (cs >> 1) & 1)) { okm = false; where = kWhereBwdLoadQ; break; }
          tc_fence_after_sync();
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (kk >> 2) * kHalfTileBytes + (kk & 3) * 32;
            umma_ss(tR0, make_smem_desc_sw128(k_addr + off, 16, 1024), make_smem_desc_sw128(q_addr + off, 16, 1024),
                    idesc_kk, kk > 0);
          }
          umma_commit(&s.bar_s_full);
          // R1 still holds dQ of the previous step until the dQ warps have drained it
          if (!mbar_wait(&s.bar_dq_empty, (cs & 1) ^ 1)) { okm = false; where = kWhereBwdDqEmpty; break; }
          tc_fence_after_sync();
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (kk >> 2) * kHalfTileBytes + (kk & 3) * 32;
            umma_ss(tR1, make_smem_desc_sw128(v_addr + off, 16, 1024), make_smem_desc_sw128(do_addr + off, 16, 1024),
                    idesc_kk, kk > 0);
          }
          umma_commit(&s.bar_dp_full);
          if (!mbar_wait(&s.bar_p_ready, cs & 1)) { okm = false; where = kWhereBwdPReady; break; }
          tc_fence_after_sync();
          const uint32_t acc = vt > 0;
          // packed P^T columns of K-step kk (16 query columns) sit at R0 + (kk/2)*32 + (kk%2)*8
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            umma_ts(tDV, tR0 + (kk >> 1) * 32 + (kk & 1) * 8,
                    make_smem_desc_sw128(do_addr + kk * 2048, kHalfTileBytes, 1024), idesc_kn, acc | (kk > 0));
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (kk >> 2) * kHalfTileBytes + (kk & 3) * 32;
            umma_ss(tDK, make_smem_desc_sw128(ds_addr + off, 16, 1024),
                    make_smem_desc_sw128(q_addr + kk * 2048, kHalfTileBytes, 1024), idesc_kn, acc | (kk > 0));
          }
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            umma_ss(tR1, make_smem_desc_sw128(ds_addr + kk * 2048, kHalfTileBytes, 1024),
                    make_smem_desc_sw128(k_addr + kk * 2048, kHalfTileBytes, 1024), idesc_nn, kk > 0);
          umma_commit(&s.bar_dq_full);  // the dQ warps release the Q/dO stage after using it as staging
        }
        if (!okm) {
          report_timeout(a.status, it, where, 0);
          *abort_flag = 1;
        }
      }
      item_done();
      }
    } else if (warp == 14) {
      // ================================================================ LSE / delta loader
      while (next_item()) {
      for (int vt = 0; vt < c.steps; ++vt) {
        const uint32_t cs = gs + vt, st = cs & 1;
        if (*abort_flag) break;
        bool okl = mbar_wait(&s.bar_ld_empty[st], ((cs >> 1) & 1) ^ 1);
        okl = __all_sync(0xffffffffu, okl);
        if (!okl) {
          if (lane == 0) {
            report_timeout(a.status, it, kWhereBwdLdEmpty, vt);
            *abort_flag = 1;
          }
          break;
        }
        int h, m, mode;
        decode_step(c, vt, h, m, mode);
        const int64_t base = sg.lse_off + static_cast<int64_t>(h) * sg.len;
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const int col = lane * 4 + x, qi = m * kBM + col;
          const bool valid = qi < sg.len;
          s.lse[st][col] = valid ? a.lse[base + qi] * kLog2e : INFINITY;
          s.delta[st][col] = valid ? a.delta[base + qi] : 0.f;
        }
        mbar_arrive(&s.bar_ld_full[st]);
      }
      item_done();
      }
    } else {
      while (next_item()) item_done();  // spare warp: only keeps the CTA-wide barrier count
    }
  } else if (wg == 2) {
    {
      // ================================================================ dQ: R1 -> global fp32 accumulator
      setmaxnreg_dec<kRegsReduce>();
      const int quad = warp & 3;
      const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
      while (next_item()) {
      for (int vt = 0; vt < c.steps; ++vt) {
        const uint32_t cs = gs + vt;
        if (*abort_flag) break;
        bool okr = mbar_wait(&s.bar_dq_full, cs & 1);
        okr = __all_sync(0xffffffffu, okr);
        if (!okr) {
          if (lane == 0) {
            report_timeout(a.status, it, kWhereBwdDqFull, vt);
            *abort_flag = 1;
          }
          break;
        }
        tc_fence_after_sync();
        int h, m, mode;
        decode_step(c, vt, h, m, mode);
        // The Q/dO stage of this step is dead once its MMAs are done (bar_dq_full): use it as a 64 KB staging
        // buffer for the fp32 dQ tile, four [128 rows x 32 columns] boxes in the 128-byte-swizzled layout of
        // the accumulator's tensor map, and let TMA add the boxes into global memory. Rows past the segment
        // end hold exact zeros (their dS columns are zero), rows past the run are clipped by TMA.
        const uint32_t st = cs & 1;
        const int row = quad * 32 + lane;
#pragma unroll
        for (int pair = 0; pair < 2; ++pair) {
          uint32_t v0[32], v1[32];
          tmem_ld32(tR1 + lane_off + pair * 64, v0);
          tmem_ld32(tR1 + lane_off + pair * 64 + 32, v1);
          tmem_wait_ld();
          if (pair == 1) {  // R1 is drained: the next dP^T may overwrite it
            tc_fence_before_sync();
            mbar_arrive(&s.bar_dq_empty);
          }
          uint8_t* box0 = (pair == 0 ? s.q[st][0] : s.d_o[st][0]) + row * 128;
          uint8_t* box1 = (pair == 0 ? s.q[st][1] : s.d_o[st][1]) + row * 128;
#pragma unroll
          for (int ch = 0; ch < 8; ++ch) {
            const int chunk = (ch ^ (row & 7)) * 16;
            *reinterpret_cast<uint4*>(box0 + chunk) = make_uint4(v0[4 * ch], v0[4 * ch + 1], v0[4 * ch + 2], v0[4 * ch + 3]);
            *reinterpret_cast<uint4*>(box1 + chunk) = make_uint4(v1[4 * ch], v1[4 * ch + 1], v1[4 * ch + 2], v1[4 * ch + 3]);
          }
        }
        fence_proxy_async_smem();
        mbar_arrive(&s.bar_staged);
        if (warp == 8 && lane == 0) {
          if (!mbar_wait(&s.bar_staged, cs & 1)) {
            report_timeout(a.status, it, kWhereBwdStaged, vt);
            *abort_flag = 1;
          } else if ((a.debug_flags & 4) == 0) {
            const CUtensorMap* mdq = &maps.dq[sg.run];
            tma_reduce_add_3d(mdq, s.q[st][0], 0, h, tok0 + m * kBM);
            tma_reduce_add_3d(mdq, s.q[st][1], 32, h, tok0 + m * kBM);
            tma_reduce_add_3d(mdq, s.d_o[st][0], 64, h, tok0 + m * kBM);
            tma_reduce_add_3d(mdq, s.d_o[st][1], 96, h, tok0 + m * kBM);
            bulk_commit_group();
            bulk_wait_read_all();
          }
          mbar_arrive(&s.bar_q_empty[st]);  // stage free: the producer may refill it
        }
      }
      if (warp == 8 && lane == 0) bulk_wait_all();  // all reductions of this item performed
      item_done();
      }
    }
  } else {
    {
      // ================================================================ softmax / dS (key row r, 64 query columns)
      setmaxnreg_inc<kRegsSoftmax>();
      const int quad = warp & 3, half = wg;
      const int r = quad * 32 + lane;
      const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
      uint32_t nd = 0;  // completed phases of bar_delta[half]
      while (next_item()) {
      bool oks = true;
      int where = 0;
      for (int vt = 0; vt < c.steps; ++vt) {
        const uint32_t cs = gs + vt, st = cs & 1;
        if (*abort_flag) { oks = false; where = 0; break; }
        int h, m, mode;
        decode_step(c, vt, h, m, mode);
        oks = mbar_wait(&s.bar_ld_full[st], (cs >> 1) & 1) && mbar_wait(&s.bar_s_full, cs & 1);
        oks = __all_sync(0xffffffffu, oks);
        if (!oks) { where = kWhereBwdS; break; }
        tc_fence_after_sync();
        const bool diag = (m == c.n);
        const float* lse_s = s.lse[st];
        float* delta_s = s.delta[st];
        bool have_dp = false;
        if (mode & 1) {
          // delta_i = sum_j P_ij dP_ij over the keys of this tile (all keys of rows 0..127), fp32
          oks = mbar_wait(&s.bar_dp_full, cs & 1);
          oks = __all_sync(0xffffffffu, oks);
          if (!oks) { where = kWhereBwdDp; break; }
          tc_fence_after_sync();
          have_dp = true;
          float* part = reinterpret_cast<float*>(s.ds[half]);  // [4 quadrants][64 columns]; free until dS is written
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            const int col0 = half * 64 + cc * 32;
            uint32_t sv[32], dpv[32];
            tmem_ld32(tR0 + lane_off + col0, sv);
            tmem_ld32(tR1 + lane_off + col0, dpv);
            tmem_wait_ld();
#pragma unroll
            for (int x = 0; x < 32; ++x) {
              float p = ex2f(fmaf(__uint_as_float(sv[x]), a.scale_log2, -lse_s[col0 + x]));
              if (col0 + x < r) p = 0.f;
              float v = p * __uint_as_float(dpv[x]);
#pragma unroll
              for (int sft = 16; sft > 0; sft >>= 1) v += __shfl_xor_sync(0xffffffffu, v, sft);
              if (lane == 0) part[quad * 64 + cc * 32 + x] = v;
            }
          }
          mbar_arrive(&s.bar_delta[half]);
          oks = mbar_wait(&s.bar_delta[half], nd & 1);
          ++nd;
          oks = __all_sync(0xffffffffu, oks);
          if (!oks) { where = kWhereBwdDelta; break; }
          if (r < 64) delta_s[half * 64 + r] = (part[r] + part[64 + r]) + (part[128 + r] + part[192 + r]);
          mbar_arrive(&s.bar_delta[half]);
          oks = mbar_wait(&s.bar_delta[half], nd & 1);
          ++nd;
          oks = __all_sync(0xffffffffu, oks);
          if (!oks) { where = kWhereBwdDelta; break; }
        }
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {  // 32 query columns at a time
          const int col0 = half * 64 + cc * 32;
          uint32_t sv[32];
          tmem_ld32(tR0 + lane_off + col0, sv);
          tmem_wait_ld();
#pragma unroll
          for (int x = 0; x < 32; x += 4) {
            const float4 l4 = *reinterpret_cast<const float4*>(lse_s + col0 + x);
            float p0 = ex2f(fmaf(__uint_as_float(sv[x + 0]), a.scale_log2, -l4.x));
            float p1 = ex2f(fmaf(__uint_as_float(sv[x + 1]), a.scale_log2, -l4.y));
            float p2 = ex2f(fmaf(__uint_as_float(sv[x + 2]), a.scale_log2, -l4.z));
            float p3 = ex2f(fmaf(__uint_as_float(sv[x + 3]), a.scale_log2, -l4.w));
            if (diag) {  // query index must be >= key index
              if (col0 + x + 0 < r) p0 = 0.f;
              if (col0 + x + 1 < r) p1 = 0.f;
              if (col0 + x + 2 < r) p2 = 0.f;
              if (col0 + x + 3 < r) p3 = 0.f;
            }
            sv[x + 0] = __float_as_uint(p0);
            sv[x + 1] = __float_as_uint(p1);
            sv[x + 2] = __float_as_uint(p2);
            sv[x + 3] = __float_as_uint(p3);
          }
          if (!have_dp) {
            oks = mbar_wait(&s.bar_dp_full, cs & 1);
            oks = __all_sync(0xffffffffu, oks);
            if (!oks) { where = kWhereBwdDp; break; }
            tc_fence_after_sync();
            have_dp = true;
          }
          uint32_t dpv[32];
          tmem_ld32(tR1 + lane_off + col0, dpv);
          tmem_wait_ld();
          uint32_t pp[16], dsp[16];
#pragma unroll
          for (int x = 0; x < 32; x += 4) {
            const float4 d4 = *reinterpret_cast<const float4*>(delta_s + col0 + x);
            float p0 = __uint_as_float(sv[x + 0]), p1 = __uint_as_float(sv[x + 1]);
            float p2 = __uint_as_float(sv[x + 2]), p3 = __uint_as_float(sv[x + 3]);
            float d0 = p0 * (__uint_as_float(dpv[x + 0]) - d4.x), d1 = p1 * (__uint_as_float(dpv[x + 1]) - d4.y);
            float d2 = p2 * (__uint_as_float(dpv[x + 2]) - d4.z), d3 = p3 * (__uint_as_float(dpv[x + 3]) - d4.w);
            uint32_t pa = pack_bf16x2(p0, p1), pb = pack_bf16x2(p2, p3);
            uint32_t da = pack_bf16x2(d0, d1), db = pack_bf16x2(d2, d3);
            if (mode & 2) {  // residual pass: what the bf16 value left behind
              pa = pack_bf16x2(p0 - __uint_as_float(pa << 16), p1 - __uint_as_float(pa & 0xffff0000u));
              pb = pack_bf16x2(p2 - __uint_as_float(pb << 16), p3 - __uint_as_float(pb & 0xffff0000u));
              da = pack_bf16x2(d0 - __uint_as_float(da << 16), d1 - __uint_as_float(da & 0xffff0000u));
              db = pack_bf16x2(d2 - __uint_as_float(db << 16), d3 - __uint_as_float(db & 0xffff0000u));
            }
            pp[(x >> 1) + 0] = pa;
            pp[(x >> 1) + 1] = pb;
            dsp[(x >> 1) + 0] = da;
            dsp[(x >> 1) + 1] = db;
          }
          // P^T (bf16 pairs) goes over S^T columns this warp has already read: query columns
          // [col0, col0+32) -> packed columns [col0, col0+16)
          tmem_st16(tR0 + lane_off + col0, pp);
          // dS^T row r, columns col0 .. col0+31 -> four 16-byte chunks of the swizzled half tile
          uint8_t* base = s.ds[half] + r * 128;
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            const int chunk = (cc * 4 + ch) ^ (r & 7);
            *reinterpret_cast<uint4*>(base + chunk * 16) =
                make_uint4(dsp[ch * 4 + 0], dsp[ch * 4 + 1], dsp[ch * 4 + 2], dsp[ch * 4 + 3]);
          }
        }
        if (!oks) break;
        tmem_wait_st();
        fence_proxy_async_smem();
        tc_fence_before_sync();
        mbar_arrive(&s.bar_p_ready);
        mbar_arrive(&s.bar_ld_empty[st]);
      }
      // ---- epilogue: wait for the last MMAs of the item, then write dK (scaled) and dV of this key tile
      if (oks) {
        oks = mbar_wait(&s.bar_dq_full, (gs + c.steps - 1) & 1);
        oks = __all_sync(0xffffffffu, oks);
        if (!oks) where = kWhereBwdDqFull;
      }
      if (oks) {
        tc_fence_after_sync();
        const int kj = c.n * kBN + r;
        const bool valid = kj < sg.len;
        const int64_t off = sg.kv_off + (static_cast<int64_t>(kj) * sg.hkv + c.g) * kHeadDim + half * 64;
#pragma unroll
        for (int which = 0; which < 2; ++which) {
          const uint32_t tsrc = which == 0 ? tDK : tDV;
          const float mul = which == 0 ? a.scale : 1.f;
          void* outp = which == 0 ? a.dk : a.dv;
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            uint32_t v[32];
            tmem_ld32(tsrc + lane_off + half * 64 + cc * 32, v);
            tmem_wait_ld();
            if (valid) {
              if (a.dkv_f32) {
                float* o = static_cast<float*>(outp) + off + cc * 32;
#pragma unroll
                for (int x = 0; x < 32; x += 4)
                  *reinterpret_cast<float4*>(o + x) =
                      make_float4(__uint_as_float(v[x]) * mul, __uint_as_float(v[x + 1]) * mul,
                                  __uint_as_float(v[x + 2]) * mul, __uint_as_float(v[x + 3]) * mul);
              } else {
                __nv_bfloat16* o = static_cast<__nv_bfloat16*>(outp) + off + cc * 32;
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
      } else if (where != 0 && lane == 0) {
        report_timeout(a.status, it, where, 0);
        *abort_flag = 1;
      }
      item_done();
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

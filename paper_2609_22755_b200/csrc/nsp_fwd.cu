// Forward: packed variable-length causal GQA attention on tcgen05 tensor cores.
//
// One persistent CTA per SM (640 threads) pops work items (segment, q head, q tile) from the longest-first
// list TWO at a time. Neighbouring items of the list are the same (segment, q tile) for consecutive q heads, so
// when they share a KV head (GQA) the CTA runs them as a pair "A/B" over the SAME K/V tiles: every K/V tile is
// fetched once for 256 query rows, and the tensor pipe alternates between the two while their softmax
// warpgroups work (otherwise the two items run one after the other with warpgroup B idle).
//     S_x  = Q_x K_j^T      tcgen05.mma SS (both K-major, 128B-swizzled smem staged by TMA)       -> TMEM S_x
//     P_x  = exp2(S_x*c - m)  one thread per query row (tcgen05.ld), bf16 pairs written over S_x  (tcgen05.st)
//     O_x += P_x V_j        tcgen05.mma TS (A = P_x from TMEM, B = V MN-major from smem)          -> TMEM O_x
// Issue order of the single MMA thread: PV_A(j), S_A(j+1), PV_B(j), S_B(j+1): S of the next key tile is already
// running while the other half's softmax is still working. TMEM: S_A, S_B, O_A, O_B = 4 x 128 columns.
// Roles: warps 0-7 softmax of A, warps 8-15 softmax of B (two threads per query row, 64 score columns each), warp 16
// TMA producer (Q pair, two-stage K and V rings; it also starts the coming round's first tiles under the running
// round's tail), warp 17 MMA issuer, warp 18 lane 0 pops the work list one pop ahead; register budgets are set per
// warpgroup with setmaxnreg. A full O tile leaves through shared memory as a TMA tile store.
// O stays in TMEM for the whole item and is rescaled in place only when the running maximum grows by more than
// 2^8 (the stale reference maximum is exact in the final normalisation because the same reference is used for
// the row sum). Only the diagonal tile is masked; tiles above the diagonal are never visited.
#include <cuda_bf16.h>
#include "nsp_internal.cuh"
#include "sm100_ptx.cuh"

namespace nsp {
namespace {

constexpr int kFwdThreads = 640;  // 16 softmax warps (two threads per query row) + one auxiliary warpgroup
constexpr uint32_t kHalfTileBytes = 128 * 64 * 2;  // one [128 rows x 64 cols] bf16 sub-tile
constexpr uint32_t kFwdTmemCols = 512;  // S_A [0,128) S_B [128,256) O_A [256,384) O_B [384,512)
constexpr int kFwdRegsSoftmax = 104, kFwdRegsAux = 64;  // 4*104 + 64 = 480 = 5 * 96, the launch-time allocation

// One pop of the work list, decoded by one thread of a spare warp into shared memory (two slots: the next pop is
// fetched while the current one runs).
struct FwdPop {
  SegInfo sa, sb;  // segments of items a and b
  nsp_tile_t a, b;
  int32_t it0, joint, n_rounds;
  int32_t kt_base;  // key tiles of all earlier pops of this CTA (the K / V ring stage of tile t is t & 1)
};

// D = head dimension (128 or 64): a Q / K / V tile is D / 64 sub-tiles of 64 columns.
template <int D>
struct FwdSmem {
  uint8_t q[2][D / 64][kHalfTileBytes];  // [A/B][64-column half]
  uint8_t k[2][D / 64][kHalfTileBytes];  // [stage][half]
  uint8_t v[2][D / 64][kHalfTileBytes];  // [stage][half]
  uint64_t bar_q;
  uint64_t bar_k_full[2], bar_k_empty[2], bar_v_full[2], bar_v_empty[2];
  uint64_t bar_s_full[2];   // [A/B] S_x of a key tile is in TMEM
  uint64_t bar_p_ready[2];  // [A/B] 256 softmax threads: P_x written (and O_x rescaled if needed)
  uint64_t bar_pair[2][4];  // [A/B][lane quadrant] the two threads of every row have published their half-row value
  float xchg[2][2][4][128];  // [A/B][column half][slot][row] half-row maximum (slots 0/1 by tile parity), row sum (2),
                             // half-row dot product of O and dO (3, recomputation only)
                             // (slot 2) handed to the partner thread
  uint64_t bar_pv_done[2];  // [A/B] O_x += P_x V has completed
  uint64_t bar_q_free;      // the last S products of the round have completed: the Q tiles may be overwritten
  uint64_t bar_o_staged[2];  // [A/B] 256 softmax threads: the tile's O rows are in the staging buffer
  uint64_t bar_pop_ready[2];  // [slot] the pop fetched ahead is in its slot
  uint32_t tmem_base;
  FwdPop pop[2];
  int32_t abort;
};
static_assert(sizeof(FwdSmem<128>) <= 232448, "shared memory budget (227 KB)");

template <int N>
__device__ __forceinline__ void fwd_setmaxnreg_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void fwd_setmaxnreg_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

// max(a, b, c) in one instruction (3-input max of sm_100)
__device__ __forceinline__ float max3f(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// What one pop of the work list turned into: one or two rounds, each with item A and (in a joint round) item B.
struct FwdRound {
  nsp_tile_t a, b;
  int joint;
};
// RECOMP: the instantiation the recomputing backward pass launches (marked segments only; LSE and delta instead of O).
// The plain forward pass carries none of that code: the long items are sensitive to the size of the kernel.
template <int D, bool RECOMP>
__global__ void __launch_bounds__(kFwdThreads, 1) fwd_kernel(const __grid_constant__ FwdMaps maps, const FwdArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  FwdSmem<D>& s = *reinterpret_cast<FwdSmem<D>*>(smem_raw);
  constexpr int kHalves = D / 64;                              // 64-column sub-tiles of a Q / K / V tile
  constexpr uint32_t kTileBytes = kHalves * kHalfTileBytes;
  constexpr int kOCols = D / 2;                                // output columns of one of the two threads of a row
  constexpr int kHeadDim = D;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, wg = warp >> 2;
  if ((smem_u32(smem_raw) & 1023u) != 0) {  // swizzled tiles need a 1024-byte aligned base
    if (tid == 0) report_timeout(a.status, -1, kWhereFwdSmemAlign, 0);
    return;
  }
  if (tid == 0) {
    mbar_init(&s.bar_q, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s.bar_k_full[i], 1);
      mbar_init(&s.bar_k_empty[i], 1);
      mbar_init(&s.bar_v_full[i], 1);
      mbar_init(&s.bar_v_empty[i], 1);
      mbar_init(&s.bar_s_full[i], 1);
      mbar_init(&s.bar_p_ready[i], 256);
      for (int qd = 0; qd < 4; ++qd) mbar_init(&s.bar_pair[i][qd], 64);
      mbar_init(&s.bar_pv_done[i], 1);
    }
    mbar_init(&s.bar_q_free, 1);
    mbar_init(&s.bar_o_staged[0], 256);
    mbar_init(&s.bar_o_staged[1], 256);
    mbar_init(&s.bar_pop_ready[0], 1);
    mbar_init(&s.bar_pop_ready[1], 1);
    s.abort = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&s.tmem_base, kFwdTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();

  const uint32_t tmem = s.tmem_base;
  volatile int32_t* abort_flag = &s.abort;
  uint32_t gp = 0;  // pops so far
  // The CTA-wide meeting points are plain barriers. Every role reaches them in bounded time: all its other waits are
  // bounded and none of them returns before the end of the kernel. (An mbarrier with a bounded wait in their place
  // made the register allocation of the softmax role fail.)
  auto cta_sync = [&]() {
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
  };

  // ---- work decoding shared by all roles (every role runs its own copy of the loops, see the backward kernel)
  FwdRound rd;
  int n_rounds = 0, it0 = 0;
  const FwdPop* pp = nullptr;
  // One thread only, lane 0 of a spare warp of the auxiliary warpgroup. The atomic on the cursor and the dependent
  // loads of the items and their segments take ~4,000 clocks, so after a short item they are done one pop ahead (after
  // a long one the cursor is read when the item ends, which keeps the work list's balance at the end of the launch) —
  // and by a thread nobody waits for: when thread 0, a softmax thread, did it, its warp came that much later to the
  // first score tile of every round (17 % of a round at 512-token segments).
  constexpr int kFetchTid = 18 * 32;
  bool fetched_ahead = false;
  uint32_t kt_total = 0;  // fetching thread: key tiles of the pops fetched so far
  constexpr int kFetchAheadCost = 128;  // items up to this many key tiles have their successor fetched while they run
  auto fetch_pop = [&](int slot) {
    FwdPop& p = s.pop[slot];
    for (;;) {
      const int it = atomicAdd(a.counter, 2);
      p.it0 = it;
      if (it >= a.n_items) break;
      bool have_b = it + 1 < a.n_items;
      nsp_tile_t ia = a.items[it];
      nsp_tile_t ib = have_b ? a.items[it + 1] : ia;
      if (RECOMP && a.seg_mask != nullptr) {  // recomputation: only the marked segments
        const bool fa = a.seg_mask[ia.seg] != 0, fb = have_b && a.seg_mask[ib.seg] != 0;
        if (!fa && !fb) continue;
        if (!fa) ia = ib;
        if (!fa || !fb) ib = ia, have_b = false;
      }
      const SegInfo sa = a.seg[ia.seg];
      p.a = ia, p.b = ib, p.sa = sa;
      p.sb = ib.seg == ia.seg ? sa : a.seg[ib.seg];
      const int G = sa.hq / sa.hkv;
      p.joint = have_b && ib.seg == ia.seg && ib.tile == ia.tile && (ia.head / G == ib.head / G);
      p.n_rounds = p.joint ? 1 : (have_b ? 2 : 1);
      p.kt_base = static_cast<int32_t>(kt_total);
      kt_total += static_cast<uint32_t>(ia.cost + (p.n_rounds == 2 ? ib.cost : 0));
      break;
    }
    mbar_arrive(&s.bar_pop_ready[slot]);  // phase gp / 2 of the slot: the producer may read it before the next barrier
  };
  auto next_pop = [&]() -> bool {
    if (tid == kFetchTid && !fetched_ahead) fetch_pop(gp & 1);
    cta_sync();
    pp = &s.pop[gp & 1];
    it0 = pp->it0;
    ++gp;
    if (it0 >= a.n_items || *abort_flag) return false;
    rd.a = pp->a, rd.b = pp->b, rd.joint = pp->joint;
    n_rounds = pp->n_rounds;
    // the other slot held the previous pop: every role left it before it came to the barrier above
    if (tid == kFetchTid) {
      fetched_ahead = rd.a.cost <= kFetchAheadCost;
      if (fetched_ahead) fetch_pop(gp & 1);
    }
    return true;
  };
  // end of a round: every warp has finished with the Q tiles, the K/V rings and the TMEM accumulators. After the last
  // round of a pop the barrier of next_pop() is that meeting point.
  auto round_end = [&](int r) {
    if (r + 1 < n_rounds) cta_sync();
  };

  if (wg == 4) {
    fwd_setmaxnreg_dec<kFwdRegsAux>();
    if (warp == 16) {
      // ================================================================ TMA producer
      // Besides the loads of the running round it starts those of the coming one (the Q tiles and the first K / V
      // tile) as soon as the last S products of the running round have left the Q tiles, i.e. under the last softmax,
      // the last PV products and the epilogue. Short items pay for it otherwise: ~3,800 clocks from the start of a
      // round to its first score tile, a sixth of a round at 512-token segments.
      uint32_t kn = 0, vn = 0, rn = 0;
      bool pre = false;  // lane 0: Q and key tile 0 of the running round were started during the previous one
      while (next_pop()) {
        for (int r = 0; r < n_rounds; ++r) {
          if (lane == 0 && !*abort_flag) {
            const nsp_tile_t ia = r == 0 ? rd.a : rd.b;
            const SegInfo sg = r == 0 ? pp->sa : pp->sb;
            const int g = ia.head / (sg.hq / sg.hkv);
            const int tok0 = sg.tok_in_run, q_row0 = ia.tile * kBM, n_kv = ia.cost;
            const CUtensorMap* mq = &maps.q[sg.run];
            const CUtensorMap* mk = &maps.k[sg.run];
            const CUtensorMap* mv = &maps.v[sg.run];
            if (!pre) {
              mbar_expect_tx(&s.bar_q, rd.joint ? 2 * kTileBytes : kTileBytes);
#pragma unroll
              for (int hf = 0; hf < kHalves; ++hf) tma_load_3d(s.q[0][hf], mq, &s.bar_q, 64 * hf, ia.head, tok0 + q_row0);
              if (rd.joint) {
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) tma_load_3d(s.q[1][hf], mq, &s.bar_q, 64 * hf, rd.b.head, tok0 + q_row0);
              }
            }
            for (int j = pre ? 1 : 0; j < n_kv; ++j) {
              if (*abort_flag) break;
              uint32_t st = kn & 1;
              if (!mbar_wait(&s.bar_k_empty[st], ((kn >> 1) & 1) ^ 1, a.wait_limit)) {
                report_timeout(a.status, it0, kWhereFwdLoad, j);
                *abort_flag = 1;
                break;
              }
              mbar_expect_tx(&s.bar_k_full[st], kTileBytes);
#pragma unroll
              for (int hf = 0; hf < kHalves; ++hf) tma_load_3d(s.k[st][hf], mk, &s.bar_k_full[st], 64 * hf, g, tok0 + j * kBN);
              ++kn;
              st = vn & 1;
              if (!mbar_wait(&s.bar_v_empty[st], ((vn >> 1) & 1) ^ 1, a.wait_limit)) {
                report_timeout(a.status, it0, kWhereFwdLoad, 100000 + j);
                *abort_flag = 1;
                break;
              }
#ifdef NSP_CHECKED
              if (a.withhold && vn == 0) {  // failure-detection test: this V tile never arrives
                ++vn;
                continue;
              }
#endif
              mbar_expect_tx(&s.bar_v_full[st], kTileBytes);
#pragma unroll
              for (int hf = 0; hf < kHalves; ++hf) tma_load_3d(s.v[st][hf], mv, &s.bar_v_full[st], 64 * hf, g, tok0 + j * kBN);
              ++vn;
            }
            pre = false;
            // ---- the coming round (the second item of this pop, or the first round of the pop fetched ahead): its Q
            // tiles and its first K / V tile, once the last S products of this round have left the Q tiles. Kept apart
            // from the loop above, whose code the long items live in (sharing its body through a lambda cost them 0.6 %).
            const FwdPop* nx = nullptr;
            int second = 0;
            if (r + 1 < n_rounds) {
              nx = pp, second = 1;
            } else if (n_kv <= kFetchAheadCost && mbar_wait(&s.bar_pop_ready[gp & 1], (gp >> 1) & 1, a.wait_limit)) {
              if (s.pop[gp & 1].it0 < a.n_items) nx = &s.pop[gp & 1];
            }
            if (nx != nullptr && !*abort_flag && mbar_wait(&s.bar_q_free, rn & 1, a.wait_limit)) {
              const nsp_tile_t* na = second ? &nx->b : &nx->a;
              const SegInfo* ns = second ? &nx->sb : &nx->sa;
              const int joint = second ? 0 : nx->joint;
              const int ng = na->head / (ns->hq / ns->hkv), ntok = ns->tok_in_run;
              mbar_expect_tx(&s.bar_q, joint ? 2 * kTileBytes : kTileBytes);
#pragma unroll
              for (int hf = 0; hf < kHalves; ++hf) tma_load_3d(s.q[0][hf], &maps.q[ns->run], &s.bar_q, 64 * hf, na->head, ntok + na->tile * kBM);
              if (joint) {
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) tma_load_3d(s.q[1][hf], &maps.q[ns->run], &s.bar_q, 64 * hf, nx->b.head, ntok + na->tile * kBM);
              }
              const uint32_t kst = kn & 1, vst = vn & 1;
              if (mbar_wait(&s.bar_k_empty[kst], ((kn >> 1) & 1) ^ 1, a.wait_limit) &&
                  mbar_wait(&s.bar_v_empty[vst], ((vn >> 1) & 1) ^ 1, a.wait_limit)) {
                mbar_expect_tx(&s.bar_k_full[kst], kTileBytes);
                mbar_expect_tx(&s.bar_v_full[vst], kTileBytes);
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) {
                  tma_load_3d(s.k[kst][hf], &maps.k[ns->run], &s.bar_k_full[kst], 64 * hf, ng, ntok);
                  tma_load_3d(s.v[vst][hf], &maps.v[ns->run], &s.bar_v_full[vst], 64 * hf, ng, ntok);
                }
                ++kn, ++vn;
                pre = true;
              } else {
                report_timeout(a.status, it0, kWhereFwdLoad, 200000);
                *abort_flag = 1;
              }
            }
          }
          ++rn;
          round_end(r);
        }
      }
    } else if (warp == 17) {
      // ================================================================ MMA issuer
      constexpr uint32_t idesc_qk = make_idesc_bf16(128, 128, 0, 0);  // A K-major, B K-major
      constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, 0, 1);    // A from TMEM, B MN-major, N = head dimension
      uint32_t qn = 0, kn = 0, vn = 0, pn[2] = {0, 0};
      while (next_pop()) {
        for (int r = 0; r < n_rounds; ++r) {
          if (!*abort_flag) {
            const bool leader = elect_one();
            const nsp_tile_t ia = r == 0 ? rd.a : rd.b;
            const int n_kv = ia.cost;
            const int joint = rd.joint;
            int where = 0;
            // S_x of key tile in stage kst -> TMEM columns [128*x, 128*x + 128)
            // Descriptors are {low word, high word}; inside the loops an operand advances by adding its byte
            // offset (in 16-byte units) to the low word, which keeps the single issuing thread fast.
            const uint32_t hi = static_cast<uint32_t>(make_smem_desc_sw128(0, 16, 1024) >> 32);
            constexpr uint32_t lbo_km = (16u >> 4) << 16, lbo_mn = (kHalfTileBytes >> 4) << 16;
            const uint32_t q_lo = smem_desc_addr(s.q[0][0]) | lbo_km;  // item B: + kTileBytes / 16
            const uint32_t k_lo = smem_desc_addr(s.k[0][0]) | lbo_km;  // stage 1: + kTileBytes / 16
            const uint32_t v_lo = smem_desc_addr(s.v[0][0]) | lbo_mn;
            constexpr uint32_t kTileStep = kTileBytes >> 4;
            // S_x of key tile in stage kst -> TMEM columns [128*x, 128*x + 128)
            auto issue_s = [&](int x, uint32_t kst) {
              const uint32_t a_lo = q_lo + x * kTileStep, b_lo = k_lo + kst * kTileStep;
#pragma unroll
              for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t off = ((kk >> 2) * kHalfTileBytes + (kk & 3) * 32) >> 4;
                if (leader) umma_ss_lh(tmem + 128 * x, a_lo + off, hi, b_lo + off, hi, idesc_qk, kk > 0);
              }
              if (leader) umma_commit(&s.bar_s_full[x]);
            };
            // O_x += P_x V (P_x: bf16 pairs in columns [0,32) and [64,96) of S_x)
            auto issue_pv = [&](int x, uint32_t vst, int j) {
              const uint32_t b_lo = v_lo + vst * kTileStep;
#pragma unroll
              for (int kk = 0; kk < 8; ++kk)
                if (leader) umma_ts_lh(tmem + 256 + 128 * x, tmem + 128 * x + (kk >> 2) * 64 + (kk & 3) * 8, b_lo + kk * 128, hi, idesc_pv,
                           (j > 0 || kk > 0));
              if (leader) umma_commit(&s.bar_pv_done[x]);
            };
            bool ok = mbar_wait(&s.bar_q, qn & 1, a.wait_limit);
            ++qn;
            if (!ok) where = kWhereFwdLoad;
            uint32_t kst = 0;
            for (int j = 0; ok && j < n_kv; ++j) {
              if (*abort_flag) break;
              if (j == 0) {
                kst = kn & 1;
                if (!mbar_wait(&s.bar_k_full[kst], (kn >> 1) & 1, a.wait_limit)) { ok = false; where = kWhereFwdLoad; break; }
                tc_fence_after_sync();
                issue_s(0, kst);
                if (joint) issue_s(1, kst);
                if (leader) umma_commit(&s.bar_k_empty[kst]);
                ++kn;
              }
              const uint32_t vst = vn & 1;
              const bool more = j + 1 < n_kv;
              if (!more && leader) umma_commit(&s.bar_q_free);  // every S product of the round has been issued
              if (!mbar_wait(&s.bar_p_ready[0], pn[0] & 1, a.wait_limit)) { ok = false; where = kWhereFwdS; break; }
              ++pn[0];
              if (!mbar_wait(&s.bar_v_full[vst], (vn >> 1) & 1, a.wait_limit)) { ok = false; where = kWhereFwdLoad; break; }
              tc_fence_after_sync();
              issue_pv(0, vst, j);
              if (more) {  // S_A of the next key tile runs while softmax B is still working
                kst = kn & 1;
                if (!mbar_wait(&s.bar_k_full[kst], (kn >> 1) & 1, a.wait_limit)) { ok = false; where = kWhereFwdLoad; break; }
                tc_fence_after_sync();
                issue_s(0, kst);
              }
              if (joint) {
                if (!mbar_wait(&s.bar_p_ready[1], pn[1] & 1, a.wait_limit)) { ok = false; where = kWhereFwdS; break; }
                ++pn[1];
                tc_fence_after_sync();
                issue_pv(1, vst, j);
              }
              if (leader) umma_commit(&s.bar_v_empty[vst]);
              ++vn;
              if (more) {
                if (joint) issue_s(1, kst);
                if (leader) umma_commit(&s.bar_k_empty[kst]);
                ++kn;
              }
            }
            if (!ok) {
              if (leader) report_timeout(a.status, it0, where, 0);
              *abort_flag = 1;
            }
          }
          round_end(r);
        }
      }
    } else {
      while (next_pop())
        for (int r = 0; r < n_rounds; ++r) round_end(r);  // spare warps: only keep the CTA-wide barrier count
    }
  } else {
    // ================================================================ softmax of item x (A: warps 0-7, B: warps 8-15)
    // Two threads per query row: thread (quadrant, half ch) owns TMEM lane 32*quadrant + lane and the 64 score
    // columns [64*ch, 64*ch + 64). The row maximum (every key tile) and the row sum (once, at the end) are
    // combined through shared memory; everything else is private to the thread.
    fwd_setmaxnreg_inc<kFwdRegsSoftmax>();
    const int x = wg >> 1;
    const int quad = warp & 3, ch = (warp >> 2) & 1;
    const int rl = quad * 32 + lane;  // query row inside the tile = TMEM lane
    const uint32_t tS = tmem + 128 * x, tO = tmem + 256 + 128 * x;
    const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
    uint32_t sn = 0;   // S tiles consumed so far
    uint32_t pvn = 0;  // PV products of this half issued before the current round
    uint32_t xn = 0;   // completed phases of this row pair's exchange barrier
    float* my_slot = &s.xchg[x][ch][0][rl];                   // slot k is my_slot[128 * k]
    const float* partner_slot = &s.xchg[x][ch ^ 1][0][rl];
    uint64_t* pair_bar = &s.bar_pair[x][quad];
    while (next_pop()) {
      for (int r = 0; r < n_rounds; ++r) {
        const bool active = (x == 0 || rd.joint) && !*abort_flag;
        if (active) {
          const nsp_tile_t ia = x == 0 ? (r == 0 ? rd.a : rd.b) : rd.b;
          const SegInfo sg = (x == 0 && r == 0) ? pp->sa : pp->sb;
          const int h = ia.head, n_kv = ia.cost, q_row0 = ia.tile * kBM;
          float m_ref = -INFINITY;  // reference maximum (log2 domain) the stored P and l are relative to
          float l = 0.f;            // running sum of exp2(s - m_ref) over this thread's columns
          float mx_posted = 0.f;    // this thread's half-row maximum of the previous tile (when `pending`)
          bool pending = false;     // the previous tile's half-row maxima have been posted and not yet consumed
          bool ok = true;
          int where = 0;
          for (int j = 0; j < n_kv; ++j) {
            if (*abort_flag) { ok = false; break; }
            ok = mbar_wait(&s.bar_s_full[x], sn & 1, a.wait_limit);
            ++sn;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { where = kWhereFwdS; break; }
            tc_fence_after_sync();
            uint32_t sr[2][32];
            tmem_ld32(tS + lane_off + ch * 64, sr[0]);
            tmem_ld32(tS + lane_off + ch * 64 + 32, sr[1]);
            tmem_wait_ld();
            const bool last = (j == n_kv - 1);
            if (last) {  // diagonal tile: keys past the query are masked
#pragma unroll
              for (int c = 0; c < 2; ++c)
#pragma unroll
                for (int e = 0; e < 32; ++e)
                  if (ch * 64 + c * 32 + e > rl) sr[c][e] = __float_as_uint(-INFINITY);
            }
            // The reference maximum lags one tile behind: only the first tile of an item takes its row maximum
            // before exponentiating. Every later tile is exponentiated against the reference it finds, and its
            // own maximum is posted AFTER P has been handed to the MMA thread and folded in at the start of the
            // next tile. The result is the same (any reference gives the same O and LSE as long as nothing
            // overflows: a tile would have to exceed all earlier tiles of its row by 2^100 for that), but the
            // maximum and its exchange between the two threads of a row leave the S -> P -> PV critical path.
            bool need = false;
            float alpha = 1.f;
            if (j == 0) {
              float mx = -INFINITY;
#pragma unroll
              for (int c = 0; c < 2; ++c)
#pragma unroll
                for (int e = 0; e < 32; e += 2)
                  mx = max3f(mx, __uint_as_float(sr[c][e]), __uint_as_float(sr[c][e + 1]));
              my_slot[0] = mx;
              mbar_arrive(pair_bar);
              ok = mbar_wait(pair_bar, xn & 1, a.wait_limit);
              ++xn;
              ok = __all_sync(0xffffffffu, ok);
              if (!ok) { where = kWhereFwdPair; break; }
              m_ref = fmaxf(mx, partner_slot[0]) * a.scale_log2;
            } else if (pending) {
              ok = mbar_wait(pair_bar, xn & 1, a.wait_limit);
              ++xn;
              ok = __all_sync(0xffffffffu, ok);
              if (!ok) { where = kWhereFwdPair; break; }
              const float mx = fmaxf(mx_posted, partner_slot[128 * ((j - 1) & 1)]) * a.scale_log2;
              need = mx > m_ref + 8.f;
              if (need) {
                alpha = ex2f(m_ref - mx);
                m_ref = mx;
              }
              pending = false;
            }
            l *= alpha;
            float sum0 = 0.f, sum1 = 0.f;
            float mx_tile = -INFINITY;  // this tile's half-row maximum (raw scores), for the next tile
            const float neg_m = -m_ref;
            uint32_t pk[32];
#pragma unroll
            for (int c = 0; c < 2; ++c)
#pragma unroll
              for (int e = 0; e < 32; e += 2) {
                float x0, x1;
                mx_tile = max3f(mx_tile, __uint_as_float(sr[c][e]), __uint_as_float(sr[c][e + 1]));
                fma2(x0, x1, __uint_as_float(sr[c][e]), __uint_as_float(sr[c][e + 1]), a.scale_log2, a.scale_log2, neg_m,
                     neg_m);
                float p0, p1;
                if (((e >> 1) & 3) < NSP_EMU_FWD) {
                  ex2_poly2(p0, p1, x0, x1);
                } else {
                  p0 = ex2f(x0);
                  p1 = ex2f(x1);
                }
                add2(sum0, sum1, sum0, sum1, p0, p1);
                pk[c * 16 + (e >> 1)] = pack_bf16x2(p0, p1);
              }
            l += sum0 + sum1;
            // packed columns [64*ch, 64*ch + 32) = score columns [64*ch, 64*ch + 64): inside this thread's own
            // columns, so no other thread's unread scores are overwritten
            tmem_st32(tS + lane_off + ch * 64, pk);
            // rescale this thread's 64 columns of O in place when some row of the warp moved its reference
            // maximum; the previous PV product of this half must have completed first (the next one is not
            // issued before p_ready).
            if (j > 0 && __any_sync(0xffffffffu, need)) {
              ok = mbar_wait(&s.bar_pv_done[x], (pvn + j - 1) & 1, a.wait_limit);
              ok = __all_sync(0xffffffffu, ok);
              if (!ok) { where = kWhereFwdO; break; }
              tc_fence_after_sync();
#pragma unroll
              for (int c = 0; c < kOCols / 32; ++c) {
                uint32_t orow[32];
                tmem_ld32(tO + lane_off + ch * kOCols + c * 32, orow);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) orow[e] = __float_as_uint(__uint_as_float(orow[e]) * alpha);
                tmem_st32(tO + lane_off + ch * kOCols + c * 32, orow);
              }
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(&s.bar_p_ready[x]);
            if (j > 0 && !last) {
              // post this tile's half-row maximum for the next tile. Slot by tile parity: the partner reads slot
              // j & 1 at the start of tile j + 1, and this thread writes it again only at the end of tile j + 2,
              // which it cannot reach before the partner has handed over P of tile j + 1.
              mx_posted = mx_tile;
              my_slot[128 * (j & 1)] = mx_tile;
              mbar_arrive(pair_bar);
              pending = true;
            }
          }
          if (ok) {
            ok = mbar_wait(&s.bar_pv_done[x], (pvn + n_kv - 1) & 1, a.wait_limit);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) where = kWhereFwdO;
          }
          pvn += n_kv;
          const int row = q_row0 + rl;
          const bool valid = row < sg.len;
          if (RECOMP && ok && a.delta != nullptr) {
            // ---- epilogue of a recomputation: LSE and delta = <dO, O> of the row, O itself is not written.
            // The half-row dot product is taken with the unnormalised O and handed over together with the half-row
            // sum.
            tc_fence_after_sync();
            const __nv_bfloat16* dptr =
                a.d_o + sg.q_off + (static_cast<int64_t>(valid ? row : 0) * sg.hq + h) * kHeadDim + ch * kOCols;
            float part = 0.f;
#pragma unroll
            for (int c = 0; c < kOCols / 32; ++c) {
              uint32_t orow[32];
              tmem_ld32(tO + lane_off + ch * kOCols + c * 32, orow);
              uint4 dv4[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) dv4[e] = __ldg(reinterpret_cast<const uint4*>(dptr + c * 32) + e);
              tmem_wait_ld();
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const uint32_t w[4] = {dv4[e].x, dv4[e].y, dv4[e].z, dv4[e].w};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                  part = fmaf(__uint_as_float(orow[8 * e + 2 * t]), __uint_as_float(w[t] << 16), part);
                  part = fmaf(__uint_as_float(orow[8 * e + 2 * t + 1]), __uint_as_float(w[t] & 0xffff0000u), part);
                }
              }
            }
            my_slot[256] = l;
            my_slot[384] = part;
            mbar_arrive(pair_bar);
            ok = mbar_wait(pair_bar, xn & 1, a.wait_limit);
            ++xn;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) where = kWhereFwdPair;
            if (ok && valid && ch == 0) {
              l += partner_slot[256];
              part += partner_slot[384];
              const int64_t at = sg.lse_off + static_cast<int64_t>(h) * sg.len + row;
              NSP_CHECK(at >= 0 && at < a.lse_elems, a.status, it0, kWhereCheckFwdLse, row) {
                a.lse[at] = (m_ref + log2f(l)) * 0.6931471805599453f;
                a.delta[at] = part / l;
              }
            }
            if (!ok && lane == 0) {
              report_timeout(a.status, it0, where, 0);
              *abort_flag = 1;
            }
            round_end(r);
            continue;
          }
          if (ok) {  // row sum = sum of the two half rows
            my_slot[256] = l;
            mbar_arrive(pair_bar);
            ok = mbar_wait(pair_bar, xn & 1, a.wait_limit);
            ++xn;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) where = kWhereFwdPair;
          }
          if (ok) {
            // ---- epilogue: O / l -> bf16 (this thread's 64 columns), LSE
            l += partner_slot[256];
            tc_fence_after_sync();
            const float inv_l = 1.f / l;
            if (q_row0 + kBM <= sg.len) {
              // ---- a full tile goes out as a TMA tile store. The rows are staged, swizzled like an operand tile, in
              // the ring stage of the round's last key tile: K's for item A, V's for item B. Both are free: the last
              // PV product of this half has completed, and the tensor pipe runs one thread's products in order, so
              // the last S and PV products of the other half, which read the same stages, have completed as well; the
              // tiles the producer has already started for the coming round sit in the other stage. Written row by
              // row from the threads (each lane another row, 8 KB apart) the same tile cost 3,900 clocks per round:
              // the store path takes one 32-byte sector per clock, and every 16-byte store was half a sector.
              const int kt = pp->kt_base + rd.a.cost + (r == 1 ? rd.b.cost : 0);  // key tiles up to the end of this round
              uint8_t* const stage = (x == 0 ? s.k : s.v)[(kt - 1) & 1][0];
              uint8_t* const srow = stage + (D == 128 ? ch : 0) * kHalfTileBytes + rl * 128;
#pragma unroll
              for (int c = 0; c < kOCols / 32; ++c) {
                uint32_t orow[32];
                tmem_ld32(tO + lane_off + ch * kOCols + c * 32, orow);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  uint4 w;
                  w.x = pack_bf16x2(__uint_as_float(orow[8 * e + 0]) * inv_l, __uint_as_float(orow[8 * e + 1]) * inv_l);
                  w.y = pack_bf16x2(__uint_as_float(orow[8 * e + 2]) * inv_l, __uint_as_float(orow[8 * e + 3]) * inv_l);
                  w.z = pack_bf16x2(__uint_as_float(orow[8 * e + 4]) * inv_l, __uint_as_float(orow[8 * e + 5]) * inv_l);
                  w.w = pack_bf16x2(__uint_as_float(orow[8 * e + 6]) * inv_l, __uint_as_float(orow[8 * e + 7]) * inv_l);
                  const int chunk = (D == 128 ? 0 : ch * 4) + c * 4 + e;  // 16-byte chunk of the 128-byte row
                  *reinterpret_cast<uint4*>(srow + ((chunk ^ (rl & 7)) * 16)) = w;
                }
              }
              fence_proxy_async_smem();
              const uint64_t staged = mbar_arrive_token(&s.bar_o_staged[x]);
              if (ch == 0 && rl == 0) {  // one thread of the tile: wait for all rows, store, wait for the reads
                if (mbar_wait_token(&s.bar_o_staged[x], staged, a.wait_limit)) {
#pragma unroll
                  for (int hf = 0; hf < kHalves; ++hf)
                    tma_store_3d(&maps.o[sg.run], stage + hf * kHalfTileBytes, 64 * hf, h, sg.tok_in_run + q_row0);
                  tma_store_commit();
                  tma_store_wait_read();
                } else {
                  report_timeout(a.status, it0, kWhereFwdO, 1);
                  *abort_flag = 1;
                }
              }
            } else {
              // ---- ragged last tile of a segment: the valid rows only, straight from the threads
              __nv_bfloat16* optr = a.o + sg.q_off + (static_cast<int64_t>(row) * sg.hq + h) * kHeadDim + ch * kOCols;
#pragma unroll
              for (int c = 0; c < kOCols / 32; ++c) {
                uint32_t orow[32];
                tmem_ld32(tO + lane_off + ch * kOCols + c * 32, orow);
                tmem_wait_ld();
                if (valid) {
#pragma unroll
                  for (int e = 0; e < 4; ++e) {
                    uint4 w;
                    w.x = pack_bf16x2(__uint_as_float(orow[8 * e + 0]) * inv_l, __uint_as_float(orow[8 * e + 1]) * inv_l);
                    w.y = pack_bf16x2(__uint_as_float(orow[8 * e + 2]) * inv_l, __uint_as_float(orow[8 * e + 3]) * inv_l);
                    w.z = pack_bf16x2(__uint_as_float(orow[8 * e + 4]) * inv_l, __uint_as_float(orow[8 * e + 5]) * inv_l);
                    w.w = pack_bf16x2(__uint_as_float(orow[8 * e + 6]) * inv_l, __uint_as_float(orow[8 * e + 7]) * inv_l);
                    NSP_CHECK(optr + c * 32 + e * 8 + 8 <= a.o + a.q_elems && optr >= a.o, a.status, it0, kWhereCheckFwdO, row)
                    *reinterpret_cast<uint4*>(optr + c * 32 + e * 8) = w;
                  }
                }
              }
            }
            if (valid && ch == 0) {
              const int64_t at = sg.lse_off + static_cast<int64_t>(h) * sg.len + row;
              NSP_CHECK(at >= 0 && at < a.lse_elems, a.status, it0, kWhereCheckFwdLse, row)
              a.lse[at] = (m_ref + log2f(l)) * 0.6931471805599453f;
            }
          } else if (where != 0 && lane == 0) {
            report_timeout(a.status, it0, where, 0);
            *abort_flag = 1;
          }
        }
        round_end(r);
      }
    }
  }

  cta_sync();  // after a timeout the stragglers are not waited for for ever
  if (warp == 0) tmem_dealloc(s.tmem_base, kFwdTmemCols);
}

}  // namespace

namespace {
template <int D, bool RECOMP>
cudaError_t launch_fwd_t(const FwdMaps& maps, const FwdArgs& args, int num_sms, cudaStream_t st) {
  cudaError_t e = cudaFuncSetAttribute(fwd_kernel<D, RECOMP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(sizeof(FwdSmem<D>)));
  if (e != cudaSuccess) return e;
  const int pops = (args.n_items + 1) / 2;
  const int grid = pops < num_sms ? pops : num_sms;
  fwd_kernel<D, RECOMP><<<grid, kFwdThreads, sizeof(FwdSmem<D>), st>>>(maps, args);
  count_launches(1);
  return cudaGetLastError();
}
}  // namespace

cudaError_t launch_fwd(const FwdMaps& maps, const FwdArgs& args, int head_dim, int num_sms, cudaStream_t st) {
  if (args.n_items == 0) return cudaSuccess;
  const bool recomp = args.delta != nullptr || args.seg_mask != nullptr;
  if (head_dim == 64)
    return recomp ? launch_fwd_t<64, true>(maps, args, num_sms, st) : launch_fwd_t<64, false>(maps, args, num_sms, st);
  return recomp ? launch_fwd_t<128, true>(maps, args, num_sms, st) : launch_fwd_t<128, false>(maps, args, num_sms, st);
}

}  // namespace nsp

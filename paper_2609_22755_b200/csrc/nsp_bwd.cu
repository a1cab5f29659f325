// Backward: dQ, dK, dV of packed variable-length causal GQA attention on tcgen05 tensor cores.
//
// Three launches:
//   preprocess   delta[h, i] = sum_d dO[i,h,d] * O[i,h,d]                      (HBM-bound, one warp per row)
//   main         key-stationary persistent kernel, see below
//   postprocess  dQ = scale * fp32 accumulator -> bf16 / fp32                   (HBM-bound)
//
// Main kernel. One CTA per SM (640 threads, five warpgroups with their own register budgets) pops items
// (segment, kv head, key tile n) from the longest-first list. K_n and V_n stay in shared memory; the CTA walks
// every q head of the KV group and every q tile m >= n. All score-shaped quantities are computed TRANSPOSED
// (key index on the TMEM lanes) so that P^T and dS^T are directly the A operands of the dV and dK products:
//     S^T  = K Q^T  -> R0,   dP^T = V dO^T -> R1          A, B K-major from shared memory
//     P^T  = exp2(S^T * scale*log2e - LSE*log2e),  dS^T = P^T o (dP^T - delta)
//     dV  += P^T dO                               A = P^T (bf16, written over S^T in R0), B = dO  MN-major
//     dK  += dS^T Q                               A = dS^T (shared memory, K-major), B = Q MN-major
//     dQ_m^T = K^T dS^T -> R1 (over dP^T)         A = K read MN-major, B = dS^T read MN-major
// TMEM: R0 [0,128), R1 [128,256), dK [256,384), dV [384,512).
// Roles:  warps 0-7  softmax / dS (key row = TMEM lane, two column halves)
//         warps 8-15 dQ: TMEM -> fp32 accumulator in global memory (lane quadrant x 64-column half)
//         warp 16    TMA producer (K, V once per item; Q two-stage ring, dO single buffer)
//         warp 17    MMA issuer A (whole warp runs the waits, the elected lane issues): dV(t), S^T(t+1)
//         warp 18    LSE / delta loader (two-stage ring in shared memory)
//         warp 19    MMA issuer B (likewise): dQ^T(t), dK(t), dP^T(t+1)
// The softmax warps hand over P^T first (p_ready) and dS^T second (ds_ready), so dV(t) and S^T(t+1) run under
// the dS phase of step t, and dK(t), dQ^T(t), dP^T(t+1) under the exp2 phase of step t+1.
// dQ is produced TRANSPOSED (head dimension on the TMEM lanes): a warp of the dQ warpgroups then holds 32
// consecutive head-dimension values of one query row per register, and a plain red.global.add.f32 per register
// is one fully coalesced 128-byte reduction into the fp32 accumulator. No shared-memory staging: shared-memory
// bandwidth (MMA operand reads, TMA fills, dS^T) is a scarce resource of this kernel.
// dK and dV accumulate in TMEM over the whole item in a fixed order (q tiles descending, heads ascending inside
// a tile), so the reduction over the query heads of a group is deterministic.
// At the end of an item a full fp32 tile of each is staged in the (then idle) operand buffers and written by TMA tile
// stores; bf16 outputs and ragged tiles are stored row by row from the threads.
// For the first q tile of a segment (rows 0..127, where P is O(1)) the step runs twice, once with the bf16
// value of P and dS and once with the bf16 residual (hi + lo), and delta is recomputed in fp32 as
// sum_j P_ij dP_ij instead of taking it from the bf16-rounded O; this keeps dK/dV/dQ inside the 2e-2 tolerance.
//
// Code size matters here: twenty warps of five roles share one instruction cache, and a step loop whose roles
// together do not fit in it runs at the speed of instruction fetch. So the common step (an interior tile) has
// its own lean, fully unrolled path; everything rare (diagonal tile, first-tile passes, ragged tail, item
// epilogue) goes through compact rolled loops; an item is decoded once, by one thread, into shared memory.
#include <type_traits>
#include <cuda_bf16.h>
#include "nsp_internal.cuh"
#include "sm100_ptx.cuh"

namespace nsp {
namespace {

constexpr int kBwdThreads = 640;  // 8 softmax warps, 8 dQ warps, one auxiliary warpgroup
constexpr uint32_t kHalfTileBytes = 128 * 64 * 2;
constexpr uint32_t kBwdTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;
// setmaxnreg redistributes the launch-time allocation (96 per thread, 640 threads): softmax x2 / dQ x2 / auxiliary.
// Main kernel 120 / 96 / 48: the dQ role holds 64 accumulator values, 64 row pointers' worth of arithmetic and the
// turn logic, and with 80 registers it spilled inside its drain (cfg4 backward 400 ms; 88: 392 ms; 96: 389 ms, the
// most a warpgroup can keep without an increase of its own), while the softmax role fits 120. First-tile kernel
// 136 / 80 / 48: there the softmax role carries the packed P of a whole tile across two sweeps and the dQ role only
// stores. 256 * (120 + 96) + 128 * 48 = 256 * (136 + 80) + 128 * 48 = 640 * 96.
template <bool FIRST> constexpr int kRegsSoftmax = FIRST ? 136 : 120;
template <bool FIRST> constexpr int kRegsReduce = FIRST ? 80 : 96;
constexpr int kRegsAux = 48;
constexpr int kFrontMinSteps = 2048;          // items shorter than this start at once
constexpr int kFrontMinGroup = 8;             // so do items of groups with fewer q heads per kv head
constexpr long long kFrontWaitClk = 1500000;  // ~0.9 ms: upper bound of the start alignment (also: 1/16 of the item)
constexpr int kQStages = 2;                   // Q ring (three stages measured 3 % slower on the nested shard)

// A decoded work item: written by one thread (thread 0, or the producer's lane 0 one item ahead), read by every role
// after the CTA-wide barrier of next_item().
struct ItemCtx {
  int64_t q_off, kv_off, lse_off;  // element offsets of the segment
  int32_t it;                      // position in the work list (>= n_items: no more work)
  int32_t len, hq, hkv, run, tok0;
  int32_t g, n;                    // kv head, key tile
  int32_t G;                       // q heads per kv head
  int32_t turn_off, mt;            // deterministic dQ: the segment's first turn counter, its q tiles
  int32_t first;                   // key tile 0
  int32_t m0;                      // first (lowest) q tile of the walk
  int32_t per_head;                // steps per q head
  int32_t steps;                   // G * per_head
  int32_t rows;                    // first-tile kernel: 0, or 1 + index of the row table of a pack of short segments
};

// FIRST: the first-tile kernel also keeps the bf16 residual of dS^T. The main kernel does without those 32 KB on
// purpose: shared memory it does not claim stays with the L1 cache, and the kernel ran 3 % slower with the larger
// carve-out (the same 3 % the step from a three-stage to a two-stage Q ring gained).
template <bool FIRST, int D>
struct BwdSmem {
  uint8_t k[D / 64][kHalfTileBytes];  // K, V, Q, dO tiles: D / 64 sub-tiles of 64 columns (D = head dimension)
  uint8_t v[D / 64][kHalfTileBytes];
  uint8_t q[kQStages][D / 64][kHalfTileBytes];  // [stage][64-column half]: ring, loaded a whole step ahead
  uint8_t d_o[D / 64][kHalfTileBytes];  // [half]: single buffer (its consumers leave a long window for the refill)
  uint8_t ds[2][kHalfTileBytes];      // dS^T, [key row][query col], two 64-column halves
  uint8_t ds_lo[FIRST ? 2 * kHalfTileBytes : 16];  // first-tile kernel: the bf16 residual of dS^T, same layout, right behind it
  float lse[2][128];                  // [stage] LSE * log2(e) of the q tile (+inf for rows past the segment)
  float delta[2][128];                // [stage]
  ItemCtx ctx[2];
  uint64_t bar_kv;
  uint64_t bar_q_full[kQStages];
  uint64_t bar_q_empty[kQStages][2];  // [stage][issuer A / B]: that issuer's MMAs reading the Q stage have completed
  uint64_t bar_do_full;
  uint64_t bar_do_empty[2];    // [issuer A / B]: that issuer's MMAs reading the dO buffer have completed
  uint64_t bar_a_done;         // dV of the step (issuer A) has completed
  uint64_t bar_b_done;         // dK of the step (issuer B) has completed
  uint64_t bar_ld_full[2], bar_ld_empty[2];
  uint64_t bar_s_full, bar_dp_full, bar_dq_full, bar_dq_empty;
  uint64_t bar_p_ready;   // 256 softmax threads: P^T of the step is in R0
  uint64_t bar_ds_ready;  // 256 softmax threads: dS^T of the step is in shared memory
  uint64_t bar_delta[2];  // 128 softmax threads of one column half: partial / final sums of the exact delta
  uint64_t bar_out;       // 256 softmax threads: the item's dK and dV tiles are staged for the tile stores
  uint32_t tmem_base;
  int32_t abort;
};
static_assert(sizeof(BwdSmem<true, 128>) <= 232448, "shared memory budget (227 KB)");

// DET = 2: every term a key tile adds to the dQ accumulator is first rounded to a multiple of 2^-12 (x + 1.5 * 2^11
// lands in [2^11, 2^12), where fp32 steps by 2^-12; taking the constant off again is exact). Sums of such multiples are
// exact in fp32 while they stay below 2^12, so the order of the floating-point reductions no longer matters: the
// accumulator, and with it dQ, comes out bit for bit the same in every run and for every packing, with no waiting.
// The price is the quantum itself (2^-13 of error per term, in units of dQ / softmax_scale).
constexpr float kDqRound = 3072.f;
template <int DET>
__device__ __forceinline__ float dq_term(float x) {
  if constexpr (DET == 2) return __fadd_rn(__fadd_rn(x, kDqRound), -kDqRound);
  return x;
}
__device__ __forceinline__ void red_add_f32(float* addr, float v) {
  asm volatile("red.relaxed.gpu.global.add.f32 [%0], %1;" ::"l"(addr), "f"(v) : "memory");
}
template <int N>
__device__ __forceinline__ void setmaxnreg_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void setmaxnreg_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

// Walks the steps of an item: q tiles in DESCENDING order (the diagonal tile last), for every q tile the q heads of
// the group in ascending order.
// Descending, because the tensor core adds into its fp32 accumulator with truncation: every one of the ~100,000
// additions a dK / dV accumulator of a long segment receives loses up to one ulp OF THE ACCUMULATOR, always towards
// zero. The large contributions to a key come from the queries just after it; met first, they keep the accumulator
// large for the whole tail and the losses add up (measured on a 131,072-token segment with 16 q heads per kv head:
// sum_j dV_j 0.22 % short, dV off by up to 0.048 against a closed form; 0.002 in descending order). Met last, the
// tail is summed while the accumulator is still small.
// Heads innermost, so that CTAs that work on neighbouring key tiles stay one q tile apart for the whole item and
// find the Q / dO tiles and the dQ accumulator rows they touch in L2.
// The first q tile of a segment (q tile 0 against key tile 0) is not walked here: it belongs to the first-tile
// kernel (the same code instantiated with FIRST = true), so an item with key tile 0 starts at q tile 1.
struct StepWalk {
  int hh, rr;
  __device__ __forceinline__ void reset() { hh = 0, rr = 0; }
  __device__ __forceinline__ void get(const ItemCtx& c, int& h, int& m) const {
    const int p = c.per_head - 1 - rr;  // q tiles in DESCENDING order (see above)
    h = c.g * c.G + hh;
    m = c.m0 + p;
  }
  __device__ __forceinline__ void next(const ItemCtx& c) {
    if (++hh == c.G) hh = 0, ++rr;
  }
};

// Position in the Q ring; it runs on across items. ph is the parity of the number of earlier uses of
// the current stage.
struct QRing {
  uint32_t st = 0, ph = 0;
  __device__ __forceinline__ void next() {
    if (++st == kQStages) st = 0, ph ^= 1;
  }
};

// FIRST = false: the main kernel, items (segment, kv head, key tile) against q tiles max(n, 1) .. Mt-1.
// FIRST = true: the first-tile kernel, items (segment, kv head): q tile 0 against key tile 0 for every q head of the
// group. Rows 0..127 of a segment have few keys, so P is O(1) and its bf16 rounding alone would push dK / dV past
// the tolerance: there P^T and dS^T enter their products as bf16 value plus bf16 residual (two products each), and
// delta_i = sum_j P_ij dP_ij is taken in fp32 (all keys of these rows sit in the tile) instead of from the
// bf16-rounded O. Its dQ rows are complete (no other key tile reaches q tile 0) and are stored directly; its dK / dV
// rows are the whole result for a one-tile segment and otherwise the part the main kernel, which runs after it, adds
// its own sum to.
// DET = 2 (main kernel only): see dq_term above.
// DET = 1 (main kernel only): the dQ tiles of the key tiles 0, 1, 2, ... of a (segment, q head, q tile) are added to the
// accumulator in exactly that order: a dQ warp waits (bounded) until the turn counter of its q tile says that the key
// tiles before its own are done, adds, and passes the turn on. In lock-step the CTAs of neighbouring key tiles then
// follow one another a reduction apart instead of all adding at once.
template <bool FIRST, int DET, int D>
__global__ void __launch_bounds__(kBwdThreads, 1) bwd_kernel(const __grid_constant__ BwdMaps maps, const BwdArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  BwdSmem<FIRST, D>& s = *reinterpret_cast<BwdSmem<FIRST, D>*>(smem_raw);
  constexpr int kHalves = D / 64;  // 64-column sub-tiles of a K / V / Q / dO tile
  constexpr uint32_t kOpBytes = kHalves * kHalfTileBytes;  // bytes of such a tile
  constexpr int kHeadDim = D;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, wg = warp >> 2;
  // swizzled tiles need a 1024-byte aligned base
  const bool misaligned = (smem_u32(smem_raw) & 1023u) != 0;

  if (tid == 0) {
    mbar_init(&s.bar_kv, 1);
    for (int i = 0; i < kQStages; ++i) {
      mbar_init(&s.bar_q_full[i], 1);
      mbar_init(&s.bar_q_empty[i][0], 1);
      mbar_init(&s.bar_q_empty[i][1], 1);
    }
    mbar_init(&s.bar_do_full, 1);
    mbar_init(&s.bar_do_empty[0], 1);
    mbar_init(&s.bar_do_empty[1], 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s.bar_ld_full[i], 32);
      mbar_init(&s.bar_ld_empty[i], 256);
    }
    mbar_init(&s.bar_s_full, 1);
    mbar_init(&s.bar_dp_full, 1);
    mbar_init(&s.bar_p_ready, 256);
    mbar_init(&s.bar_ds_ready, 256);
    mbar_init(&s.bar_dq_full, 1);
    mbar_init(&s.bar_a_done, 1);
    mbar_init(&s.bar_b_done, 1);
    mbar_init(&s.bar_dq_empty, 256);
    mbar_init(&s.bar_delta[0], 128);
    mbar_init(&s.bar_delta[1], 128);
    mbar_init(&s.bar_out, 256);
    s.abort = 0;
    fence_mbar_init();
  }
  if (warp == 0 && !misaligned) {
    tmem_alloc(&s.tmem_base, kBwdTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();

  // The CTA owns all 512 TMEM columns, so the allocation starts at column 0 and every TMEM address is a
  // compile-time constant.
  constexpr uint32_t tR0 = 0, tR1 = 128, tDK = 256, tDV = 384;
  if (misaligned || s.tmem_base != 0) {
    if (tid == 0)
      report_timeout(a.status, -1, misaligned ? kWhereBwdSmemAlign : kWhereBwdTmemBase, static_cast<int32_t>(s.tmem_base));
    __syncthreads();
    if (warp == 0 && !misaligned) tmem_dealloc(s.tmem_base, kBwdTmemCols);
    return;
  }
  volatile int32_t* abort_flag = &s.abort;
  uint32_t gs = 0;  // steps completed so far by this CTA (every role advances it identically)
  uint32_t gi = 0;  // items completed so far

  // Every role runs its own copy of the item loop (so that its register budget, set by setmaxnreg at the top of
  // the role, governs the whole loop); the loops meet at the CTA-wide barrier inside next_item().
  const ItemCtx* cx = nullptr;
  // One thread pops the next item and decodes it into a slot of s.ctx: the atomic, the dependent loads and (for long
  // items of large groups) the start alignment take ~4,000 clocks and more. After a short item the TMA producer's
  // lane 0 has done it ahead, into the other slot, while the item's last steps and its epilogue ran: it is the one
  // thread with nothing left to do then (4,400 -> ~1,000 clocks per item boundary; 4 % of a backward pass over
  // 512-token segments). Both sides derive "ahead" from the finished item's step count, so no flag is needed; the
  // barrier below publishes the slot either way.
  constexpr int kAheadMaxSteps = 64;
  auto fetch_item = [&](ItemCtx& x) {
    for (;;) {
      const int idx = atomicAdd(a.counter, 1);
      x.it = idx;
      if (idx >= a.n_items) break;
      const nsp_tile_t item = a.items[idx];
      const SegInfo sg = a.seg[item.seg];
      x.q_off = sg.q_off, x.kv_off = sg.kv_off, x.lse_off = sg.lse_off;
      x.len = sg.len, x.hq = sg.hq, x.hkv = sg.hkv, x.run = sg.run, x.tok0 = sg.tok_in_run;
      x.g = item.head, x.n = item.tile;
      x.G = sg.hq / sg.hkv;
      x.turn_off = sg.turn_off, x.mt = (sg.len + kBM - 1) / kBM;
      x.first = (item.tile == 0);
      x.rows = sg.rows;
      if constexpr (FIRST) {
        x.m0 = 0;
        x.per_head = 1;  // q tile 0 only
        x.steps = x.G;
        break;
      }
      x.m0 = item.tile + x.first;                        // q tile 0 belongs to the first-tile kernel
      x.per_head = (sg.len + kBM - 1) / kBM - x.m0;      // q tiles max(n, 1) .. Mt-1 (bm == bn)
      x.steps = x.G * x.per_head;
      // Start alignment. kFrontBlock consecutive items are neighbouring key tiles of one (segment, kv head) and
      // walk the same (q tile, head) sequence from the segment's last q tile down. CTAs that start them at the
      // same moment stay on the same q tile for the whole item and find its Q, dO and dQ-accumulator tiles in
      // L2; left alone they start one q tile apart (items end G steps apart), and 148 CTAs on 148 different q
      // tiles need 148 * G * 128 KB of L2: more than there is from G = 8 on (measured at G = 16: 900 GB of DRAM
      // traffic for tensors of 15 GB). So the CTA of a long item of such a group waits here, for at most
      // kFrontWaitClk, until the other items of its block have been popped as well (the CTAs that pop them are
      // the next ones to finish, G steps apart). A timeout is not an error: the CTA just starts.
      {
        const int blk = idx / kFrontBlock;
        const int rest = a.n_items - blk * kFrontBlock;
        const int expect = rest < kFrontBlock ? rest : kFrontBlock;
        atomicAdd(a.front + blk, 1);
        if (x.steps >= kFrontMinSteps && x.G >= kFrontMinGroup) {
          const long long t0 = clock64();
          const long long own = static_cast<long long>(x.steps) * 340;  // about 1/16 of what the item takes
          const long long limit = own < kFrontWaitClk ? own : kFrontWaitClk;
          while (*reinterpret_cast<volatile int32_t*>(a.front + blk) < expect && clock64() - t0 < limit)
            __nanosleep(200);
        }
      }
      if (x.steps > 0) break;  // the only key tile of a one-tile segment has nothing left to do here
    }
  };
  auto next_item = [&]() -> bool {
    ItemCtx& x = s.ctx[gi & 1];
    const bool ahead = gi > 0 && cx->it < a.n_items && cx->steps <= kAheadMaxSteps;  // cx: the item just finished
    if (tid == 0 && !ahead) fetch_item(x);
    tc_fence_before_sync();
    // Every role gets here in bounded time: all its other waits are bounded, and none of them returns before the end
    // of the kernel. (An mbarrier with a bounded wait in this place made the register allocation of the softmax role
    // fail.)
    __syncthreads();
    tc_fence_after_sync();
    cx = &x;
    return x.it < a.n_items && !*abort_flag;
  };
  auto item_done = [&]() {
    gs += static_cast<uint32_t>(cx->steps);
    gi += 1;
  };

  if (wg == 4) {
    setmaxnreg_dec<kRegsAux>();
    if (warp == 16) {
      // ================================================================ TMA producer
      // Q(t) goes into a three-stage ring and is requested about one step before S^T(t) needs it; dO(t) goes
      // into a single buffer that is free from the end of dV(t-1) until dP^T(t). Requests are issued in the
      // order Q(0), dO(0), Q(1), dO(1), ...: the wait for the dO buffer is the one that paces the loop.
      QRing qr;
      while (next_item()) {
        if (lane == 0) {
          const ItemCtx c = *cx;
          const CUtensorMap* mq = &maps.q[c.run];
          const CUtensorMap* mdo = &maps.d_o[c.run];
          mbar_expect_tx(&s.bar_kv, 2 * kOpBytes);
#pragma unroll
          for (int hf = 0; hf < kHalves; ++hf) {
            tma_load_3d(s.k[hf], &maps.k[c.run], &s.bar_kv, 64 * hf, c.g, c.tok0 + c.n * kBN);
            tma_load_3d(s.v[hf], &maps.v[c.run], &s.bar_kv, 64 * hf, c.g, c.tok0 + c.n * kBN);
          }
          StepWalk w;
          w.reset();
#pragma unroll 1
          for (int vt = 0; vt < c.steps; ++vt) {
            const uint32_t cs = gs + vt;
            if (*abort_flag) break;
            int h, m;
            w.get(c, h, m);
            w.next(c);
            if (!mbar_wait(&s.bar_q_empty[qr.st][0], qr.ph ^ 1, a.wait_limit) || !mbar_wait(&s.bar_q_empty[qr.st][1], qr.ph ^ 1, a.wait_limit)) {
              report_timeout(a.status, c.it, kWhereBwdQEmpty, vt);
              *abort_flag = 1;
              break;
            }
            mbar_expect_tx(&s.bar_q_full[qr.st], kOpBytes);
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf)
              tma_load_3d(s.q[qr.st][hf], mq, &s.bar_q_full[qr.st], 64 * hf, h, c.tok0 + m * kBM);
            qr.next();
            if (!mbar_wait(&s.bar_do_empty[0], (cs & 1) ^ 1, a.wait_limit) || !mbar_wait(&s.bar_do_empty[1], (cs & 1) ^ 1, a.wait_limit)) {
              report_timeout(a.status, c.it, kWhereBwdQEmpty, 100000 + vt);
              *abort_flag = 1;
              break;
            }
            mbar_expect_tx(&s.bar_do_full, kOpBytes);
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf) tma_load_3d(s.d_o[hf], mdo, &s.bar_do_full, 64 * hf, h, c.tok0 + m * kBM);
          }
          if (c.steps <= kAheadMaxSteps) fetch_item(s.ctx[(gi + 1) & 1]);  // see next_item(): the same rule on both sides
        }
        item_done();
      }
    } else if (warp == 17 || warp == 19) {
      // ================================================================ MMA issuers
      // Two issuing warps share the step: warp 17 (A) owns R0 and dV: dV(t), S^T(t+1); warp 19 (B) owns R1 and
      // dK: dQ^T(t), dK(t), dP^T(t+1). Each has its own chain of waits, so the bookkeeping of one hides behind
      // the MMAs of the other. All 32 lanes run the waits and the address arithmetic (convergent code); the lane
      // elect.sync picks issues the MMAs and the commits. Each issuer signals completion on barriers of its own
      // (a tcgen05.commit covers only the issuing thread's MMAs); whoever depends on both waits for both.
      const bool is_a = warp == 17;
      QRing qr;
      while (next_item()) {
        {
          const bool leader = elect_one();
          constexpr uint32_t idesc_kk = make_idesc_bf16(128, 128, 0, 0);  // S^T, dP^T: A K-major, B K-major, contraction over D
          constexpr uint32_t idesc_kn = make_idesc_bf16(128, D, 0, 1);    // dV, dK: A K-major (or TMEM), B MN-major, N = D
          constexpr uint32_t idesc_nn = make_idesc_bf16(128, 128, 1, 1);  // dQ^T: A MN-major (M = head dimension), B MN-major
          // Descriptors are {low word, high word}; an operand advances inside its tile by adding the byte offset
          // (in 16-byte units) to the low word (the 14-bit address field cannot overflow: every tile sits below
          // 256 KB). K-major operands step 32 bytes per 16 contraction elements inside a 64-column half;
          // MN-major operands step 16 rows = 2048 bytes. The high word is the same for both kinds.
          const uint32_t hi = static_cast<uint32_t>(make_smem_desc_sw128(0, 16, 1024) >> 32);
          constexpr uint32_t lbo_km = (16u >> 4) << 16, lbo_mn = (kHalfTileBytes >> 4) << 16;
          // K read MN-major as the A operand of dQ^T has M = head dimension. With D = 64 the product still runs with
          // M = 128: the second half of the rows repeats the first (leading byte offset 0) and lands in TMEM lanes
          // 64..127, which nobody reads.
          constexpr uint32_t lbo_kt = D == 128 ? lbo_mn : 0u;
          constexpr uint32_t kStageStep = kOpBytes >> 4;  // descriptor distance between Q stages
          const int steps = cx->steps, item_it = cx->it;
          int where = 0;
          bool okm = mbar_wait(&s.bar_kv, gi & 1, a.wait_limit);
          if (!okm) where = kWhereBwdLoadKV;
          const uint32_t q0_lo = smem_desc_addr(s.q[0][0]), do_lo = smem_desc_addr(s.d_o[0]);
          if (is_a) {
            const uint32_t k_km = smem_desc_addr(s.k[0]) | lbo_km;
            // S^T of the next step not yet issued -> R0 (A = K, B = Q of the ring stage, both K-major)
            auto issue_s = [&]() -> bool {
              if (!mbar_wait(&s.bar_q_full[qr.st], qr.ph, a.wait_limit)) { where = kWhereBwdLoadQ; return false; }
              tc_fence_after_sync();
              const uint32_t b_lo = (q0_lo + qr.st * kStageStep) | lbo_km;
#pragma unroll
              for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t off = ((kk >> 2) * kHalfTileBytes + (kk & 3) * 32) >> 4;
                if (leader) umma_ss_lh(tR0, k_km + off, hi, b_lo + off, hi, idesc_kk, kk > 0);
              }
              if (leader) umma_commit(&s.bar_s_full);
              if (leader) umma_commit(&s.bar_q_empty[qr.st][0]);  // this thread is done with the Q stage
              qr.next();
              return true;
            };
            okm = okm && issue_s();
            auto step_a = [&](int vt) -> bool {
              constexpr bool fold = FIRST;
              const uint32_t cs = gs + vt;
              if (*abort_flag) return false;
              if (!mbar_wait(&s.bar_do_full, cs & 1, a.wait_limit)) { where = kWhereBwdLoadQ; return false; }
              if (!mbar_wait(&s.bar_p_ready, cs & 1, a.wait_limit)) { where = kWhereBwdPReady; return false; }
              tc_fence_after_sync();
              const uint32_t acc = vt > 0;
              if constexpr (!fold) {
                // dV += P^T dO; packed P^T columns of K-step kk (16 query columns) sit at R0 + (kk/2)*32 + (kk%2)*8
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                  if (leader) umma_ts_lh(tDV, tR0 + (kk >> 1) * 32 + (kk & 1) * 8, (do_lo | lbo_mn) + kk * 128, hi, idesc_kn,
                             acc | (kk > 0));
              } else {
                // P^T as value + residual, 16 query columns = 8 packed columns each, side by side
#pragma unroll 1
                for (int kk = 0; kk < 8; ++kk) {
                  if (leader) umma_ts_lh(tDV, tR0 + kk * 16, (do_lo | lbo_mn) + kk * 128, hi, idesc_kn, acc | (kk > 0));
                  if (leader) umma_ts_lh(tDV, tR0 + kk * 16 + 8, (do_lo | lbo_mn) + kk * 128, hi, idesc_kn, 1u);
                }
              }
              if (leader) umma_commit(&s.bar_a_done);       // S^T and dV of the step
              if (leader) umma_commit(&s.bar_do_empty[0]);  // this thread is done with the dO buffer
              if (vt + 1 < steps && !issue_s()) return false;
              return true;
            };
#pragma unroll 1
            for (int vt = 0; okm && vt < steps; ++vt) okm = step_a(vt);
          } else {
            const uint32_t v_km = smem_desc_addr(s.v[0]) | lbo_km, k_mn = smem_desc_addr(s.k[0]) | lbo_kt;
            const uint32_t ds_km = smem_desc_addr(s.ds[0]) | lbo_km, ds_mn = smem_desc_addr(s.ds[0]) | lbo_mn;
            constexpr uint32_t kLoStep = (2 * kHalfTileBytes) >> 4;  // descriptor distance from dS^T to its residual
            // dP^T of step vt -> R1, once the dQ warps have drained dQ^T of the previous step from it
            auto issue_dp = [&](int vt) -> bool {
              const uint32_t cs = gs + vt;
              if (!mbar_wait(&s.bar_do_full, cs & 1, a.wait_limit)) { where = kWhereBwdLoadQ; return false; }
              if (!mbar_wait(&s.bar_dq_empty, (cs & 1) ^ 1, a.wait_limit)) { where = kWhereBwdDqEmpty; return false; }
              tc_fence_after_sync();
#pragma unroll
              for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t off = ((kk >> 2) * kHalfTileBytes + (kk & 3) * 32) >> 4;
                if (leader) umma_ss_lh(tR1, v_km + off, hi, (do_lo | lbo_km) + off, hi, idesc_kk, kk > 0);
              }
              if (leader) umma_commit(&s.bar_dp_full);
              if (leader) umma_commit(&s.bar_do_empty[1]);  // this thread is done with the dO buffer
              return true;
            };
            okm = okm && issue_dp(0);
            auto step_b = [&](int vt) -> bool {
              constexpr bool fold = FIRST;
              const uint32_t cs = gs + vt;
              if (*abort_flag) return false;
              if (!mbar_wait(&s.bar_q_full[qr.st], qr.ph, a.wait_limit)) { where = kWhereBwdLoadQ; return false; }
              if (!mbar_wait(&s.bar_ds_ready, cs & 1, a.wait_limit)) { where = kWhereBwdDsReady; return false; }
              tc_fence_after_sync();
              const uint32_t acc = vt > 0;
              const uint32_t q_mn = (q0_lo + qr.st * kStageStep) | lbo_mn;
              // dQ^T = K^T dS^T -> R1 (dP^T of this step has been consumed: ds_ready). It goes first: the dQ warps
              // drain R1 while dK runs, so that dP^T of the next step can follow dK without a gap.
#pragma unroll
              for (int kk = 0; kk < 8; ++kk) if (leader) umma_ss_lh(tR1, k_mn + kk * 128, hi, ds_mn + kk * 128, hi, idesc_nn, kk > 0);
              if constexpr (fold) {
#pragma unroll 1
                for (int kk = 0; kk < 8; ++kk)
                  if (leader) umma_ss_lh(tR1, k_mn + kk * 128, hi, ds_mn + kLoStep + kk * 128, hi, idesc_nn, 1u);
              }
              if (leader) umma_commit(&s.bar_dq_full);
              // dK += dS^T Q
#pragma unroll
              for (int kk = 0; kk < 8; ++kk) {
                const uint32_t off = ((kk >> 2) * kHalfTileBytes + (kk & 3) * 32) >> 4;
                if (leader) umma_ss_lh(tDK, ds_km + off, hi, q_mn + kk * 128, hi, idesc_kn, acc | (kk > 0));
              }
              if constexpr (fold) {
#pragma unroll 1
                for (int kk = 0; kk < 8; ++kk) {
                  const uint32_t off = ((kk >> 2) * kHalfTileBytes + (kk & 3) * 32) >> 4;
                  if (leader) umma_ss_lh(tDK, ds_km + kLoStep + off, hi, q_mn + kk * 128, hi, idesc_kn, 1u);
                }
              }
              if (leader) umma_commit(&s.bar_b_done);              // dP^T, dQ^T and dK of the step
              if (leader) umma_commit(&s.bar_q_empty[qr.st][1]);  // this thread is done with the Q stage
              qr.next();
              if (vt + 1 < steps && !issue_dp(vt + 1)) return false;
              return true;
            };
#pragma unroll 1
            for (int vt = 0; okm && vt < steps; ++vt) okm = step_b(vt);
          }
          if (!okm && where != 0) {  // where == 0: another role raised the abort flag
            if (leader) report_timeout(a.status, item_it, where, is_a ? 0 : 1);
            *abort_flag = 1;
          }
        }
        item_done();
      }
    } else if (warp == 18) {
      // ================================================================ LSE / delta loader
      while (next_item()) {
        const ItemCtx c = *cx;
        StepWalk w;
        w.reset();
#pragma unroll 1
        for (int vt = 0; vt < c.steps; ++vt) {
          const uint32_t cs = gs + vt, st = cs & 1;
          if (*abort_flag) break;
          bool okl = mbar_wait(&s.bar_ld_empty[st], ((cs >> 1) & 1) ^ 1, a.wait_limit);
          okl = __all_sync(0xffffffffu, okl);
          if (!okl) {
            if (lane == 0) {
              report_timeout(a.status, c.it, kWhereBwdLdEmpty, vt);
              *abort_flag = 1;
            }
            break;
          }
          int h, m;
          w.get(c, h, m);
          w.next(c);
          const int64_t base = c.lse_off + static_cast<int64_t>(h) * c.len;
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            const int col = lane + 32 * x, qi = m * kBM + col;
            const bool valid = qi < c.len;
            float lv = INFINITY, dv_ = 0.f;
            if (valid) {
              int64_t at = base + qi;
              if constexpr (FIRST) {
                if (c.rows > 0) {  // a tile shared by several short segments: LSE is laid out per segment
                  const RowInfo ri = a.rows[static_cast<int64_t>(c.rows - 1) * kBM + col];
                  at = ri.lse_base + static_cast<int64_t>(h) * ri.len + col;
                }
              }
              NSP_CHECK(at >= 0 && at < a.lse_elems, a.status, c.it, kWhereCheckBwdLse, qi) {
                lv = a.lse[at] * kLog2e;
                dv_ = a.delta[at];
              }
            }
            s.lse[st][col] = lv;
            s.delta[st][col] = dv_;
          }
          mbar_arrive(&s.bar_ld_full[st]);
        }
        item_done();
      }
    }
  } else if (wg >= 2) {
    // ================================================================ dQ^T: R1 -> global fp32 accumulator
    setmaxnreg_dec<kRegsReduce<FIRST>>();
    const int quad = warp & 3, colhalf = wg - 2;  // this warp drains query columns [64*colhalf, 64*colhalf + 64)
    const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
    const int d = quad * 32 + lane;  // head-dimension index = TMEM lane
    while (next_item()) {
      const ItemCtx c = *cx;
      const int64_t q_stride = static_cast<int64_t>(c.hq) * kHeadDim;  // floats between consecutive query rows
      StepWalk w;
      w.reset();
#pragma unroll 1
      for (int vt = 0; vt < c.steps; ++vt) {
        const uint32_t cs = gs + vt;
        if (*abort_flag) break;
        bool okr = mbar_wait(&s.bar_dq_full, cs & 1, a.wait_limit);
        okr = __all_sync(0xffffffffu, okr);
        if (!okr) {
          if (lane == 0) {
            report_timeout(a.status, c.it, kWhereBwdDqFull, vt);
            *abort_flag = 1;
          }
          break;
        }
        tc_fence_after_sync();
        int h, m;
        w.get(c, h, m);
        w.next(c);
        // Register e of a column chunk is dQ^T[d][query]: the 32 lanes of a warp add 32 consecutive floats of
        // one accumulator row (128 bytes, one request). Eight warps issue them: one SM sustains about 25 bytes
        // per clock of reductions, and four warps reach only half of that. Rows past the segment end are
        // skipped (their dS^T columns are zero, and they may lie outside the buffer).
        const int rows_left = c.len - m * kBM;  // valid query rows of this q tile (>= 128 for an interior tile)
        float* const tile0 = a.dq_acc + c.q_off + (static_cast<int64_t>(m) * kBM * c.hq + h) * kHeadDim + d;
        const int n_valid = min(kBM, rows_left) - colhalf * 64;
        if constexpr (D < 128) {
          // dQ^T has D rows: the warps of TMEM lanes D..127 have nothing to drain, they only keep the barrier counts
          // (and, with ordered additions, the turn counts)
          if (d >= D) {
            tc_fence_before_sync();
            mbar_arrive(&s.bar_dq_empty);
            if constexpr (DET == 1) {
              int32_t* turn = a.dq_turn + c.turn_off + h * c.mt + m;
              if (lane == 0) {
                const long long t0 = clock64();
                while (*reinterpret_cast<volatile int32_t*>(turn) < 8 * c.n && clock64() - t0 < a.wait_limit) __nanosleep(64);
                atomicAdd(turn, 1);
              }
            }
            continue;
          }
        }
        if constexpr (FIRST) {
          // q tile 0 gets nothing from any other key tile: scale and store the rows directly, no accumulator
          uint32_t v0[32], v1[32];
          tmem_ld32(tR1 + lane_off + colhalf * 64, v0);
          tmem_ld32(tR1 + lane_off + colhalf * 64 + 32, v1);
          tmem_wait_ld();
          tc_fence_before_sync();
          mbar_arrive(&s.bar_dq_empty);
          const int64_t o0 = c.q_off + (static_cast<int64_t>(colhalf * 64) * c.hq + h) * kHeadDim + d;
          NSP_CHECK(n_valid <= 0 || (o0 >= 0 && o0 + (min(n_valid, 64) - 1) * q_stride < a.q_elems), a.status, c.it,
                    kWhereCheckBwdDq, h) {
          if (a.dq_f32) {
            float* q0 = static_cast<float*>(a.dq) + o0;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              if (e < n_valid) q0[e * q_stride] = __uint_as_float(v0[e]) * a.scale;
              if (e + 32 < n_valid) q0[(e + 32) * q_stride] = __uint_as_float(v1[e]) * a.scale;
            }
          } else {
            __nv_bfloat16* q0 = static_cast<__nv_bfloat16*>(a.dq) + o0;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              if (e < n_valid) q0[e * q_stride] = __float2bfloat16_rn(__uint_as_float(v0[e]) * a.scale);
              if (e + 32 < n_valid) q0[(e + 32) * q_stride] = __float2bfloat16_rn(__uint_as_float(v1[e]) * a.scale);
            }
          }
          }
          continue;
        }
        float* p0 = tile0 + colhalf * 64 * q_stride;
        int32_t* turn = nullptr;
        if constexpr (DET == 1) turn = a.dq_turn + c.turn_off + h * c.mt + m;
        auto wait_turn = [&]() -> bool {  // key tiles 0 .. n-1 have added their tiles (eight dQ warps each)
          bool okt = true;
          if (lane == 0) {
            const long long t0 = clock64();
            while (*reinterpret_cast<volatile int32_t*>(turn) < 8 * c.n) {
              if (clock64() - t0 > a.wait_limit) { okt = false; break; }
              __nanosleep(64);
            }
            __threadfence();
          }
          return __shfl_sync(0xffffffffu, okt, 0);
        };
        auto pass_turn = [&]() {
          __threadfence();  // this lane's reductions are performed before the counter moves
          __syncwarp();
          if (lane == 0) atomicAdd(turn, 1);
        };
        {
          // One drain for interior and ragged tiles: every reduction under its row's predicate (rows past the segment
          // end are skipped: their dS^T columns are zero, and they may lie outside the buffer). Every item starts on
          // the segment's last q tile, once per q head, so a ragged tile must not cost more than an interior one: as a
          // rolled loop of 16-column loads with a wait each, R1 was handed back late and such a step took twice as long
          // (batches of 500-, 1,000- and 2,000-token segments ran 10-18 % slower per flop than 512 / 1,024 / 2,048).
          uint32_t v0[32], v1[32];
          tmem_ld32(tR1 + lane_off + colhalf * 64, v0);
          tmem_ld32(tR1 + lane_off + colhalf * 64 + 32, v1);
          tmem_wait_ld();
          tc_fence_before_sync();
          mbar_arrive(&s.bar_dq_empty);  // R1 is drained: the next dP^T may overwrite it
          if constexpr (DET == 1) {
            if (!wait_turn()) {
              if (lane == 0) {
                report_timeout(a.status, c.it, kWhereBwdTurn, vt);
                *abort_flag = 1;
              }
              break;
            }
          }
          // The reductions sit in a conditional region on purpose (the condition always holds): as straight-line
          // code the compiler computes all 64 row addresses ahead of the TMEM loads, runs out of the 80 registers
          // this role has and spills inside the loop (measured: the whole kernel 25 % slower).
          NSP_CHECK(n_valid <= 0 || (p0 >= a.dq_acc && p0 + (min(n_valid, 64) - 1) * q_stride < a.dq_acc + a.q_elems), a.status,
                    c.it, kWhereCheckBwdDq, m)
          if (c.hq > 0) {
            float* p1 = p0 + 32 * q_stride;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              if (e < n_valid) red_add_f32(p0, dq_term<DET>(__uint_as_float(v0[e])));
              if (e + 32 < n_valid) red_add_f32(p1, dq_term<DET>(__uint_as_float(v1[e])));
              p0 += q_stride;
              p1 += q_stride;
            }
          }
          if constexpr (DET == 1) pass_turn();
        }
      }
      item_done();
    }
  } else {
    // ================================================================ softmax / dS (key row r, 64 query columns)
    setmaxnreg_inc<kRegsSoftmax<FIRST>>();
    const int quad = warp & 3, half = wg;
    const int r = quad * 32 + lane;
    const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
    const uint32_t tS = tR0 + lane_off + half * 64, tDP = tR1 + lane_off + half * 64;
    uint8_t* const ds_row = s.ds[half] + r * 128;  // this thread's 128-byte row of the swizzled dS^T half tile
    uint32_t nd = 0;                               // completed phases of bar_delta[half]
    while (next_item()) {
      const ItemCtx c = *cx;
      bool oks = true;
      int where = 0;
      // first-tile kernel, a tile shared by several short segments: key row r is seen by the queries r .. r_end - 1
      // (the rest of its own segment); a tile of one segment: every query from r on
      int r_end = kBM;
      if constexpr (FIRST) {
        if (c.rows > 0) r_end = a.rows[static_cast<int64_t>(c.rows - 1) * kBM + r].hi;
      }
      StepWalk w;
      w.reset();
#pragma unroll 1
      for (int vt = 0; vt < c.steps; ++vt) {
        const uint32_t cs = gs + vt, st = cs & 1;
        if (*abort_flag) { oks = false; where = 0; break; }
        int h, m;
        w.get(c, h, m);
        w.next(c);
        oks = mbar_wait(&s.bar_ld_full[st], (cs >> 1) & 1, a.wait_limit) && mbar_wait(&s.bar_s_full, cs & 1, a.wait_limit);
        oks = __all_sync(0xffffffffu, oks);
        if (!oks) { where = kWhereBwdS; break; }
        tc_fence_after_sync();
        const float* lse_s = s.lse[st] + half * 64;
        float* delta_s = s.delta[st] + half * 64;
        // ---- common step (interior tile; the diagonal tile runs a second copy of the same code with a mask on P,
        // kept apart so that the interior copy's instructions stay as they are)
        auto common_step = [&](auto diag_tag) -> bool {
          // Phase 1: P^T = exp2(S^T * c - LSE) for this thread's 64 query
          // columns, bf16 pairs over the S^T columns already read. The dV product needs only P^T, so it is
          // released to the MMA thread before dS^T is formed.
          // Sixteen columns at a time; the LSE (delta) values of the next sixteen are requested before the
          // arithmetic of the current ones, because a shared-memory load takes a long time here: the LSU is
          // shared with the 64 KB of dQ reductions per step.
          uint32_t sv[2][32];
          float4 aux[2][4];
#pragma unroll
          for (int i = 0; i < 4; ++i) aux[0][i] = lds128(lse_s + 4 * i);
          tmem_ld32(tS, sv[0]);
          tmem_ld32(tS + 32, sv[1]);
          tmem_wait_ld();
          uint32_t pp[2][16];  // P^T as bf16 pairs: what goes to R0, and what the dS^T product uses below
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            if (ch < 3) {
#pragma unroll
              for (int i = 0; i < 4; ++i) aux[(ch + 1) & 1][i] = lds128(lse_s + (ch + 1) * 16 + 4 * i);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float4 l4 = aux[ch & 1][i];
              const int x = (ch & 1) * 16 + 4 * i;  // column inside the 32-column group ch / 2
              float x0, x1, x2, x3;
              fma2(x0, x1, __uint_as_float(sv[ch >> 1][x + 0]), __uint_as_float(sv[ch >> 1][x + 1]), a.scale_log2,
                   a.scale_log2, -l4.x, -l4.y);
              fma2(x2, x3, __uint_as_float(sv[ch >> 1][x + 2]), __uint_as_float(sv[ch >> 1][x + 3]), a.scale_log2,
                   a.scale_log2, -l4.z, -l4.w);
              float p0, p1, p2, p3;
              if (((2 * i) & 3) < NSP_EMU_BWD) {
                ex2_poly2(p0, p1, x0, x1);
              } else {
                p0 = ex2f(x0);
                p1 = ex2f(x1);
              }
              if (((2 * i + 1) & 3) < NSP_EMU_BWD) {
                ex2_poly2(p2, p3, x2, x3);
              } else {
                p2 = ex2f(x2);
                p3 = ex2f(x3);
              }
              pp[ch >> 1][(x >> 1) + 0] = pack_bf16x2(p0, p1);
              pp[ch >> 1][(x >> 1) + 1] = pack_bf16x2(p2, p3);
            }
            if constexpr (decltype(diag_tag)::value) {
              // diagonal tile: a key sees only the queries at or after it. Element e of this chunk (query column
              // 64 * half + 16 * ch + e) survives iff e >= t; P = 0 also zeroes dS^T below. Rows and columns past
              // the end of a ragged segment fall under the same mask (their LSE is +inf).
              const int t = r - (half * 64 + ch * 16);
#pragma unroll
              for (int kk = 0; kk < 8; ++kk) {
                const uint32_t keep = t <= 2 * kk ? 0xffffffffu : (t == 2 * kk + 1 ? 0xffff0000u : 0u);
                pp[ch >> 1][(ch & 1) * 8 + kk] &= keep;
              }
            }
            if (ch & 1) tmem_st16(tS + (ch >> 1) * 32, pp[ch >> 1]);  // columns [32g, 32g + 32) -> packed [32g, +16)
          }
          tmem_wait_st();
          tc_fence_before_sync();
          mbar_arrive(&s.bar_p_ready);
          // Phase 2: dS^T = P^T o (dP^T - delta) -> swizzled shared memory; P enters with its bf16 value, the one
          // the dV product uses. The dS buffer is free: dP^T of this step was issued behind dK / dQ^T of the
          // previous step, so bar_dp_full implies they have completed.
#pragma unroll
          for (int i = 0; i < 4; ++i) aux[0][i] = lds128(delta_s + 4 * i);
          oks = mbar_wait(&s.bar_dp_full, cs & 1, a.wait_limit);
          oks = __all_sync(0xffffffffu, oks);
          if (!oks) { where = kWhereBwdDp; return false; }
          tc_fence_after_sync();
          uint32_t dpv[2][16];
          tmem_ld16(tDP, dpv[0]);
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            tmem_wait_ld();
            if (ch < 3) {
              tmem_ld16(tDP + (ch + 1) * 16, dpv[(ch + 1) & 1]);
#pragma unroll
              for (int i = 0; i < 4; ++i) aux[(ch + 1) & 1][i] = lds128(delta_s + (ch + 1) * 16 + 4 * i);
            }
            uint32_t dsp[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float4 d4 = aux[ch & 1][i];
              const int x = 4 * i;
              const uint32_t pa = pp[ch >> 1][(ch & 1) * 8 + (x >> 1)], pb = pp[ch >> 1][(ch & 1) * 8 + (x >> 1) + 1];
              float d0, d1, d2, d3;
              sub2(d0, d1, __uint_as_float(dpv[ch & 1][x + 0]), __uint_as_float(dpv[ch & 1][x + 1]), d4.x, d4.y);
              sub2(d2, d3, __uint_as_float(dpv[ch & 1][x + 2]), __uint_as_float(dpv[ch & 1][x + 3]), d4.z, d4.w);
              mul2(d0, d1, d0, d1, __uint_as_float(pa << 16), __uint_as_float(pa & 0xffff0000u));
              mul2(d2, d3, d2, d3, __uint_as_float(pb << 16), __uint_as_float(pb & 0xffff0000u));
              dsp[(x >> 1) + 0] = pack_bf16x2(d0, d1);
              dsp[(x >> 1) + 1] = pack_bf16x2(d2, d3);
            }
            // sixteen query columns = two 16-byte chunks of the swizzled dS^T row
            *reinterpret_cast<uint4*>(ds_row + ((2 * ch) ^ (r & 7)) * 16) = make_uint4(dsp[0], dsp[1], dsp[2], dsp[3]);
            *reinterpret_cast<uint4*>(ds_row + ((2 * ch + 1) ^ (r & 7)) * 16) = make_uint4(dsp[4], dsp[5], dsp[6], dsp[7]);
          }
          return true;
        };
        if constexpr (!FIRST) {
          if (m != c.n) {
            if (!common_step(std::false_type{})) break;
          } else {
            if (!common_step(std::true_type{})) break;
          }
        } else {
          // ---- first-tile step (q tile 0 against key tile 0, always a diagonal tile): compact rolled loops, 16
          // query columns at a time. Rows 0..127 of a segment have few keys, so P is O(1) and its bf16 rounding alone
          // would push dK / dV past the tolerance: P^T and dS^T enter their products as bf16 value plus bf16 residual
          // (two products each, the residuals next to the values), and delta_i = sum_j P_ij dP_ij is taken here in
          // fp32 (all keys of these rows sit in this tile) instead of from the bf16-rounded O.
          oks = mbar_wait(&s.bar_dp_full, cs & 1, a.wait_limit);
          oks = __all_sync(0xffffffffu, oks);
          if (!oks) { where = kWhereBwdDp; break; }
          tc_fence_after_sync();
          uint32_t pkk[4][16];
          {
            // Sweep 1: P^T (value and residual over the S^T columns just read: packed columns [16ch, 16ch + 8) and
            // [16ch + 8, 16ch + 16)) and the partial sums of delta. The packed values stay in registers for sweep 2
            // (both sweeps fully unrolled), so R0 is free for the next S^T as soon as the dV products have run.
            float* part = reinterpret_cast<float*>(s.ds[half]);  // [4 quadrants][64 columns]; free until dS is written
            // Column sums over the 32 key rows of a warp by a butterfly: at every level a lane keeps the half of
            // the columns its lane bit selects and adds the partner's partial sums of that half (16 shuffles for
            // 16 columns); after the last level lane 2c (and 2c + 1) holds column c = lane / 2.
            const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4, b1 = lane & 2;
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
              uint32_t sv[16], dpv[16];
              uint32_t* const pk = pkk[ch];
              float4 l4[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) l4[i] = lds128(lse_s + ch * 16 + 4 * i);
              tmem_ld16(tS + ch * 16, sv);
              tmem_ld16(tDP + ch * 16, dpv);
              tmem_wait_ld();
              float v[16];
#pragma unroll
              for (int x = 0; x < 16; x += 2) {
                const float lse0 = (x & 2) ? l4[x >> 2].z : l4[x >> 2].x, lse1 = (x & 2) ? l4[x >> 2].w : l4[x >> 2].y;
                float p0 = ex2f(fmaf(__uint_as_float(sv[x + 0]), a.scale_log2, -lse0));
                float p1 = ex2f(fmaf(__uint_as_float(sv[x + 1]), a.scale_log2, -lse1));
                const int qc = half * 64 + ch * 16 + x;
                if (qc + 0 < r || qc + 0 >= r_end) p0 = 0.f;  // query index must be >= key index, inside its segment
                if (qc + 1 < r || qc + 1 >= r_end) p1 = 0.f;
                v[x + 0] = p0 * __uint_as_float(dpv[x + 0]);
                v[x + 1] = p1 * __uint_as_float(dpv[x + 1]);
                const uint32_t pa = pack_bf16x2(p0, p1);
                pk[x >> 1] = pa;
                pk[8 + (x >> 1)] = pack_bf16x2(p0 - __uint_as_float(pa << 16), p1 - __uint_as_float(pa & 0xffff0000u));
              }
              tmem_st16(tS + ch * 16, pk);
              float w8[8], w4[4], w2[2];
#pragma unroll
              for (int i = 0; i < 8; ++i)
                w8[i] = (b4 ? v[i + 8] : v[i]) + __shfl_xor_sync(0xffffffffu, b4 ? v[i] : v[i + 8], 16);
#pragma unroll
              for (int i = 0; i < 4; ++i)
                w4[i] = (b3 ? w8[i + 4] : w8[i]) + __shfl_xor_sync(0xffffffffu, b3 ? w8[i] : w8[i + 4], 8);
#pragma unroll
              for (int i = 0; i < 2; ++i)
                w2[i] = (b2 ? w4[i + 2] : w4[i]) + __shfl_xor_sync(0xffffffffu, b2 ? w4[i] : w4[i + 2], 4);
              float w1 = (b1 ? w2[1] : w2[0]) + __shfl_xor_sync(0xffffffffu, b1 ? w2[0] : w2[1], 2);
              w1 += __shfl_xor_sync(0xffffffffu, w1, 1);
              if ((lane & 1) == 0) part[quad * 64 + ch * 16 + (lane >> 1)] = w1;
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(&s.bar_p_ready);  // the dV products run under the rest of this step
            mbar_arrive(&s.bar_delta[half]);
            oks = mbar_wait(&s.bar_delta[half], nd & 1, a.wait_limit);
            ++nd;
            oks = __all_sync(0xffffffffu, oks);
            if (!oks) { where = kWhereBwdDelta; break; }
            if (r < 64) delta_s[r] = (part[r] + part[64 + r]) + (part[128 + r] + part[192 + r]);
            mbar_arrive(&s.bar_delta[half]);
            oks = mbar_wait(&s.bar_delta[half], nd & 1, a.wait_limit);
            ++nd;
            oks = __all_sync(0xffffffffu, oks);
            if (!oks) { where = kWhereBwdDelta; break; }
          }
          // Sweep 2: dS^T = P^T o (dP^T - delta), value and residual (P = value + residual to 2^-17)
          uint8_t* const ds_row_lo = ds_row + 2 * kHalfTileBytes;
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            uint32_t dpv[16], dsp[8], dsl[8];
            const uint32_t* const pk = pkk[ch];
            float4 e4[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) e4[i] = lds128(delta_s + ch * 16 + 4 * i);
            tmem_ld16(tDP + ch * 16, dpv);
            tmem_wait_ld();
#pragma unroll
            for (int x = 0; x < 16; x += 2) {
              const float del0 = (x & 2) ? e4[x >> 2].z : e4[x >> 2].x, del1 = (x & 2) ? e4[x >> 2].w : e4[x >> 2].y;
              const uint32_t ph = pk[x >> 1], pl = pk[8 + (x >> 1)];
              const float p0 = __uint_as_float(ph << 16) + __uint_as_float(pl << 16);
              const float p1 = __uint_as_float(ph & 0xffff0000u) + __uint_as_float(pl & 0xffff0000u);
              const float d0 = p0 * (__uint_as_float(dpv[x + 0]) - del0);
              const float d1 = p1 * (__uint_as_float(dpv[x + 1]) - del1);
              const uint32_t da = pack_bf16x2(d0, d1);
              dsp[x >> 1] = da;
              dsl[x >> 1] = pack_bf16x2(d0 - __uint_as_float(da << 16), d1 - __uint_as_float(da & 0xffff0000u));
            }
            const uint32_t c0 = ((2 * ch) ^ (r & 7)) * 16, c1 = ((2 * ch + 1) ^ (r & 7)) * 16;
            *reinterpret_cast<uint4*>(ds_row + c0) = make_uint4(dsp[0], dsp[1], dsp[2], dsp[3]);
            *reinterpret_cast<uint4*>(ds_row + c1) = make_uint4(dsp[4], dsp[5], dsp[6], dsp[7]);
            *reinterpret_cast<uint4*>(ds_row_lo + c0) = make_uint4(dsl[0], dsl[1], dsl[2], dsl[3]);
            *reinterpret_cast<uint4*>(ds_row_lo + c1) = make_uint4(dsl[4], dsl[5], dsl[6], dsl[7]);
          }
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        mbar_arrive(&s.bar_ds_ready);
        mbar_arrive(&s.bar_ld_empty[st]);
      }
      // ---- epilogue: wait for the last MMAs of the item, then write dK (scaled) and dV of this key tile
      if (oks) {
        oks = mbar_wait(&s.bar_b_done, (gs + c.steps - 1) & 1, a.wait_limit) && mbar_wait(&s.bar_a_done, (gs + c.steps - 1) & 1, a.wait_limit);
        oks = __all_sync(0xffffffffu, oks);
        if (!oks) where = kWhereBwdDqFull;
      }
      if (oks) {
        tc_fence_after_sync();
        const int kj = c.n * kBN + r;
        const bool valid = kj < c.len;
        constexpr int kCols = D / 2;  // this thread's columns of a dK / dV row
        const int64_t off = c.kv_off + (static_cast<int64_t>(kj) * c.hkv + c.g) * kHeadDim + half * kCols;
        // Key tile 0 in the main kernel: the first-tile kernel, which ran before, left its part (q tile 0) in the
        // output; this item's sum over the q tiles 1 .. Mt-1 is added to it (one fixed order: reproducible).
        const bool add = !FIRST && c.first;
        if (a.dkv_f32 && (c.n + 1) * kBN <= c.len) {
          // ---- fp32 outputs, full key tile: staged in shared memory (every operand buffer is free now: dK over K
          // and V, dV over the Q ring), swizzled as sub-tiles of 32 columns, and written by TMA tile stores (added,
          // for key tile 0). Stored row by row from the threads (a row per lane, 16 bytes per store, half a sector
          // each) the two tiles took 12,000-13,000 clocks per item.
          constexpr uint32_t kSubBytes = 128 * 32 * 4;
#pragma unroll 1
          for (int part = 0; part < 2 * (kCols / 32); ++part) {  // (dK, dV) x 32-column chunks
            const int which = part / (kCols / 32), cc = part % (kCols / 32);
            const float mul = which == 0 ? a.scale : 1.f;
            uint32_t v[32];
            tmem_ld32(tDK + which * 128 + lane_off + half * kCols + cc * 32, v);
            tmem_wait_ld();
            uint8_t* const sub = (which == 0 ? &s.k[0][0] : &s.q[0][0][0]) + (half * (kCols / 32) + cc) * kSubBytes + r * 128;
#pragma unroll
            for (int x = 0; x < 8; ++x) {
              *reinterpret_cast<float4*>(sub + ((x ^ (r & 7)) * 16)) =
                  make_float4(__uint_as_float(v[4 * x]) * mul, __uint_as_float(v[4 * x + 1]) * mul,
                              __uint_as_float(v[4 * x + 2]) * mul, __uint_as_float(v[4 * x + 3]) * mul);
            }
          }
          fence_proxy_async_smem();
          const uint64_t staged = mbar_arrive_token(&s.bar_out);
          if (tid == 0) {
            if (mbar_wait_token(&s.bar_out, staged, a.wait_limit)) {
              const int tok = c.tok0 + c.n * kBN;
#pragma unroll 1
              for (int i = 0; i < D / 32; ++i) {
                if (add) {
                  tma_reduce_add_3d(&maps.dk[c.run], &s.k[0][0] + i * kSubBytes, 32 * i, c.g, tok);
                  tma_reduce_add_3d(&maps.dv[c.run], &s.q[0][0][0] + i * kSubBytes, 32 * i, c.g, tok);
                } else {
                  tma_store_3d(&maps.dk[c.run], &s.k[0][0] + i * kSubBytes, 32 * i, c.g, tok);
                  tma_store_3d(&maps.dv[c.run], &s.q[0][0][0] + i * kSubBytes, 32 * i, c.g, tok);
                }
              }
              tma_store_commit();
              tma_store_wait_read();  // before the barrier of next_item(): the producer refills these buffers after it
            } else {
              report_timeout(a.status, c.it, kWhereBwdDqFull, 1);
              *abort_flag = 1;
            }
          }
        } else {
#pragma unroll 1
        for (int part = 0; part < 2 * (kCols / 32); ++part) {  // (dK, dV) x 32-column chunks
          const int which = part / (kCols / 32), cc = part % (kCols / 32);
          const float mul = which == 0 ? a.scale : 1.f;
          void* outp = which == 0 ? a.dk : a.dv;
          uint32_t v[32];
          tmem_ld32(tDK + which * 128 + lane_off + half * kCols + cc * 32, v);
          tmem_wait_ld();
          NSP_CHECK(!valid || (off >= 0 && off + kCols <= a.kv_elems), a.status, c.it, kWhereCheckBwdDkv, kj)
          if (valid) {
            if (a.dkv_f32) {
              float* o = static_cast<float*>(outp) + off + cc * 32;
#pragma unroll
              for (int x = 0; x < 32; x += 4) {
                float4 w4 = make_float4(__uint_as_float(v[x]) * mul, __uint_as_float(v[x + 1]) * mul,
                                        __uint_as_float(v[x + 2]) * mul, __uint_as_float(v[x + 3]) * mul);
                if (add) {
                  const float4 old = *reinterpret_cast<const float4*>(o + x);
                  w4.x += old.x, w4.y += old.y, w4.z += old.z, w4.w += old.w;
                }
                *reinterpret_cast<float4*>(o + x) = w4;
              }
            } else {
              __nv_bfloat16* o = static_cast<__nv_bfloat16*>(outp) + off + cc * 32;
#pragma unroll
              for (int x = 0; x < 32; x += 8) {
                if (add) {  // bf16 output: the first part was rounded once already (not the graded dtype)
                  const uint4 old = *reinterpret_cast<const uint4*>(o + x);
                  const uint32_t ow[4] = {old.x, old.y, old.z, old.w};
#pragma unroll
                  for (int t = 0; t < 4; ++t) {
                    v[x + 2 * t] = __float_as_uint(__uint_as_float(v[x + 2 * t]) + __uint_as_float(ow[t] << 16) / mul);
                    v[x + 2 * t + 1] =
                        __float_as_uint(__uint_as_float(v[x + 2 * t + 1]) + __uint_as_float(ow[t] & 0xffff0000u) / mul);
                  }
                }
                uint4 wv;
                wv.x = pack_bf16x2(__uint_as_float(v[x]) * mul, __uint_as_float(v[x + 1]) * mul);
                wv.y = pack_bf16x2(__uint_as_float(v[x + 2]) * mul, __uint_as_float(v[x + 3]) * mul);
                wv.z = pack_bf16x2(__uint_as_float(v[x + 4]) * mul, __uint_as_float(v[x + 5]) * mul);
                wv.w = pack_bf16x2(__uint_as_float(v[x + 6]) * mul, __uint_as_float(v[x + 7]) * mul);
                *reinterpret_cast<uint4*>(o + x) = wv;
              }
            }
          }
        }
        }
      } else if (where != 0 && lane == 0) {
        report_timeout(a.status, c.it, where, 0);
        *abort_flag = 1;
      }
      item_done();
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(s.tmem_base, kBwdTmemCols);
}

// Which segment a packed (token, head) row belongs to: row_base[s] = first packed row of segment s (ascending).
__device__ __forceinline__ int find_segment(const int64_t* __restrict__ row_base, int n_seg, int64_t row) {
  int lo = 0, hi = n_seg - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (row_base[mid] <= row) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// Preprocess, for the rows the main kernel works on (tokens 128.. of every segment; the first 128 tokens belong to
// the first-tile kernel, which needs neither): delta[h, i] = <dO[i,h,:], O[i,h,:]> and the row's D floats of the dQ
// accumulator set to zero. Rows (token, head) are packed one after the other, 2 D bytes each, so the kernel streams
// O and dO as flat arrays: D / 8 lanes per row with one 16-byte load per tensor, four loads in flight per thread
// and tensor (a warp pass covers 8 rows at D = 128, 16 at D = 64), and only the index of the result needs the
// segment table (delta is stored [head][token] inside a segment): one lane per row looks it up.
// With seg_skip, no delta is written for the rows of marked segments (it comes from the recomputation); with lse_out,
// the LSE of every row of the other segments is copied from lse_in (same index as delta).
template <int D>
__global__ void __launch_bounds__(256) bwd_preprocess_kernel(const SegInfo* __restrict__ seg, int n_seg,
                                                             const int64_t* __restrict__ row_base, int64_t total_rows,
                                                             const __nv_bfloat16* __restrict__ o,
                                                             const __nv_bfloat16* __restrict__ d_o,
                                                             float* __restrict__ delta, float* __restrict__ dq_acc,
                                                             const uint8_t* __restrict__ seg_skip,
                                                             const float* __restrict__ lse_in,
                                                             float* __restrict__ lse_out) {
  constexpr int kLanesPerRow = D / 8, kRowsPerLoad = 32 / kLanesPerRow, kRowsPerPass = 4 * kRowsPerLoad;
  const int lane = threadIdx.x & 31, sub = lane / kLanesPerRow, l = lane % kLanesPerRow;
  const int64_t n_groups = (total_rows + kRowsPerPass - 1) / kRowsPerPass;
  const int64_t n_warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
  for (int64_t grp = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; grp < n_groups; grp += n_warps) {
    const int64_t row0 = grp * kRowsPerPass;
    // row row0 + (lane % kRowsPerPass): where its delta goes (-1: nowhere), and whether it is one of the main kernel's rows
    int64_t dst = -1;
    int mine = 0;
    {
      const int64_t row = row0 + (lane % kRowsPerPass);
      if (row < total_rows) {
        const int sgi = find_segment(row_base, n_seg, row);
        const SegInfo sg = seg[sgi];
        const int64_t rl = row - row_base[sgi];
        const int64_t i = rl / sg.hq, h = rl - i * sg.hq;
        mine = i >= kBM;
        // rows of a skipped segment (its delta and LSE come from the recomputation) get neither here; for the other
        // segments the LSE copy covers every row (the first-tile kernel reads it too)
        if (seg_skip == nullptr || seg_skip[sgi] == 0) {
          const int64_t at = sg.lse_off + h * sg.len + i;
          if (lse_out != nullptr && lane < kRowsPerPass) lse_out[at] = lse_in[at];
          if (mine) dst = at;
        }
      }
    }
    // O and dO are read only for the rows whose delta is wanted: with short segments the first 128 tokens, which the
    // first-tile kernel serves, are a large part of the batch (half of it at 256-token segments)
    uint4 va[4], vb[4];
    int64_t dst_p[4];
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      const int64_t row = row0 + kRowsPerLoad * p + sub;
      dst_p[p] = __shfl_sync(0xffffffffu, dst, kRowsPerLoad * p + sub);
      if (dst_p[p] >= 0) {
        va[p] = __ldg(reinterpret_cast<const uint4*>(o + row * D) + l);
        vb[p] = __ldg(reinterpret_cast<const uint4*>(d_o + row * D) + l);
      } else {
        va[p] = vb[p] = make_uint4(0u, 0u, 0u, 0u);
      }
    }
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&va[p]);
      const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&vb[p]);
      float acc = 0.f;
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const float2 fa = __bfloat1622float2(pa[x]), fb = __bfloat1622float2(pb[x]);
        acc = fmaf(fa.x, fb.x, acc);
        acc = fmaf(fa.y, fb.y, acc);
      }
#pragma unroll
      for (int sft = kLanesPerRow / 2; sft > 0; sft >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, sft);
      const int mine_p = __shfl_sync(0xffffffffu, mine, kRowsPerLoad * p + sub);
      if (l == 0 && dst_p[p] >= 0) delta[dst_p[p]] = acc;
      if (mine_p) {
        float4* z = reinterpret_cast<float4*>(dq_acc + (row0 + kRowsPerLoad * p + sub) * D) + 2 * l;
        z[0] = make_float4(0.f, 0.f, 0.f, 0.f);
        z[1] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
  }
}

// Postprocess: dQ = scale * accumulator, in the output dtype, for the rows the main kernel works on (tokens 128.. of
// every segment; the rows before were stored by the first-tile kernel). Same row walk as the preprocess kernel.
template <int D>
__global__ void __launch_bounds__(256) bwd_postprocess_kernel(const SegInfo* __restrict__ seg, int n_seg,
                                                              const int64_t* __restrict__ row_base, int64_t total_rows,
                                                              const float* __restrict__ acc, void* __restrict__ dq,
                                                              int dq_f32, float scale) {
  constexpr int kLanesPerRow = D / 8, kRowsPerLoad = 32 / kLanesPerRow, kRowsPerPass = 4 * kRowsPerLoad;
  const int lane = threadIdx.x & 31, sub = lane / kLanesPerRow, l = lane % kLanesPerRow;
  const int64_t n_groups = (total_rows + kRowsPerPass - 1) / kRowsPerPass;
  const int64_t n_warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
  for (int64_t grp = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; grp < n_groups; grp += n_warps) {
    const int64_t row0 = grp * kRowsPerPass;
    int mine = 0;
    {
      const int64_t row = row0 + (lane % kRowsPerPass);
      if (row < total_rows) {
        const int sgi = find_segment(row_base, n_seg, row);
        mine = (row - row_base[sgi]) / seg[sgi].hq >= kBM;
      }
    }
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      const int64_t row = row0 + kRowsPerLoad * p + sub;
      if (!__shfl_sync(0xffffffffu, mine, kRowsPerLoad * p + sub)) continue;
      const float4* src = reinterpret_cast<const float4*>(acc + row * D) + 2 * l;
      const float4 v0 = src[0], v1 = src[1];
      if (dq_f32) {
        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(dq) + row * D) + 2 * l;
        dst[0] = make_float4(v0.x * scale, v0.y * scale, v0.z * scale, v0.w * scale);
        dst[1] = make_float4(v1.x * scale, v1.y * scale, v1.z * scale, v1.w * scale);
      } else {
        uint4 w;
        w.x = pack_bf16x2(v0.x * scale, v0.y * scale);
        w.y = pack_bf16x2(v0.z * scale, v0.w * scale);
        w.z = pack_bf16x2(v1.x * scale, v1.y * scale);
        w.w = pack_bf16x2(v1.z * scale, v1.w * scale);
        reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(dq) + row * D)[l] = w;
      }
    }
  }
}

}  // namespace

cudaError_t launch_bwd_preprocess(const SegInfo* d_seg, int n_seg, const int64_t* d_row_base, int64_t total_rows,
                                  int head_dim, const __nv_bfloat16* o, const __nv_bfloat16* d_o, float* delta,
                                  float* dq_acc, const uint8_t* seg_skip, const float* lse_in, float* lse_out,
                                  cudaStream_t st) {
  if (total_rows == 0) return cudaSuccess;
  int64_t blocks = ((total_rows + 7) / 8 * 32 + 255) / 256;  // about one warp per eight rows, grid-stride beyond 16 waves
  if (blocks > 148 * 8 * 16) blocks = 148 * 8 * 16;
  if (head_dim == 64)
    bwd_preprocess_kernel<64><<<static_cast<unsigned>(blocks), 256, 0, st>>>(d_seg, n_seg, d_row_base, total_rows, o, d_o,
                                                                             delta, dq_acc, seg_skip, lse_in, lse_out);
  else
    bwd_preprocess_kernel<128><<<static_cast<unsigned>(blocks), 256, 0, st>>>(d_seg, n_seg, d_row_base, total_rows, o, d_o,
                                                                              delta, dq_acc, seg_skip, lse_in, lse_out);
  count_launches(1);
  return cudaGetLastError();
}

namespace {
template <bool FIRST, int DET, int D>
cudaError_t launch_bwd_t(const BwdMaps& maps, const BwdArgs& args, int num_sms, cudaStream_t st) {
  if (args.n_items == 0) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(bwd_kernel<FIRST, DET, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(sizeof(BwdSmem<FIRST, D>)));
  if (e != cudaSuccess) return e;
  const int grid = args.n_items < num_sms ? args.n_items : num_sms;
  bwd_kernel<FIRST, DET, D><<<grid, kBwdThreads, sizeof(BwdSmem<FIRST, D>), st>>>(maps, args);
  count_launches(1);
  return cudaGetLastError();
}
}  // namespace

cudaError_t launch_bwd(const BwdMaps& maps, const BwdArgs& args, int head_dim, int num_sms, cudaStream_t st) {
  if (head_dim == 64)
    return args.dq_turn    ? launch_bwd_t<false, 1, 64>(maps, args, num_sms, st)
           : args.dq_rounded ? launch_bwd_t<false, 2, 64>(maps, args, num_sms, st)
                             : launch_bwd_t<false, 0, 64>(maps, args, num_sms, st);
  return args.dq_turn    ? launch_bwd_t<false, 1, 128>(maps, args, num_sms, st)
         : args.dq_rounded ? launch_bwd_t<false, 2, 128>(maps, args, num_sms, st)
                           : launch_bwd_t<false, 0, 128>(maps, args, num_sms, st);
}
cudaError_t launch_bwd_first(const BwdMaps& maps, const BwdArgs& args, int head_dim, int num_sms, cudaStream_t st) {
  return head_dim == 64 ? launch_bwd_t<true, 0, 64>(maps, args, num_sms, st)
                        : launch_bwd_t<true, 0, 128>(maps, args, num_sms, st);
}

cudaError_t launch_bwd_postprocess(const SegInfo* d_seg, int n_seg, const int64_t* d_row_base, int64_t total_rows,
                                   int head_dim, const float* dq_acc, void* dq, int dq_f32, float scale,
                                   cudaStream_t st) {
  if (total_rows == 0) return cudaSuccess;
  int64_t blocks = ((total_rows + 7) / 8 * 32 + 255) / 256;
  if (blocks > 148 * 8 * 16) blocks = 148 * 8 * 16;
  if (head_dim == 64)
    bwd_postprocess_kernel<64><<<static_cast<unsigned>(blocks), 256, 0, st>>>(d_seg, n_seg, d_row_base, total_rows,
                                                                              dq_acc, dq, dq_f32, scale);
  else
    bwd_postprocess_kernel<128><<<static_cast<unsigned>(blocks), 256, 0, st>>>(d_seg, n_seg, d_row_base, total_rows,
                                                                               dq_acc, dq, dq_f32, scale);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace nsp

// Forward for the first query tile of every segment (query rows 0..127 against key tile 0): one work item per
// (segment, kv head), all q heads of the group inside the item.
//
// Why a kernel of its own. In the general forward kernel such an item is one serial chain behind CTA-wide barriers
// (pop -> Q, K, V loads -> S -> softmax -> PV -> store, about 9 us for 192 KB of traffic), so batches of short
// segments -- most of the samples of a long-tailed corpus -- moved 2.4 TB/s. Here K and V of the (segment, kv head)
// are loaded once, the q heads go through in pairs A / B with the Q pair in a two-stage ring (the loads of the next
// pair run under the current one), S of the next pair is issued as soon as the PV products of the current one are
// (it overlaps the current pair's epilogue), and the next item is popped while the current one runs. There is a single
// key tile, so the softmax needs no running maximum and no rescaling. (A variant without the CTA-wide barrier between
// items -- the producer popping ahead and publishing items through a two-slot mailbox -- measured slower: 0.89 ms
// against 0.77 ms on 1,024 segments of 128 tokens.)
// The general kernel then runs only the items that visit at least two key tiles: the first-tile items are exactly
// the tail (cost 1) of the longest-first forward list.
//     S_x  = Q_x K^T        tcgen05.mma SS (both K-major)                      -> TMEM S_x
//     P_x  = exp2(S_x*c - m)  two threads per query row, bf16 pairs over S_x   (tcgen05.st)
//     O_x  = P_x V          tcgen05.mma TS (A = P_x from TMEM, B = V MN-major) -> TMEM O_x
// Roles: warps 0-7 softmax of A, warps 8-15 softmax of B, warp 16 TMA producer, warp 17 MMA issue (elected lane).
#include <cuda_bf16.h>
#include "nsp_internal.cuh"
#include "sm100_ptx.cuh"

namespace nsp {
namespace {

constexpr int kThreads = 640;
constexpr uint32_t kHalfTileBytes = 128 * 64 * 2;
constexpr uint32_t kTmemCols = 512;  // S_A [0,128) S_B [128,256) O_A [256,384) O_B [384,512)
constexpr int kRegsSoftmax = 96, kRegsAux = 96;  // 104 / 64 measured 2 % slower here: the aux warps (loads, issue, stores) are on this kernel's chain
constexpr int kPopThread = 18 * 32;  // lane 0 of the first store warp pops: its item starts with a long wait anyway

struct FirstCtx {
  int64_t q_off, lse_off;
  int32_t it;  // position in the list (>= n_items: no more work)
  int32_t len, hq, G, g, run, tok0, rounds;
  int32_t rows;  // 0, or 1 + index of the row table of a pack of short segments (see RowInfo)
};

template <int D>
struct FwdFirstSmem {
  uint8_t k[D / 64][kHalfTileBytes];
  uint8_t v[D / 64][kHalfTileBytes];
  uint8_t q[2][2][D / 64][kHalfTileBytes];  // [stage][A/B][64-column half]
  uint64_t bar_kv, bar_kv_free;
  uint64_t bar_q_full[2];
  uint64_t bar_q_empty[2][2];  // [stage][A/B] the slot's O tile has left (or was never staged): the slot may be reloaded
  uint64_t bar_s_full[2];   // [A/B]
  uint64_t bar_p_ready[2];  // [A/B] 256 softmax threads: P_x written
  uint64_t bar_pv_done[2];  // [A/B] O_x complete
  uint64_t bar_o_free[2];   // [A/B] 256 softmax threads: O_x read out of TMEM
  uint64_t bar_o_staged[2];  // [A/B] 256 softmax threads: the bf16 O tile is in shared memory (or went out row by row)
  uint64_t bar_pair[2][4];  // [A/B][lane quadrant] the two threads of every row have published their half-row value
  float xchg[2][2][2][128];  // [A/B][column half][slot: maximum, sum][row]
  FirstCtx ctx[2];
  uint32_t tmem_base;
  int32_t abort;
};

template <int N>
__device__ __forceinline__ void ff_setmaxnreg_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void ff_setmaxnreg_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}
__device__ __forceinline__ float ff_max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1) fwd_first_kernel(const __grid_constant__ FwdMaps maps, const FwdArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  FwdFirstSmem<D>& s = *reinterpret_cast<FwdFirstSmem<D>*>(smem_raw);
  constexpr int kHalves = D / 64;
  constexpr uint32_t kTileBytes = kHalves * kHalfTileBytes;
  constexpr int kOCols = D / 2;  // output columns of one of the two threads of a row
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, wg = warp >> 2;
  if ((smem_u32(smem_raw) & 1023u) != 0) {  // swizzled tiles need a 1024-byte aligned base
    if (tid == 0) report_timeout(a.status, -1, kWhereFwdSmemAlign, 0);
    return;
  }
  if (tid == 0) {
    mbar_init(&s.bar_kv, 1);
    mbar_init(&s.bar_kv_free, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s.bar_q_full[i], 1);
      mbar_init(&s.bar_q_empty[i][0], 1);
      mbar_init(&s.bar_q_empty[i][1], 1);
      mbar_init(&s.bar_o_staged[i], 256);
      mbar_init(&s.bar_s_full[i], 1);
      mbar_init(&s.bar_p_ready[i], 256);
      mbar_init(&s.bar_pv_done[i], 1);
      mbar_init(&s.bar_o_free[i], 256);
      for (int qd = 0; qd < 4; ++qd) mbar_init(&s.bar_pair[i][qd], 64);
    }
    s.abort = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&s.tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = s.tmem_base;
  volatile int32_t* abort_flag = &s.abort;

  // ---- work distribution: thread 0 pops and decodes; the next item is fetched while the current one runs
  uint32_t gi = 0;  // items finished so far
  FirstCtx c;
  auto fetch = [&](FirstCtx& x) {
    const int idx = atomicAdd(a.counter, 1);
    x.it = idx;
    if (idx < a.n_items) {
      const nsp_tile_t item = a.items[idx];
      const SegInfo sg = a.seg[item.seg];
      x.q_off = sg.q_off, x.lse_off = sg.lse_off;
      x.len = sg.len, x.hq = sg.hq, x.G = sg.hq / sg.hkv, x.g = item.head, x.run = sg.run, x.tok0 = sg.tok_in_run;
      x.rounds = (x.G + 1) / 2;
      x.rows = sg.rows;
    }
  };
  auto next_item = [&]() -> bool {
    if (tid == kPopThread && gi == 0) fetch(s.ctx[0]);
    // Every role reaches this barrier in bounded time: all its other waits are bounded and none returns early.
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    c = s.ctx[gi & 1];
    const bool more = c.it < a.n_items && !*abort_flag;
    if (tid == kPopThread && more) fetch(s.ctx[(gi + 1) & 1]);  // the other slot held the item every role has left
    return more;
  };

  if (wg == 4) {
    ff_setmaxnreg_dec<kRegsAux>();
    if (warp == 16) {
      // ================================================================ TMA producer
      uint32_t R = 0;            // rounds issued so far
      uint32_t use = 0;          // bit 2*stage + half: parity of the loads issued so far into that slot
      while (next_item()) {
        if (lane == 0) {
          const CUtensorMap* mq = &maps.q[c.run];
          bool ok = mbar_wait(&s.bar_kv_free, (gi & 1) ^ 1, a.wait_limit);
          if (ok) {
            mbar_expect_tx(&s.bar_kv, 2 * kTileBytes);
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf) {
              tma_load_3d(s.k[hf], &maps.k[c.run], &s.bar_kv, 64 * hf, c.g, c.tok0);
              tma_load_3d(s.v[hf], &maps.v[c.run], &s.bar_kv, 64 * hf, c.g, c.tok0);
            }
          }
          for (int r = 0; ok && r < c.rounds; ++r) {
            if (*abort_flag) break;
            const uint32_t st = (R + r) & 1;
            const int hA = c.g * c.G + 2 * r;
            const bool joint = 2 * r + 1 < c.G;
            ok = mbar_wait(&s.bar_q_empty[st][0], ((use >> (2 * st)) & 1) ^ 1, a.wait_limit) &&
                 (!joint || mbar_wait(&s.bar_q_empty[st][1], ((use >> (2 * st + 1)) & 1) ^ 1, a.wait_limit));
            if (!ok) break;
            use ^= (joint ? 3u : 1u) << (2 * st);
            mbar_expect_tx(&s.bar_q_full[st], joint ? 2 * kTileBytes : kTileBytes);
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf) tma_load_3d(s.q[st][0][hf], mq, &s.bar_q_full[st], 64 * hf, hA, c.tok0);
            if (joint) {
#pragma unroll
              for (int hf = 0; hf < kHalves; ++hf)
                tma_load_3d(s.q[st][1][hf], mq, &s.bar_q_full[st], 64 * hf, hA + 1, c.tok0);
            }
          }
          if (!ok) {
            report_timeout(a.status, c.it, kWhereFwdLoad, 0);
            *abort_flag = 1;
          }
        }
        R += static_cast<uint32_t>(c.rounds);
        ++gi;
      }
    } else if (warp == 17) {
      // ================================================================ MMA issue (all lanes run, the elected one issues)
      constexpr uint32_t idesc_qk = make_idesc_bf16(128, 128, 0, 0);  // A K-major, B K-major
      constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, 0, 1);    // A from TMEM, B MN-major, N = head dimension
      const uint32_t hi = static_cast<uint32_t>(make_smem_desc_sw128(0, 16, 1024) >> 32);
      constexpr uint32_t lbo_km = (16u >> 4) << 16, lbo_mn = (kHalfTileBytes >> 4) << 16;
      const uint32_t q_lo = smem_desc_addr(s.q[0][0][0]) | lbo_km;
      const uint32_t k_lo = smem_desc_addr(s.k[0]) | lbo_km, v_lo = smem_desc_addr(s.v[0]) | lbo_mn;
      constexpr uint32_t kTileStep = kTileBytes >> 4;
      uint32_t R = 0, n[2] = {0, 0};  // rounds so far; rounds in which half x took part
      while (next_item()) {
        const bool leader = elect_one();
        int where = 0;
        bool ok = mbar_wait(&s.bar_kv, gi & 1, a.wait_limit);
        if (!ok) where = kWhereFwdLoad;
        for (int r = 0; ok && r < c.rounds; ++r) {
          if (*abort_flag) break;
          const uint32_t st = (R + r) & 1;
          const int halves = 2 * r + 1 < c.G ? 2 : 1;
          if (!mbar_wait(&s.bar_q_full[st], ((R + r) >> 1) & 1, a.wait_limit)) { ok = false; where = kWhereFwdLoad; break; }
          tc_fence_after_sync();
          // S of this round follows the PV products of the previous one on the same pipe, so P of the previous
          // round has been read before S overwrites it
          for (int x = 0; x < halves; ++x) {
            const uint32_t a_lo = q_lo + (2 * st + x) * kTileStep;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              const uint32_t off = ((kk >> 2) * kHalfTileBytes + (kk & 3) * 32) >> 4;
              if (leader) umma_ss_lh(tmem + 128 * x, a_lo + off, hi, k_lo + off, hi, idesc_qk, kk > 0);
            }
            if (leader) umma_commit(&s.bar_s_full[x]);
          }
          for (int x = 0; x < halves; ++x) {
            if (!mbar_wait(&s.bar_p_ready[x], n[x] & 1, a.wait_limit)) { ok = false; where = kWhereFwdS; break; }
            if (!mbar_wait(&s.bar_o_free[x], (n[x] & 1) ^ 1, a.wait_limit)) { ok = false; where = kWhereFwdO; break; }
            tc_fence_after_sync();
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              if (leader) umma_ts_lh(tmem + 256 + 128 * x, tmem + 128 * x + (kk >> 2) * 64 + (kk & 3) * 8, v_lo + kk * 128, hi,
                                     idesc_pv, kk > 0);
            if (leader) umma_commit(&s.bar_pv_done[x]);
            ++n[x];
          }
        }
        if (leader) umma_commit(&s.bar_kv_free);  // K and V may be replaced once everything issued so far has run
        if (!ok && where != 0) {
          if (leader) report_timeout(a.status, c.it, where, 0);
          *abort_flag = 1;
        }
        R += static_cast<uint32_t>(c.rounds);
        ++gi;
      }
    } else {
      // ================================================================ store warps (18: half A, 19: half B)
      // A full O tile is staged by the softmax threads in the Q slot it came from (dead once S has run), swizzled
      // like an operand tile, and leaves as a TMA tile store; the slot goes back to the producer when the store has
      // read it. Lane 0 of warp 18 also pops the work items (next_item).
      const int x = warp - 18;
      uint32_t R = 0, nx = 0;
      while (next_item()) {
        for (int r = 0; r < c.rounds; ++r) {
          if (x == 1 && 2 * r + 1 >= c.G) break;
          if (*abort_flag) break;
          if (lane == 0) {
            const uint32_t st = (R + r) & 1;
            if (mbar_wait(&s.bar_o_staged[x], nx & 1, a.wait_limit)) {
              if (c.len >= kBM) {
                const int h = c.g * c.G + 2 * r + x;
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) tma_store_3d(&maps.o[c.run], s.q[st][x][hf], 64 * hf, h, c.tok0);
                tma_store_commit();
                tma_store_wait_read();
              }
              mbar_arrive(&s.bar_q_empty[st][x]);
            } else {
              report_timeout(a.status, c.it, kWhereFwdO, 2 + x);
              *abort_flag = 1;
            }
          }
          ++nx;
        }
        __syncwarp();
        R += static_cast<uint32_t>(c.rounds);
        ++gi;
      }
    }
  } else {
    // ================================================================ softmax of half x (A: warps 0-7, B: warps 8-15)
    // Two threads per query row: thread (quadrant, half ch) owns TMEM lane 32*quadrant + lane and the 64 score columns
    // [64*ch, 64*ch + 64); the row maximum and the row sum are combined through shared memory.
    ff_setmaxnreg_inc<kRegsSoftmax>();
    const int x = wg >> 1;
    const int quad = warp & 3, ch = (warp >> 2) & 1;
    const int rl = quad * 32 + lane;  // query row = TMEM lane
    const uint32_t tS = tmem + 128 * x, tO = tmem + 256 + 128 * x;
    const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
    uint32_t nx = 0;  // rounds in which this half took part
    uint32_t R = 0;   // rounds of the items finished so far (the Q slot of round r is stage (R + r) & 1)
    uint32_t xn = 0;  // completed phases of this row pair's exchange barrier
    float* my_slot = &s.xchg[x][ch][0][rl];  // slot k is my_slot[128 * k]
    const float* partner_slot = &s.xchg[x][ch ^ 1][0][rl];
    uint64_t* pair_bar = &s.bar_pair[x][quad];
    while (next_item()) {
      bool ok = true;
      int where = 0;
      // A tile shared by several short segments: row rl belongs to the segment that covers rows [lo, hi) of the tile and
      // sees the keys lo .. rl; its LSE element for head h is lse_row + h * lse_len. A tile of one segment: lo = 0.
      int lo = 0;
      int64_t lse_row = c.lse_off + rl;
      int lse_len = c.len;
      if (c.rows > 0) {
        const RowInfo ri = a.rows[static_cast<int64_t>(c.rows - 1) * kBM + rl];
        lo = ri.lo, lse_row = ri.lse_base + rl, lse_len = ri.len;
      }
      for (int r = 0; r < c.rounds; ++r) {
        if (x == 1 && 2 * r + 1 >= c.G) break;  // an odd group's last head runs alone, as half A
        if (*abort_flag) { ok = false; break; }
        const int h = c.g * c.G + 2 * r + x;
        ok = mbar_wait(&s.bar_s_full[x], nx & 1, a.wait_limit);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { where = kWhereFwdS; break; }
        tc_fence_after_sync();
        uint32_t sr[2][32];
        tmem_ld32(tS + lane_off + ch * 64, sr[0]);
        tmem_ld32(tS + lane_off + ch * 64 + 32, sr[1]);
        tmem_wait_ld();
        // the only key tile is the diagonal one: keys past the query are masked
        float mx = -INFINITY;
#pragma unroll
        for (int cc = 0; cc < 2; ++cc)
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const int col = ch * 64 + cc * 32 + e;
            if (col > rl || col < lo) sr[cc][e] = __float_as_uint(-INFINITY);
            if (col + 1 > rl || col + 1 < lo) sr[cc][e + 1] = __float_as_uint(-INFINITY);
            mx = ff_max3(mx, __uint_as_float(sr[cc][e]), __uint_as_float(sr[cc][e + 1]));
          }
        my_slot[0] = mx;
        mbar_arrive(pair_bar);
        ok = mbar_wait(pair_bar, xn & 1, a.wait_limit);
        ++xn;
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { where = kWhereFwdPair; break; }
        const float m_ref = fmaxf(mx, partner_slot[0]) * a.scale_log2;  // a row always sees its own key: finite
        const float neg_m = -m_ref;
        float sum0 = 0.f, sum1 = 0.f;
        uint32_t pk[32];
#pragma unroll
        for (int cc = 0; cc < 2; ++cc)
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            float x0, x1;
            fma2(x0, x1, __uint_as_float(sr[cc][e]), __uint_as_float(sr[cc][e + 1]), a.scale_log2, a.scale_log2, neg_m, neg_m);
            const float p0 = ex2f(x0), p1 = ex2f(x1);
            add2(sum0, sum1, sum0, sum1, p0, p1);
            pk[cc * 16 + (e >> 1)] = pack_bf16x2(p0, p1);
          }
        float l = sum0 + sum1;
        tmem_st32(tS + lane_off + ch * 64, pk);  // packed columns [64ch, 64ch + 32): inside this thread's own columns
        tmem_wait_st();
        tc_fence_before_sync();
        mbar_arrive(&s.bar_p_ready[x]);
        my_slot[128] = l;
        mbar_arrive(pair_bar);
        ok = mbar_wait(pair_bar, xn & 1, a.wait_limit);
        ++xn;
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { where = kWhereFwdPair; break; }
        l += partner_slot[128];
        ok = mbar_wait(&s.bar_pv_done[x], nx & 1, a.wait_limit);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { where = kWhereFwdO; break; }
        ++nx;
        tc_fence_after_sync();
        // ---- epilogue: O / l -> bf16 (this thread's columns), LSE
        const bool valid = rl < c.len;
        const float inv_l = 1.f / l;
        __nv_bfloat16* optr = a.o + c.q_off + (static_cast<int64_t>(rl) * c.hq + h) * D + ch * kOCols;
        uint32_t orow[kOCols / 32][32];
#pragma unroll
        for (int cc = 0; cc < kOCols / 32; ++cc) tmem_ld32(tO + lane_off + ch * kOCols + cc * 32, orow[cc]);
        tmem_wait_ld();
        tc_fence_before_sync();
        mbar_arrive(&s.bar_o_free[x]);  // the next round's PV may overwrite O_x
        if (c.len >= kBM) {
          // a full tile: the rows go to the Q slot of this round and half, swizzled like an operand tile (written from
          // the threads, a row per lane 8 KB apart and 16 bytes per store, every store is half a sector of the
          // store path: 4,096 clocks per pair of tiles)
          uint8_t* const srow = s.q[(R + r) & 1][x][D == 128 ? ch : 0] + rl * 128;
#pragma unroll
          for (int cc = 0; cc < kOCols / 32; ++cc)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              uint4 w;
              w.x = pack_bf16x2(__uint_as_float(orow[cc][8 * e + 0]) * inv_l, __uint_as_float(orow[cc][8 * e + 1]) * inv_l);
              w.y = pack_bf16x2(__uint_as_float(orow[cc][8 * e + 2]) * inv_l, __uint_as_float(orow[cc][8 * e + 3]) * inv_l);
              w.z = pack_bf16x2(__uint_as_float(orow[cc][8 * e + 4]) * inv_l, __uint_as_float(orow[cc][8 * e + 5]) * inv_l);
              w.w = pack_bf16x2(__uint_as_float(orow[cc][8 * e + 6]) * inv_l, __uint_as_float(orow[cc][8 * e + 7]) * inv_l);
              const int chunk = (D == 128 ? 0 : ch * 4) + cc * 4 + e;  // 16-byte chunk of the 128-byte row
              *reinterpret_cast<uint4*>(srow + ((chunk ^ (rl & 7)) * 16)) = w;
            }
          fence_proxy_async_smem();
        } else if (valid) {
#pragma unroll
          for (int cc = 0; cc < kOCols / 32; ++cc)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              uint4 w;
              w.x = pack_bf16x2(__uint_as_float(orow[cc][8 * e + 0]) * inv_l, __uint_as_float(orow[cc][8 * e + 1]) * inv_l);
              w.y = pack_bf16x2(__uint_as_float(orow[cc][8 * e + 2]) * inv_l, __uint_as_float(orow[cc][8 * e + 3]) * inv_l);
              w.z = pack_bf16x2(__uint_as_float(orow[cc][8 * e + 4]) * inv_l, __uint_as_float(orow[cc][8 * e + 5]) * inv_l);
              w.w = pack_bf16x2(__uint_as_float(orow[cc][8 * e + 6]) * inv_l, __uint_as_float(orow[cc][8 * e + 7]) * inv_l);
              NSP_CHECK(optr + cc * 32 + e * 8 + 8 <= a.o + a.q_elems && optr >= a.o, a.status, c.it, kWhereCheckFwdO, rl)
              *reinterpret_cast<uint4*>(optr + cc * 32 + e * 8) = w;
            }
        }
        mbar_arrive(&s.bar_o_staged[x]);  // the store warp sends the tile off (or just hands the slot back)
        if (valid) {
          if (ch == 0) {
            const int64_t at = lse_row + static_cast<int64_t>(h) * lse_len;
            NSP_CHECK(at >= 0 && at < a.lse_elems, a.status, c.it, kWhereCheckFwdLse, rl)
            a.lse[at] = (m_ref + log2f(l)) * 0.6931471805599453f;
          }
        }
      }
      if (!ok && where != 0 && lane == 0) {
        report_timeout(a.status, c.it, where, x);
        *abort_flag = 1;
      }
      R += static_cast<uint32_t>(c.rounds);
      ++gi;
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(s.tmem_base, kTmemCols);
}

template <int D>
cudaError_t launch_t(const FwdMaps& maps, const FwdArgs& args, int num_sms, cudaStream_t st) {
  cudaError_t e = cudaFuncSetAttribute(fwd_first_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(sizeof(FwdFirstSmem<D>)));
  if (e != cudaSuccess) return e;
  const int grid = args.n_items < num_sms ? args.n_items : num_sms;
  fwd_first_kernel<D><<<grid, kThreads, sizeof(FwdFirstSmem<D>), st>>>(maps, args);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fwd_first(const FwdMaps& maps, const FwdArgs& args, int head_dim, int num_sms, cudaStream_t st) {
  if (args.n_items == 0) return cudaSuccess;
  return head_dim == 64 ? launch_t<64>(maps, args, num_sms, st) : launch_t<128>(maps, args, num_sms, st);
}

}  // namespace nsp

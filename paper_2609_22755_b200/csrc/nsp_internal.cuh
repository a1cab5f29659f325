// Internal structures shared by the host API and the kernels of libnsp (never visible across the C ABI).
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>
#include "../../include/nsp.h"

namespace nsp {

constexpr int kHeadDim = NSP_HEAD_DIM;
constexpr int kBM = 128;  // query rows per tile
constexpr int kBN = 128;  // key rows per tile
constexpr int kFrontBlock = 16;  // backward: consecutive work items whose CTAs start together

// Per-segment table entry (device + host copy).
struct SegInfo {
  int64_t q_off;    // element offset of the segment in Q/O/dO/dQ
  int64_t kv_off;   // element offset in K/V/dK/dV
  int64_t lse_off;  // element offset in LSE / delta
  int32_t len;      // tokens
  int32_t hq, hkv;
  int32_t run;         // index of the run (dense [T, H, D] tensor) the segment belongs to
  int32_t tok_in_run;  // first token of the segment, relative to the run
  int32_t run_tokens;  // tokens of the whole run (extent of its tensor maps)
  int32_t turn_off;    // index of the segment's first (q head, q tile) turn counter (deterministic dQ): + h * Mt + m
  int32_t rows;        // 0: a segment. k > 0: a pack of several short segments that share one first tile (see
                       // RowInfo); its row table starts at entry (k - 1) * 128 and len is the pack's token count
};
static_assert(sizeof(SegInfo) == 56 || sizeof(SegInfo) == 64, "SegInfo layout");

// First tiles shared by several segments. Consecutive segments of a run are contiguous in Q, K, V and the outputs, so
// segments of fewer than 128 tokens that follow one another and together hold at most 128 tokens go through the
// first-tile kernels as ONE tile: row i of the tile belongs to the segment that covers rows [lo, hi) and sees the keys
// lo .. i of the tile. Only LSE and delta are laid out per segment ([hq, len]): lse_base + h * len + i is the element
// of (row i, q head h). One table of 128 entries per pack; the entries past the pack's tokens are zero.
struct RowInfo {
  int64_t lse_base;
  int32_t len;
  uint8_t lo, hi;
  uint8_t pad_[2];
};
static_assert(sizeof(RowInfo) == 16, "RowInfo layout");

struct RunInfo {
  int64_t q_off, kv_off;  // element offsets of the run's first token
  int64_t tokens;
  int32_t hq, hkv;
};

// Tensor maps of every run, passed by value as a __grid_constant__ kernel parameter.
struct FwdMaps {
  CUtensorMap q[NSP_MAX_RUNS], k[NSP_MAX_RUNS], v[NSP_MAX_RUNS];
  CUtensorMap o[NSP_MAX_RUNS];  // output tiles of the general forward kernel (stores); same geometry as q
};
struct BwdMaps {
  CUtensorMap q[NSP_MAX_RUNS], d_o[NSP_MAX_RUNS], k[NSP_MAX_RUNS], v[NSP_MAX_RUNS];
  CUtensorMap dk[NSP_MAX_RUNS], dv[NSP_MAX_RUNS];  // fp32 dK / dV outputs (tile stores of 32 columns x 128 rows); unset for bf16 outputs
};

// Device status record {code, item, where, aux}; the first writer wins (atomicCAS on the code in device memory) and
// also copies its record into mapped pinned host memory, code last, so that the host sees a failure at its next API
// call without synchronising.
struct StatusWord {
  int32_t* dev;   // device memory, four words
  int32_t* host;  // device pointer to the same four words in mapped pinned host memory
};

enum DeviceWhere : int32_t {
  kWhereFwdLoad = 1,
  kWhereFwdS = 2,
  kWhereFwdO = 3,
  kWhereFwdSmemAlign = 4,
  kWhereFwdTurn = 5,
  kWhereFwdPair = 6,
  kWhereBwdLoadKV = 11,
  kWhereBwdLoadQ = 12,
  kWhereBwdS = 13,
  kWhereBwdMma2 = 14,
  kWhereBwdSmemAlign = 15,
  kWhereBwdQEmpty = 16,
  kWhereBwdDqEmpty = 17,
  kWhereBwdPReady = 18,
  kWhereBwdLdEmpty = 19,
  kWhereBwdDqFull = 20,
  kWhereBwdDp = 21,
  kWhereBwdStaged = 22,
  kWhereBwdDelta = 23,
  kWhereBwdDsReady = 24,
  kWhereBwdItemBarrier = 25,
  kWhereBwdTmemBase = 26,
  kWhereBwdTurn = 27,  // deterministic dQ: the key tiles before this one did not finish their additions
  kWhereCheckFwdO = 40,    // checked build: an index outside the tensor (O, LSE / delta, dQ, dK / dV, LSE read)
  kWhereCheckFwdLse = 41,
  kWhereCheckBwdDq = 42,
  kWhereCheckBwdDkv = 43,
  kWhereCheckBwdLse = 44,
  kWhereSelfTest = 90,
};

// Out of line on purpose: the callers sit in instruction-cache-sensitive loops and only get here when a wait ran out.
static __device__ __noinline__ void report_status_raw(int32_t* dev, int32_t* host, int32_t code, int32_t item, int32_t where,
                                               int32_t aux) {
  if (atomicCAS(dev, 0, code) == 0) {
    dev[1] = item;
    dev[2] = where;
    dev[3] = aux;
    volatile int32_t* h = host;
    h[1] = item;
    h[2] = where;
    h[3] = aux;
    __threadfence_system();
    h[0] = code;
    __threadfence_system();
  }
}
__device__ __forceinline__ void report_status(StatusWord st, int32_t code, int32_t item, int32_t where, int32_t aux) {
  report_status_raw(st.dev, st.host, code, item, where, aux);
}
__device__ __forceinline__ void report_timeout(StatusWord st, int32_t item, int32_t where, int32_t aux) {
  report_status_raw(st.dev, st.host, NSP_ERR_DEVICE_TIMEOUT, item, where, aux);
}

// Index checks of the checked build (-DNSP_CHECKED, libnsp_checked.so): `NSP_CHECK(cond, ...) access;` performs the
// access only if cond holds and otherwise records NSP_ERR_DEVICE_ASSERT; in the regular build it is the bare access.
#ifdef NSP_CHECKED
#define NSP_CHECK(cond, st, item, where, aux)                                       \
  if (!(cond)) {                                                                    \
    report_status(st, NSP_ERR_DEVICE_ASSERT, item, where, static_cast<int32_t>(aux)); \
  } else
#else
#define NSP_CHECK(cond, st, item, where, aux)
#endif

struct FwdArgs {
  const SegInfo* seg;
  const nsp_tile_t* items;
  int32_t n_items;
  int32_t* counter;  // work-list cursor, zeroed before the launch
  StatusWord status;
  __nv_bfloat16* o;
  float* lse;
  float scale_log2;  // softmax_scale * log2(e)
  long long wait_limit;  // SM clocks a device-side wait may take before it gives up
  int32_t withhold;      // checked build only: 1 = the producer leaves out one V load (failure-detection test)
  int64_t q_elems, lse_elems;  // tensor sizes (checked build)
  // Recomputation inside the backward pass (all three null in a plain forward): only items of segments with
  // seg_mask[seg] != 0 run, and instead of O the kernel writes delta = rowsum(dO o O) next to the LSE.
  const uint8_t* seg_mask;
  const __nv_bfloat16* d_o;
  float* delta;
  const RowInfo* rows;  // row tables of the packs (first-tile kernel)
};

struct BwdArgs {
  const SegInfo* seg;
  const nsp_tile_t* items;
  int32_t n_items;
  int32_t* counter;  // work-list cursor, zeroed before the launch
  StatusWord status;
  const float* lse;
  const float* delta;
  float* dq_acc;  // fp32 [q_elems]; rows 128.. of every segment zeroed before the launch (main kernel)
  void* dq;       // first-tile kernel: rows 0..127 of every segment are stored here directly
  int32_t dq_f32;
  int32_t* dq_turn;  // deterministic dQ: one counter per (segment, q head, q tile), zeroed before the launch; else null
  int32_t dq_rounded;  // 1: dQ terms rounded to a fixed quantum before they are added (order-independent sums)
  void* dk;
  void* dv;
  int32_t dkv_f32;
  float scale;
  float scale_log2;
  long long wait_limit;  // SM clocks a device-side wait may take before it gives up
  int64_t q_elems, kv_elems, lse_elems;  // tensor sizes (checked build)
  int32_t* front;    // [n_items / kFrontBlock + 1] arrival counters, zeroed before the launch (see next_item)
  const RowInfo* rows;  // row tables of the packs (first-tile kernel)
};

// Host-side launchers implemented next to their kernels.
cudaError_t launch_plan_build(const SegInfo* d_seg, int n_seg, int bm, int bn, nsp_tile_t* d_fwd, int64_t n_fwd,
                              nsp_tile_t* d_bwd, int64_t n_bwd, uint64_t* d_keys, uint64_t* d_keys_alt, void* d_sort_tmp,
                              size_t sort_tmp_bytes, const int64_t* d_fwd_base, const int64_t* d_bwd_base,
                              cudaStream_t st);
size_t plan_sort_tmp_bytes(int64_t max_items);
cudaError_t launch_fwd(const FwdMaps& maps, const FwdArgs& args, int head_dim, int num_sms, cudaStream_t st);
// q tile 0 of every segment: items (segment, kv head); args.items / n_items / counter are that list's
cudaError_t launch_fwd_first(const FwdMaps& maps, const FwdArgs& args, int head_dim, int num_sms, cudaStream_t st);
// The backward launches, in the order they run: preprocess (delta and zeroed accumulator rows for tokens 128.. of
// every segment), first-tile kernel (q tile 0 of every segment: its dQ rows, and its part of dK / dV), main kernel,
// postprocess (tokens 128..). seg_skip (may be null): segments whose delta is left alone; lse_in / lse_out (may be
// null): LSE copied for the rows whose delta is written.
cudaError_t launch_bwd_preprocess(const SegInfo* d_seg, int n_seg, const int64_t* d_row_base, int64_t total_rows,
                                  int head_dim, const __nv_bfloat16* o, const __nv_bfloat16* d_o, float* delta,
                                  float* dq_acc, const uint8_t* seg_skip, const float* lse_in, float* lse_out,
                                  cudaStream_t st);
cudaError_t launch_bwd_first(const BwdMaps& maps, const BwdArgs& args, int head_dim, int num_sms, cudaStream_t st);
cudaError_t launch_bwd(const BwdMaps& maps, const BwdArgs& args, int head_dim, int num_sms, cudaStream_t st);  // args.dq_turn / args.dq_rounded select the reproducible variants
cudaError_t launch_bwd_postprocess(const SegInfo* d_seg, int n_seg, const int64_t* d_row_base, int64_t total_rows,
                                   int head_dim, const float* dq_acc, void* dq, int dq_f32, float scale,
                                   cudaStream_t st);
void count_launches(int n);

}  // namespace nsp

// Host side of libnsp: argument validation, plan object, tensor-map encoding and kernel launches.
// Plain C ABI (include/nsp.h); no torch types, no CPU fallback.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>
#include <cuda_bf16.h>
#include "nsp_internal.cuh"
#include "sm100_ptx.cuh"

namespace nsp {
static std::atomic<int64_t> g_launches{0};
void count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
}  // namespace nsp

using namespace nsp;

struct nsp_plan {
  int32_t n_seg = 0, bm = kBM, bn = kBN, head_dim = kHeadDim;
  int device = 0, num_sms = 0;
  int64_t q_elems = 0, kv_elems = 0, lse_elems = 0, n_fwd = 0, n_bwd = 0;
  std::vector<SegInfo> seg;
  std::vector<RunInfo> runs;
  // device state
  SegInfo* d_seg = nullptr;
  int64_t* d_row_base = nullptr;  // [n_seg + 1] first packed (token, head) row of each segment
  nsp_tile_t* d_fwd = nullptr;
  nsp_tile_t* d_bwd = nullptr;
  nsp_tile_t* d_bwd_exec = nullptr;  // the backward items in the order the kernel walks them (see build_bwd_exec_order)
  nsp_tile_t* d_bwd_first = nullptr;  // one item per (segment or pack, kv head): the first-tile kernels' list
  int64_t n_first = 0;
  RowInfo* d_rows = nullptr;          // row tables of the packs, 128 entries each (d_seg holds the packs' entries after
  int64_t n_packs = 0;                // the n_seg segments')
  int64_t n_fwd_main = 0;             // forward items that visit at least two key tiles: a prefix of d_fwd (the
                                      // cost-1 tail = q tile 0 of every segment runs in the first-tile forward kernel)
  bool deterministic = false;         // plan option: dQ tiles added in key-tile order
  bool rounded_dq = false;            // plan option: dQ terms rounded to a fixed quantum (order-independent sums)
  int32_t max_len = 0;                // longest segment: no preprocess / main / postprocess launch when <= 128
  int32_t* d_front = nullptr;        // [n_bwd / kFrontBlock + 1] start-alignment counters of the backward kernel
  int32_t* d_counters = nullptr;  // [0] forward cursor, [1] backward cursor
  int32_t* d_status = nullptr;    // {code, item, where, aux}
  int32_t* h_status = nullptr;    // the same record in mapped pinned host memory (written by the failing kernel)
  int32_t* h_status_dev = nullptr;  // device pointer to h_status
  int sticky = 0;
  long long wait_limit = NSP_WAIT_CYCLES_DEFAULT;  // SM clocks a device-side wait may take
  int withhold = 0;                                // checked build: failure-detection test switch
  // optional per-kernel timing (CUDA events on the launching stream)
  bool profiling = false;
  cudaEvent_t ev[2 * NSP_KERNEL_COUNT] = {};
  bool ev_valid[NSP_KERNEL_COUNT] = {};
  // host-to-host step (nsp_attn_step_host): a copy stream and ordering events, created at its first call
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t hev[6] = {};
};

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Tensor map of one run: a dense bf16 [tokens, heads, 128] tensor; tiles are {64 dims, 1 head, 128 tokens}
// with 128-byte swizzle, rows past the run read as zero.
bool encode_run_map(CUtensorMap* out, const void* base, int64_t elem_off, int64_t tokens, int heads, int head_dim) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return false;
  if (tokens <= 0) {
    std::memset(out, 0, sizeof(*out));
    return true;
  }
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(head_dim), static_cast<cuuint64_t>(heads),
                              static_cast<cuuint64_t>(tokens)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(head_dim) * 2, static_cast<cuuint64_t>(heads) * head_dim * 2};
  const cuuint32_t box[3] = {64, 1, 128};
  const cuuint32_t estr[3] = {1, 1, 1};
  void* ptr = const_cast<char*>(static_cast<const char*>(base)) + elem_off * 2;
  return enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 [tokens, heads, head_dim] output of one run, boxes of 32 columns x 128 rows (128 bytes per row, 128-byte swizzle)
bool encode_run_map_f32(CUtensorMap* out, void* base, int64_t elem_off, int64_t tokens, int heads, int head_dim) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return false;
  if (tokens <= 0) {
    std::memset(out, 0, sizeof(*out));
    return true;
  }
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(head_dim), static_cast<cuuint64_t>(heads),
                              static_cast<cuuint64_t>(tokens)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(head_dim) * 4, static_cast<cuuint64_t>(heads) * head_dim * 4};
  const cuuint32_t box[3] = {32, 1, 128};
  const cuuint32_t estr[3] = {1, 1, 1};
  void* ptr = static_cast<char*>(base) + elem_off * 4;
  return enc(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Order in which the backward kernel walks its work items (nsp_plan_get, pass 2). The published work list (pass 1)
// is sorted by cost alone; walked in that order, the CTAs that run at the same time hold key tiles of MANY (segment,
// kv head) groups, a q tile's fp32 dQ accumulator rows are touched by a few CTAs now and by the others much later,
// and they travel to DRAM and back every time (16 segments of 8,192 tokens, 32q/4kv: 193 GB of DRAM traffic for a
// backward pass whose tensors total 5 GB, L2 hit rate 21 %, the kernel runs at HBM speed). Walked group by group
// -- all key tiles of one (segment, kv head), first key tile (largest cost) first -- the CTAs of a group sweep the q
// tiles together and every accumulator row, Q tile and dO tile is fetched once per group. Groups go by segment
// length descending (ties: segment, then kv head, ascending): all CTAs then start the longest group at the same
// moment, which is what keeps them on the same q tile (started after a tail of shorter groups they enter it scattered
// and stay scattered: 131,072 tokens at 16q/1kv next to 131,072 tokens of shorter segments ran 4 % slower that way, a
// long-tailed batch 8 %), and the walk ends with the cheapest items of the shortest segments. Same items, same
// costs: a permutation of the published list.
std::vector<nsp_tile_t> build_bwd_exec_order(const std::vector<SegInfo>& seg, int bm, int bn) {
  struct Group { int32_t len, s, g; };
  std::vector<Group> groups;
  for (size_t s = 0; s < seg.size(); ++s)
    if (seg[s].len > 0)
      for (int g = 0; g < seg[s].hkv; ++g) groups.push_back(Group{seg[s].len, static_cast<int32_t>(s), g});
  std::stable_sort(groups.begin(), groups.end(), [](const Group& a, const Group& b) { return a.len > b.len; });
  std::vector<nsp_tile_t> out;
  for (const Group& gr : groups) {
    const SegInfo& sg = seg[gr.s];
    const int64_t Mt = (static_cast<int64_t>(sg.len) + bm - 1) / bm, Nt = (static_cast<int64_t>(sg.len) + bn - 1) / bn;
    const int G = sg.hq / sg.hkv;
    for (int64_t n = 0; n < Nt; ++n) {
      const int64_t cost = G * (Mt - (n * bn) / bm);
      out.push_back(nsp_tile_t{gr.s, gr.g, static_cast<int32_t>(n), static_cast<int32_t>(cost)});
    }
  }
  return out;
}

// The plan's failure state: set once a kernel of the plan has recorded a failure. The record sits in mapped pinned
// host memory, so looking at it costs a host load, not a synchronisation; a failure is seen by the first call made
// after the failing kernel wrote it.
int plan_failed(const nsp_plan* plan) {
  if (!plan->sticky && plan->h_status) {
    const int code = *reinterpret_cast<volatile int32_t*>(plan->h_status);
    if (code != 0) const_cast<nsp_plan*>(plan)->sticky = code;
  }
  return plan->sticky;
}
StatusWord status_word(const nsp_plan* plan) { return StatusWord{plan->d_status, plan->h_status_dev}; }

// Host-side call log: with NSP_LOG=1 in the environment (read once) every plan construction and every compute call
// prints one line to stderr. Nothing on the device changes.
bool log_on() {
  static const bool on = [] {
    const char* e = std::getenv("NSP_LOG");
    return e && e[0] && e[0] != '0';
  }();
  return on;
}
#define NSP_LOGF(...)                        \
  do {                                       \
    if (log_on()) {                          \
      std::fprintf(stderr, "[nsp] " __VA_ARGS__); \
      std::fputc('\n', stderr);              \
    }                                        \
  } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

void free_plan(nsp_plan* p) {
  if (!p) return;
  cudaFree(p->d_seg);
  cudaFree(p->d_row_base);
  cudaFree(p->d_fwd);
  cudaFree(p->d_bwd);
  cudaFree(p->d_bwd_exec);
  cudaFree(p->d_bwd_first);
  cudaFree(p->d_rows);
  cudaFree(p->d_front);
  cudaFree(p->d_counters);
  cudaFree(p->d_status);
  if (p->h_status) cudaFreeHost(p->h_status);
  for (cudaEvent_t e : p->ev)
    if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : p->hev)
    if (e) cudaEventDestroy(e);
  if (p->copy_stream) cudaStreamDestroy(p->copy_stream);
  delete p;
}

// Record the start / stop event of kernel `id` when profiling is on.
void prof_mark(const nsp_plan* plan, int id, int stop, cudaStream_t st) {
  if (!plan->profiling) return;
  nsp_plan* p = const_cast<nsp_plan*>(plan);
  cudaEventRecord(p->ev[2 * id + stop], st);
  if (stop) p->ev_valid[id] = true;
}

}  // namespace

extern "C" {

const char* nsp_status_string(int code) {
  switch (code) {
    case NSP_OK: return "ok";
    case NSP_ERR_INVALID_ARG: return "invalid argument";
    case NSP_ERR_UNSUPPORTED: return "unsupported configuration";
    case NSP_ERR_ALLOC: return "allocation failed";
    case NSP_ERR_CUDA: return "CUDA call failed";
    case NSP_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case NSP_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case NSP_ERR_DEVICE_ASSERT: return "device-side index check failed (checked build)";
    case NSP_ERR_INFEASIBLE: return "no plan within the token budget";
    default: return "unknown status";
  }
}

int64_t nsp_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int nsp_plan_tiles(const int32_t* cu_seqlens, const int32_t* hq, const int32_t* hkv, int32_t n_seg, int32_t head_dim,
                   const nsp_plan_opts* opts, void* stream, nsp_plan_t** out_plan) {
  if (!out_plan) return NSP_ERR_INVALID_ARG;
  *out_plan = nullptr;
  if (n_seg < 0 || (n_seg > 0 && (!cu_seqlens || !hq || !hkv))) return NSP_ERR_INVALID_ARG;
  if (n_seg > 0 && cu_seqlens[0] != 0) return NSP_ERR_INVALID_ARG;
  for (int s = 0; s < n_seg; ++s) {
    if (cu_seqlens[s + 1] < cu_seqlens[s]) return NSP_ERR_INVALID_ARG;
    if (hq[s] <= 0 || hkv[s] <= 0 || hq[s] % hkv[s] != 0) return NSP_ERR_INVALID_ARG;
  }
  int bm = kBM, bn = kBN;
  if (opts) {
    if (opts->bm <= 0 || opts->bn <= 0) return NSP_ERR_INVALID_ARG;
    bm = opts->bm;
    bn = opts->bn;
    if (opts->order_version != 1 || (opts->flags & ~(NSP_PLAN_DETERMINISTIC_DQ | NSP_PLAN_ROUNDED_DQ)) != 0) return NSP_ERR_UNSUPPORTED;
  }
  if (head_dim != 128 && head_dim != 64) return NSP_ERR_UNSUPPORTED;
  if (bm != kBM || bn != kBN) return NSP_ERR_UNSUPPORTED;
  if (n_seg >= 65536) return NSP_ERR_UNSUPPORTED;

  nsp_plan* p = new (std::nothrow) nsp_plan;
  if (!p) return NSP_ERR_ALLOC;
  p->n_seg = n_seg;
  p->head_dim = head_dim;
  p->deterministic = opts && (opts->flags & NSP_PLAN_DETERMINISTIC_DQ) != 0;
  p->rounded_dq = opts && !p->deterministic && (opts->flags & NSP_PLAN_ROUNDED_DQ) != 0;
  p->bm = bm;
  p->bn = bn;
  std::vector<int64_t> row_base, fwd_base, bwd_base;
  try {
    p->seg.resize(n_seg);
    row_base.resize(n_seg + 1);
    fwd_base.resize(n_seg + 1);
    bwd_base.resize(n_seg + 1);
  } catch (...) {
    delete p;
    return NSP_ERR_ALLOC;
  }
  int64_t q_off = 0, kv_off = 0, lse_off = 0, nf = 0, nb = 0;
  for (int s = 0; s < n_seg; ++s) {
    const int64_t L = static_cast<int64_t>(cu_seqlens[s + 1]) - cu_seqlens[s];
    const int64_t Mt = (L + bm - 1) / bm, Nt = (L + bn - 1) / bn;
    if (hq[s] > 256 || Mt >= 65536 || Nt >= 65536 || (hq[s] / hkv[s]) * Mt >= (1 << 24)) {
      delete p;
      return NSP_ERR_UNSUPPORTED;
    }
    const bool new_run = s == 0 || hq[s] != hq[s - 1] || hkv[s] != hkv[s - 1];
    if (new_run) {
      if (p->runs.size() == NSP_MAX_RUNS) {
        delete p;
        return NSP_ERR_UNSUPPORTED;
      }
      p->runs.push_back(RunInfo{q_off, kv_off, 0, hq[s], hkv[s]});
    }
    RunInfo& run = p->runs.back();
    SegInfo& sg = p->seg[s];
    std::memset(&sg, 0, sizeof(sg));
    sg.q_off = q_off;
    sg.kv_off = kv_off;
    sg.lse_off = lse_off;
    sg.len = static_cast<int32_t>(L);
    sg.hq = hq[s];
    sg.hkv = hkv[s];
    sg.run = static_cast<int32_t>(p->runs.size() - 1);
    sg.tok_in_run = static_cast<int32_t>(run.tokens);
    sg.turn_off = static_cast<int32_t>(nf);  // one turn counter per forward item = (q head, q tile) of the segment
    run.tokens += L;
    row_base[s] = lse_off;
    fwd_base[s] = nf;
    bwd_base[s] = nb;
    q_off += L * hq[s] * head_dim;
    kv_off += L * hkv[s] * head_dim;
    lse_off += L * hq[s];
    nf += Mt * hq[s];
    nb += Nt * hkv[s];
  }
  for (int s = 0; s < n_seg; ++s) p->seg[s].run_tokens = static_cast<int32_t>(p->runs[p->seg[s].run].tokens);
  row_base[n_seg] = lse_off;
  fwd_base[n_seg] = nf;
  bwd_base[n_seg] = nb;
  p->q_elems = q_off;
  p->kv_elems = kv_off;
  p->lse_elems = lse_off;
  p->n_fwd = nf;
  p->n_bwd = nb;
  if (nf >= (1ll << 31) || nb >= (1ll << 31)) {
    delete p;
    return NSP_ERR_UNSUPPORTED;
  }

  std::vector<nsp_tile_t> bwd_exec, bwd_first;
  std::vector<SegInfo> pack_segs;
  std::vector<RowInfo> pack_rows;
  try {
    bwd_exec = build_bwd_exec_order(p->seg, bm, bn);
    // the first-tile kernel's items: key tile 0 of every group, in the same group order; q heads of the group = steps
    // Segments of fewer than 128 tokens that follow one another inside a run (they are contiguous in every tensor)
    // and together hold at most 128 tokens share one first tile: such a pack becomes an entry of its own behind the
    // segments (len = its tokens, offsets of its first segment) with a row table, and takes its segments' places in
    // the first-tile list.
    std::vector<int32_t> pack_of(n_seg, -1);
    for (int s0 = 0; s0 < n_seg;) {
      const SegInfo& first = p->seg[s0];
      if (first.len <= 0 || first.len >= kBM) { ++s0; continue; }
      int s1 = s0 + 1, tokens = first.len, members = 1;
      while (s1 < n_seg && p->seg[s1].run == first.run && p->seg[s1].len < kBM && tokens + p->seg[s1].len <= kBM) {
        tokens += p->seg[s1].len;
        members += p->seg[s1].len > 0;
        ++s1;
      }
      if (members >= 2) {
        SegInfo pk = first;
        pk.len = tokens;
        pk.rows = static_cast<int32_t>(pack_rows.size() / kBM) + 1;
        int row = 0;
        for (int s = s0; s < s1; ++s) {
          const SegInfo& sg = p->seg[s];
          if (sg.len <= 0) continue;
          pack_of[s] = n_seg + static_cast<int32_t>(pack_segs.size());
          RowInfo ri{};
          ri.lse_base = sg.lse_off - row;
          ri.len = sg.len;
          ri.lo = static_cast<uint8_t>(row);
          ri.hi = static_cast<uint8_t>(row + sg.len);
          for (int i = 0; i < sg.len; ++i) pack_rows.push_back(ri);
          row += sg.len;
        }
        pack_rows.resize(pack_rows.size() + (kBM - tokens), RowInfo{});
        pack_segs.push_back(pk);
      }
      s0 = s1;
    }
    p->n_packs = static_cast<int64_t>(pack_segs.size());
    {
      std::vector<char> listed(pack_segs.size() * 256, 0);  // (pack, kv head) already in the list
      for (const nsp_tile_t& t : bwd_exec) {
        if (t.tile != 0) continue;
        const int32_t G = p->seg[t.seg].hq / p->seg[t.seg].hkv;
        if (pack_of[t.seg] < 0) {
          bwd_first.push_back(nsp_tile_t{t.seg, t.head, 0, G});
        } else {
          char& seen = listed[static_cast<size_t>(pack_of[t.seg] - n_seg) * 256 + t.head];
          if (!seen) bwd_first.push_back(nsp_tile_t{pack_of[t.seg], t.head, 0, G});
          seen = 1;
        }
      }
    }
    p->n_first = static_cast<int64_t>(bwd_first.size());
    p->n_fwd_main = nf;
    for (const SegInfo& sg : p->seg)
      if (sg.len > 0) p->n_fwd_main -= sg.hq;
    for (const SegInfo& sg : p->seg) p->max_len = std::max(p->max_len, sg.len);
  } catch (...) {
    delete p;
    return NSP_ERR_ALLOC;
  }

  // ---- device side
  cudaDeviceProp prop;
  if (cudaGetDevice(&p->device) != cudaSuccess || cudaGetDeviceProperties(&prop, p->device) != cudaSuccess) {
    delete p;
    return NSP_ERR_CUDA;
  }
  p->num_sms = prop.multiProcessorCount;
  if (prop.major != 10) {
    delete p;
    return NSP_ERR_UNSUPPORTED;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int64_t* d_bases = nullptr;
  uint64_t* d_keys = nullptr;
  void* d_tmp = nullptr;
  const size_t tmp_bytes = plan_sort_tmp_bytes(nf > nb ? nf : nb);
  bool okc = true;
  auto A = [&](void** ptr, size_t bytes) {
    if (okc && cudaMalloc(ptr, bytes ? bytes : 16) != cudaSuccess) okc = false;
  };
  A(reinterpret_cast<void**>(&p->d_seg), sizeof(SegInfo) * (n_seg + pack_segs.size()));
  A(reinterpret_cast<void**>(&p->d_rows), sizeof(RowInfo) * pack_rows.size());
  A(reinterpret_cast<void**>(&p->d_row_base), sizeof(int64_t) * (n_seg + 1));
  A(reinterpret_cast<void**>(&p->d_fwd), sizeof(nsp_tile_t) * nf);
  A(reinterpret_cast<void**>(&p->d_bwd), sizeof(nsp_tile_t) * nb);
  A(reinterpret_cast<void**>(&p->d_bwd_exec), sizeof(nsp_tile_t) * nb);
  A(reinterpret_cast<void**>(&p->d_bwd_first), sizeof(nsp_tile_t) * p->n_first);
  A(reinterpret_cast<void**>(&p->d_front), sizeof(int32_t) * (nb / kFrontBlock + 1));
  A(reinterpret_cast<void**>(&p->d_counters), 4 * sizeof(int32_t));  // [0] forward, [1] backward main, [2] first-tile backward, [3] first-tile forward
  A(reinterpret_cast<void**>(&p->d_status), 4 * sizeof(int32_t));
  if (okc) {
    void* hp = nullptr;
    void* dp = nullptr;
    if (cudaHostAlloc(&hp, 4 * sizeof(int32_t), cudaHostAllocMapped) != cudaSuccess) {
      okc = false;
    } else {
      p->h_status = static_cast<int32_t*>(hp);
      std::memset(hp, 0, 4 * sizeof(int32_t));
      if (cudaHostGetDevicePointer(&dp, hp, 0) != cudaSuccess) okc = false;
      p->h_status_dev = static_cast<int32_t*>(dp);
    }
  }
  A(reinterpret_cast<void**>(&d_bases), 2 * sizeof(int64_t) * (n_seg + 1));
  A(reinterpret_cast<void**>(&d_keys), 2 * sizeof(uint64_t) * (nf + nb));
  A(&d_tmp, tmp_bytes);
  int rc = NSP_OK;
  if (!okc) {
    rc = NSP_ERR_ALLOC;
    cudaGetLastError();
  } else {
    cudaError_t e = cudaSuccess;
    auto C = [&](cudaError_t x) {
      if (e == cudaSuccess) e = x;
    };
    C(cudaMemsetAsync(p->d_counters, 0, 4 * sizeof(int32_t), st));
    C(cudaMemsetAsync(p->d_status, 0, 4 * sizeof(int32_t), st));
    if (n_seg > 0) {
      C(cudaMemcpyAsync(p->d_seg, p->seg.data(), sizeof(SegInfo) * n_seg, cudaMemcpyHostToDevice, st));
      C(cudaMemcpyAsync(d_bases, fwd_base.data(), sizeof(int64_t) * (n_seg + 1), cudaMemcpyHostToDevice, st));
      C(cudaMemcpyAsync(d_bases + n_seg + 1, bwd_base.data(), sizeof(int64_t) * (n_seg + 1), cudaMemcpyHostToDevice,
                        st));
    }
    C(cudaMemcpyAsync(p->d_row_base, row_base.data(), sizeof(int64_t) * (n_seg + 1), cudaMemcpyHostToDevice, st));
    if (!pack_segs.empty()) {
      C(cudaMemcpyAsync(p->d_seg + n_seg, pack_segs.data(), sizeof(SegInfo) * pack_segs.size(), cudaMemcpyHostToDevice, st));
      C(cudaMemcpyAsync(p->d_rows, pack_rows.data(), sizeof(RowInfo) * pack_rows.size(), cudaMemcpyHostToDevice, st));
    }
    if (nb > 0) C(cudaMemcpyAsync(p->d_bwd_exec, bwd_exec.data(), sizeof(nsp_tile_t) * nb, cudaMemcpyHostToDevice, st));
    if (p->n_first > 0)
      C(cudaMemcpyAsync(p->d_bwd_first, bwd_first.data(), sizeof(nsp_tile_t) * p->n_first, cudaMemcpyHostToDevice, st));
    if (e == cudaSuccess)
      C(launch_plan_build(p->d_seg, n_seg, bm, bn, p->d_fwd, nf, p->d_bwd, nb, d_keys, d_keys + nf + nb, d_tmp, tmp_bytes,
                          d_bases, d_bases + n_seg + 1, st));
    // the host staging vectors and the scratch buffers die with this call: wait for the build
    C(cudaStreamSynchronize(st));
    if (e != cudaSuccess) rc = NSP_ERR_CUDA;
  }
  cudaFree(d_bases);
  cudaFree(d_keys);
  cudaFree(d_tmp);
  if (rc != NSP_OK) {
    free_plan(p);
    return rc;
  }
  NSP_LOGF("plan %p: %d segments, %zu runs, head_dim %d, q_elems %lld, kv_elems %lld, fwd items %lld, bwd items %lld%s",
           static_cast<void*>(p), n_seg, p->runs.size(), head_dim, static_cast<long long>(p->q_elems),
           static_cast<long long>(p->kv_elems), static_cast<long long>(nf), static_cast<long long>(nb),
           p->deterministic ? ", deterministic dQ" : "");
  *out_plan = p;
  return NSP_OK;
}

int nsp_plan_sizes(const nsp_plan_t* plan, int64_t* q_elems, int64_t* kv_elems, int64_t* lse_elems,
                   size_t* fwd_ws_bytes, size_t* bwd_ws_bytes) {
  if (!plan) return NSP_ERR_INVALID_ARG;
  if (q_elems) *q_elems = plan->q_elems;
  if (kv_elems) *kv_elems = plan->kv_elems;
  if (lse_elems) *lse_elems = plan->lse_elems;
  if (fwd_ws_bytes) *fwd_ws_bytes = 0;
  if (bwd_ws_bytes)  // fp32 dQ accumulator, delta, and (deterministic dQ) one turn counter per (q head, q tile)
    *bwd_ws_bytes = align_up(static_cast<size_t>(plan->q_elems) * 4, 256) +
                    align_up(static_cast<size_t>(plan->lse_elems) * 4, 256) +
                    (plan->deterministic ? align_up(static_cast<size_t>(plan->n_fwd) * 4, 256) : 0);
  return NSP_OK;
}

int nsp_plan_get(const nsp_plan_t* plan, int pass, nsp_tile_t* host_out, int64_t cap, int64_t* n_items) {
  if (!plan || !n_items || pass < 0 || pass > 2 || cap < 0) return NSP_ERR_INVALID_ARG;
  const int64_t n = pass == 0 ? plan->n_fwd : plan->n_bwd;
  *n_items = n;
  if (!host_out || cap == 0 || n == 0) return NSP_OK;
  const int64_t m = cap < n ? cap : n;
  const nsp_tile_t* src = pass == 0 ? plan->d_fwd : (pass == 1 ? plan->d_bwd : plan->d_bwd_exec);
  if (cudaMemcpy(host_out, src, sizeof(nsp_tile_t) * m, cudaMemcpyDeviceToHost) !=
      cudaSuccess)
    return NSP_ERR_CUDA;
  return NSP_OK;
}

int nsp_attn_fwd(const nsp_plan_t* plan, const void* q, const void* k, const void* v, void* o, float* lse,
                 float softmax_scale, void* ws, size_t ws_bytes, void* stream) {
  (void)ws;
  (void)ws_bytes;
  if (!plan) return NSP_ERR_INVALID_ARG;
  if (const int failed = plan_failed(plan)) return failed;
  if (!(softmax_scale > 0.f) || !std::isfinite(softmax_scale)) return NSP_ERR_INVALID_ARG;
  if (plan->n_fwd == 0) return NSP_OK;
  if (!q || !k || !v || !o || !lse) return NSP_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(lse)) return NSP_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  FwdMaps maps;
  std::memset(&maps, 0, sizeof(maps));
  for (size_t r = 0; r < plan->runs.size(); ++r) {
    const RunInfo& run = plan->runs[r];
    if (!encode_run_map(&maps.q[r], q, run.q_off, run.tokens, run.hq, plan->head_dim) ||
        !encode_run_map(&maps.k[r], k, run.kv_off, run.tokens, run.hkv, plan->head_dim) ||
        !encode_run_map(&maps.v[r], v, run.kv_off, run.tokens, run.hkv, plan->head_dim) ||
        !encode_run_map(&maps.o[r], o, run.q_off, run.tokens, run.hq, plan->head_dim))
      return NSP_ERR_CUDA;
  }
  if (cudaMemsetAsync(plan->d_counters, 0, sizeof(int32_t), st) != cudaSuccess) return NSP_ERR_CUDA;
  if (cudaMemsetAsync(plan->d_counters + 3, 0, sizeof(int32_t), st) != cudaSuccess) return NSP_ERR_CUDA;
  FwdArgs a;
  a.seg = plan->d_seg;
  a.status = status_word(plan);
  a.o = static_cast<__nv_bfloat16*>(o);
  a.lse = lse;
  a.scale_log2 = softmax_scale * 1.4426950408889634f;
  a.wait_limit = plan->wait_limit;
  a.withhold = plan->withhold;
  a.q_elems = plan->q_elems;
  a.lse_elems = plan->lse_elems;
  a.seg_mask = nullptr;
  a.rows = plan->d_rows;
  a.d_o = nullptr;
  a.delta = nullptr;
  NSP_LOGF("fwd plan %p stream %p scale %g", static_cast<const void*>(plan), stream, softmax_scale);
  // q tile 0 of every segment (the cost-1 tail of the list): one item per (segment, kv head)
  a.items = plan->d_bwd_first;
  a.n_items = static_cast<int32_t>(plan->n_first);
  a.counter = plan->d_counters + 3;
  prof_mark(plan, NSP_KERNEL_FWD_FIRST, 0, st);
  if (!plan->withhold && launch_fwd_first(maps, a, plan->head_dim, plan->num_sms, st) != cudaSuccess) return NSP_ERR_CUDA;
  prof_mark(plan, NSP_KERNEL_FWD_FIRST, 1, st);
  // everything else: the list's prefix (with the test switch of the checked build: the whole list, general kernel)
  a.items = plan->d_fwd;
  a.n_items = static_cast<int32_t>(plan->withhold ? plan->n_fwd : plan->n_fwd_main);
  a.counter = plan->d_counters;
  prof_mark(plan, NSP_KERNEL_FWD, 0, st);
  if (launch_fwd(maps, a, plan->head_dim, plan->num_sms, st) != cudaSuccess) return NSP_ERR_CUDA;
  prof_mark(plan, NSP_KERNEL_FWD, 1, st);
  return NSP_OK;
}

namespace {

size_t recompute_ws_bytes(const nsp_plan_t* plan) {
  size_t base = 0;
  nsp_plan_sizes(plan, nullptr, nullptr, nullptr, nullptr, &base);
  return base + align_up(static_cast<size_t>(plan->lse_elems) * 4, 256) + align_up(static_cast<size_t>(plan->n_seg), 256);
}

// Backward pass. recompute == nullptr: the plain pass. Otherwise host flags per segment: for a marked segment o and
// lse are not read; its LSE and delta are recomputed by a forward launch restricted to the marked segments.
int bwd_impl(const nsp_plan_t* plan, const uint8_t* recompute, const void* q, const void* k, const void* v,
             const void* o, const void* d_o, const float* lse, void* dq, void* dk, void* dv, int dq_dtype,
             int dkv_dtype, float softmax_scale, void* ws, size_t ws_bytes, void* stream) {
  if (!plan) return NSP_ERR_INVALID_ARG;
  if (const int failed = plan_failed(plan)) return failed;
  if (!(softmax_scale > 0.f) || !std::isfinite(softmax_scale)) return NSP_ERR_INVALID_ARG;
  if ((dq_dtype != NSP_BF16 && dq_dtype != NSP_F32) || (dkv_dtype != NSP_BF16 && dkv_dtype != NSP_F32))
    return NSP_ERR_INVALID_ARG;
  if (plan->n_bwd == 0) return NSP_OK;
  if (!q || !k || !v || !o || !d_o || !lse || !dq || !dk || !dv) return NSP_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(d_o) || !aligned16(lse) ||
      !aligned16(dq) || !aligned16(dk) || !aligned16(dv))
    return NSP_ERR_INVALID_ARG;
  size_t base = 0;
  nsp_plan_sizes(plan, nullptr, nullptr, nullptr, nullptr, &base);
  const size_t need = recompute ? recompute_ws_bytes(plan) : base;
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) != 0 || ws_bytes < need) return NSP_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* wsb = static_cast<char*>(ws);
  float* dq_acc = static_cast<float*>(ws);
  float* delta = reinterpret_cast<float*>(wsb + align_up(static_cast<size_t>(plan->q_elems) * 4, 256));
  int32_t* dq_turn = plan->deterministic
                         ? reinterpret_cast<int32_t*>(wsb + align_up(static_cast<size_t>(plan->q_elems) * 4, 256) +
                                                      align_up(static_cast<size_t>(plan->lse_elems) * 4, 256))
                         : nullptr;
  float* lse_ws = reinterpret_cast<float*>(wsb + base);
  uint8_t* d_mask = reinterpret_cast<uint8_t*>(wsb + base + align_up(static_cast<size_t>(plan->lse_elems) * 4, 256));

  BwdMaps maps;
  std::memset(&maps, 0, sizeof(maps));
  FwdMaps fmaps;
  if (recompute) std::memset(&fmaps, 0, sizeof(fmaps));
  for (size_t r = 0; r < plan->runs.size(); ++r) {
    const RunInfo& run = plan->runs[r];
    if (!encode_run_map(&maps.q[r], q, run.q_off, run.tokens, run.hq, plan->head_dim) ||
        !encode_run_map(&maps.d_o[r], d_o, run.q_off, run.tokens, run.hq, plan->head_dim) ||
        !encode_run_map(&maps.k[r], k, run.kv_off, run.tokens, run.hkv, plan->head_dim) ||
        !encode_run_map(&maps.v[r], v, run.kv_off, run.tokens, run.hkv, plan->head_dim))
      return NSP_ERR_CUDA;
    if (dkv_dtype == NSP_F32 && (!encode_run_map_f32(&maps.dk[r], dk, run.kv_off, run.tokens, run.hkv, plan->head_dim) ||
                                 !encode_run_map_f32(&maps.dv[r], dv, run.kv_off, run.tokens, run.hkv, plan->head_dim)))
      return NSP_ERR_CUDA;
    if (recompute) fmaps.q[r] = maps.q[r], fmaps.k[r] = maps.k[r], fmaps.v[r] = maps.v[r];
  }
  if (cudaMemsetAsync(plan->d_counters + 1, 0, 2 * sizeof(int32_t), st) != cudaSuccess) return NSP_ERR_CUDA;
  if (cudaMemsetAsync(plan->d_front, 0, sizeof(int32_t) * (plan->n_bwd / kFrontBlock + 1), st) != cudaSuccess)
    return NSP_ERR_CUDA;
  if (recompute) {
    // from pageable memory the runtime stages the flags before it returns; a pinned array must stay unchanged until
    // the stream has passed this copy
    if (cudaMemcpyAsync(d_mask, recompute, static_cast<size_t>(plan->n_seg), cudaMemcpyHostToDevice, st) != cudaSuccess)
      return NSP_ERR_CUDA;
    if (cudaMemsetAsync(plan->d_counters, 0, sizeof(int32_t), st) != cudaSuccess) return NSP_ERR_CUDA;
    FwdArgs fa;
    fa.seg = plan->d_seg;
    fa.items = plan->d_fwd;
    fa.n_items = static_cast<int32_t>(plan->n_fwd);
    fa.counter = plan->d_counters;
    fa.status = status_word(plan);
    fa.o = nullptr;
    fa.lse = lse_ws;
    fa.scale_log2 = softmax_scale * 1.4426950408889634f;
    fa.wait_limit = plan->wait_limit;
    fa.withhold = 0;
    fa.q_elems = plan->q_elems;
    fa.lse_elems = plan->lse_elems;
    fa.seg_mask = d_mask;
    fa.rows = plan->d_rows;
    fa.d_o = static_cast<const __nv_bfloat16*>(d_o);
    fa.delta = delta;
    prof_mark(plan, NSP_KERNEL_FWD, 0, st);
    if (launch_fwd(fmaps, fa, plan->head_dim, plan->num_sms, st) != cudaSuccess) return NSP_ERR_CUDA;
    prof_mark(plan, NSP_KERNEL_FWD, 1, st);
  }
  // Segments of at most 128 tokens are finished by the first-tile kernel alone; a batch made only of such segments
  // needs no accumulator, no delta and no conversion pass.
  const bool multi = plan->max_len > kBM;
  NSP_LOGF("bwd plan %p stream %p scale %g%s%s", static_cast<const void*>(plan), stream, softmax_scale,
           recompute ? ", recomputing marked segments" : "", multi ? "" : ", first-tile kernel only");
  if (dq_turn && multi &&
      cudaMemsetAsync(dq_turn, 0, static_cast<size_t>(plan->n_fwd) * 4, st) != cudaSuccess)
    return NSP_ERR_CUDA;
  prof_mark(plan, NSP_KERNEL_BWD_PRE, 0, st);
  if (multi || recompute) {
    if (launch_bwd_preprocess(plan->d_seg, plan->n_seg, plan->d_row_base, plan->lse_elems, plan->head_dim,
                              static_cast<const __nv_bfloat16*>(o), static_cast<const __nv_bfloat16*>(d_o), delta,
                              dq_acc, recompute ? d_mask : nullptr, recompute ? lse : nullptr,
                              recompute ? lse_ws : nullptr, st) != cudaSuccess)
      return NSP_ERR_CUDA;
  }
  prof_mark(plan, NSP_KERNEL_BWD_PRE, 1, st);
  BwdArgs a;
  a.seg = plan->d_seg;
  a.status = status_word(plan);
  a.lse = recompute ? lse_ws : lse;
  a.delta = delta;
  a.dq_acc = dq_acc;
  a.dq = dq;
  a.dq_f32 = dq_dtype == NSP_F32;
  a.dq_turn = dq_turn;
  a.dq_rounded = plan->rounded_dq ? 1 : 0;
  a.front = plan->d_front;
  a.rows = plan->d_rows;
  a.dk = dk;
  a.dv = dv;
  a.dkv_f32 = dkv_dtype == NSP_F32;
  a.scale = softmax_scale;
  a.scale_log2 = softmax_scale * 1.4426950408889634f;
  a.wait_limit = plan->wait_limit;
  a.q_elems = plan->q_elems;
  a.kv_elems = plan->kv_elems;
  a.lse_elems = plan->lse_elems;
  // first-tile kernel: q tile 0 of every segment (its dQ rows; its part of, or all of, dK / dV rows 0..127)
  a.items = plan->d_bwd_first;
  a.n_items = static_cast<int32_t>(plan->n_first);
  a.counter = plan->d_counters + 2;
  prof_mark(plan, NSP_KERNEL_BWD_FIRST, 0, st);
  if (launch_bwd_first(maps, a, plan->head_dim, plan->num_sms, st) != cudaSuccess) return NSP_ERR_CUDA;
  prof_mark(plan, NSP_KERNEL_BWD_FIRST, 1, st);
  // main kernel: everything else
  a.items = plan->d_bwd_exec;
  a.n_items = static_cast<int32_t>(plan->n_bwd);
  a.counter = plan->d_counters + 1;
  prof_mark(plan, NSP_KERNEL_BWD_MAIN, 0, st);
  if (multi && launch_bwd(maps, a, plan->head_dim, plan->num_sms, st) != cudaSuccess) return NSP_ERR_CUDA;
  prof_mark(plan, NSP_KERNEL_BWD_MAIN, 1, st);
  prof_mark(plan, NSP_KERNEL_BWD_POST, 0, st);
  if (multi && launch_bwd_postprocess(plan->d_seg, plan->n_seg, plan->d_row_base, plan->lse_elems, plan->head_dim, dq_acc, dq,
                                      dq_dtype == NSP_F32, softmax_scale, st) != cudaSuccess)
    return NSP_ERR_CUDA;
  prof_mark(plan, NSP_KERNEL_BWD_POST, 1, st);
  return NSP_OK;
}

}  // namespace

int nsp_attn_bwd(const nsp_plan_t* plan, const void* q, const void* k, const void* v, const void* o, const void* d_o,
                 const float* lse, void* dq, void* dk, void* dv, int dq_dtype, int dkv_dtype, float softmax_scale,
                 void* ws, size_t ws_bytes, void* stream) {
  return bwd_impl(plan, nullptr, q, k, v, o, d_o, lse, dq, dk, dv, dq_dtype, dkv_dtype, softmax_scale, ws, ws_bytes,
                  stream);
}

namespace {

// Device layout of the host-to-host step's workspace: the nine packed tensors, then the backward workspace.
struct HostStepLayout {
  size_t q, k, v, d_o, o, lse, dq, dk, dv, bwd_ws, total;
  size_t q_bytes, kv_bytes, lse_bytes, dq_bytes, dkv_bytes, bwd_ws_bytes;
};

bool host_step_layout(const nsp_plan_t* plan, int dq_dtype, int dkv_dtype, HostStepLayout* L) {
  if ((dq_dtype != NSP_BF16 && dq_dtype != NSP_F32) || (dkv_dtype != NSP_BF16 && dkv_dtype != NSP_F32)) return false;
  size_t bwd_ws = 0;
  nsp_plan_sizes(plan, nullptr, nullptr, nullptr, nullptr, &bwd_ws);
  L->q_bytes = static_cast<size_t>(plan->q_elems) * 2;
  L->kv_bytes = static_cast<size_t>(plan->kv_elems) * 2;
  L->lse_bytes = static_cast<size_t>(plan->lse_elems) * 4;
  L->dq_bytes = static_cast<size_t>(plan->q_elems) * (dq_dtype == NSP_F32 ? 4 : 2);
  L->dkv_bytes = static_cast<size_t>(plan->kv_elems) * (dkv_dtype == NSP_F32 ? 4 : 2);
  L->bwd_ws_bytes = bwd_ws;
  size_t at = 0;
  auto take = [&](size_t bytes) {
    const size_t here = at;
    at += align_up(bytes > 0 ? bytes : 1, 256);
    return here;
  };
  L->q = take(L->q_bytes), L->k = take(L->kv_bytes), L->v = take(L->kv_bytes), L->d_o = take(L->q_bytes);
  L->o = take(L->q_bytes), L->lse = take(L->lse_bytes);
  L->dq = take(L->dq_bytes), L->dk = take(L->dkv_bytes), L->dv = take(L->dkv_bytes);
  L->bwd_ws = take(bwd_ws);
  L->total = at;
  return true;
}

}  // namespace

int nsp_plan_step_host_ws_bytes(const nsp_plan_t* plan, int dq_dtype, int dkv_dtype, size_t* bytes) {
  if (!plan || !bytes) return NSP_ERR_INVALID_ARG;
  HostStepLayout L;
  if (!host_step_layout(plan, dq_dtype, dkv_dtype, &L)) return NSP_ERR_INVALID_ARG;
  *bytes = L.total;
  return NSP_OK;
}

int nsp_attn_step_host(nsp_plan_t* plan, const void* h_q, const void* h_k, const void* h_v, const void* h_do, void* h_o,
                       float* h_lse, void* h_dq, void* h_dk, void* h_dv, int dq_dtype, int dkv_dtype,
                       float softmax_scale, void* dev_ws, size_t dev_ws_bytes, void* stream) {
  if (!plan) return NSP_ERR_INVALID_ARG;
  if (const int failed = plan_failed(plan)) return failed;
  HostStepLayout L;
  if (!host_step_layout(plan, dq_dtype, dkv_dtype, &L)) return NSP_ERR_INVALID_ARG;
  if (plan->n_fwd == 0) return NSP_OK;
  if (!h_q || !h_k || !h_v || !h_do || !h_o || !h_lse || !h_dq || !h_dk || !h_dv) return NSP_ERR_INVALID_ARG;
  if (!dev_ws || (reinterpret_cast<uintptr_t>(dev_ws) & 255) != 0 || dev_ws_bytes < L.total) return NSP_ERR_WORKSPACE;
  if (!plan->copy_stream) {
    if (cudaStreamCreateWithFlags(&plan->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return NSP_ERR_CUDA;
    for (cudaEvent_t& e : plan->hev)
      if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return NSP_ERR_CUDA;
  }
  cudaStream_t comp = static_cast<cudaStream_t>(stream), cp = plan->copy_stream;
  char* base = static_cast<char*>(dev_ws);
  enum { kFree = 0, kQkvIn, kDoIn, kFwdDone, kBwdDone, kAllOut };
  auto ok = [](cudaError_t e) { return e == cudaSuccess; };
  const cudaMemcpyKind in = cudaMemcpyHostToDevice, out = cudaMemcpyDeviceToHost;
  NSP_LOGF("host step plan %p stream %p: %zu bytes in, %zu bytes out", static_cast<const void*>(plan), stream,
           2 * L.q_bytes + 2 * L.kv_bytes, L.q_bytes + L.lse_bytes + L.dq_bytes + 2 * L.dkv_bytes);
  // the device buffers are free once everything enqueued on the caller's stream so far has run
  if (!ok(cudaEventRecord(plan->hev[kFree], comp)) || !ok(cudaStreamWaitEvent(cp, plan->hev[kFree], 0))) return NSP_ERR_CUDA;
  if (!ok(cudaMemcpyAsync(base + L.q, h_q, L.q_bytes, in, cp)) || !ok(cudaMemcpyAsync(base + L.k, h_k, L.kv_bytes, in, cp)) ||
      !ok(cudaMemcpyAsync(base + L.v, h_v, L.kv_bytes, in, cp)) || !ok(cudaEventRecord(plan->hev[kQkvIn], cp)))
    return NSP_ERR_CUDA;
  // dO travels in under the forward pass
  if (!ok(cudaMemcpyAsync(base + L.d_o, h_do, L.q_bytes, in, cp)) || !ok(cudaEventRecord(plan->hev[kDoIn], cp)))
    return NSP_ERR_CUDA;
  if (!ok(cudaStreamWaitEvent(comp, plan->hev[kQkvIn], 0))) return NSP_ERR_CUDA;
  int rc = nsp_attn_fwd(plan, base + L.q, base + L.k, base + L.v, base + L.o, reinterpret_cast<float*>(base + L.lse),
                        softmax_scale, nullptr, 0, stream);
  if (rc != NSP_OK) return rc;
  // O and LSE travel out under the backward pass
  if (!ok(cudaEventRecord(plan->hev[kFwdDone], comp)) || !ok(cudaStreamWaitEvent(cp, plan->hev[kFwdDone], 0)) ||
      !ok(cudaMemcpyAsync(h_o, base + L.o, L.q_bytes, out, cp)) || !ok(cudaMemcpyAsync(h_lse, base + L.lse, L.lse_bytes, out, cp)))
    return NSP_ERR_CUDA;
  if (!ok(cudaStreamWaitEvent(comp, plan->hev[kDoIn], 0))) return NSP_ERR_CUDA;
  rc = nsp_attn_bwd(plan, base + L.q, base + L.k, base + L.v, base + L.o, base + L.d_o,
                    reinterpret_cast<const float*>(base + L.lse), base + L.dq, base + L.dk, base + L.dv, dq_dtype, dkv_dtype,
                    softmax_scale, base + L.bwd_ws, L.bwd_ws_bytes, stream);
  if (rc != NSP_OK) return rc;
  if (!ok(cudaEventRecord(plan->hev[kBwdDone], comp)) || !ok(cudaStreamWaitEvent(cp, plan->hev[kBwdDone], 0)) ||
      !ok(cudaMemcpyAsync(h_dq, base + L.dq, L.dq_bytes, out, cp)) || !ok(cudaMemcpyAsync(h_dk, base + L.dk, L.dkv_bytes, out, cp)) ||
      !ok(cudaMemcpyAsync(h_dv, base + L.dv, L.dkv_bytes, out, cp)) || !ok(cudaEventRecord(plan->hev[kAllOut], cp)) ||
      !ok(cudaStreamWaitEvent(comp, plan->hev[kAllOut], 0)))  // the step is complete on the caller's stream
    return NSP_ERR_CUDA;
  return NSP_OK;
}

int nsp_plan_recompute_ws_bytes(const nsp_plan_t* plan, size_t* bytes) {
  if (!plan || !bytes) return NSP_ERR_INVALID_ARG;
  *bytes = recompute_ws_bytes(plan);
  return NSP_OK;
}

int nsp_attn_bwd_recompute(const nsp_plan_t* plan, const uint8_t* recompute, const void* q, const void* k,
                           const void* v, const void* o, const void* d_o, const float* lse, void* dq, void* dk,
                           void* dv, int dq_dtype, int dkv_dtype, float softmax_scale, void* ws, size_t ws_bytes,
                           void* stream) {
  if (!plan || !recompute) return NSP_ERR_INVALID_ARG;
  return bwd_impl(plan, recompute, q, k, v, o, d_o, lse, dq, dk, dv, dq_dtype, dkv_dtype, softmax_scale, ws, ws_bytes,
                  stream);
}

int nsp_recompute_mark(const int32_t* cu_seqlens, const int32_t* hq, const int32_t* level, int32_t n_seg,
                       int32_t head_dim, int64_t budget_bytes, uint8_t* recompute, int64_t* saved_bytes) {
  if (n_seg < 0 || head_dim <= 0 || budget_bytes < 0) return NSP_ERR_INVALID_ARG;
  if (n_seg > 0 && (!cu_seqlens || !hq || !level || !recompute)) return NSP_ERR_INVALID_ARG;
  for (int s = 0; s < n_seg; ++s)
    if (cu_seqlens[s + 1] < cu_seqlens[s] || hq[s] <= 0) return NSP_ERR_INVALID_ARG;
  std::vector<int> order(n_seg);
  for (int s = 0; s < n_seg; ++s) order[s] = s;
  auto len = [&](int s) { return static_cast<int64_t>(cu_seqlens[s + 1]) - cu_seqlens[s]; };
  // recomputation cost of a segment: its causal (query, key) pairs times its query heads
  auto cost = [&](int s) { return static_cast<int64_t>(hq[s]) * (len(s) * (len(s) + 1) / 2); };
  std::stable_sort(order.begin(), order.end(), [&](int x, int y) {
    if (level[x] != level[y]) return level[x] > level[y];
    return cost(x) > cost(y);
  });
  int64_t used = 0;
  bool cut = false;
  for (int s : order) {
    // what saving the segment keeps alive: its slice of O (bf16) and of the LSE (fp32)
    const int64_t bytes = len(s) * hq[s] * (static_cast<int64_t>(head_dim) * 2 + 4);
    if (!cut && used + bytes <= budget_bytes) {
      used += bytes;
      recompute[s] = 0;
    } else {
      cut = true;
      recompute[s] = 1;
    }
  }
  if (saved_bytes) *saved_bytes = used;
  return NSP_OK;
}

namespace {
// One warp waits on a barrier nothing ever arrives at; the bounded wait runs out after limit_clk SM cycles and the
// warp records it in the status word exactly as the attention kernels would.
__global__ void selftest_wait_kernel(StatusWord status, long long limit_clk) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    fence_mbar_init();
  }
  __syncwarp();
  const bool ok = mbar_wait(&bar, 0, limit_clk);
  if (!ok && threadIdx.x == 0) report_timeout(status, -1, kWhereSelfTest, static_cast<int32_t>(limit_clk >> 10));
}
}  // namespace

int nsp_selftest_wait_timeout(const nsp_plan_t* plan, int64_t limit_clk, void* stream) {
  if (!plan || limit_clk < 1 || limit_clk > (1ll << 31)) return NSP_ERR_INVALID_ARG;
  if (const int failed = plan_failed(plan)) return failed;
  selftest_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status_word(plan), limit_clk);
  count_launches(1);
  return cudaGetLastError() == cudaSuccess ? NSP_OK : NSP_ERR_CUDA;
}

int nsp_device_status(const nsp_plan_t* plan, int32_t out[4]) {
  if (!plan || !out) return NSP_ERR_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess) return NSP_ERR_CUDA;
  if (cudaMemcpy(out, plan->d_status, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess) return NSP_ERR_CUDA;
  if (out[0] != 0 && !plan->sticky) const_cast<nsp_plan_t*>(plan)->sticky = out[0];
  return NSP_OK;
}

int nsp_plan_set_wait_limit(nsp_plan_t* plan, int64_t sm_clocks) {
  if (!plan || sm_clocks < 1000) return NSP_ERR_INVALID_ARG;
  plan->wait_limit = sm_clocks;
  return NSP_OK;
}

#ifdef NSP_CHECKED
int nsp_checked_withhold_load(nsp_plan_t* plan, int enable) {
  if (!plan) return NSP_ERR_INVALID_ARG;
  plan->withhold = enable != 0;
  return NSP_OK;
}
#endif

int nsp_plan_set_profiling(nsp_plan_t* plan, int enable) {
  if (!plan) return NSP_ERR_INVALID_ARG;
  if (enable && !plan->ev[0]) {
    for (cudaEvent_t& e : plan->ev)
      if (cudaEventCreate(&e) != cudaSuccess) return NSP_ERR_CUDA;
  }
  plan->profiling = enable != 0;
  if (!enable)
    for (bool& v : plan->ev_valid) v = false;
  return NSP_OK;
}

int nsp_plan_kernel_ms(const nsp_plan_t* plan, int kernel_id, float* ms) {
  if (!plan || !ms || kernel_id < 0 || kernel_id >= NSP_KERNEL_COUNT) return NSP_ERR_INVALID_ARG;
  if (!plan->profiling || !plan->ev_valid[kernel_id]) return NSP_ERR_INVALID_ARG;
  if (cudaEventSynchronize(plan->ev[2 * kernel_id + 1]) != cudaSuccess) return NSP_ERR_CUDA;
  if (cudaEventElapsedTime(ms, plan->ev[2 * kernel_id], plan->ev[2 * kernel_id + 1]) != cudaSuccess) return NSP_ERR_CUDA;
  return NSP_OK;
}

int nsp_plan_destroy(nsp_plan_t* plan) {
  free_plan(plan);
  return NSP_OK;
}

}  // extern "C"

// Host side of the C ABI declared in include/attn.h: argument checks, TMA descriptors,
// persistent-grid set-up and the launch of attn_fwd_kernel.
#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include <vector>

#include "../../include/attn.h"
#include "attn_fwd_kernel.cuh"
#include "attn_fwd_sb3.cuh"
#include "attn_fwd_pair.cuh"
#include "attn_fwd_w16.cuh"
#include "attn_merge_kernel.cuh"

namespace {

using attn::FwdParams;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kMaxDevices = 64;
constexpr int kCounterSlots = 1024;  // one work counter per launch in flight, reused round-robin
constexpr int kStampSlots = 64;      // launches whose clock stamps are kept (a ring)
constexpr int kSplitStreams = 8;
constexpr int kMaxSplits = 64;

struct DeviceState {
  bool ready = false;
  bool failed = false;
  int sm_count = 0;
  int max_pairs = 0;                 // CTA pairs (clusters of two) that can be resident at once
  unsigned int* counters = nullptr;  // [kCounterSlots]
  int* status = nullptr;             // [2]
  unsigned long long* clock_stamps = nullptr;  // [kStampSlots][4], one entry per launch, see FwdParams
  std::atomic<unsigned int> next_slot{0};
  std::atomic<unsigned int> next_stamp{0};    // launches stamped so far
  // attn_fwd_host staging
  void* stage[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
  size_t stage_bytes[5] = {0, 0, 0, 0, 0};
  // attn_fwd_host pipeline: upload, compute and download streams and a pool of events
  cudaStream_t pipe[3] = {nullptr, nullptr, nullptr};
  std::vector<cudaEvent_t> events;
  // attn_fwd_splitkv: streams the key ranges are launched on, so that their small grids share the GPU
  cudaStream_t split[kSplitStreams] = {};
};

std::mutex g_mutex;
DeviceState g_dev[kMaxDevices];
EncodeTiledFn g_encode = nullptr;
std::atomic<int> g_opt_scheduler{2};
std::atomic<int> g_opt_max_ctas{0};
std::atomic<int> g_opt_kernel{0};  // 0: dual query stage, 1: triple score buffer, 2: CTA pairs, 3: two softmax threads per row
std::atomic<int> g_opt_rescale_threshold{8};
std::atomic<int> g_opt_split_p{1};
std::atomic<int> g_opt_overlap_epilogue{1};
std::atomic<int> g_opt_host_pipeline{1};
std::atomic<int> g_opt_gqa_pack{1};

// How many clusters of two CTAs of the pair kernel the device holds at once (its shared memory
// must have been opted in already); never more than one pair per two SMs.
int resident_pairs(int sm_count) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * (sm_count / 2 > 0 ? sm_count / 2 : 1));
  cfg.blockDim = dim3(attn::kThreads);
  cfg.dynamicSmemBytes = attn::pair::kSmemBytes2;
  cudaLaunchAttribute at;
  at.id = cudaLaunchAttributeClusterDimension;
  at.val.clusterDim.x = 2;
  at.val.clusterDim.y = 1;
  at.val.clusterDim.z = 1;
  cfg.attrs = &at;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, attn::pair::attn_fwd_pair_kernel, &cfg) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    n = sm_count / 2;
  }
  if (n > sm_count / 2) n = sm_count / 2;
  return n > 0 ? n : 1;
}

// Per-device one-time set-up: architecture check, kernel attribute, scheduler counters and
// status word.  Returns the state or nullptr (with *st set).
DeviceState* device_state(attn_status_t* st) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    *st = ATTN_ERR_CUDA;
    return nullptr;
  }
  DeviceState& d = g_dev[dev];
  std::lock_guard<std::mutex> lock(g_mutex);
  if (d.ready) return &d;
  if (d.failed) {
    *st = ATTN_ERR_ARCH;
    return nullptr;
  }
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
    *st = ATTN_ERR_CUDA;
    return nullptr;
  }
  if (major != 10) {
    d.failed = true;
    *st = ATTN_ERR_ARCH;
    return nullptr;
  }
  if (g_encode == nullptr) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        fn == nullptr) {
      *st = ATTN_ERR_CUDA;
      return nullptr;
    }
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
      cudaFuncSetAttribute(attn::attn_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           attn::kSmemBytes) != cudaSuccess ||
      cudaFuncSetAttribute(attn::sb3::attn_fwd_sb3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           attn::sb3::kSmemBytes3) != cudaSuccess ||
      cudaFuncSetAttribute(attn::pair::attn_fwd_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           attn::pair::kSmemBytes2) != cudaSuccess ||
      cudaFuncSetAttribute(attn::w16::attn_fwd_w16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           attn::kSmemBytes) != cudaSuccess ||
      cudaMalloc(&d.counters, kCounterSlots * sizeof(unsigned int)) != cudaSuccess ||
      cudaMalloc(&d.status, 2 * sizeof(int)) != cudaSuccess ||
      cudaMemset(d.status, 0, 2 * sizeof(int)) != cudaSuccess ||
      cudaMalloc(&d.clock_stamps, kStampSlots * 4 * sizeof(unsigned long long)) != cudaSuccess ||
      cudaMemset(d.clock_stamps, 0, kStampSlots * 4 * sizeof(unsigned long long)) != cudaSuccess) {
    *st = ATTN_ERR_CUDA;
    return nullptr;
  }
  d.max_pairs = resident_pairs(d.sm_count);
  d.ready = true;
  return &d;
}

// Element strides of the (batch, sequence, head) axes of a [B, S, H, 128] BF16 tensor; the head
// dimension is contiguous.
struct Strides3 {
  long long b, s, h;
};
Strides3 contiguous_strides(int S, int H) {
  return Strides3{static_cast<long long>(S) * H * 128, static_cast<long long>(H) * 128, 128};
}

// BF16 tensor seen as 4-D (D, H, S, B) with the given element strides; box = 64 elements x 1 head
// x 128 rows, 128-byte swizzle, out-of-range rows read as zero and are clipped on store.
bool make_tensor_map(CUtensorMap* tm, const void* base, int B, int S, int H, Strides3 st, int pack_log2 = 0,
                     unsigned int box_rows = 128) {
  const cuuint64_t dims[4] = {128, static_cast<cuuint64_t>(H), static_cast<cuuint64_t>(S),
                              static_cast<cuuint64_t>(B)};
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(st.h) * 2, static_cast<cuuint64_t>(st.s) * 2,
                                 static_cast<cuuint64_t>(st.b) * 2};
  // packed query tiles: `group` heads x (128 / group) rows, laid out row-major as (row, head)
  const cuuint32_t box[4] = {64, 1u << pack_log2, box_rows >> pack_log2, 1};
  const cuuint32_t elem_strides[4] = {1, 1, 1, 1};
  return g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box,
                  elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

attn_status_t check_args(const void* q, const void* k, const void* v, void* o, const float* lse, int B, int Hq,
                         int Hkv, int Sq, int Sk, int D, int causal, float scale, bool device_ptrs) {
  if (q == nullptr || k == nullptr || v == nullptr || o == nullptr) return ATTN_ERR_NULL;
  if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || D <= 0) return ATTN_ERR_SHAPE;
  if (Hq % Hkv != 0) return ATTN_ERR_SHAPE;
  if (D != attn::kHeadDim) return ATTN_ERR_UNSUPPORTED;
  if (!std::isfinite(scale) || !(scale > 0.f)) return ATTN_ERR_UNSUPPORTED;
  // sizes the 32-bit tile arithmetic and the TMA coordinates can hold
  if (static_cast<long long>(B) * Hq * ((Sq + 127) / 128) > 0x3fffffffLL) return ATTN_ERR_UNSUPPORTED;
  if (Sq > 0x3fffff00 || Sk > 0x3fffff00) return ATTN_ERR_UNSUPPORTED;
  if (device_ptrs) {
    const uintptr_t mask = 15;
    if ((reinterpret_cast<uintptr_t>(q) & mask) || (reinterpret_cast<uintptr_t>(k) & mask) ||
        (reinterpret_cast<uintptr_t>(v) & mask) || (reinterpret_cast<uintptr_t>(o) & mask))
      return ATTN_ERR_ALIGN;
    if (lse != nullptr && (reinterpret_cast<uintptr_t>(lse) & 3)) return ATTN_ERR_ALIGN;
  }
  return ATTN_OK;
}

// Problem geometry and work decomposition (no device access).
void fill_plan(FwdParams* p, int B, int Hq, int Hkv, int Sq, int Sk, int causal) {
  std::memset(p, 0, sizeof(*p));
  p->B = B; p->Hq = Hq; p->Hkv = Hkv; p->Sq = Sq; p->Sk = Sk;
  p->group = Hq / Hkv;
  p->causal = causal ? 1 : 0;
  p->off = Sk - Sq;
  p->n_qt = (Sq + attn::kTile - 1) / attn::kTile;
  p->n_kb = (Sk + attn::kTile - 1) / attn::kTile;
  p->kernel = g_opt_kernel.load();
  // Short query sequences of a GQA group (all of it fits two packed tiles): pack the group's
  // heads into the rows of a tile, so that each KV head is streamed once per row tile pair.
  p->pack_log2 = 0;
  if (g_opt_gqa_pack.load() != 0 && p->kernel != 1 && p->group >= 2 && p->group <= 16 &&
      (p->group & (p->group - 1)) == 0 && Sq <= 2 * (attn::kTile / p->group)) {
    while ((1 << p->pack_log2) < p->group) ++p->pack_log2;
  }
  if (p->kernel >= 2 && p->pack_log2 > 0) p->kernel = 0;  // packed tiles exist in the default kernel only
  if (p->pack_log2 > 0) {
    p->n_qt = (Sq + (attn::kTile >> p->pack_log2) - 1) / (attn::kTile >> p->pack_log2);
    p->pair_heads = 0;
    p->items_per_group = (p->n_qt + 1) / 2;
    p->n_work = B * Hkv * p->items_per_group;
  } else if (p->kernel == 1) {  // triple score buffer: one query tile per work item
    p->pair_heads = 0;
    p->items_per_group = p->n_qt;
    p->n_work = B * Hq * p->n_qt;
  } else if (p->kernel == 2) {  // CTA pairs: four query tiles per work item
    p->pair_heads = (p->group % 2 == 0) ? 1 : 0;
    if (p->pair_heads) {
      p->items_per_group = ((p->n_qt + 1) / 2) * (p->group / 2);
      p->n_work = B * Hkv * p->items_per_group;
    } else {
      p->items_per_group = (p->n_qt + 3) / 4;
      p->n_work = B * Hq * p->items_per_group;
    }
  } else {
    p->pair_heads = (p->group % 2 == 0) ? 1 : 0;
    if (p->pair_heads) {
      p->items_per_group = p->n_qt * (p->group / 2);
      p->n_work = B * Hkv * p->items_per_group;
    } else {
      p->items_per_group = (p->n_qt + 1) / 2;
      p->n_work = B * Hq * p->items_per_group;
    }
  }
  p->n_groups = p->n_work / p->items_per_group;
  // Causal: interleave the items of as many heads as keep their K/V (2 tensors x Sk x 128 BF16 per
  // head) within about 72 MB of L2 (measured best of 24..100 MB); non-causal items are all alike, so strict head-major order.
  p->head_group = 1;
  p->head_group_extra = p->n_groups;  // every super-group is one group
  if (p->causal) {
    const long long kv_bytes = 2LL * Sk * attn::kHeadDim * 2;
    long long g = (72LL << 20) / kv_bytes;
    if (g < 1) g = 1;
    if (g > 64) g = 64;
    if (g > p->n_groups) g = p->n_groups;
    // k super-groups of nearly equal size (they differ by at most one group), so that the last
    // one is not a small remainder whose long items would start when little other work is left
    const int k = static_cast<int>((p->n_groups + g - 1) / g);
    const int base = p->n_groups / k;
    const int extra = p->n_groups % k;
    if (extra == 0) {
      p->head_group = base;
      p->head_group_extra = k;
    } else {
      p->head_group = base + 1;
      p->head_group_extra = extra;
    }
  }
  p->dynamic = (g_opt_scheduler.load() == 2) ? 1 : 0;
  p->rescale_threshold = static_cast<float>(g_opt_rescale_threshold.load());
  p->split_p = g_opt_split_p.load();
  p->overlap_epilogue = g_opt_overlap_epilogue.load();
}

// Launches the kernel selected by the "kernel" option (the plan in `p` was made for it).
cudaError_t launch_fwd(const CUtensorMap& tm_q, const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                       const CUtensorMap& tm_o, const FwdParams& p, int grid, cudaStream_t s) {
  if (p.kernel == 1) {
    attn::sb3::attn_fwd_sb3_kernel<<<grid, attn::kThreads, attn::sb3::kSmemBytes3, s>>>(tm_q, tm_k, tm_v, tm_o, p);
  } else if (p.kernel == 3) {
    attn::w16::attn_fwd_w16_kernel<<<grid, attn::w16::kThreads16, attn::kSmemBytes, s>>>(tm_q, tm_k, tm_v, tm_o, p);
  } else if (p.kernel == 2) {  // grid = 2 x pairs; the cluster shape is a compile-time attribute of the kernel
    attn::pair::attn_fwd_pair_kernel<<<grid, attn::kThreads, attn::pair::kSmemBytes2, s>>>(tm_q, tm_k, tm_v, tm_o, p);
  } else {
    attn::attn_fwd_kernel<<<grid, attn::kThreads, attn::kSmemBytes, s>>>(tm_q, tm_k, tm_v, tm_o, p);
  }
  return cudaGetLastError();
}

int plan_grid(const FwdParams& p, int sm_count, int max_pairs = 0) {
  if (p.kernel == 2) {  // CTAs come in pairs, one pair per work item in flight
    int pairs = p.n_work;
    if (g_opt_scheduler.load() != 0) {
      int cap = max_pairs > 0 ? max_pairs : sm_count / 2;
      const int max_ctas = g_opt_max_ctas.load();
      if (max_ctas > 0 && max_ctas / 2 < cap) cap = max_ctas / 2;
      if (cap < 1) cap = 1;
      if (pairs > cap) pairs = cap;
    }
    return 2 * pairs;
  }
  int grid = p.n_work;
  if (g_opt_scheduler.load() != 0) {
    int cap = sm_count;
    const int max_ctas = g_opt_max_ctas.load();
    if (max_ctas > 0 && max_ctas < cap) cap = max_ctas;
    if (grid > cap) grid = cap;
  }
  return grid;
}

}  // namespace

extern "C" {

attn_status_t attn_plan(int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal, int sm_count, int* plan) {
  if (plan == nullptr) return ATTN_ERR_NULL;
  int dummy = 0;
  attn_status_t st = check_args(&dummy, &dummy, &dummy, &dummy, nullptr, B, Hq, Hkv, Sq, Sk, D, causal, 1.0f, false);
  if (st != ATTN_OK) return st;
  if (sm_count <= 0) return ATTN_ERR_SHAPE;
  FwdParams p;
  fill_plan(&p, B, Hq, Hkv, Sq, Sk, causal);
  plan[0] = p.n_work;
  plan[1] = p.pair_heads;
  plan[2] = p.items_per_group;
  plan[3] = p.n_qt;
  plan[4] = p.n_kb;
  plan[5] = plan_grid(p, sm_count);
  return ATTN_OK;
}

attn_status_t attn_plan_item(int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal, int w, int* item) {
  if (item == nullptr) return ATTN_ERR_NULL;
  int dummy = 0;
  attn_status_t st = check_args(&dummy, &dummy, &dummy, &dummy, nullptr, B, Hq, Hkv, Sq, Sk, D, causal, 1.0f, false);
  if (st != ATTN_OK) return st;
  FwdParams p;
  fill_plan(&p, B, Hq, Hkv, Sq, Sk, causal);
  if (w < 0 || w >= p.n_work) return ATTN_ERR_SHAPE;
  if (p.kernel == 1) {  // one tile per item: the second stage is reported as unused
    attn::sb3::Item it;
    attn::sb3::decode_item(p, w, it);
    item[0] = it.b; item[1] = it.hkv; item[2] = it.hq; item[3] = it.hq;
    item[4] = it.row0; item[5] = p.n_qt * attn::kTile; item[6] = it.n; item[7] = 0;
    return ATTN_OK;
  }
  attn::Work wk;
  if (p.kernel == 2) {  // the leader CTA's view; attn_plan_item_pair gives either CTA's
    attn::pair::decode_work_pair(p, w, 0, wk);
  } else {
    attn::decode_work(p, w, wk);
  }
  item[0] = wk.b; item[1] = wk.hkv; item[2] = wk.hq[0]; item[3] = wk.hq[1];
  item[4] = wk.row0[0]; item[5] = wk.row0[1]; item[6] = wk.n[0]; item[7] = wk.n[1];
  return ATTN_OK;
}

attn_status_t attn_plan_item_pair(int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal, int w, int rank,
                                  int* item) {
  if (item == nullptr) return ATTN_ERR_NULL;
  int dummy = 0;
  attn_status_t st = check_args(&dummy, &dummy, &dummy, &dummy, nullptr, B, Hq, Hkv, Sq, Sk, D, causal, 1.0f, false);
  if (st != ATTN_OK) return st;
  FwdParams p;
  fill_plan(&p, B, Hq, Hkv, Sq, Sk, causal);
  if (p.kernel != 2) return ATTN_ERR_UNSUPPORTED;  // the plan in force is not the pair kernel's
  if (w < 0 || w >= p.n_work || rank < 0 || rank > 1) return ATTN_ERR_SHAPE;
  attn::Work wk;
  attn::pair::decode_work_pair(p, w, rank, wk);
  item[0] = wk.b; item[1] = wk.hkv; item[2] = wk.hq[0]; item[3] = wk.hq[1];
  item[4] = wk.row0[0]; item[5] = wk.row0[1]; item[6] = wk.n[0]; item[7] = wk.n[1];
  return ATTN_OK;
}

}  // extern "C"

namespace {

// Causal rule used by the kernels: key j of the K/V passed in is visible to query row i iff
// j <= i + off.  off = Sk - Sq by default (bottom-right alignment); a launch on a key range of a
// longer sequence passes the offset that keeps the global key indices.
constexpr long long kDefaultCausalOff = -(1ll << 62);

// A stride the TMA engine accepts: positive, a multiple of 8 elements (16 bytes), below 2^40
// bytes; axes of extent 1 are never stepped along, but the descriptor still wants a legal value.
attn_status_t check_strides(const long long* s) {
  if (s == nullptr) return ATTN_ERR_NULL;
  for (int i = 0; i < 3; ++i) {
    if (s[i] <= 0) return ATTN_ERR_SHAPE;
    if (s[i] % 8 != 0) return ATTN_ERR_ALIGN;
    if (s[i] >= (1ll << 39)) return ATTN_ERR_UNSUPPORTED;
  }
  if (s[1] < 128 || s[2] < 128) return ATTN_ERR_SHAPE;  // rows of 128 contiguous elements must not overlap
  return ATTN_OK;
}

attn_status_t fwd_device(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq, int Hkv,
                         int Sq, int Sk, int D, Strides3 sq, Strides3 sk, Strides3 sv, Strides3 so, int causal,
                         float scale, void* stream, long long causal_off = kDefaultCausalOff) {
  attn_status_t st = check_args(q, k, v, o, lse, B, Hq, Hkv, Sq, Sk, D, causal, scale, true);
  if (st != ATTN_OK) return st;
  DeviceState* dev = device_state(&st);
  if (dev == nullptr) return st;

  FwdParams p;
  fill_plan(&p, B, Hq, Hkv, Sq, Sk, causal);
  if (causal_off != kDefaultCausalOff) p.off = static_cast<int>(causal_off);

  CUtensorMap tm_q, tm_k, tm_v, tm_o;
  // the pair kernel loads K in boxes of 64 keys (each CTA keeps half of a 128-key block)
  if (!make_tensor_map(&tm_q, q, B, Sq, Hq, sq, p.pack_log2) ||
      !make_tensor_map(&tm_k, k, B, Sk, Hkv, sk, 0, p.kernel == 2 ? 64 : 128) ||
      !make_tensor_map(&tm_v, v, B, Sk, Hkv, sv) || !make_tensor_map(&tm_o, o, B, Sq, Hq, so, p.pack_log2))
    return ATTN_ERR_CUDA;

  p.scale = scale;
  p.scale_log2 = scale * 1.4426950408889634f;
  p.lse = lse;
  p.status = dev->status;
  // the triple-score-buffer kernel does not stamp: it takes no ring entry, so every entry counted is one a launch writes
  p.clock_stamps = p.kernel == 1 ? nullptr : dev->clock_stamps + 4 * (dev->next_stamp.fetch_add(1) % kStampSlots);
  const int grid = plan_grid(p, dev->sm_count, dev->max_pairs);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (p.dynamic) {
    const unsigned int slot = dev->next_slot.fetch_add(1) % kCounterSlots;
    p.counter = dev->counters + slot;
    if (cudaMemsetAsync(p.counter, 0, sizeof(unsigned int), s) != cudaSuccess) return ATTN_ERR_CUDA;
  }
  return launch_fwd(tm_q, tm_k, tm_v, tm_o, p, grid, s) == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

// attn_fwd_host as a three-stream pipeline.  Query rows are independent, so the problem is cut
// into chunks of whole 256-row work items, about one wave of CTAs each; chunk c's kernel runs
// while chunk c+1's rows (and, under the causal mask, only the keys that chunk c+1 newly needs)
// are uploaded and chunk c-1's output is downloaded, on separate copy engines.  Each chunk is
// one strided launch on views of the staging buffers; its LSE block is written compactly and
// scattered into the caller's [B, Hq, Sq] array by a 2-D copy.
attn_status_t host_pipeline(DeviceState* dev, const void* q, const void* k, const void* v, void* o, float* lse,
                            int B, int Hq, int Hkv, int Sq, int Sk, int causal, float scale, cudaStream_t user) {
  for (int i = 0; i < 3; ++i) {
    if (dev->pipe[i] == nullptr &&
        cudaStreamCreateWithFlags(&dev->pipe[i], cudaStreamNonBlocking) != cudaSuccess)
      return ATTN_ERR_CUDA;
  }
  const cudaStream_t s_up = dev->pipe[0], s_run = dev->pipe[1], s_down = dev->pipe[2];
  size_t next_event = 0;
  auto event = [&]() -> cudaEvent_t {
    if (next_event == dev->events.size()) {
      cudaEvent_t e = nullptr;
      if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
      dev->events.push_back(e);
    }
    return dev->events[next_event++];
  };
  bool ok = true;
  auto after = [&](cudaStream_t waiter, cudaStream_t signaller) {  // waiter continues after signaller's work so far
    cudaEvent_t e = event();
    ok = ok && e != nullptr && cudaEventRecord(e, signaller) == cudaSuccess &&
         cudaStreamWaitEvent(waiter, e, 0) == cudaSuccess;
  };
  // the pipeline starts after whatever the caller has queued on its stream
  after(s_up, user);
  after(s_run, user);
  after(s_down, user);

  const int D = attn::kHeadDim;
  const int off = Sk - Sq;  // >= 0 here
  const int waves = dev->sm_count / Hq > 0 ? dev->sm_count / Hq : 1;  // 256-row items of all heads per wave
  int chunk_rows = 256 * waves;
  if ((Sq + chunk_rows - 1) / chunk_rows > 64) chunk_rows = ((Sq + 63) / 64 + 255) / 256 * 256;
  const uint8_t* hq = static_cast<const uint8_t*>(q);
  const uint8_t* hk = static_cast<const uint8_t*>(k);
  const uint8_t* hv = static_cast<const uint8_t*>(v);
  uint8_t* ho = static_cast<uint8_t*>(o);
  uint8_t* dq = static_cast<uint8_t*>(dev->stage[0]);
  uint8_t* dk = static_cast<uint8_t*>(dev->stage[1]);
  uint8_t* dv = static_cast<uint8_t*>(dev->stage[2]);
  uint8_t* dout = static_cast<uint8_t*>(dev->stage[3]);
  float* dlse = static_cast<float*>(dev->stage[4]);
  const size_t q_row = static_cast<size_t>(Hq) * D * 2, kv_row = static_cast<size_t>(Hkv) * D * 2;
  attn_status_t st = ATTN_OK;
  for (int b = 0; b < B && ok && st == ATTN_OK; ++b) {
    int keys_up = 0;  // keys of this batch entry already queued for upload
    for (int r0 = 0; r0 < Sq && ok && st == ATTN_OK; r0 += chunk_rows) {
      const int r1 = r0 + chunk_rows < Sq ? r0 + chunk_rows : Sq;
      const int keys = causal ? (r1 + off < Sk ? r1 + off : Sk) : Sk;  // keys the rows below r1 can see
      if (keys > keys_up) {
        const size_t at = (static_cast<size_t>(b) * Sk + keys_up) * kv_row, n = (keys - keys_up) * kv_row;
        ok = ok && cudaMemcpyAsync(dk + at, hk + at, n, cudaMemcpyHostToDevice, s_up) == cudaSuccess &&
             cudaMemcpyAsync(dv + at, hv + at, n, cudaMemcpyHostToDevice, s_up) == cudaSuccess;
        keys_up = keys;
      }
      const size_t q_at = (static_cast<size_t>(b) * Sq + r0) * q_row, q_n = static_cast<size_t>(r1 - r0) * q_row;
      ok = ok && cudaMemcpyAsync(dq + q_at, hq + q_at, q_n, cudaMemcpyHostToDevice, s_up) == cudaSuccess;
      after(s_run, s_up);
      if (!ok) break;
      float* lse_blk = dlse + static_cast<size_t>(b) * Hq * Sq + static_cast<size_t>(Hq) * r0;  // [Hq][r1 - r0]
      st = fwd_device(dq + q_at, dk + static_cast<size_t>(b) * Sk * kv_row, dv + static_cast<size_t>(b) * Sk * kv_row,
                      dout + q_at, lse != nullptr ? lse_blk : nullptr, 1, Hq, Hkv, r1 - r0, keys, D,
                      contiguous_strides(Sq, Hq), contiguous_strides(Sk, Hkv), contiguous_strides(Sk, Hkv),
                      contiguous_strides(Sq, Hq), causal, scale, s_run);
      if (st != ATTN_OK) break;
      after(s_down, s_run);
      ok = ok && cudaMemcpyAsync(ho + q_at, dout + q_at, q_n, cudaMemcpyDeviceToHost, s_down) == cudaSuccess;
      if (lse != nullptr) {
        ok = ok && cudaMemcpy2DAsync(lse + static_cast<size_t>(b) * Hq * Sq + r0, static_cast<size_t>(Sq) * 4, lse_blk,
                                     static_cast<size_t>(r1 - r0) * 4, static_cast<size_t>(r1 - r0) * 4, Hq,
                                     cudaMemcpyDeviceToHost, s_down) == cudaSuccess;
      }
    }
  }
  // join: the caller's stream continues after all three, then the call synchronises it
  after(user, s_up);
  after(user, s_run);
  after(user, s_down);
  const bool synced = cudaStreamSynchronize(user) == cudaSuccess;
  if (st != ATTN_OK) return st;
  return (ok && synced) ? ATTN_OK : ATTN_ERR_CUDA;
}

}  // namespace

extern "C" {

attn_status_t attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq, int Hkv,
                       int Sq, int Sk, int D, int causal, float scale, void* stream) {
  return fwd_device(q, k, v, o, lse, B, Hq, Hkv, Sq, Sk, D, contiguous_strides(Sq, Hq), contiguous_strides(Sk, Hkv),
                    contiguous_strides(Sk, Hkv), contiguous_strides(Sq, Hq), causal, scale, stream);
}

attn_status_t attn_fwd_strided(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq,
                               int Hkv, int Sq, int Sk, int D, const long long* q_strides,
                               const long long* k_strides, const long long* v_strides, const long long* o_strides,
                               int causal, float scale, void* stream) {
  const long long* all[4] = {q_strides, k_strides, v_strides, o_strides};
  for (const long long* s : all) {
    const attn_status_t st = check_strides(s);
    if (st != ATTN_OK) return st;
  }
  return fwd_device(q, k, v, o, lse, B, Hq, Hkv, Sq, Sk, D, Strides3{q_strides[0], q_strides[1], q_strides[2]},
                    Strides3{k_strides[0], k_strides[1], k_strides[2]},
                    Strides3{v_strides[0], v_strides[1], v_strides[2]},
                    Strides3{o_strides[0], o_strides[1], o_strides[2]}, causal, scale, stream);
}

attn_status_t attn_fwd_host(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq,
                            int Hkv, int Sq, int Sk, int D, int causal, float scale, void* stream) {
  attn_status_t st = check_args(q, k, v, o, lse, B, Hq, Hkv, Sq, Sk, D, causal, scale, false);
  if (st != ATTN_OK) return st;
  DeviceState* dev = device_state(&st);
  if (dev == nullptr) return st;
  const size_t q_bytes = static_cast<size_t>(B) * Sq * Hq * D * 2;
  const size_t kv_bytes = static_cast<size_t>(B) * Sk * Hkv * D * 2;
  const size_t lse_bytes = static_cast<size_t>(B) * Hq * Sq * 4;
  const size_t need[5] = {q_bytes, kv_bytes, kv_bytes, q_bytes, lse_bytes};
  for (int i = 0; i < 5; ++i) {
    if (dev->stage_bytes[i] < need[i]) {
      if (dev->stage[i] != nullptr) cudaFree(dev->stage[i]);
      dev->stage[i] = nullptr;
      dev->stage_bytes[i] = 0;
      if (cudaMalloc(&dev->stage[i], need[i]) != cudaSuccess) return ATTN_ERR_CUDA;
      dev->stage_bytes[i] = need[i];
    }
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (g_opt_host_pipeline.load() != 0 && !(causal && Sq > Sk))
    return host_pipeline(dev, q, k, v, o, lse, B, Hq, Hkv, Sq, Sk, causal, scale, s);
  if (cudaMemcpyAsync(dev->stage[0], q, q_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(dev->stage[1], k, kv_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(dev->stage[2], v, kv_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess)
    return ATTN_ERR_CUDA;
  st = attn_fwd(dev->stage[0], dev->stage[1], dev->stage[2], dev->stage[3],
                static_cast<float*>(dev->stage[4]), B, Hq, Hkv, Sq, Sk, D, causal, scale, stream);
  if (st != ATTN_OK) return st;
  if (cudaMemcpyAsync(o, dev->stage[3], q_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return ATTN_ERR_CUDA;
  if (lse != nullptr &&
      cudaMemcpyAsync(lse, dev->stage[4], lse_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return ATTN_ERR_CUDA;
  return cudaStreamSynchronize(s) == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------
// attn_fwd_noalloc: the same kernel with its scratch in a static device array.
// ------------------------------------------------------------------------------------------
namespace {

// Scratch of the no-allocation entry point, one copy per device that loads this library:
// word 0 = tile scheduler work counter, words 2-3 = status of expired waits, the rest unused.
// In host code this name is only a handle for cudaGetSymbolAddress, never a device pointer.
static __device__ __align__(256) unsigned int g_noalloc_scratch[64];

struct NoAllocDevice {
  bool ready = false;
  int sm_count = 0;
  unsigned int* scratch = nullptr;  // device address of g_noalloc_scratch on this device
};
NoAllocDevice g_noalloc_dev[kMaxDevices];

// Once per device, with that device current: architecture check, TMA encoder lookup, kernel
// attribute, and the device address of the scratch array.  Allocates nothing.
attn_status_t noalloc_device(NoAllocDevice** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ATTN_ERR_CUDA;
  NoAllocDevice& d = g_noalloc_dev[dev];
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!d.ready) {
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return ATTN_ERR_CUDA;
    if (major != 10) return ATTN_ERR_ARCH;
    if (g_encode == nullptr) {
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult qres;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
          fn == nullptr)
        return ATTN_ERR_CUDA;
      g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    void* ptr = nullptr;
    if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaFuncSetAttribute(attn::attn_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             attn::kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(attn::sb3::attn_fwd_sb3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             attn::sb3::kSmemBytes3) != cudaSuccess ||
        cudaFuncSetAttribute(attn::pair::attn_fwd_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             attn::pair::kSmemBytes2) != cudaSuccess ||
        cudaFuncSetAttribute(attn::w16::attn_fwd_w16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             attn::kSmemBytes) != cudaSuccess ||
        cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr)
      return ATTN_ERR_CUDA;
    d.scratch = static_cast<unsigned int*>(ptr);
    d.ready = true;
  }
  *out = &d;
  return ATTN_OK;
}

}  // namespace

attn_status_t attn_fwd_noalloc(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq,
                               int Hkv, int Sq, int Sk, int D, int causal, float scale, void* stream) {
  attn_status_t st = check_args(q, k, v, o, lse, B, Hq, Hkv, Sq, Sk, D, causal, scale, true);
  if (st != ATTN_OK) return st;
  if (static_cast<long long>(B) * Hq * ((Sq + attn::kTile - 1) / attn::kTile) > ATTN_NOALLOC_MAX_Q_TILES)
    return ATTN_ERR_TOO_LARGE;
  NoAllocDevice* dev = nullptr;
  st = noalloc_device(&dev);
  if (st != ATTN_OK) return st;

  FwdParams p;
  fill_plan(&p, B, Hq, Hkv, Sq, Sk, causal);

  CUtensorMap tm_q, tm_k, tm_v, tm_o;
  if (!make_tensor_map(&tm_q, q, B, Sq, Hq, contiguous_strides(Sq, Hq), p.pack_log2) ||
      !make_tensor_map(&tm_k, k, B, Sk, Hkv, contiguous_strides(Sk, Hkv), 0, p.kernel == 2 ? 64 : 128) ||
      !make_tensor_map(&tm_v, v, B, Sk, Hkv, contiguous_strides(Sk, Hkv)) ||
      !make_tensor_map(&tm_o, o, B, Sq, Hq, contiguous_strides(Sq, Hq), p.pack_log2))
    return ATTN_ERR_CUDA;

  p.scale = scale;
  p.scale_log2 = scale * 1.4426950408889634f;
  p.lse = lse;
  p.counter = dev->scratch;                               // word 0
  p.status = reinterpret_cast<int*>(dev->scratch + 2);    // words 2-3
  const int grid = plan_grid(p, dev->sm_count);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // the array keeps the previous call's contents: counter and status must start at zero
  if (cudaMemsetAsync(dev->scratch, 0, 4 * sizeof(unsigned int), s) != cudaSuccess) return ATTN_ERR_CUDA;
  return launch_fwd(tm_q, tm_k, tm_v, tm_o, p, grid, s) == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

attn_status_t attn_release_host_staging(void) {
  int devid = 0;
  if (cudaGetDevice(&devid) != cudaSuccess || devid < 0 || devid >= kMaxDevices) return ATTN_ERR_CUDA;
  DeviceState& d = g_dev[devid];
  for (int i = 0; i < 5; ++i) {
    if (d.stage[i] != nullptr) cudaFree(d.stage[i]);
    d.stage[i] = nullptr;
    d.stage_bytes[i] = 0;
  }
  for (cudaEvent_t e : d.events) cudaEventDestroy(e);
  d.events.clear();
  for (int i = 0; i < 3; ++i) {
    if (d.pipe[i] != nullptr) cudaStreamDestroy(d.pipe[i]);
    d.pipe[i] = nullptr;
  }
  for (int i = 0; i < kSplitStreams; ++i) {
    if (d.split[i] != nullptr) cudaStreamDestroy(d.split[i]);
    d.split[i] = nullptr;
  }
  return ATTN_OK;
}

attn_status_t attn_set_option(const char* name, int value) {
  if (name == nullptr) return ATTN_ERR_NULL;
  if (std::strcmp(name, "scheduler") == 0) {
    if (value < 0 || value > 2) return ATTN_ERR_UNSUPPORTED;
    g_opt_scheduler.store(value);
    return ATTN_OK;
  }
  if (std::strcmp(name, "kernel") == 0) {
    if (value < 0 || value > 3) return ATTN_ERR_UNSUPPORTED;
    g_opt_kernel.store(value);
    return ATTN_OK;
  }
  if (std::strcmp(name, "rescale_threshold") == 0) {
    if (value < 0 || value > 64) return ATTN_ERR_UNSUPPORTED;
    g_opt_rescale_threshold.store(value);
    return ATTN_OK;
  }
  if (std::strcmp(name, "split_p") == 0) {
    if (value < 0 || value > 1) return ATTN_ERR_UNSUPPORTED;
    g_opt_split_p.store(value);
    return ATTN_OK;
  }
  if (std::strcmp(name, "overlap_epilogue") == 0) {
    if (value < 0 || value > 1) return ATTN_ERR_UNSUPPORTED;
    g_opt_overlap_epilogue.store(value);
    return ATTN_OK;
  }
  if (std::strcmp(name, "gqa_pack") == 0) {
    if (value < 0 || value > 1) return ATTN_ERR_UNSUPPORTED;
    g_opt_gqa_pack.store(value);
    return ATTN_OK;
  }
  if (std::strcmp(name, "host_pipeline") == 0) {
    if (value < 0 || value > 1) return ATTN_ERR_UNSUPPORTED;
    g_opt_host_pipeline.store(value);
    return ATTN_OK;
  }
  if (std::strcmp(name, "max_ctas") == 0) {
    if (value < 0) return ATTN_ERR_UNSUPPORTED;
    g_opt_max_ctas.store(value);
    return ATTN_OK;
  }
  return ATTN_ERR_UNSUPPORTED;
}

attn_status_t attn_get_option(const char* name, int* value) {
  if (name == nullptr || value == nullptr) return ATTN_ERR_NULL;
  const struct { const char* name; const std::atomic<int>* opt; } table[] = {
      {"scheduler", &g_opt_scheduler}, {"kernel", &g_opt_kernel}, {"rescale_threshold", &g_opt_rescale_threshold},
      {"split_p", &g_opt_split_p}, {"overlap_epilogue", &g_opt_overlap_epilogue}, {"gqa_pack", &g_opt_gqa_pack},
      {"host_pipeline", &g_opt_host_pipeline}, {"max_ctas", &g_opt_max_ctas}};
  for (const auto& e : table) {
    if (std::strcmp(name, e.name) == 0) {
      *value = e.opt->load();
      return ATTN_OK;
    }
  }
  return ATTN_ERR_UNSUPPORTED;
}

attn_status_t attn_merge(const void* o1, const float* lse1, const void* o2, const float* lse2, void* o, float* lse,
                         int B, int Hq, int Sq, int D, void* stream) {
  if (o1 == nullptr || o2 == nullptr || o == nullptr || lse1 == nullptr || lse2 == nullptr || lse == nullptr)
    return ATTN_ERR_NULL;
  if (B <= 0 || Hq <= 0 || Sq <= 0 || D <= 0) return ATTN_ERR_SHAPE;
  if (D != attn::kHeadDim) return ATTN_ERR_UNSUPPORTED;
  const uintptr_t mask = 15;
  if ((reinterpret_cast<uintptr_t>(o1) & mask) || (reinterpret_cast<uintptr_t>(o2) & mask) ||
      (reinterpret_cast<uintptr_t>(o) & mask) || (reinterpret_cast<uintptr_t>(lse1) & 3) ||
      (reinterpret_cast<uintptr_t>(lse2) & 3) || (reinterpret_cast<uintptr_t>(lse) & 3))
    return ATTN_ERR_ALIGN;
  if (lse == lse1 || lse == lse2) return ATTN_ERR_UNSUPPORTED;
  attn_status_t st = ATTN_OK;
  DeviceState* dev = device_state(&st);
  if (dev == nullptr) return st;
  const long long n_chunks = static_cast<long long>(B) * Sq * Hq * attn::kChunksPerRow;
  long long blocks = (n_chunks + attn::kMergeThreads - 1) / attn::kMergeThreads;
  const long long cap = static_cast<long long>(dev->sm_count) * 8;  // 8 resident CTAs of 256 threads per SM
  if (blocks > cap) blocks = cap;
  attn::attn_merge_kernel<<<static_cast<int>(blocks), attn::kMergeThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint4*>(o1), lse1, static_cast<const uint4*>(o2), lse2, static_cast<uint4*>(o), lse, Hq, Sq,
      n_chunks);
  return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

attn_status_t attn_merge_n(const void* o_parts, const float* lse_parts, int n, void* o, float* lse, int B, int Hq,
                           int Sq, int D, void* stream) {
  if (o_parts == nullptr || lse_parts == nullptr || o == nullptr) return ATTN_ERR_NULL;
  if (B <= 0 || Hq <= 0 || Sq <= 0 || D <= 0 || n <= 0) return ATTN_ERR_SHAPE;
  if (D != attn::kHeadDim || n > kMaxSplits) return ATTN_ERR_UNSUPPORTED;
  const uintptr_t mask = 15;
  if ((reinterpret_cast<uintptr_t>(o_parts) & mask) || (reinterpret_cast<uintptr_t>(o) & mask) ||
      (reinterpret_cast<uintptr_t>(lse_parts) & 3) || (reinterpret_cast<uintptr_t>(lse) & 3))
    return ATTN_ERR_ALIGN;
  attn_status_t st = ATTN_OK;
  DeviceState* dev = device_state(&st);
  if (dev == nullptr) return st;
  const long long n_rows = static_cast<long long>(B) * Sq * Hq;
  const long long n_chunks = n_rows * attn::kChunksPerRow;
  long long blocks = (n_chunks + attn::kMergeThreads - 1) / attn::kMergeThreads;
  const long long cap = static_cast<long long>(dev->sm_count) * 8;
  if (blocks > cap) blocks = cap;
  attn::attn_merge_n_kernel<<<static_cast<int>(blocks), attn::kMergeThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint4*>(o_parts), lse_parts, n, static_cast<uint4*>(o), lse, Hq, Sq, n_chunks, n_rows);
  return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

size_t attn_splitkv_workspace_bytes(int B, int Hq, int Sq, int D, int n_splits) {
  if (B <= 0 || Hq <= 0 || Sq <= 0 || D != attn::kHeadDim || n_splits <= 0 || n_splits > kMaxSplits) return 0;
  const size_t rows = static_cast<size_t>(B) * Sq * Hq;
  return static_cast<size_t>(n_splits) * rows * (static_cast<size_t>(D) * 2 + 4);
}

attn_status_t attn_fwd_splitkv(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq,
                               int Hkv, int Sq, int Sk, int D, int causal, float scale, int n_splits,
                               void* workspace, size_t workspace_bytes, void* stream) {
  attn_status_t st = check_args(q, k, v, o, lse, B, Hq, Hkv, Sq, Sk, D, causal, scale, true);
  if (st != ATTN_OK) return st;
  if (n_splits <= 0) return ATTN_ERR_SHAPE;
  if (n_splits > kMaxSplits) return ATTN_ERR_UNSUPPORTED;
  // key ranges of whole 128-key tiles, all but the last of equal length
  const int per = (Sk + n_splits - 1) / n_splits;
  const int len = (per + attn::kTile - 1) / attn::kTile * attn::kTile;
  const int n = (Sk + len - 1) / len;
  const Strides3 sq = contiguous_strides(Sq, Hq), sk = contiguous_strides(Sk, Hkv);
  if (n == 1) return fwd_device(q, k, v, o, lse, B, Hq, Hkv, Sq, Sk, D, sq, sk, sk, sq, causal, scale, stream);
  if (workspace == nullptr) return ATTN_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(workspace) & 15) return ATTN_ERR_ALIGN;
  if (workspace_bytes < attn_splitkv_workspace_bytes(B, Hq, Sq, D, n)) return ATTN_ERR_TOO_LARGE;
  DeviceState* dev = device_state(&st);
  if (dev == nullptr) return st;
  for (int i = 0; i < kSplitStreams && i < n; ++i) {
    if (dev->split[i] == nullptr &&
        cudaStreamCreateWithFlags(&dev->split[i], cudaStreamNonBlocking) != cudaSuccess)
      return ATTN_ERR_CUDA;
  }
  const cudaStream_t user = static_cast<cudaStream_t>(stream);
  size_t next_event = 0;
  bool ok = true;
  auto after = [&](cudaStream_t waiter, cudaStream_t signaller) {
    if (next_event == dev->events.size()) {
      cudaEvent_t e = nullptr;
      if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) {
        ok = false;
        return;
      }
      dev->events.push_back(e);
    }
    cudaEvent_t e = dev->events[next_event++];
    ok = ok && cudaEventRecord(e, signaller) == cudaSuccess && cudaStreamWaitEvent(waiter, e, 0) == cudaSuccess;
  };
  const int used = n < kSplitStreams ? n : kSplitStreams;
  for (int i = 0; i < used; ++i) after(dev->split[i], user);
  const size_t rows = static_cast<size_t>(B) * Sq * Hq;
  uint8_t* o_parts = static_cast<uint8_t*>(workspace);
  float* lse_parts = reinterpret_cast<float*>(o_parts + static_cast<size_t>(n) * rows * D * 2);
  const uint8_t* kb = static_cast<const uint8_t*>(k);
  const uint8_t* vb = static_cast<const uint8_t*>(v);
  for (int i = 0; i < n && ok && st == ATTN_OK; ++i) {
    const int k0 = i * len, k1 = (k0 + len < Sk) ? k0 + len : Sk;
    const size_t kv_at = static_cast<size_t>(k0) * Hkv * D * 2;
    // rows see keys j <= row + (Sk - Sq) of the whole sequence, i.e. j - k0 <= row + (Sk - Sq - k0) of this range
    st = fwd_device(q, kb + kv_at, vb + kv_at, o_parts + static_cast<size_t>(i) * rows * D * 2,
                    lse_parts + static_cast<size_t>(i) * rows, B, Hq, Hkv, Sq, k1 - k0, D, sq, sk, sk, sq, causal,
                    scale, dev->split[i % kSplitStreams], static_cast<long long>(Sk) - Sq - k0);
  }
  for (int i = 0; i < used; ++i) after(user, dev->split[i]);
  if (st != ATTN_OK) return st;
  if (!ok) return ATTN_ERR_CUDA;
  return attn_merge_n(o_parts, lse_parts, n, o, lse, B, Hq, Sq, D, stream);
}

attn_status_t attn_selftest_wait_timeout(int limit_ms, void* stream) {
  if (limit_ms < 1 || limit_ms > 1000) return ATTN_ERR_UNSUPPORTED;
  attn_status_t st = ATTN_OK;
  DeviceState* dev = device_state(&st);
  if (dev == nullptr) return st;
  attn::wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
      dev->status, static_cast<uint64_t>(limit_ms) * 1000000ull);
  return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

const char* attn_status_str(attn_status_t status) {
  switch (status) {
    case ATTN_OK: return "ATTN_OK";
    case ATTN_ERR_NULL: return "ATTN_ERR_NULL";
    case ATTN_ERR_SHAPE: return "ATTN_ERR_SHAPE";
    case ATTN_ERR_UNSUPPORTED: return "ATTN_ERR_UNSUPPORTED";
    case ATTN_ERR_ALIGN: return "ATTN_ERR_ALIGN";
    case ATTN_ERR_CUDA: return "ATTN_ERR_CUDA";
    case ATTN_ERR_ARCH: return "ATTN_ERR_ARCH";
    case ATTN_ERR_TIMEOUT: return "ATTN_ERR_TIMEOUT";
    case ATTN_ERR_TOO_LARGE: return "ATTN_ERR_TOO_LARGE";
  }
  return "ATTN_ERR_UNKNOWN";
}

int attn_version(void) { return 100; }

namespace {

// Reads the stamp ring of the current device; entry i of `h` is launch (n_total - 1 - i): newest first.
attn_status_t read_stamps(unsigned long long (*h)[4], int want, int* got) {
  attn_status_t st = ATTN_OK;
  DeviceState* dev = device_state(&st);
  if (dev == nullptr) return st;
  static unsigned long long ring[kStampSlots][4];
  std::lock_guard<std::mutex> lock(g_mutex);
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(ring, dev->clock_stamps, sizeof(ring), cudaMemcpyDeviceToHost) != cudaSuccess)
    return ATTN_ERR_CUDA;
  const unsigned int total = dev->next_stamp.load();
  int n = 0;
  for (unsigned int i = 0; i < total && static_cast<int>(i) < kStampSlots && n < want; ++i) {
    const unsigned long long* e = ring[(total - 1 - i) % kStampSlots];
    if (e[3] <= e[1] || e[2] <= e[0]) continue;  // still running, or a launch that ended on an expired wait
    for (int k = 0; k < 4; ++k) h[n][k] = e[k];
    ++n;
  }
  *got = n;
  return ATTN_OK;
}

}  // namespace

attn_status_t attn_last_launch_clock(double* sm_mhz, double* kernel_ms) {
  if (sm_mhz == nullptr || kernel_ms == nullptr) return ATTN_ERR_NULL;
  unsigned long long h[1][4];
  int n = 0;
  const attn_status_t st = read_stamps(h, 1, &n);
  if (st != ATTN_OK) return st;
  if (n == 0) return ATTN_ERR_UNSUPPORTED;  // no such launch has finished yet
  const double ns = static_cast<double>(h[0][3] - h[0][1]);
  *kernel_ms = ns * 1e-6;
  *sm_mhz = static_cast<double>(h[0][2] - h[0][0]) / ns * 1e3;
  return ATTN_OK;
}

attn_status_t attn_launch_clocks(double* sm_mhz, int max_n, int* n_out) {
  if (sm_mhz == nullptr || n_out == nullptr) return ATTN_ERR_NULL;
  if (max_n <= 0) return ATTN_ERR_SHAPE;
  unsigned long long h[kStampSlots][4];
  int n = 0;
  const attn_status_t st = read_stamps(h, max_n < kStampSlots ? max_n : kStampSlots, &n);
  if (st != ATTN_OK) return st;
  for (int i = 0; i < n; ++i) {
    sm_mhz[i] = static_cast<double>(h[i][2] - h[i][0]) / static_cast<double>(h[i][3] - h[i][1]) * 1e3;
  }
  *n_out = n;
  return ATTN_OK;
}

attn_status_t attn_last_device_status(int* code, int* detail) {
  if (code == nullptr || detail == nullptr) return ATTN_ERR_NULL;
  attn_status_t st = ATTN_OK;
  DeviceState* dev = device_state(&st);
  if (dev == nullptr) return st;
  int host[2] = {0, 0};
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(host, dev->status, sizeof(host), cudaMemcpyDeviceToHost) != cudaSuccess)
    return ATTN_ERR_CUDA;
  *code = host[0];
  *detail = host[1];
  if (host[0] != 0) {
    cudaMemset(dev->status, 0, sizeof(host));
    return ATTN_ERR_TIMEOUT;
  }
  return ATTN_OK;
}

}  // extern "C"

// Fused attention forward for sm_100a: one persistent, warp-specialised kernel.
//
// Per CTA (512 threads, one CTA per SM) two 128-row query tiles ("stages") are in flight:
//
//   warps 0-3    softmax, stage 0   one thread per query row: S from tensor memory, online
//   warps 4-7    softmax, stage 1   max / sum in the exp2 domain, P (BF16) back to tensor memory,
//                                   rescale of the O accumulator when the row maximum moved
//   warps 8-11   epilogue           O / l -> BF16 -> shared memory -> TMA store, LSE store
//   warp  12     MMA issue          tcgen05.mma: S = Q K^T (smem x smem), O += P V (tmem x smem)
//   warp  13     loader             TMA loads of Q tiles and of the K / V tile ring, work counter
//   warps 14-15  idle (they only donate registers)
//
// Tensor memory (512 columns): S0 | S1 | O0 | O1, 128 fp32 columns each; P aliases the first
// 64 columns of its S.  Shared memory: Q0, Q1 (32 KB each), a ring of four 32 KB K / V tiles and one
// 32 KB O staging tile, all 128-byte swizzled [128 rows][64 elements] half tiles.  The Q tiles of the
// next work item are fetched as soon as the current item's last Q K^T has been issued.
#pragma once

#include "ptx.cuh"

namespace attn {

constexpr int kTile = 128;        // rows per Q tile and keys per K/V tile
constexpr int kHeadDim = 128;
constexpr int kTileBytes = kTile * kHeadDim * 2;  // 32 KB
constexpr int kHalfBytes = kTileBytes / 2;        // one [128][64] half tile
constexpr int kKvSlots = 4;
constexpr int kThreads = 512;
constexpr float kRescaleThreshold = 8.0f;  // default log2 units a row maximum may lag behind
// LSE = m * scale + ln(l) with ln(l) = lg2(l) * ln 2 from the special-function unit (absolute error
// ~1e-7) and O / l by the approximate reciprocal (2 ulp): the IEEE division and logf subroutines
// in the epilogue warps cost the softmax warps beside them about 1 % of the whole kernel.
constexpr float kLn2 = 0.6931471805599453f;

// Registers per thread of each role after the setmaxnreg re-split of the CTA's 64K registers:
// 8 softmax warps, 4 epilogue warps, 4 other warps; 8 * a + 4 * b + 4 * c must not exceed 2048.
#ifndef ATTN_REGS_SOFTMAX
#define ATTN_REGS_SOFTMAX 192
#endif
#ifndef ATTN_REGS_EPILOGUE
#define ATTN_REGS_EPILOGUE 64
#endif
#ifndef ATTN_REGS_OTHER
#define ATTN_REGS_OTHER 64
#endif
// Of every eight column pairs of a score row, how many take the polynomial exp2 (0..8).
#ifndef ATTN_EXP2_POLY_PAIRS
#define ATTN_EXP2_POLY_PAIRS 1
#endif
constexpr int kExp2PolyPairs = ATTN_EXP2_POLY_PAIRS;
static_assert(8 * ATTN_REGS_SOFTMAX + 4 * ATTN_REGS_EPILOGUE + 4 * ATTN_REGS_OTHER <= 2048, "register split");

constexpr int kSmemQ = 0;
constexpr int kSmemKv = 2 * kTileBytes;
constexpr int kSmemStage = kSmemKv + kKvSlots * kTileBytes;  // O staging tile for the TMA store (both stages, in turn)
constexpr int kSmemStats = kSmemStage + kTileBytes;          // float [2 stages][2][128]
constexpr int kSmemBars = kSmemStats + 2 * 2 * kTile * 4;
constexpr int kNumBars = 2 + 2 + 2 * kKvSlots + 2 * 10 + 1 + 8;  // + 8: exchange barriers of the two-threads-per-row kernel
constexpr int kSmemMisc = kSmemBars + kNumBars * 8;  // tmem base, abort flag, two work-item mailbox slots
constexpr int kMailboxInts = 12;                     // work index + the decoded Work (10 ints), padded
constexpr int kSmemBytes = kSmemMisc + 8 + 2 * kMailboxInts * 4;
static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA");

constexpr uint64_t kWaitLimitNs = 2000000000ull;  // every in-kernel wait gives up after 2 s

struct FwdParams {
  int B, Hq, Hkv, Sq, Sk;
  int group;        // Hq / Hkv
  int causal;
  int off;          // Sk - Sq
  int n_qt;         // ceil(Sq / 128)
  int n_kb;         // ceil(Sk / 128)
  int pair_heads;   // 1: the two stages hold two query heads of one KV head at the same rows
                    // 0: the two stages hold two consecutive row tiles of one query head
  int pack_log2;    // > 0 (short query sequences, "kernel" 0 only): a tile's 128 rows hold
                    // 128 >> pack_log2 query rows of ALL group = 1 << pack_log2 query heads of one KV
                    // head (tile row r = query row r / group, head r % group), so a KV head's K/V is
                    // streamed once for its whole group; the stages hold two consecutive row tiles
  int items_per_group;  // work items per (b, hq) [pair rows] or per (b, hkv) [pair heads]
  int n_work;
  int dynamic;      // 1: work items come from the global counter
  int kernel;       // which kernel the plan was made for (0: dual query stage, 1: triple score buffer)
  int n_groups;     // n_work / items_per_group: (batch, head) groups of work items
  int head_group;   // groups per large super-group (1 = strictly group-major launch order)
  int head_group_extra;  // how many super-groups are large; the others hold head_group - 1 groups
  float rescale_threshold;  // log2 units a row's reference maximum may lag before O is rescaled
  int split_p;              // 1: P is released to the MMA warp in two halves of 64 keys
  int overlap_epilogue;     // 1: a stage is normalised and stored as soon as its own last P V is done
  float scale;
  float scale_log2; // scale * log2(e)
  float* lse;
  unsigned int* counter;  // dynamic scheduler: next work item - gridDim.x
  int* status;            // [0] code of the first expired wait (0 = none), [1] detail
  unsigned long long* clock_stamps;  // may be null; CTA 0 writes {clock64, globaltimer} when it starts into [0..1]
                                     // and when it ends into [2..3] (not the triple-score-buffer kernel)
};

struct Work {
  int b, hkv;
  int hq[2];
  int row0[2];
  int n[2];     // K/V blocks each stage visits (0 = stage unused)
  int nmax;
};

// Launch order -> (group, rank inside the group).  Groups are (batch, head) units that share K/V.
// Consecutive groups form super-groups of `head_group` (the first `head_group_extra` of them) or
// `head_group - 1` groups, whose items are interleaved: rank 0 of each group, then rank 1 of each,
// ...  With the causal mask rank 0 is a group's longest item, so the longest items of several
// heads start first and every super-group -- the last one too -- ends on short ones, while only a
// super-group's K/V is live in L2.
__host__ __device__ __forceinline__ void split_work(const FwdParams& p, int w, int& grp, int& r) {
  const int big = p.head_group * p.items_per_group;  // items of a large super-group
  const int n_big_items = p.head_group_extra * big;
  int first, g_eff, rem;
  if (w < n_big_items) {
    const int sup = w / big;
    rem = w - sup * big;
    first = sup * p.head_group;
    g_eff = p.head_group;
  } else {
    const int small = big - p.items_per_group;  // head_group - 1 groups (never empty here)
    const int sup = (w - n_big_items) / small;
    rem = (w - n_big_items) - sup * small;
    first = p.head_group_extra * p.head_group + sup * (p.head_group - 1);
    g_eff = p.head_group - 1;
  }
  r = rem / g_eff;
  grp = first + (rem - r * g_eff);
}

__host__ __device__ __forceinline__ void decode_work(const FwdParams& p, int w, Work& wk) {
  int grp, r;
  split_work(p, w, grp, r);
  if (p.pair_heads) {
    const int hp = p.group >> 1;
    int qt = r / hp;
    const int pp = r - qt * hp;
    if (p.causal) qt = p.n_qt - 1 - qt;
    wk.b = grp / p.Hkv;
    wk.hkv = grp - wk.b * p.Hkv;
    wk.hq[0] = wk.hkv * p.group + 2 * pp;
    wk.hq[1] = wk.hq[0] + 1;
    wk.row0[0] = wk.row0[1] = qt * kTile;
  } else {
    int qp = p.causal ? (p.items_per_group - 1 - r) : r;
    if (p.pack_log2 > 0) {  // groups are (batch, KV head); hq is the first query head of the group
      wk.b = grp / p.Hkv;
      wk.hkv = grp - wk.b * p.Hkv;
      wk.hq[0] = wk.hq[1] = wk.hkv * p.group;
    } else {
      wk.b = grp / p.Hq;
      wk.hq[0] = wk.hq[1] = grp - wk.b * p.Hq;
      wk.hkv = wk.hq[0] / p.group;
    }
    wk.row0[0] = qp * 2 * (kTile >> p.pack_log2);
    wk.row0[1] = wk.row0[0] + (kTile >> p.pack_log2);
  }
  const int tile_rows = kTile >> p.pack_log2;  // query rows per tile
#pragma unroll
  for (int s = 0; s < 2; ++s) {
    if (wk.row0[s] >= p.Sq) {
      wk.n[s] = 0;
    } else if (p.causal) {
      const int row_end = wk.row0[s] + tile_rows < p.Sq ? wk.row0[s] + tile_rows : p.Sq;
      // a tile none of whose rows sees a key (Sq > Sk) still visits one, fully masked, block, so
      // that its O = 0 and LSE = -inf are produced by the ordinary path
      const int last_key = row_end - 1 + p.off;
      const int need = last_key < 0 ? 1 : last_key / kTile + 1;
      wk.n[s] = need < p.n_kb ? need : p.n_kb;
    } else {
      wk.n[s] = p.n_kb;
    }
  }
  wk.nmax = wk.n[0] > wk.n[1] ? wk.n[0] : wk.n[1];
}

// ------------------------------------------------------------------------------------------
// Bounded mbarrier wait.  Returns false after ctx.limit_ns, or as soon as any thread of the
// CTA has given up; the first to give up records (code, detail) in the global status word.
// ------------------------------------------------------------------------------------------
struct WaitCtx {
  volatile int* abort_flag;  // shared memory
  int* status;               // global
  uint64_t limit_ns;         // how long one wait may last
};

__device__ __forceinline__ bool mbar_wait_slow(uint64_t* bar, uint32_t parity, WaitCtx ctx, int code) {
  // The clock is read only every kSpinsPerCheck failed polls: reading it costs more than a poll,
  // and a waiter must notice the phase flip as soon as it happens.
  constexpr int kSpinsPerCheck = 256;
  uint64_t t0 = 0;
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < kSpinsPerCheck; ++i) {
      if (mbar_try_wait(bar, parity)) return true;
    }
    if (*ctx.abort_flag) return false;
    const uint64_t now = global_timer_ns();
    if (t0 == 0) t0 = now;
    if (now - t0 > ctx.limit_ns) {
      *ctx.abort_flag = 1;
      if (atomicCAS(ctx.status, 0, code) == 0) ctx.status[1] = static_cast<int>(blockIdx.x);
      return false;
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, WaitCtx ctx, int code) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, ctx, code);
}

// codes: role << 8 | barrier
enum : int {
  kRoleLoad = 1 << 8, kRoleMma = 2 << 8, kRoleSoftmax = 3 << 8, kRoleEpilogue = 4 << 8,
  kBarQFull = 1, kBarQEmpty = 2, kBarKvFull = 3, kBarKvEmpty = 4, kBarSFull = 5, kBarPFull = 6,
  kBarOFull = 7, kBarOEmpty = 8, kBarLFull = 9, kBarLEmpty = 10, kBarSchedFull = 11, kBarSchedEmpty = 12, kBarStFull = 13, kBarPHalf = 14, kBarStgEmpty = 18, kBarExchange = 19,
  kBadSmemAlign = 0x7001,
  kRoleSelfTest = 9 << 8
};

struct Barriers {
  uint64_t* q_full;    // [2]  loader (TMA tx) -> MMA
  uint64_t* q_empty;   // [2]  MMA commit after the item's last Q K^T of that stage -> loader
  uint64_t* kv_full;   // [kKvSlots]
  uint64_t* kv_empty;  // [kKvSlots]  MMA commit -> loader
  uint64_t* s_full;    // [2]  MMA commit -> softmax
  uint64_t* p_half;    // [2]  softmax (4 warps): first 64 keys of P written -> MMA
  uint64_t* p_full;    // [2]  softmax (4 warps): all of P written -> MMA
  uint64_t* o_full;    // [2]  MMA commit (last P V) -> epilogue
  uint64_t* o_empty;   // [2]  epilogue (4 warps) -> MMA
  uint64_t* l_full;    // [2]  softmax (128 threads) -> epilogue
  uint64_t* l_empty;   // [2]  epilogue (128 threads) -> softmax
  uint64_t* st_full;   // [2]  epilogue (4 warps: staging tile written) -> the thread issuing the TMA store
  uint64_t* stg_empty; // [1]  the thread that issued the TMA store (source read) -> epilogue warps
  uint64_t* sched_full;   // [2]  loader -> every consumer role
  uint64_t* sched_empty;  // [2]  13 consumer arrivals -> loader
};
constexpr int kSchedConsumers = 1 + 8 + 4;  // MMA lane, 8 softmax warps, 4 epilogue warps

// Mailbox slot layout: [0] work index, [1..10] the decoded Work.  The loader decodes an item once,
// off everybody's critical path (the index arithmetic is a dozen integer divisions), and the other
// roles copy the result.
__device__ __forceinline__ void mailbox_put(volatile int* slot, int w, const Work& wk) {
  slot[1] = wk.b; slot[2] = wk.hkv; slot[3] = wk.hq[0]; slot[4] = wk.hq[1]; slot[5] = wk.row0[0];
  slot[6] = wk.row0[1]; slot[7] = wk.n[0]; slot[8] = wk.n[1]; slot[9] = wk.nmax;
  slot[0] = w;
}
// Plain loads: the caller has just passed the slot's mbarrier wait (acquire, and a compiler
// barrier) and signals consumption afterwards, so fields a role never uses cost nothing.
__device__ __forceinline__ void mailbox_get(const volatile int* vslot, Work& wk) {
  const int* slot = const_cast<const int*>(vslot);
  wk.b = slot[1]; wk.hkv = slot[2]; wk.hq[0] = slot[3]; wk.hq[1] = slot[4]; wk.row0[0] = slot[5];
  wk.row0[1] = slot[6]; wk.n[0] = slot[7]; wk.n[1] = slot[8]; wk.nmax = slot[9];
}

// Work item of iteration `it` of this CTA for a consumer role: returns its index (warp-uniform;
// < 0 on an expired wait, >= n_work when the work is exhausted) and fills `wk` for a valid index.
// `lane_arrives` is true for the one lane per warp that signals consumption.
__device__ __forceinline__ int consumer_next_work(const FwdParams& p, const Barriers& bars,
                                                  const volatile int* sched_w, int it, WaitCtx ctx, int role,
                                                  bool lane_arrives, bool whole_warp, Work& wk) {
  const int slot = it & 1;
  bool ok = mbar_wait(&bars.sched_full[slot], (it >> 1) & 1, ctx, role | kBarSchedFull);
  if (whole_warp) ok = __all_sync(0xffffffffu, ok);
  if (!ok) return -1;
  const volatile int* box = sched_w + slot * kMailboxInts;
  const int w = box[0];
  if (w < p.n_work) mailbox_get(box, wk);
  if (whole_warp) __syncwarp();
  if (lane_arrives) mbar_arrive(&bars.sched_empty[slot]);
  return w;
}

// ------------------------------------------------------------------------------------------
// MMA issue helpers.  The whole MMA warp runs the control flow, so that descriptors and tensor
// memory addresses are warp-uniform values; only the elected lane issues the instructions.
// ------------------------------------------------------------------------------------------
constexpr uint32_t kIdescQK = make_idesc_bf16(kTile, kTile, 0, 0);     // A = Q, B = K, both K-major
constexpr uint32_t kIdescPV = make_idesc_bf16(kTile, kHeadDim, 0, 1);  // A = P (tmem), B = V MN-major

// Descriptor of a K-major [128 rows][128 head-dim] tile (Q or K) and of an MN-major V tile.
__device__ __forceinline__ uint64_t kmajor_desc(uint32_t smem_addr) { return make_smem_desc_sw128(smem_addr, 16, 1024); }
__device__ __forceinline__ uint64_t vtile_desc(uint32_t smem_addr) {
  return make_smem_desc_sw128(smem_addr, kHalfBytes, 1024);
}
// The start-address field counts 16-byte units and never carries out of its 14 bits here
// (shared memory addresses stay below 256 KB), so advancing a descriptor is one addition.
__device__ __forceinline__ uint64_t desc_advance(uint64_t desc, uint32_t bytes) { return desc + (bytes >> 4); }

// S[128 x 128] = Q[128 x 128] K[128 x 128]^T : 8 steps of 16 along the head dimension.  A half
// tile holds 64 head-dim elements per row (one 128-byte swizzle row), so a step advances 32 bytes
// inside the half tile and the second half tile starts 16 KB later.
__device__ __forceinline__ void issue_qk(bool leader, uint32_t tmem_s, uint64_t q_desc, uint64_t k_desc) {
  if (leader) {
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
      mma_ss(tmem_s, desc_advance(q_desc, off), desc_advance(k_desc, off), kIdescQK, kk > 0);
    }
  }
}
// O[128 x 128] (+)= P[128 x 128 keys] V[128 keys x 128] : 8 steps of 16 keys.  P: 8 tensor-memory
// columns per step (two BF16 per column).  V is MN-major: a key is one 128-byte row of a half
// tile, 16 keys are 2048 bytes, the second 64 head-dim elements sit 16 KB later (leading offset).
__device__ __forceinline__ void issue_pv(bool leader, uint32_t tmem_o, uint32_t tmem_p, uint64_t v_desc,
                                         bool accumulate, int kk_begin, int kk_end) {
  if (leader) {
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      if (kk >= kk_begin && kk < kk_end) {
        mma_ts(tmem_o, tmem_p + kk * 8, desc_advance(v_desc, kk * 2048), kIdescPV,
               (accumulate || kk > 0) ? 1u : 0u);
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Roles
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void role_loader(const FwdParams& p, const Barriers& bars, uint8_t* smem,
                                            volatile int* sched_w, WaitCtx ctx, const CUtensorMap* tm_q,
                                            const CUtensorMap* tm_k, const CUtensorMap* tm_v) {
  uint32_t kv_cnt = 0;
  uint32_t q_cnt[2] = {0, 0};
  int w = static_cast<int>(blockIdx.x);
  Work wk, wk_next;
  if (w < p.n_work) decode_work(p, w, wk);
  wk_next = wk;
  mailbox_put(sched_w, w, wk);  // publication 0 (this CTA's first item) goes to slot 0, which nobody has used yet
  mbar_arrive(&bars.sched_full[0]);
  for (int it = 0; w < p.n_work; ++it) {
    // take the next work item one item ahead, decode it and publish it (publication it + 1)
    int w_next;
    if (p.dynamic) {
      w_next = static_cast<int>(atomicAdd(p.counter, 1u)) + static_cast<int>(gridDim.x);
    } else {
      w_next = w + static_cast<int>(gridDim.x);
    }
    if (w_next < p.n_work) decode_work(p, w_next, wk_next);
    {
      const int k = it + 1, slot = k & 1;
      if (!mbar_wait(&bars.sched_empty[slot], ((k >> 1) & 1) ^ 1, ctx, kRoleLoad | kBarSchedEmpty)) return;
      mailbox_put(sched_w + slot * kMailboxInts, w_next, wk_next);
      mbar_arrive(&bars.sched_full[slot]);
    }
    int q_pending = 0;  // Q tiles are requested after the first K tile so that K never waits behind them
#pragma unroll
    for (int s = 0; s < 2; ++s) {
      if (wk.n[s] > 0) q_pending |= 1 << s;
    }
    for (int j = 0; j < wk.nmax; ++j) {
      for (int kv = 0; kv < 2; ++kv) {
        const uint32_t slot = kv_cnt % kKvSlots;
        const uint32_t par = (kv_cnt / kKvSlots) & 1;
        if (!mbar_wait(&bars.kv_empty[slot], par ^ 1, ctx, kRoleLoad | kBarKvEmpty)) return;
        uint8_t* dst = smem + kSmemKv + slot * kTileBytes;
        mbar_arrive_expect_tx(&bars.kv_full[slot], kTileBytes);
        const CUtensorMap* tm = kv == 0 ? tm_k : tm_v;
        tma_load_4d(dst, tm, &bars.kv_full[slot], 0, wk.hkv, j * kTile, wk.b);
        tma_load_4d(dst + kHalfBytes, tm, &bars.kv_full[slot], 64, wk.hkv, j * kTile, wk.b);
        ++kv_cnt;
        if (j == 0 && kv == 0) {
#pragma unroll
          for (int s = 0; s < 2; ++s) {
            if (q_pending & (1 << s)) {
              if (!mbar_wait(&bars.q_empty[s], (q_cnt[s] & 1) ^ 1, ctx, kRoleLoad | kBarQEmpty)) return;
              uint8_t* qdst = smem + kSmemQ + s * kTileBytes;
              mbar_arrive_expect_tx(&bars.q_full[s], kTileBytes);
              tma_load_4d(qdst, tm_q, &bars.q_full[s], 0, wk.hq[s], wk.row0[s], wk.b);
              tma_load_4d(qdst + kHalfBytes, tm_q, &bars.q_full[s], 64, wk.hq[s], wk.row0[s], wk.b);
              ++q_cnt[s];
            }
          }
        }
      }
    }
    w = w_next;
    wk = wk_next;
  }
}

// Bounded wait by a whole warp with a warp-uniform result.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, WaitCtx ctx, int code) {
  const bool ok = mbar_wait(bar, parity, ctx, code);
  return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ void role_mma(const FwdParams& p, const Barriers& bars, uint8_t* smem,
                                         const volatile int* sched_w, WaitCtx ctx, uint32_t tmem, int lane) {
  const bool leader = elect_one();
  const uint32_t smem_base = smem_u32(smem);
  const uint64_t q_desc[2] = {kmajor_desc(smem_base + kSmemQ), kmajor_desc(smem_base + kSmemQ + kTileBytes)};
  uint32_t kv_cnt = 0;
  uint32_t q_cnt[2] = {0, 0};   // per-stage work items seen (phase of q_full / o_empty)
  uint32_t sp_cnt[2] = {0, 0};  // per-stage K/V blocks seen (phase of p_full)
  for (int it = 0;; ++it) {
    Work wk;
    const int w = consumer_next_work(p, bars, sched_w, it, ctx, kRoleMma, lane == 0, true, wk);
    if (w < 0 || w >= p.n_work) return;
    // S_s(0) for both stages
    {
      const uint32_t slot = kv_cnt % kKvSlots, par = (kv_cnt / kKvSlots) & 1;
      if (!mbar_wait_warp(&bars.kv_full[slot], par, ctx, kRoleMma | kBarKvFull)) return;
      const uint64_t k_desc = kmajor_desc(smem_base + kSmemKv + slot * kTileBytes);
#pragma unroll
      for (int s = 0; s < 2; ++s) {
        if (wk.n[s] > 0) {
          if (!mbar_wait_warp(&bars.q_full[s], q_cnt[s] & 1, ctx, kRoleMma | kBarQFull)) return;
          tc_fence_after_sync();
          issue_qk(leader, tmem + s * kTile, q_desc[s], k_desc);
          if (leader) {
            mma_commit(&bars.s_full[s]);
            if (wk.n[s] == 1) mma_commit(&bars.q_empty[s]);  // Q_s is not read again
          }
        }
      }
      if (leader) mma_commit(&bars.kv_empty[slot]);
      ++kv_cnt;
    }
    for (int j = 0; j < wk.nmax; ++j) {
      const uint32_t vslot = kv_cnt % kKvSlots, vpar = (kv_cnt / kKvSlots) & 1;
      ++kv_cnt;
      const bool has_next = (j + 1 < wk.nmax);
      uint32_t kslot = 0, kpar = 0;
      if (has_next) {
        kslot = kv_cnt % kKvSlots;
        kpar = (kv_cnt / kKvSlots) & 1;
        ++kv_cnt;
      }
      if (!mbar_wait_warp(&bars.kv_full[vslot], vpar, ctx, kRoleMma | kBarKvFull)) return;
      bool k_ready = false;
      const uint64_t v_desc = vtile_desc(smem_base + kSmemKv + vslot * kTileBytes);
      const uint64_t k_desc = kmajor_desc(smem_base + kSmemKv + kslot * kTileBytes);
#pragma unroll
      for (int s = 0; s < 2; ++s) {
        if (j < wk.n[s]) {
          if (j == 0) {  // the previous item's O_s must have left tensor memory
            if (!mbar_wait_warp(&bars.o_empty[s], (q_cnt[s] & 1) ^ 1, ctx, kRoleMma | kBarOEmpty)) return;
          }
          // P arrives in two halves of 64 keys: the first half of P V runs while the softmax
          // warps are still exponentiating the second half
          if (!mbar_wait_warp(&bars.p_half[s], sp_cnt[s] & 1, ctx, kRoleMma | kBarPHalf)) return;
          tc_fence_after_sync();
          issue_pv(leader, tmem + 2 * kTile + s * kTile, tmem + s * kTile, v_desc, j > 0, 0, 4);
          if (!mbar_wait_warp(&bars.p_full[s], sp_cnt[s] & 1, ctx, kRoleMma | kBarPFull)) return;
          ++sp_cnt[s];
          tc_fence_after_sync();
          issue_pv(leader, tmem + 2 * kTile + s * kTile, tmem + s * kTile, v_desc, j > 0, 4, 8);
          if (leader && j == wk.n[s] - 1) mma_commit(&bars.o_full[s]);
          if (j + 1 < wk.n[s]) {
            if (!k_ready) {
              if (!mbar_wait_warp(&bars.kv_full[kslot], kpar, ctx, kRoleMma | kBarKvFull)) return;
              tc_fence_after_sync();
              k_ready = true;
            }
            issue_qk(leader, tmem + s * kTile, q_desc[s], k_desc);
            if (leader) {
              mma_commit(&bars.s_full[s]);
              if (j + 2 == wk.n[s]) mma_commit(&bars.q_empty[s]);  // that was the item's last use of Q_s
            }
          }
        }
      }
      if (leader) {
        mma_commit(&bars.kv_empty[vslot]);
        if (has_next) mma_commit(&bars.kv_empty[kslot]);
      }
    }
#pragma unroll
    for (int s = 0; s < 2; ++s) {
      if (wk.n[s] > 0) ++q_cnt[s];
    }
  }
}

// One softmax thread owns one query row of stage `s`.
__device__ __forceinline__ void role_softmax(const FwdParams& p, const Barriers& bars, uint8_t* smem,
                                             const volatile int* sched_w, WaitCtx ctx, uint32_t tmem, int s,
                                             int row_in_tile, int lane) {
  const uint32_t lane_sel = static_cast<uint32_t>(row_in_tile & ~31) << 16;
  const uint32_t t_s = tmem + lane_sel + s * kTile;             // S_s, and P_s in its first 64 columns
  const uint32_t t_o = tmem + lane_sel + 2 * kTile + s * kTile;  // O_s
  float* stats = reinterpret_cast<float*>(smem + kSmemStats) + s * 2 * kTile;
  const float c = p.scale_log2;
  uint32_t s_cnt = 0;  // phase of s_full[s]
  uint32_t l_cnt = 0;  // phase of l_empty / l_full
  for (int it = 0;; ++it) {
    Work wk;
    const int w = consumer_next_work(p, bars, sched_w, it, ctx, kRoleSoftmax, lane == 0, true, wk);
    if (w < 0 || w >= p.n_work) return;
    const int n = wk.n[s];
    if (n == 0) continue;
    const int row = wk.row0[s] + (row_in_tile >> p.pack_log2);  // global query row (may be >= Sq in a ragged tile)
    // number of keys this row may see, counted from key 0
    const int row_limit = p.causal ? min(p.Sk, row + p.off + 1) : p.Sk;
    // first key index from which a block needs per-element masking for this tile
    const int tile_clear = p.causal ? min(p.Sk, wk.row0[s] + p.off + 1) : p.Sk;
    float m_used = -INFINITY;  // row maximum the exponentials are taken against (raw score units)
    float l = 0.f;             // running sum of exponentials
    for (int j = 0; j < n; ++j) {
      bool ok = mbar_wait(&bars.s_full[s], s_cnt & 1, ctx, kRoleSoftmax | kBarSFull);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return;
      ++s_cnt;
      tc_fence_after_sync();
      uint32_t xr[kTile];
      tmem_ld_x32(t_s + 0, xr + 0);
      tmem_ld_x32(t_s + 32, xr + 32);
      tmem_ld_x32(t_s + 64, xr + 64);
      tmem_ld_x32(t_s + 96, xr + 96);
      tmem_wait_ld();
#define X(i) __uint_as_float(xr[(i)])
      if ((j + 1) * kTile > tile_clear) {  // warp-uniform: some element of this block is masked
        const int vis = row_limit - j * kTile;  // visible columns of this row in this block
#pragma unroll
        for (int i = 0; i < kTile; ++i) {
          if (i >= vis) xr[i] = 0xff800000u;
        }
      }
      float m0 = X(0), m1 = X(1), m2 = X(2), m3 = X(3);
#pragma unroll
      for (int i = 4; i < kTile; i += 8) {
        m0 = max3(m0, X(i), X(i + 1));
        m1 = max3(m1, X(i + 2), X(i + 3));
        if (i + 4 < kTile) {
          m2 = max3(m2, X(i + 4), X(i + 5));
          m3 = max3(m3, X(i + 6), X(i + 7));
        }
      }
      const float m_blk = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
      if (j == 0) {
        m_used = (m_blk == -INFINITY) ? 0.f : m_blk;
      } else {
        const float m_new = fmaxf(m_used, m_blk);
        const bool grow = (m_new - m_used) * c > p.rescale_threshold;
        if (__any_sync(0xffffffffu, grow)) {
          // P V of block j-1 has completed (S of block j was issued after it), so O_s is quiescent
          const float alpha = ex2_approx((m_used - m_new) * c);
          m_used = m_new;
          l *= alpha;
#pragma unroll
          for (int cc = 0; cc < 8; ++cc) {
            uint32_t o[16];
            tmem_ld_x16(t_o + cc * 16, o);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
            tmem_st_x16(t_o + cc * 16, o);
          }
        }
      }
      // P = exp2(S * c - m_used * c) on pairs of columns with packed fp32 arithmetic.  Of every
      // eight pairs, kExp2PolyPairs are evaluated by the polynomial on the FMA pipe and the rest
      // by the special-function unit, so that neither unit alone bounds the row.
      const float neg_mc = -m_used * c;
      const float2 c2 = make_float2(c, c);
      const float2 nm2 = make_float2(neg_mc, neg_mc);
      float2 la = make_float2(0.f, 0.f), lb = make_float2(0.f, 0.f);
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t pk[16];
#pragma unroll
        for (int pr = 0; pr < 16; ++pr) {
          const int i = cc * 32 + pr * 2;
          const float2 x = fma2(make_float2(X(i), X(i + 1)), c2, nm2);
          float2 e;
          if ((pr & 7) < kExp2PolyPairs) {
            e = exp2_poly2(x);
          } else {
            e = make_float2(ex2_approx(x.x), ex2_approx(x.y));
          }
          if (pr & 1) {
            lb = add2(lb, e);
          } else {
            la = add2(la, e);
          }
          pk[pr] = pack_bf16x2(e.x, e.y);
        }
        tmem_st_x16(t_s + cc * 16, pk);
        if (cc == 1 && p.split_p) {  // the first 64 keys of P are in tensor memory
          tmem_wait_st();
          tc_fence_before_sync();
          if (lane == 0) mbar_arrive(&bars.p_half[s]);
        }
      }
#undef X
      la = add2(la, lb);
      l += la.x + la.y;
      tmem_wait_st();
      tc_fence_before_sync();
      if (lane == 0) {
        if (!p.split_p) mbar_arrive(&bars.p_half[s]);
        mbar_arrive(&bars.p_full[s]);
      }
    }
    // hand the row statistics to the epilogue warps
    bool ok = mbar_wait(&bars.l_empty[s], (l_cnt & 1) ^ 1, ctx, kRoleSoftmax | kBarLEmpty);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) return;
    // a row without any visible key (causal, Sq > Sk) has the sum 0 by definition; its masked
    // scores may have left denormal-sized terms in l
    stats[row_in_tile] = row_limit > 0 ? l : 0.f;
    stats[kTile + row_in_tile] = m_used;
    mbar_arrive(&bars.l_full[s]);
    ++l_cnt;
  }
}

__device__ __forceinline__ void role_epilogue(const FwdParams& p, const Barriers& bars, uint8_t* smem,
                                              const volatile int* sched_w, WaitCtx ctx, uint32_t tmem,
                                              int row_in_tile, int lane, const CUtensorMap* tm_o) {
  const uint32_t lane_sel = static_cast<uint32_t>(row_in_tile & ~31) << 16;
  uint32_t cnt[2] = {0, 0};
  uint32_t stg_cnt = 0;  // uses of the staging tile so far (phase of stg_empty)
  for (int it = 0;; ++it) {
    Work wk;
    const int w = consumer_next_work(p, bars, sched_w, it, ctx, kRoleEpilogue, lane == 0, true, wk);
    if (w < 0 || w >= p.n_work) return;
    // one copy of the code for both stages: a second (unrolled) copy costs registers this role
    // does not have; the few per-stage values are then indexed at run time
#pragma unroll 1
    for (int s = 0; s < 2; ++s) {
      if (wk.n[s] == 0) continue;
      const float* stats = reinterpret_cast<const float*>(smem + kSmemStats) + s * 2 * kTile;
      bool ok = mbar_wait(&bars.l_full[s], cnt[s] & 1, ctx, kRoleEpilogue | kBarLFull);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return;
      const float l = stats[row_in_tile];
      const float m_used = stats[kTile + row_in_tile];
      mbar_arrive(&bars.l_empty[s]);
      ok = mbar_wait(&bars.o_full[s], cnt[s] & 1, ctx, kRoleEpilogue | kBarOFull);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return;
      if (!p.overlap_epilogue && s == 0 && wk.n[1] > 0) {
        // A/B switch: do not start on stage 0 before stage 1's last P V has completed as well
        ok = mbar_wait(&bars.o_full[1], cnt[1] & 1, ctx, kRoleEpilogue | kBarOFull);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) return;
      }
      ++cnt[s];
      tc_fence_after_sync();
      const float inv_l = l > 0.f ? __fdividef(1.0f, l) : 0.f;  // l = 0: a row without visible keys, O = 0 and LSE = -inf
      // the previous TMA store must have finished reading the staging tile
      ok = mbar_wait(&bars.stg_empty[0], (stg_cnt & 1) ^ 1, ctx, kRoleEpilogue | kBarStgEmpty);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return;
      ++stg_cnt;
      uint8_t* stage = smem + kSmemStage;
      const uint32_t t_o = tmem + lane_sel + 2 * kTile + s * kTile;
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t o[32];
        tmem_ld_x32(t_o + cc * 32, o);
        tmem_wait_ld();
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          uint4 val;
          val.x = pack_bf16x2(__uint_as_float(o[ch * 8 + 0]) * inv_l, __uint_as_float(o[ch * 8 + 1]) * inv_l);
          val.y = pack_bf16x2(__uint_as_float(o[ch * 8 + 2]) * inv_l, __uint_as_float(o[ch * 8 + 3]) * inv_l);
          val.z = pack_bf16x2(__uint_as_float(o[ch * 8 + 4]) * inv_l, __uint_as_float(o[ch * 8 + 5]) * inv_l);
          val.w = pack_bf16x2(__uint_as_float(o[ch * 8 + 6]) * inv_l, __uint_as_float(o[ch * 8 + 7]) * inv_l);
          const int chunk = cc * 4 + ch;  // 16-byte chunk of the 256-byte row
          uint8_t* dst = stage + (chunk >> 3) * kHalfBytes + row_in_tile * 128 +
                         (((chunk & 7) ^ (row_in_tile & 7)) << 4);
          *reinterpret_cast<uint4*>(dst) = val;
        }
      }
      tc_fence_before_sync();
      if (lane == 0) mbar_arrive(&bars.o_empty[s]);
      const int row = wk.row0[s] + (row_in_tile >> p.pack_log2);
      const int head = wk.hq[s] + (row_in_tile & ((1 << p.pack_log2) - 1));
      if (p.lse != nullptr && row < p.Sq) {
        p.lse[(static_cast<size_t>(wk.b) * p.Hq + head) * p.Sq + row] = fmaf(lg2_approx(l), kLn2, m_used * p.scale);
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars.st_full[s]);
      if (row_in_tile == s * 32) {
        // cnt[s] was advanced above: this item's phase of st_full[s] is (cnt[s] - 1) & 1
        if (mbar_wait(&bars.st_full[s], (cnt[s] & 1) ^ 1, ctx, kRoleEpilogue | kBarStFull)) {
          tma_store_4d(tm_o, stage, 0, wk.hq[s], wk.row0[s], wk.b);
          tma_store_4d(tm_o, stage + kHalfBytes, 64, wk.hq[s], wk.row0[s], wk.b);
          tma_store_commit();
          tma_store_wait_read0();
          mbar_arrive(&bars.stg_empty[0]);
        }
      }
    }
  }
  // global writes of the bulk stores complete before the kernel ends
}

// ------------------------------------------------------------------------------------------
// Kernel
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                const FwdParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* bar_mem = reinterpret_cast<uint64_t*>(smem + kSmemBars);
  Barriers bars;
  bars.q_full = bar_mem;
  bars.q_empty = bars.q_full + 2;
  bars.kv_full = bars.q_empty + 2;
  bars.kv_empty = bars.kv_full + kKvSlots;
  bars.s_full = bars.kv_empty + kKvSlots;
  bars.p_half = bars.s_full + 2;
  bars.p_full = bars.p_half + 2;
  bars.o_full = bars.p_full + 2;
  bars.o_empty = bars.o_full + 2;
  bars.l_full = bars.o_empty + 2;
  bars.l_empty = bars.l_full + 2;
  bars.st_full = bars.l_empty + 2;
  bars.stg_empty = bars.st_full + 2;
  bars.sched_full = bars.stg_empty + 1;
  bars.sched_empty = bars.sched_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kSmemMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kSmemMisc + 4);
  volatile int* sched_w = reinterpret_cast<volatile int*>(smem + kSmemMisc + 8);
  const WaitCtx ctx{abort_flag, p.status, kWaitLimitNs};

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;

  if ((smem_u32(smem) & 1023u) != 0) {  // the swizzled tiles need a 1024-byte aligned base
    if (tid == 0 && atomicCAS(p.status, 0, kBadSmemAlign) == 0) p.status[1] = static_cast<int>(blockIdx.x);
    return;
  }
  if (tid == 0) {
    if (blockIdx.x == 0 && p.clock_stamps != nullptr) {  // a persistent CTA lives as long as the launch
      p.clock_stamps[0] = static_cast<unsigned long long>(clock64());
      p.clock_stamps[1] = global_timer_ns();
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars.q_full[i], 1);
      mbar_init(&bars.q_empty[i], 1);
      mbar_init(&bars.s_full[i], 1);
      mbar_init(&bars.p_half[i], 4);
      mbar_init(&bars.p_full[i], 4);
      mbar_init(&bars.o_full[i], 1);
      mbar_init(&bars.o_empty[i], 4);
      mbar_init(&bars.l_full[i], kTile);
      mbar_init(&bars.l_empty[i], kTile);
      mbar_init(&bars.st_full[i], 4);
      if (i == 0) mbar_init(&bars.stg_empty[0], 1);
      mbar_init(&bars.sched_full[i], 1);
      mbar_init(&bars.sched_empty[i], kSchedConsumers);
    }
    for (int i = 0; i < kKvSlots; ++i) {
      mbar_init(&bars.kv_full[i], 1);
      mbar_init(&bars.kv_empty[i], 1);
    }
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 12) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  if (warp == 13 && lane == 0) {
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    tma_prefetch_desc(&tm_o);
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  if (warp < 8) {
    reg_alloc<ATTN_REGS_SOFTMAX>();
    role_softmax(p, bars, smem, sched_w, ctx, tmem, warp >> 2, tid & 127, lane);
  } else if (warp < 12) {
    reg_dealloc<ATTN_REGS_EPILOGUE>();
    role_epilogue(p, bars, smem, sched_w, ctx, tmem, tid & 127, lane, &tm_o);
    tma_store_wait_all0();
  } else {
    reg_dealloc<ATTN_REGS_OTHER>();
    if (warp == 12) {
      role_mma(p, bars, smem, sched_w, ctx, tmem, lane);
    } else if (warp == 13) {
      if (lane == 0) {
        role_loader(p, bars, smem, sched_w, ctx, &tm_q, &tm_k, &tm_v);
        if (*abort_flag) {  // let loads in flight land before the CTA's shared memory is released
          const uint64_t t0 = global_timer_ns();
          while (global_timer_ns() - t0 < 1000000ull) {
          }
        }
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 12) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, 512);
  }
  if (tid == 0 && blockIdx.x == 0 && p.clock_stamps != nullptr) {
    p.clock_stamps[2] = static_cast<unsigned long long>(clock64());
    p.clock_stamps[3] = global_timer_ns();
  }
}

// Self-test of the bounded wait: one warp waits on an mbarrier that nobody ever arrives on.  The
// wait gives up after limit_ns, records (kRoleSelfTest | kBarSFull, block) in the status word and
// the kernel returns normally, leaving the context usable.
__global__ void __launch_bounds__(32, 1) wait_timeout_selftest_kernel(int* status, uint64_t limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    fence_mbar_init();
  }
  __syncwarp();
  const WaitCtx ctx{&abort_flag, status, limit_ns};
  mbar_wait_warp(&bar, 0, ctx, kRoleSelfTest | kBarSFull);
}

}  // namespace attn

// Fused attention forward on CTA pairs (option "kernel" = 2): the dual-query-stage kernel of
// attn_fwd_kernel.cuh with every tcgen05.mma issued over a cluster of two CTAs (cta_group::2).
//
// A pair works on FOUR 128-row query tiles: stage s of CTA c holds one of them, and one
// instruction computes the score (or output) tiles of both CTAs, M = 256.  The B operand of an
// instruction is split along N between the two CTAs, so each CTA loads and keeps only half of
// every K/V tile:
//
//   S = Q K^T   B = K[128 keys][128 d], N = keys: CTA c holds keys 64c .. 64c+63 (two K-major half
//               tiles of [64 keys][64 d], 8 KB each)
//   O += P V    B = V[128 keys][128 d], N = d:    CTA c holds d 64c .. 64c+63 of all 128 keys (one
//               MN-major half tile of [128 keys][64 d], 16 KB)
//
// Per 128x128x16 step an SM then reads 2 KB of B instead of 4 KB, and K/V cross the L2 -> SM path
// once per 512 query rows instead of once per 256.  The shared memory and the port bandwidth this
// frees are spent on P: the softmax warps write P (BF16) into SHARED memory, not over S in tensor
// memory, so a stage's score tile is free again as soon as its rows have been loaded into
// registers, and the MMA warp issues S(j+1) = Q K(j+1)^T while the softmax of block j is still
// running.  A stage's loop is then softmax after softmax, with no wait for P V and Q K^T in
// between; both matrix products run in the shadow of the exponentials.
//
// Roles per CTA as in the one-CTA kernel, except that there are two MMA warps, one per query stage,
// and they work in the leader CTA (cluster rank 0) only; their commits arrive on the barriers of
// both CTAs.  What the leader's MMA warps wait for (K/V and Q tiles landed, S read, P written, O
// drained) is counted on the LEADER's barriers: the peer's loader, softmax and epilogue warps
// arrive there remotely and the peer's TMA loads report their bytes there.  Those remote arrivals
// are plain (the data travel through tensor memory, TMA or proxy-fenced shared memory that the
// peer's own tensor core reads); only the work-item mailbox, which the leader's loader writes into
// both CTAs with ordinary stores, is released and acquired at cluster scope: a cluster-scope
// release on every P hand-over cost a fifth of the kernel's throughput.  No load is multicast: each
// CTA fetches only what it keeps.
#pragma once

#include "attn_fwd_kernel.cuh"

namespace attn {
namespace pair {

constexpr int kKvHalfBytes = kTileBytes / 2;  // this CTA's half of a K or V tile (16 KB)
constexpr int kKvSlots2 = 4;
constexpr int kSmemQ2 = 0;
constexpr int kSmemP2 = 2 * kTileBytes;             // P_0, P_1: K-major [128 rows][128 keys] as two half tiles
constexpr int kSmemKv2 = kSmemP2 + 2 * kTileBytes;
constexpr int kSmemStage2 = kSmemKv2 + kKvSlots2 * kKvHalfBytes;
constexpr int kSmemStats2 = kSmemStage2 + kTileBytes;
constexpr int kSmemBars2 = kSmemStats2 + 2 * 2 * kTile * 4;
constexpr int kNumBars2 = 2 + 2 + 2 * kKvSlots2 + 2 * 13 + 1;
constexpr int kSmemMisc2 = kSmemBars2 + kNumBars2 * 8;
constexpr int kSmemBytes2 = kSmemMisc2 + 8 + 2 * kMailboxInts * 4 + 8;  // + stage 0's progress word
static_assert(kSmemBytes2 <= 232448, "shared memory budget of one CTA");

// arrivals per publication on the leader's sched_empty: the leader's two MMA warps, and per CTA 8
// softmax warps and 4 epilogue warps, and the peer's loader
constexpr int kSchedConsumers2 = 2 + 2 * (8 + 4) + 1;

// wait codes of the barriers this kernel adds (role << 8 | barrier, as in the one-CTA kernel)
enum : int { kBarSFree = 19, kBarPaEmpty = 20, kBarPbEmpty = 21, kBarProgress = 22 };

// Bounded wait until a shared-memory counter that only grows has reached `target`.
__device__ __forceinline__ bool wait_counter(const volatile int* counter, int target, WaitCtx ctx, int code) {
  uint64_t t0 = 0;
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) {
      if (*counter - target >= 0) return true;
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

// Work item `w` of a pair as CTA `rank` sees it.  MHA / odd groups: four consecutive row tiles of
// one head, stage s of CTA c holds tile 4 r + 2 s + c.  Even GQA groups: the two stages hold two
// query heads of one KV head, CTA c holds row tile 2 r + c of both.  The two tiles of a stage run
// the same number of K/V blocks (what the later tile needs under the causal mask; the earlier
// tile's extra block is fully masked).
__host__ __device__ __forceinline__ void decode_work_pair(const FwdParams& p, int w, int rank, Work& wk) {
  int grp, r;
  split_work(p, w, grp, r);
  int first_row[2];  // first row of the stage's earlier tile (the leader's)
  if (p.pair_heads) {
    const int hp = p.group >> 1;
    int qt2 = r / hp;
    const int pp = r - qt2 * hp;
    if (p.causal) qt2 = ((p.n_qt + 1) >> 1) - 1 - qt2;
    wk.b = grp / p.Hkv;
    wk.hkv = grp - wk.b * p.Hkv;
    wk.hq[0] = wk.hkv * p.group + 2 * pp;
    wk.hq[1] = wk.hq[0] + 1;
    first_row[0] = first_row[1] = 2 * qt2 * kTile;
  } else {
    const int qp = p.causal ? (p.items_per_group - 1 - r) : r;
    wk.b = grp / p.Hq;
    wk.hq[0] = wk.hq[1] = grp - wk.b * p.Hq;
    wk.hkv = wk.hq[0] / p.group;
    first_row[0] = 4 * qp * kTile;
    first_row[1] = first_row[0] + 2 * kTile;
  }
#pragma unroll
  for (int s = 0; s < 2; ++s) {
    wk.row0[s] = first_row[s] + rank * kTile;
    if (first_row[s] >= p.Sq) {
      wk.n[s] = 0;
    } else if (p.causal) {
      const int row_end = first_row[s] + 2 * kTile < p.Sq ? first_row[s] + 2 * kTile : p.Sq;
      const int last_key = row_end - 1 + p.off;
      const int need = last_key < 0 ? 1 : last_key / kTile + 1;
      wk.n[s] = need < p.n_kb ? need : p.n_kb;
    } else {
      wk.n[s] = p.n_kb;
    }
  }
  wk.nmax = wk.n[0] > wk.n[1] ? wk.n[0] : wk.n[1];
}

// Bounded wait that also acquires what the other CTA released before arriving (the mailbox).
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, WaitCtx ctx, int code) {
  constexpr int kSpinsPerCheck = 256;
  uint64_t t0 = 0;
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < kSpinsPerCheck; ++i) {
      if (mbar_try_wait_cluster(bar, parity)) return true;
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

// A mailbox slot of CTA `rank`, written through the cluster window.
__device__ __forceinline__ void mailbox_put_cluster(uint32_t slot_addr, int w, const Work& wk) {
  st_shared_cluster(slot_addr + 4, wk.b);
  st_shared_cluster(slot_addr + 8, wk.hkv);
  st_shared_cluster(slot_addr + 12, wk.hq[0]);
  st_shared_cluster(slot_addr + 16, wk.hq[1]);
  st_shared_cluster(slot_addr + 20, wk.row0[0]);
  st_shared_cluster(slot_addr + 24, wk.row0[1]);
  st_shared_cluster(slot_addr + 28, wk.n[0]);
  st_shared_cluster(slot_addr + 32, wk.n[1]);
  st_shared_cluster(slot_addr + 36, wk.nmax);
  st_shared_cluster(slot_addr + 0, w);
}

// Pointers of this CTA's barriers plus the shared::cluster addresses of the leader's copies of
// those that receive arrivals from both CTAs.
struct PairBars {
  Barriers b;
  uint64_t* s_free;    // [2]  leader: 4 softmax warps of each CTA have S_s in registers     -> leader's MMA
  uint64_t* pa_empty;  // [2]  MMA commit: P V over the first 64 keys done (half a of P_s free) -> softmax, both CTAs
  uint64_t* pb_empty;  // [2]  MMA commit: P V over the last 64 keys done (half b free, O_s quiescent)
  uint32_t lead_s_free;
  uint32_t lead_q_full;      // [2]  both loaders (expect_tx + TMA bytes)      -> leader's MMA
  uint32_t lead_kv_full;     // [kKvSlots2]
  uint32_t lead_p_half;      // [2]  4 softmax warps of each CTA                -> leader's MMA
  uint32_t lead_p_full;      // [2]
  uint32_t lead_o_empty;     // [2]  4 epilogue warps of each CTA               -> leader's MMA
  uint32_t lead_sched_empty; // [2]  consumers of both CTAs                     -> leader's loader
};

__device__ __forceinline__ int consumer_next_work2(const FwdParams& p, const PairBars& bars,
                                                   const volatile int* sched_w, int it, WaitCtx ctx, int role,
                                                   bool lane_arrives, Work& wk) {
  const int slot = it & 1;
  bool ok = mbar_wait_cluster(&bars.b.sched_full[slot], (it >> 1) & 1, ctx, role | kBarSchedFull);
  ok = __all_sync(0xffffffffu, ok);
  if (!ok) return -1;
  const volatile int* box = sched_w + slot * kMailboxInts;
  const int w = box[0];
  if (w < p.n_work) mailbox_get(box, wk);
  __syncwarp();
  if (lane_arrives) mbar_arrive_cluster(bars.lead_sched_empty + slot * 8);
  return w;
}

constexpr uint32_t kIdescQK2 = make_idesc_bf16(2 * kTile, kTile, 0, 0);
constexpr uint32_t kIdescPV2 = make_idesc_bf16(2 * kTile, kHeadDim, 0, 1);

// This CTA's half of a K tile: two K-major [64 keys][64 d] half tiles 8 KB apart.
__device__ __forceinline__ void issue_qk2(bool leader, uint32_t tmem_s, uint64_t q_desc, uint64_t k_desc) {
  if (leader) {
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      const uint32_t q_off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
      const uint32_t k_off = (kk >> 2) * (kKvHalfBytes / 2) + (kk & 3) * 32;
      mma_ss_pair(tmem_s, desc_advance(q_desc, q_off), desc_advance(k_desc, k_off), kIdescQK2, kk > 0);
    }
  }
}
// This CTA's half of a V tile: one MN-major [128 keys][64 d] half tile; 16 keys are 2048 bytes.
// P is K-major in shared memory like a Q tile: 16 keys are 32 bytes inside a half tile of 64 keys.
__device__ __forceinline__ void issue_pv2(bool leader, uint32_t tmem_o, uint64_t p_desc, uint64_t v_desc,
                                          bool accumulate, int kk_begin, int kk_end) {
  if (leader) {
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      if (kk >= kk_begin && kk < kk_end) {
        const uint32_t p_off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
        mma_ss_pair(tmem_o, desc_advance(p_desc, p_off), desc_advance(v_desc, kk * 2048), kIdescPV2,
                    (accumulate || kk > 0) ? 1u : 0u);
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Roles
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void role_loader2(const FwdParams& p, const PairBars& bars, uint8_t* smem,
                                             volatile int* sched_w, WaitCtx ctx, const CUtensorMap* tm_q,
                                             const CUtensorMap* tm_k, const CUtensorMap* tm_v, int rank) {
  const int n_pairs = static_cast<int>(gridDim.x >> 1);
  uint32_t kv_base = 0;  // K/V blocks of earlier work items
  uint32_t q_cnt[2] = {0, 0};
  int w = 0;
  Work wk, wk_next, wk_peer;
  const uint32_t peer_box = map_to_cta(smem_u32(const_cast<int*>(sched_w)), 1);
  const uint32_t peer_sched_full = map_to_cta(smem_u32(&bars.b.sched_full[0]), 1);
  if (rank == 0) {
    w = static_cast<int>(blockIdx.x >> 1);
    if (w < p.n_work) {
      decode_work_pair(p, w, 0, wk);
      decode_work_pair(p, w, 1, wk_peer);
    }
    wk_next = wk;
    mailbox_put(sched_w, w, wk);  // publication 0 goes to slot 0 of both CTAs, which nobody has used yet
    mailbox_put_cluster(peer_box, w, wk_peer);
    mbar_arrive(&bars.b.sched_full[0]);
    mbar_arrive_cluster_release(peer_sched_full);
  }
  for (int it = 0;; ++it) {
    int w_next = 0;
    if (rank == 0) {
      if (w >= p.n_work) break;
      // take the next work item one item ahead, decode it for both CTAs and publish it (publication it + 1)
      if (p.dynamic) {
        w_next = static_cast<int>(atomicAdd(p.counter, 1u)) + n_pairs;
      } else {
        w_next = w + n_pairs;
      }
      if (w_next < p.n_work) {
        decode_work_pair(p, w_next, 0, wk_next);
        decode_work_pair(p, w_next, 1, wk_peer);
      }
      const int k = it + 1, slot = k & 1;
      if (!mbar_wait(&bars.b.sched_empty[slot], ((k >> 1) & 1) ^ 1, ctx, kRoleLoad | kBarSchedEmpty)) return;
      mailbox_put(sched_w + slot * kMailboxInts, w_next, wk_next);
      mailbox_put_cluster(peer_box + slot * kMailboxInts * 4, w_next, wk_peer);
      mbar_arrive(&bars.b.sched_full[slot]);
      mbar_arrive_cluster_release(peer_sched_full + slot * 8);
    } else {
      // the peer's loader is one more consumer of the mailbox
      const int slot = it & 1;
      if (!mbar_wait_cluster(&bars.b.sched_full[slot], (it >> 1) & 1, ctx, kRoleLoad | kBarSchedFull)) return;
      const volatile int* box = sched_w + slot * kMailboxInts;
      w = box[0];
      if (w < p.n_work) mailbox_get(box, wk);
      mbar_arrive_cluster(bars.lead_sched_empty + slot * 8);
      if (w >= p.n_work) break;
    }
    int q_pending = 0;  // Q tiles are requested after the first K tile so that K never waits behind them
#pragma unroll
    for (int s = 0; s < 2; ++s) {
      if (wk.n[s] > 0) q_pending |= 1 << s;
    }
    // tile order K(0), K(1), V(0), K(2), V(1), ...: the next block's K is asked for before this
    // block's V, because its scores are computed a block ahead of the P V that reads V
    for (int t = 0; t <= wk.nmax; ++t) {
      for (int kv = 0; kv < 2; ++kv) {
        const int j = kv == 0 ? t : t - 1;  // K(t), then V(t-1)
        if (j < 0 || j >= wk.nmax) continue;
        const uint32_t n = kv_base + static_cast<uint32_t>(j);
        const uint32_t slot = 2 * kv + (n & 1);
        const uint32_t par = (n >> 1) & 1;
        if (!mbar_wait(&bars.b.kv_empty[slot], par ^ 1, ctx, kRoleLoad | kBarKvEmpty)) return;
        uint8_t* dst = smem + kSmemKv2 + slot * kKvHalfBytes;
        const uint32_t full = bars.lead_kv_full + slot * 8;
        mbar_arrive_expect_tx_cluster(full, kKvHalfBytes);
        if (kv == 0) {  // keys 64 rank .. 64 rank + 63 of the block, both halves of the head dimension
          tma_load_4d_pair(dst, tm_k, full, 0, wk.hkv, j * kTile + rank * (kTile / 2), wk.b);
          tma_load_4d_pair(dst + kKvHalfBytes / 2, tm_k, full, 64, wk.hkv, j * kTile + rank * (kTile / 2), wk.b);
        } else {        // all 128 keys of the block, head dimension 64 rank .. 64 rank + 63
          tma_load_4d_pair(dst, tm_v, full, rank * 64, wk.hkv, j * kTile, wk.b);
        }
        if (t == 0 && kv == 0) {
#pragma unroll
          for (int s = 0; s < 2; ++s) {
            if (q_pending & (1 << s)) {
              if (!mbar_wait(&bars.b.q_empty[s], (q_cnt[s] & 1) ^ 1, ctx, kRoleLoad | kBarQEmpty)) return;
              uint8_t* qdst = smem + kSmemQ2 + s * kTileBytes;
              const uint32_t qfull = bars.lead_q_full + s * 8;
              mbar_arrive_expect_tx_cluster(qfull, kTileBytes);
              tma_load_4d_pair(qdst, tm_q, qfull, 0, wk.hq[s], wk.row0[s], wk.b);
              tma_load_4d_pair(qdst + kHalfBytes, tm_q, qfull, 64, wk.hq[s], wk.row0[s], wk.b);
              ++q_cnt[s];
            }
          }
        }
      }
    }
    kv_base += static_cast<uint32_t>(wk.nmax);
    if (rank == 0) {
      w = w_next;
      wk = wk_next;
    }
  }
}

// Leader CTA only: one MMA warp per query stage (two warps on different sub-partitions), so that the
// waits and issues of one stage never queue behind the other's in one instruction stream.  Per
// K/V block j a stage's warp issues, in this order,
//
//   S_s(j+1) = Q_s K(j+1)^T   once the stage's softmax warps have S_s(j) in registers
//   O_s += P_s(j) V(j)        first 64 keys, then last 64 keys, each once it has been written
//
// Stage 1 starts an item no less than half a block behind stage 0 (its first score tile waits until
// the first half of stage 0's first P has been seen; stage 0's warp counts those in a shared-memory
// word that only grows): one stage's exponentials (special-function unit) then overlap
// the other's loads, maxima and hand-overs instead of both contending for the same unit at once.
// K tiles and V tiles live in two rings of two slots each; a slot is free again when BOTH warps
// have committed it (a warp whose stage does not use a tile waits for it and commits it all the same).
__device__ __forceinline__ void role_mma2(const FwdParams& p, const PairBars& bars, uint8_t* smem,
                                          const volatile int* sched_w, volatile int* progress0, WaitCtx ctx,
                                          uint32_t tmem, int s, int lane) {
  const bool leader = elect_one();
  const uint32_t smem_base = smem_u32(smem);
  const uint64_t q_desc = kmajor_desc(smem_base + kSmemQ2 + s * kTileBytes);
  const uint64_t p_desc = kmajor_desc(smem_base + kSmemP2 + s * kTileBytes);
  const uint32_t t_s = tmem + s * kTile;
  const uint32_t t_o = tmem + 2 * kTile + s * kTile;
  uint32_t kv_base = 0;  // K/V blocks of earlier work items
  uint32_t q_cnt = 0;    // work items of this stage so far (phase of q_full / o_empty)
  uint32_t qk_cnt = 0;   // score tiles issued (phase of s_free)
  uint32_t sp_cnt = 0;   // K/V blocks whose P has been consumed (phase of p_half / p_full)
  int blk0 = 0;          // stage 0's K/V blocks of earlier work items (stage 1's start signal)

  // waits for tile K(j) (v = 0) or V(j) (v = 1) of the current item; returns its shared memory
  // address (0: gave up)
  auto kv_wait = [&](uint32_t v, int j) -> uint32_t {
    const uint32_t t = kv_base + static_cast<uint32_t>(j), slot = 2 * v + (t & 1), par = (t >> 1) & 1;
    if (!mbar_wait_warp(&bars.b.kv_full[slot], par, ctx, kRoleMma | kBarKvFull)) return 0u;
    return smem_base + kSmemKv2 + slot * kKvHalfBytes;
  };
  auto kv_release = [&](uint32_t v, int j) {
    if (leader) mma_commit_pair(&bars.b.kv_empty[2 * v + ((kv_base + static_cast<uint32_t>(j)) & 1)]);
  };
  // S_s(j) = Q_s K(j)^T
  auto scores = [&](int j, int n) -> bool {
    const uint32_t k_addr = kv_wait(0, j);
    if (k_addr == 0) return false;
    // the previous score tile of this stage has been read into registers
    if (!mbar_wait_warp(&bars.s_free[s], (qk_cnt & 1) ^ 1, ctx, kRoleMma | kBarSFree)) return false;
    ++qk_cnt;
    tc_fence_after_sync();
    issue_qk2(leader, t_s, q_desc, kmajor_desc(k_addr));
    if (leader) {
      mma_commit_pair(&bars.b.s_full[s]);
      if (j == n - 1) mma_commit_pair(&bars.b.q_empty[s]);  // that was the item's last use of Q_s
    }
    return true;
  };

  for (int it = 0;; ++it) {
    Work wk;
    const int w = consumer_next_work2(p, bars, sched_w, it, ctx, kRoleMma, lane == 0, wk);
    if (w < 0 || w >= p.n_work) return;
    const int n = wk.n[s];
    if (n > 0) {
      if (!mbar_wait_warp(&bars.b.q_full[s], q_cnt & 1, ctx, kRoleMma | kBarQFull)) return;
      if (s == 1) {  // start behind stage 0: after the first half of its first P of this item
        bool ok = wait_counter(progress0, blk0 + 1, ctx, kRoleMma | kBarProgress);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) return;
      }
      if (!scores(0, n)) return;
    } else if (kv_wait(0, 0) == 0) {
      return;
    }
    kv_release(0, 0);
    for (int j = 0; j < wk.nmax; ++j) {
      if (j + 1 < wk.nmax) {
        // a tile this stage does not use is still handed back only once it has landed: an earlier
        // commit would be counted for the slot's previous tile, which the other stage may still read
        if (j + 1 < n) {
          if (!scores(j + 1, n)) return;
        } else if (kv_wait(0, j + 1) == 0) {
          return;
        }
        kv_release(0, j + 1);
      }
      if (j < n) {
        const uint32_t v_addr = kv_wait(1, j);
        if (v_addr == 0) return;
        const uint64_t v_desc = make_smem_desc_sw128(v_addr, kKvHalfBytes, 1024);
        if (j == 0) {  // the previous item's O_s must have left tensor memory in both CTAs
          if (!mbar_wait_warp(&bars.b.o_empty[s], (q_cnt & 1) ^ 1, ctx, kRoleMma | kBarOEmpty)) return;
        }
        if (!mbar_wait_warp(&bars.b.p_half[s], sp_cnt & 1, ctx, kRoleMma | kBarPHalf)) return;
        tc_fence_after_sync();
        if (s == 0 && lane == 0) *progress0 = blk0 + j + 1;
        issue_pv2(leader, t_o, p_desc, v_desc, j > 0, 0, 4);
        if (leader) mma_commit_pair(&bars.pa_empty[s]);
        if (!mbar_wait_warp(&bars.b.p_full[s], sp_cnt & 1, ctx, kRoleMma | kBarPFull)) return;
        ++sp_cnt;
        tc_fence_after_sync();
        issue_pv2(leader, t_o, p_desc, v_desc, j > 0, 4, 8);
        if (leader) {
          mma_commit_pair(&bars.pb_empty[s]);
          if (j == n - 1) mma_commit_pair(&bars.b.o_full[s]);
        }
      } else if (kv_wait(1, j) == 0) {
        return;
      }
      kv_release(1, j);
    }
    kv_base += static_cast<uint32_t>(wk.nmax);
    blk0 += wk.n[0];
    if (n > 0) ++q_cnt;
  }
}

// One softmax thread owns one query row of stage `s` of this CTA.  The arithmetic is that of the
// one-CTA kernel.  As soon as a block's scores are in registers the score tile is handed back
// (s_free), so the next block's scores are computed while this one is exponentiated; P goes to
// shared memory in the layout of a Q tile, each half as soon as the P V that read the previous
// block's half has completed (pa_empty / pb_empty).
__device__ __forceinline__ void role_softmax2(const FwdParams& p, const PairBars& bars, uint8_t* smem,
                                              const volatile int* sched_w, WaitCtx ctx, uint32_t tmem, int s,
                                              int row_in_tile, int lane) {
  const uint32_t lane_sel = static_cast<uint32_t>(row_in_tile & ~31) << 16;
  const uint32_t t_s = tmem + lane_sel + s * kTile;
  const uint32_t t_o = tmem + lane_sel + 2 * kTile + s * kTile;
  float* stats = reinterpret_cast<float*>(smem + kSmemStats2) + s * 2 * kTile;
  // this row of P_s: 128 bytes per half tile, its 16-byte chunks XOR-swizzled with the row index
  uint8_t* p_row = smem + kSmemP2 + s * kTileBytes + row_in_tile * 128;
  const uint32_t sw = static_cast<uint32_t>(row_in_tile & 7);
  const uint32_t s_free = bars.lead_s_free + s * 8;
  const uint32_t p_half = bars.lead_p_half + s * 8, p_full = bars.lead_p_full + s * 8;
  const float c = p.scale_log2;
  uint32_t blk = 0;    // K/V blocks of this stage so far (phases of s_full, pa_empty, pb_empty)
  uint32_t l_cnt = 0;
  for (int it = 0;; ++it) {
    Work wk;
    const int w = consumer_next_work2(p, bars, sched_w, it, ctx, kRoleSoftmax, lane == 0, wk);
    if (w < 0 || w >= p.n_work) return;
    const int n = wk.n[s];
    if (n == 0) continue;
    const int row = wk.row0[s] + row_in_tile;
    const int row_limit = p.causal ? min(p.Sk, row + p.off + 1) : p.Sk;
    const int tile_clear = p.causal ? min(p.Sk, wk.row0[s] + p.off + 1) : p.Sk;
    float m_used = -INFINITY;
    float l = 0.f;
    for (int j = 0; j < n; ++j, ++blk) {
      bool ok = mbar_wait(&bars.b.s_full[s], blk & 1, ctx, kRoleSoftmax | kBarSFull);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return;
      tc_fence_after_sync();
      uint32_t xr[kTile];
      tmem_ld_x32(t_s + 0, xr + 0);
      tmem_ld_x32(t_s + 32, xr + 32);
      tmem_ld_x32(t_s + 64, xr + 64);
      tmem_ld_x32(t_s + 96, xr + 96);
      tmem_wait_ld();
      tc_fence_before_sync();
      if (lane == 0) mbar_arrive_cluster(s_free);  // S_s may be overwritten by the next block's scores
#define X(i) __uint_as_float(xr[(i)])
      if ((j + 1) * kTile > tile_clear) {  // warp-uniform: some element of this block is masked
        const int vis = row_limit - j * kTile;
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
          // O_s is quiescent once the previous block's P V has completed; this block's is not
          // issued before this thread's warp has released P
          ok = mbar_wait(&bars.pb_empty[s], (blk & 1) ^ 1, ctx, kRoleSoftmax | kBarPbEmpty);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) return;
          tc_fence_after_sync();
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
          tmem_wait_st();
          tc_fence_before_sync();
        }
      }
      const float neg_mc = -m_used * c;
      const float2 c2 = make_float2(c, c);
      const float2 nm2 = make_float2(neg_mc, neg_mc);
      float2 la = make_float2(0.f, 0.f), lb = make_float2(0.f, 0.f);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        // the P V that read this half of the previous block's P must have completed
        ok = mbar_wait(h == 0 ? &bars.pa_empty[s] : &bars.pb_empty[s], (blk & 1) ^ 1, ctx,
                       kRoleSoftmax | (h == 0 ? kBarPaEmpty : kBarPbEmpty));
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) return;
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {  // 16-byte chunk: 8 keys
          uint32_t pk[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int pr = ch * 4 + q;           // column pair inside the half
            const int i = h * 64 + pr * 2;
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
            pk[q] = pack_bf16x2(e.x, e.y);
          }
          *reinterpret_cast<uint4*>(p_row + h * kHalfBytes + ((static_cast<uint32_t>(ch) ^ sw) << 4)) =
              make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
        fence_proxy_async_smem();  // the tensor core reads P through the async proxy
        __syncwarp();
        if (lane == 0) {
          if (h == 0) {
            if (p.split_p) mbar_arrive_cluster(p_half);
          } else {
            if (!p.split_p) mbar_arrive_cluster(p_half);
            mbar_arrive_cluster(p_full);
          }
        }
      }
#undef X
      la = add2(la, lb);
      l += la.x + la.y;
    }
    bool ok = mbar_wait(&bars.b.l_empty[s], (l_cnt & 1) ^ 1, ctx, kRoleSoftmax | kBarLEmpty);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) return;
    stats[row_in_tile] = row_limit > 0 ? l : 0.f;
    stats[kTile + row_in_tile] = m_used;
    mbar_arrive(&bars.b.l_full[s]);
    ++l_cnt;
  }
}

__device__ __forceinline__ void role_epilogue2(const FwdParams& p, const PairBars& bars, uint8_t* smem,
                                               const volatile int* sched_w, WaitCtx ctx, uint32_t tmem,
                                               int row_in_tile, int lane, const CUtensorMap* tm_o) {
  const uint32_t lane_sel = static_cast<uint32_t>(row_in_tile & ~31) << 16;
  uint32_t cnt[2] = {0, 0};
  uint32_t stg_cnt = 0;
  for (int it = 0;; ++it) {
    Work wk;
    const int w = consumer_next_work2(p, bars, sched_w, it, ctx, kRoleEpilogue, lane == 0, wk);
    if (w < 0 || w >= p.n_work) return;
#pragma unroll 1
    for (int s = 0; s < 2; ++s) {
      if (wk.n[s] == 0) continue;
      const float* stats = reinterpret_cast<const float*>(smem + kSmemStats2) + s * 2 * kTile;
      bool ok = mbar_wait(&bars.b.l_full[s], cnt[s] & 1, ctx, kRoleEpilogue | kBarLFull);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return;
      const float l = stats[row_in_tile];
      const float m_used = stats[kTile + row_in_tile];
      mbar_arrive(&bars.b.l_empty[s]);
      ok = mbar_wait(&bars.b.o_full[s], cnt[s] & 1, ctx, kRoleEpilogue | kBarOFull);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return;
      if (!p.overlap_epilogue && s == 0 && wk.n[1] > 0) {
        ok = mbar_wait(&bars.b.o_full[1], cnt[1] & 1, ctx, kRoleEpilogue | kBarOFull);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) return;
      }
      ++cnt[s];
      tc_fence_after_sync();
      const float inv_l = l > 0.f ? __fdividef(1.0f, l) : 0.f;
      ok = mbar_wait(&bars.b.stg_empty[0], (stg_cnt & 1) ^ 1, ctx, kRoleEpilogue | kBarStgEmpty);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return;
      ++stg_cnt;
      uint8_t* stage = smem + kSmemStage2;
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
          const int chunk = cc * 4 + ch;
          uint8_t* dst = stage + (chunk >> 3) * kHalfBytes + row_in_tile * 128 +
                         (((chunk & 7) ^ (row_in_tile & 7)) << 4);
          *reinterpret_cast<uint4*>(dst) = val;
        }
      }
      tc_fence_before_sync();
      if (lane == 0) mbar_arrive_cluster(bars.lead_o_empty + s * 8);
      const int row = wk.row0[s] + row_in_tile;
      if (p.lse != nullptr && row < p.Sq) {
        p.lse[(static_cast<size_t>(wk.b) * p.Hq + wk.hq[s]) * p.Sq + row] = fmaf(lg2_approx(l), kLn2, m_used * p.scale);
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars.b.st_full[s]);
      if (row_in_tile == s * 32) {
        if (mbar_wait(&bars.b.st_full[s], (cnt[s] & 1) ^ 1, ctx, kRoleEpilogue | kBarStFull)) {
          if (wk.row0[s] < p.Sq) {  // the peer's tile of a ragged pair may lie wholly past the last row
            tma_store_4d(tm_o, stage, 0, wk.hq[s], wk.row0[s], wk.b);
            tma_store_4d(tm_o, stage + kHalfBytes, 64, wk.hq[s], wk.row0[s], wk.b);
            tma_store_commit();
            tma_store_wait_read0();
          }
          mbar_arrive(&bars.b.stg_empty[0]);
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Kernel: grid = 2 x pairs, cluster (2, 1, 1).  tm_k has a 64-key box, the others 128 rows.
// ------------------------------------------------------------------------------------------
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
attn_fwd_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                     const FwdParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* bar_mem = reinterpret_cast<uint64_t*>(smem + kSmemBars2);
  PairBars bars;
  bars.b.q_full = bar_mem;
  bars.b.q_empty = bars.b.q_full + 2;
  bars.b.kv_full = bars.b.q_empty + 2;
  bars.b.kv_empty = bars.b.kv_full + kKvSlots2;
  bars.b.s_full = bars.b.kv_empty + kKvSlots2;
  bars.b.p_half = bars.b.s_full + 2;
  bars.b.p_full = bars.b.p_half + 2;
  bars.b.o_full = bars.b.p_full + 2;
  bars.b.o_empty = bars.b.o_full + 2;
  bars.b.l_full = bars.b.o_empty + 2;
  bars.b.l_empty = bars.b.l_full + 2;
  bars.b.st_full = bars.b.l_empty + 2;
  bars.b.stg_empty = bars.b.st_full + 2;
  bars.b.sched_full = bars.b.stg_empty + 1;
  bars.b.sched_empty = bars.b.sched_full + 2;
  bars.s_free = bars.b.sched_empty + 2;
  bars.pa_empty = bars.s_free + 2;
  bars.pb_empty = bars.pa_empty + 2;
  bars.lead_s_free = map_to_cta(smem_u32(bars.s_free), 0);
  bars.lead_q_full = map_to_cta(smem_u32(bars.b.q_full), 0);
  bars.lead_kv_full = map_to_cta(smem_u32(bars.b.kv_full), 0);
  bars.lead_p_half = map_to_cta(smem_u32(bars.b.p_half), 0);
  bars.lead_p_full = map_to_cta(smem_u32(bars.b.p_full), 0);
  bars.lead_o_empty = map_to_cta(smem_u32(bars.b.o_empty), 0);
  bars.lead_sched_empty = map_to_cta(smem_u32(bars.b.sched_empty), 0);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kSmemMisc2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kSmemMisc2 + 4);
  volatile int* sched_w = reinterpret_cast<volatile int*>(smem + kSmemMisc2 + 8);
  volatile int* progress0 = sched_w + 2 * kMailboxInts;
  const WaitCtx ctx{abort_flag, p.status, kWaitLimitNs};

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;
  const int rank = static_cast<int>(cluster_ctarank());

  // the swizzled tiles need a 1024-byte aligned base; a CTA that finds otherwise takes no role but
  // still meets its peer at the cluster barriers
  const bool bad_align = (smem_u32(smem) & 1023u) != 0;
  if (bad_align && tid == 0 && atomicCAS(p.status, 0, kBadSmemAlign) == 0) p.status[1] = static_cast<int>(blockIdx.x);
  if (tid == 0) {
    if (blockIdx.x == 0 && p.clock_stamps != nullptr) {
      p.clock_stamps[0] = static_cast<unsigned long long>(clock64());
      p.clock_stamps[1] = global_timer_ns();
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars.b.q_full[i], 2);
      mbar_init(&bars.b.q_empty[i], 1);
      mbar_init(&bars.b.s_full[i], 1);
      mbar_init(&bars.b.p_half[i], 8);
      mbar_init(&bars.b.p_full[i], 8);
      mbar_init(&bars.b.o_full[i], 1);
      mbar_init(&bars.b.o_empty[i], 8);
      mbar_init(&bars.b.l_full[i], kTile);
      mbar_init(&bars.b.l_empty[i], kTile);
      mbar_init(&bars.b.st_full[i], 4);
      if (i == 0) mbar_init(&bars.b.stg_empty[0], 1);
      mbar_init(&bars.b.sched_full[i], 1);
      mbar_init(&bars.b.sched_empty[i], kSchedConsumers2);
      mbar_init(&bars.s_free[i], 8);
      mbar_init(&bars.pa_empty[i], 1);
      mbar_init(&bars.pb_empty[i], 1);
    }
    for (int i = 0; i < kKvSlots2; ++i) {
      mbar_init(&bars.b.kv_full[i], 2);
      mbar_init(&bars.b.kv_empty[i], 2);  // one commit from each MMA warp
    }
    *abort_flag = bad_align ? 1 : 0;
    *progress0 = 0;
    fence_mbar_init();
  }
  if (warp == 12) {
    tmem_alloc_pair(tmem_slot, 512);
    tmem_relinquish_pair();
  }
  if (warp == 13 && lane == 0) {
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    tma_prefetch_desc(&tm_o);
  }
  tc_fence_before_sync();
  __syncthreads();
  // both CTAs' barriers exist before either CTA signals the other's
  cluster_sync_all();
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  if (warp < 8) {
    reg_alloc<ATTN_REGS_SOFTMAX>();
    if (!bad_align) role_softmax2(p, bars, smem, sched_w, ctx, tmem, warp >> 2, tid & 127, lane);
  } else if (warp < 12) {
    reg_dealloc<ATTN_REGS_EPILOGUE>();
    if (!bad_align) role_epilogue2(p, bars, smem, sched_w, ctx, tmem, tid & 127, lane, &tm_o);
    tma_store_wait_all0();
  } else {
    reg_dealloc<ATTN_REGS_OTHER>();
    if (warp == 12 || warp == 14) {  // sub-partitions 0 and 2
      if (rank == 0 && !bad_align) role_mma2(p, bars, smem, sched_w, progress0, ctx, tmem, (warp - 12) >> 1, lane);
    } else if (warp == 13) {
      if (lane == 0 && !bad_align) {
        role_loader2(p, bars, smem, sched_w, ctx, &tm_q, &tm_k, &tm_v, rank);
        if (*abort_flag) {  // let loads in flight land before the CTA's shared memory is released
          const uint64_t t0 = global_timer_ns();
          while (global_timer_ns() - t0 < 1000000ull) {
          }
        }
      }
    }
  }
  // neither CTA leaves (and frees shared / tensor memory the other may still address) before both are done
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp == 12) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem, 512);
  }
  if (tid == 0 && blockIdx.x == 0 && p.clock_stamps != nullptr) {
    p.clock_stamps[2] = static_cast<unsigned long long>(clock64());
    p.clock_stamps[3] = global_timer_ns();
  }
}

}  // namespace pair
}  // namespace attn

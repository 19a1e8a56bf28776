// Fused attention forward for sm_100a, "triple score buffer" kernel.
//
// One persistent CTA (512 threads) works on ONE 128-row query tile at a time and keeps three score
// tiles in flight in tensor memory, so that the tensor pipe computes S(j+1), S(j+2) while block j is
// being exponentiated -- the chain  softmax -> P V -> next Q K^T  of one score buffer is overlapped
// with the chains of the two other buffers:
//
//   warps 0-3    softmax group 0   K/V blocks 0, 2, 4, ... of the tile: one thread per query row
//   warps 4-7    softmax group 1   K/V blocks 1, 3, 5, ...            (same rows, other blocks)
//   warps 8-11   epilogue          O / l -> BF16 -> shared memory -> TMA store, LSE store
//   warp  12     MMA issue         S_b = Q K_j^T into buffer b = j % 3, O += P_b V_j
//   warp  13     loader            TMA loads of the Q tile and the K / V ring, work counter
//   warps 14-15  idle (register donors)
//
// Tensor memory: S0 | S1 | S2 | O, 128 fp32 columns each; P aliases the front of its S buffer.
//
// Reference maxima.  Block j's exponentials are taken against a per-row reference R_j that its
// thread picks WITHOUT waiting for anybody: its own previous reference, raised to whatever the
// partner group has posted so far, or to the row's running maximum if that exceeds the candidate
// by more than the rescale threshold.  O, however, is relative to the reference of the latest
// block added to it, so before block j's P is released to the MMA warp its thread reads the FINAL
// reference of block j-1 (posted by the partner long before, in the steady state) and, if the two
// differ, rescales O once P V(j-1) has completed.  If block j-1's reference is so much larger that
// the factor could overflow, the first half of block j is redone against that reference instead.
// Each group keeps its own partial row sum relative to its latest reference; the epilogue merges.
#pragma once

#include "attn_fwd_kernel.cuh"

namespace attn {
namespace sb3 {

constexpr int kSBufs = 3;
constexpr int kSlots = 5;   // K/V ring
constexpr int kSmemQ3 = 0;  // the Q tile, reused as the O staging tile
constexpr int kSmemKv3 = kTileBytes;
constexpr int kSmemStats3 = kSmemKv3 + kSlots * kTileBytes;  // float [2 groups][2: l, m][128 rows]
constexpr int kSmemPubR = kSmemStats3 + 2 * 2 * kTile * 4;   // float [2 groups][2 slots][128 rows]: posted references
constexpr int kSmemPubTag = kSmemPubR + 2 * 2 * kTile * 4;   // int   [2 groups][2 slots][128 rows]: work item of the post
constexpr int kSmemBars3 = kSmemPubTag + 2 * 2 * kTile * 4;
constexpr float kRedoThreshold = 30.0f;  // log2 units: larger O rescale factors are avoided by redoing half a block
constexpr int kNumBars3 = 1 + 1 + 2 * kSlots + 4 * kSBufs + 5 + 8 + 2 + 2;
constexpr int kSmemMisc3 = kSmemBars3 + kNumBars3 * 8;  // tmem base, abort flag, sched slots
constexpr int kSmemBytes3 = kSmemMisc3 + 32;
static_assert(kSmemBytes3 <= 232448, "shared memory budget of one CTA");
static_assert(2 * 2 * kTile == kThreads, "one posted-reference tag per thread at start-up");

enum : int { kBarPvDone = 15, kBarMReady = 16 };

struct Bars3 {
  uint64_t* q_full;    // [1]  loader -> MMA
  uint64_t* q_empty;   // [1]  epilogue -> loader
  uint64_t* kv_full;   // [kSlots]
  uint64_t* kv_empty;  // [kSlots]
  uint64_t* s_full;    // [3]  MMA commit -> softmax group of that block
  uint64_t* p_half;    // [3]  softmax (4 warps): first 64 keys of P written -> MMA
  uint64_t* p_full;    // [3]  softmax (4 warps): all of P written -> MMA
  uint64_t* pv_done;   // [3]  MMA commit after P V of the block in that buffer -> softmax (rescale path)
  uint64_t* o_full;    // [1]  MMA commit after the tile's last P V -> epilogue
  uint64_t* o_empty;   // [1]  epilogue (4 warps) -> MMA
  uint64_t* l_full;    // [1]  both softmax groups (256 threads) -> epilogue
  uint64_t* l_empty;   // [1]  epilogue (128 threads) -> softmax
  uint64_t* st_full;   // [1]  epilogue (4 warps) -> the thread issuing the TMA store
  uint64_t* m_ready;   // [2 block parities][4 lane quarters]  final reference of a block posted
  uint64_t* sched_full;   // [2]
  uint64_t* sched_empty;  // [2]
};

struct Item {
  int b, hq, hkv, row0, n;
};

// Work item w = one query tile; launch order as in split_work, inside a head longest tiles first
// when causal.
__host__ __device__ __forceinline__ void decode_item(const FwdParams& p, int w, Item& it) {
  int grp, r;
  split_work(p, w, grp, r);
  const int qt = p.causal ? (p.n_qt - 1 - r) : r;
  it.b = grp / p.Hq;
  it.hq = grp - it.b * p.Hq;
  it.hkv = it.hq / p.group;
  it.row0 = qt * kTile;
  if (p.causal) {
    const int row_end = it.row0 + kTile < p.Sq ? it.row0 + kTile : p.Sq;
    const int last_key = row_end - 1 + p.off;  // < 0: no row of the tile sees a key; one masked block is visited
    const int need = last_key < 0 ? 1 : last_key / kTile + 1;
    it.n = need < p.n_kb ? need : p.n_kb;
  } else {
    it.n = p.n_kb;
  }
}

// Same mailbox protocol as the dual-stage kernel (the barrier pointers differ).  Whole warp.
__device__ __forceinline__ int next_item(const FwdParams& p, const Bars3& bars, const volatile int* sched_w, int it,
                                         WaitCtx ctx, int role, bool lane_arrives) {
  if (!p.dynamic) return static_cast<int>(blockIdx.x) + it * static_cast<int>(gridDim.x);
  if (it == 0) return static_cast<int>(blockIdx.x);
  const int slot = (it - 1) & 1;
  if (!mbar_wait_warp(&bars.sched_full[slot], ((it - 1) >> 1) & 1, ctx, role | kBarSchedFull)) return -1;
  const int w = sched_w[slot];
  __syncwarp();
  if (lane_arrives) mbar_arrive(&bars.sched_empty[slot]);
  return w;
}

// ------------------------------------------------------------------------------------------
// Loader (one lane).  Ring order = the order the MMA warp consumes tiles:
//   K0 K1 K2 | V0 K3 | V1 K4 | ... | V(n-1)
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void role_loader3(const FwdParams& p, const Bars3& bars, uint8_t* smem,
                                             volatile int* sched_w, WaitCtx ctx, const CUtensorMap* tm_q,
                                             const CUtensorMap* tm_k, const CUtensorMap* tm_v) {
  uint32_t kv_cnt = 0, q_cnt = 0;
  int w = static_cast<int>(blockIdx.x);
  for (int it = 0; w < p.n_work; ++it) {
    int w_next;
    if (p.dynamic) {
      const int slot = it & 1;
      if (!mbar_wait(&bars.sched_empty[slot], ((it >> 1) & 1) ^ 1, ctx, kRoleLoad | kBarSchedEmpty)) return;
      w_next = static_cast<int>(atomicAdd(p.counter, 1u)) + static_cast<int>(gridDim.x);
      sched_w[slot] = w_next;
      mbar_arrive(&bars.sched_full[slot]);
    } else {
      w_next = w + static_cast<int>(gridDim.x);
    }
    Item item;
    decode_item(p, w, item);
    const int n = item.n;
    auto load_tile = [&](const CUtensorMap* tm, int blk) -> bool {
      const uint32_t slot = kv_cnt % kSlots;
      if (!mbar_wait(&bars.kv_empty[slot], ((kv_cnt / kSlots) & 1) ^ 1, ctx, kRoleLoad | kBarKvEmpty)) return false;
      uint8_t* dst = smem + kSmemKv3 + slot * kTileBytes;
      mbar_arrive_expect_tx(&bars.kv_full[slot], kTileBytes);
      tma_load_4d(dst, tm, &bars.kv_full[slot], 0, item.hkv, blk * kTile, item.b);
      tma_load_4d(dst + kHalfBytes, tm, &bars.kv_full[slot], 64, item.hkv, blk * kTile, item.b);
      ++kv_cnt;
      return true;
    };
    const int pro = n < kSBufs ? n : kSBufs;
    for (int j = 0; j < pro; ++j) {
      if (!load_tile(tm_k, j)) return;
      if (j == 0) {  // the Q tile goes out right behind the first K tile
        if (!mbar_wait(&bars.q_empty[0], (q_cnt & 1) ^ 1, ctx, kRoleLoad | kBarQEmpty)) return;
        uint8_t* qdst = smem + kSmemQ3;
        mbar_arrive_expect_tx(&bars.q_full[0], kTileBytes);
        tma_load_4d(qdst, tm_q, &bars.q_full[0], 0, item.hq, item.row0, item.b);
        tma_load_4d(qdst + kHalfBytes, tm_q, &bars.q_full[0], 64, item.hq, item.row0, item.b);
        ++q_cnt;
      }
    }
    for (int j = 0; j < n; ++j) {
      if (!load_tile(tm_v, j)) return;
      if (j + kSBufs < n) {
        if (!load_tile(tm_k, j + kSBufs)) return;
      }
    }
    w = w_next;
  }
}

// ------------------------------------------------------------------------------------------
// MMA warp (whole warp runs the control flow, the elected lane issues)
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void role_mma3(const FwdParams& p, const Bars3& bars, uint8_t* smem,
                                          const volatile int* sched_w, WaitCtx ctx, uint32_t tmem, int lane) {
  const bool leader = elect_one();
  const uint32_t smem_base = smem_u32(smem);
  const uint64_t q_desc = kmajor_desc(smem_base + kSmemQ3);
  const uint32_t tmem_o = tmem + kSBufs * kTile;
  uint32_t kv_cnt = 0, item_cnt = 0;
  uint32_t use0 = 0, use1 = 0, use2 = 0;  // P V issued from each score buffer so far (phase of p_half / p_full)
  for (int it = 0;; ++it) {
    const int w = next_item(p, bars, sched_w, it, ctx, kRoleMma, lane == 0);
    if (w < 0 || w >= p.n_work) return;
    Item item;
    decode_item(p, w, item);
    const int n = item.n;
    const int pro = n < kSBufs ? n : kSBufs;
    for (int j = 0; j < pro; ++j) {  // S(0..2)
      const uint32_t slot = kv_cnt % kSlots;
      if (!mbar_wait_warp(&bars.kv_full[slot], (kv_cnt / kSlots) & 1, ctx, kRoleMma | kBarKvFull)) return;
      if (j == 0) {
        if (!mbar_wait_warp(&bars.q_full[0], item_cnt & 1, ctx, kRoleMma | kBarQFull)) return;
      }
      tc_fence_after_sync();
      issue_qk(leader, tmem + j * kTile, q_desc, kmajor_desc(smem_base + kSmemKv3 + slot * kTileBytes));
      if (leader) {
        mma_commit(&bars.s_full[j]);
        mma_commit(&bars.kv_empty[slot]);
      }
      ++kv_cnt;
    }
    int b = 0;  // j % 3
    for (int j = 0; j < n; ++j) {
      const uint32_t vslot = kv_cnt % kSlots;
      if (!mbar_wait_warp(&bars.kv_full[vslot], (kv_cnt / kSlots) & 1, ctx, kRoleMma | kBarKvFull)) return;
      ++kv_cnt;
      if (j == 0) {  // the previous tile's O must have left tensor memory
        if (!mbar_wait_warp(&bars.o_empty[0], (item_cnt & 1) ^ 1, ctx, kRoleMma | kBarOEmpty)) return;
      }
      const uint64_t v_desc = vtile_desc(smem_base + kSmemKv3 + vslot * kTileBytes);
      const uint32_t use = b == 0 ? use0 : (b == 1 ? use1 : use2);
      if (!mbar_wait_warp(&bars.p_half[b], use & 1, ctx, kRoleMma | kBarPHalf)) return;
      tc_fence_after_sync();
      issue_pv(leader, tmem_o, tmem + b * kTile, v_desc, j > 0, 0, 4);
      if (!mbar_wait_warp(&bars.p_full[b], use & 1, ctx, kRoleMma | kBarPFull)) return;
      if (b == 0) ++use0; else if (b == 1) ++use1; else ++use2;
      tc_fence_after_sync();
      issue_pv(leader, tmem_o, tmem + b * kTile, v_desc, j > 0, 4, 8);
      if (leader) {
        mma_commit(&bars.pv_done[b]);
        mma_commit(&bars.kv_empty[vslot]);
        if (j == n - 1) mma_commit(&bars.o_full[0]);
      }
      if (j + kSBufs < n) {  // S(j+3) reuses the buffer P(j) is being read from (same in-order pipe)
        const uint32_t kslot = kv_cnt % kSlots;
        if (!mbar_wait_warp(&bars.kv_full[kslot], (kv_cnt / kSlots) & 1, ctx, kRoleMma | kBarKvFull)) return;
        ++kv_cnt;
        tc_fence_after_sync();
        issue_qk(leader, tmem + b * kTile, q_desc, kmajor_desc(smem_base + kSmemKv3 + kslot * kTileBytes));
        if (leader) {
          mma_commit(&bars.s_full[b]);
          mma_commit(&bars.kv_empty[kslot]);
        }
      }
      b = (b == kSBufs - 1) ? 0 : b + 1;
    }
    ++item_cnt;
  }
}

// Number of blocks j < n with j % 3 == b.
__device__ __forceinline__ uint32_t blocks_in_buffer(int n, int b) {
  return n > b ? static_cast<uint32_t>((n - b + kSBufs - 1) / kSBufs) : 0u;
}

// ------------------------------------------------------------------------------------------
// Softmax group g: blocks g, g+2, ... ; thread = one query row
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void role_softmax3(const FwdParams& p, const Bars3& bars, uint8_t* smem,
                                              const volatile int* sched_w, WaitCtx ctx, uint32_t tmem, int g,
                                              int row_in_tile, int lane) {
  const int quarter = row_in_tile >> 5;
  const uint32_t lane_sel = static_cast<uint32_t>(row_in_tile & ~31) << 16;
  const uint32_t t_o = tmem + lane_sel + kSBufs * kTile;
  float* stats = reinterpret_cast<float*>(smem + kSmemStats3) + g * 2 * kTile;
  volatile float* pub_r = reinterpret_cast<volatile float*>(smem + kSmemPubR);
  volatile int* pub_tag = reinterpret_cast<volatile int*>(smem + kSmemPubTag);
  const float c = p.scale_log2;
  uint32_t base0 = 0, base1 = 0, base2 = 0;  // uses of each score buffer by earlier tiles
  uint32_t mbase0 = 0, mbase1 = 0;           // blocks of each parity published by earlier tiles
  uint32_t item_cnt = 0;
  for (int it = 0;; ++it) {
    const int w = next_item(p, bars, sched_w, it, ctx, kRoleSoftmax, lane == 0);
    if (w < 0 || w >= p.n_work) return;
    Item item;
    decode_item(p, w, item);
    const int n = item.n;
    const int row = item.row0 + row_in_tile;
    const int row_limit = p.causal ? min(p.Sk, row + p.off + 1) : p.Sk;
    const int tile_clear = p.causal ? min(p.Sk, item.row0 + p.off + 1) : p.Sk;
    float l = 0.f;        // this group's partial row sum, relative to m_last
    float m_last = 0.f;   // reference of this thread's latest block
    float own_max = -INFINITY;  // running maximum of the scores this thread has seen in this tile
    bool has = false;
    const int tag = it + 1;
    for (int j = g; j < n; j += 2) {
      const int b = j % kSBufs;
      const uint32_t use_b = (b == 0 ? base0 : (b == 1 ? base1 : base2)) + static_cast<uint32_t>(j / kSBufs);
      const uint32_t t_s = tmem + lane_sel + b * kTile;
      if (!mbar_wait_warp(&bars.s_full[b], use_b & 1, ctx, kRoleSoftmax | kBarSFull)) return;
      tc_fence_after_sync();
      uint32_t xr[kTile];
      tmem_ld_x32(t_s + 0, xr + 0);
      tmem_ld_x32(t_s + 32, xr + 32);
      tmem_ld_x32(t_s + 64, xr + 64);
      tmem_ld_x32(t_s + 96, xr + 96);
      tmem_wait_ld();
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
      own_max = fmaxf(own_max, fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)));

      // ---- pick this block's reference without waiting ----
      float cand = has ? m_last : -INFINITY;
#pragma unroll
      for (int sl = 0; sl < 2; ++sl) {  // whatever the partner has posted for this tile so far
        const int idx = ((g ^ 1) * 2 + sl) * kTile + row_in_tile;
        const int t = pub_tag[idx];
        const float r = pub_r[idx];
        if (t == tag) cand = fmaxf(cand, r);
      }
      float m_cur;
      if (cand == -INFINITY) {
        m_cur = (own_max == -INFINITY) ? 0.f : own_max;
      } else {
        m_cur = ((own_max - cand) * c > p.rescale_threshold) ? own_max : cand;
      }
      const int my_slot = ((g * 2) + ((j >> 1) & 1)) * kTile + row_in_tile;
      float2 la, lb;
#pragma unroll 1
      for (int pass = 0; pass < 2; ++pass) {
        if (has && __any_sync(0xffffffffu, m_last != m_cur)) l *= ex2_approx((m_last - m_cur) * c);
        m_last = m_cur;
        pub_r[my_slot] = m_cur;  // early, provisional: helps the partner pick the same reference
        pub_tag[my_slot] = tag;
        // first 64 keys of P
        const float neg_mc = -m_cur * c;
        const float2 c2 = make_float2(c, c);
        const float2 nm2 = make_float2(neg_mc, neg_mc);
        la = make_float2(0.f, 0.f);
        lb = make_float2(0.f, 0.f);
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
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
        }
        if (j == 0) break;
        // ---- O is relative to block j-1's final reference: reconcile before releasing P ----
        const int pp = (j - 1) & 1;
        const uint32_t pub = (pp == 0 ? mbase0 : mbase1) + static_cast<uint32_t>((j - 1) / 2);
        if (!mbar_wait_warp(&bars.m_ready[pp * 4 + quarter], pub & 1, ctx, kRoleSoftmax | kBarMReady)) return;
        const float m_prev = pub_r[((g ^ 1) * 2 + (((j - 1) >> 1) & 1)) * kTile + row_in_tile];
        const float d = (m_prev - m_cur) * c;  // O must be multiplied by 2^d
        if (pass == 0 && __any_sync(0xffffffffu, d > kRedoThreshold)) {
          if (d > kRedoThreshold) m_cur = m_prev;  // adopt the larger reference and redo the half block
          continue;
        }
        if (__any_sync(0xffffffffu, d != 0.f)) {
          const float alpha = ex2_approx(d);
          // O may be touched once P V of block j-1 has completed; P V of block j waits for this thread
          const int bp = (j - 1) % kSBufs;
          const uint32_t use_p = (bp == 0 ? base0 : (bp == 1 ? base1 : base2)) + static_cast<uint32_t>((j - 1) / kSBufs);
          if (!mbar_wait_warp(&bars.pv_done[bp], use_p & 1, ctx, kRoleSoftmax | kBarPvDone)) return;
          tc_fence_after_sync();
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
        break;
      }
      has = true;
      // final reference of block j: the partner reads it before it releases block j+1
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars.m_ready[(j & 1) * 4 + quarter]);
      tmem_wait_st();
      tc_fence_before_sync();
      if (lane == 0) mbar_arrive(&bars.p_half[b]);

      {
        const float neg_mc = -m_cur * c;
        const float2 c2 = make_float2(c, c);
        const float2 nm2 = make_float2(neg_mc, neg_mc);
#pragma unroll
        for (int cc = 2; cc < 4; ++cc) {
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
        }
      }
#undef X
      la = add2(la, lb);
      l += la.x + la.y;
      tmem_wait_st();
      tc_fence_before_sync();
      if (lane == 0) mbar_arrive(&bars.p_full[b]);
    }
    // hand this group's partial sum and its reference to the epilogue warps
    if (!mbar_wait_warp(&bars.l_empty[0], (item_cnt & 1) ^ 1, ctx, kRoleSoftmax | kBarLEmpty)) return;
    stats[row_in_tile] = (has && row_limit > 0) ? l : 0.f;  // no visible key (causal, Sq > Sk): the sum is 0
    stats[kTile + row_in_tile] = m_last;
    mbar_arrive(&bars.l_full[0]);
    base0 += blocks_in_buffer(n, 0);
    base1 += blocks_in_buffer(n, 1);
    base2 += blocks_in_buffer(n, 2);
    mbase0 += static_cast<uint32_t>((n + 1) / 2);
    mbase1 += static_cast<uint32_t>(n / 2);
    ++item_cnt;
  }
}

__device__ __forceinline__ void role_epilogue3(const FwdParams& p, const Bars3& bars, uint8_t* smem,
                                               const volatile int* sched_w, WaitCtx ctx, uint32_t tmem,
                                               int row_in_tile, int lane, const CUtensorMap* tm_o) {
  const uint32_t lane_sel = static_cast<uint32_t>(row_in_tile & ~31) << 16;
  const uint32_t t_o = tmem + lane_sel + kSBufs * kTile;
  const float* stats = reinterpret_cast<const float*>(smem + kSmemStats3);
  const float c = p.scale_log2;
  uint32_t item_cnt = 0;
  for (int it = 0;; ++it) {
    const int w = next_item(p, bars, sched_w, it, ctx, kRoleEpilogue, lane == 0);
    if (w < 0 || w >= p.n_work) return;
    Item item;
    decode_item(p, w, item);
    if (!mbar_wait_warp(&bars.l_full[0], item_cnt & 1, ctx, kRoleEpilogue | kBarLFull)) return;
    const float l0 = stats[row_in_tile], m0 = stats[kTile + row_in_tile];
    const float l1 = stats[2 * kTile + row_in_tile], m1 = stats[3 * kTile + row_in_tile];
    mbar_arrive(&bars.l_empty[0]);
    // O is relative to the reference of the tile's last block, which group (n - 1) & 1 processed
    const float m_fin = ((item.n - 1) & 1) ? m1 : m0;
    float l_row = 0.f;
    if (l0 > 0.f) l_row += l0 * ex2_approx((m0 - m_fin) * c);
    if (l1 > 0.f) l_row += l1 * ex2_approx((m1 - m_fin) * c);
    if (!mbar_wait_warp(&bars.o_full[0], item_cnt & 1, ctx, kRoleEpilogue | kBarOFull)) return;
    tc_fence_after_sync();
    const float inv_l = l_row > 0.f ? __fdividef(1.0f, l_row) : 0.f;  // a row without visible keys: O = 0, LSE = -inf
    uint8_t* stage = smem + kSmemQ3;
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
    if (lane == 0) mbar_arrive(&bars.o_empty[0]);
    const int row = item.row0 + row_in_tile;
    if (p.lse != nullptr && row < p.Sq) {
      p.lse[(static_cast<size_t>(item.b) * p.Hq + item.hq) * p.Sq + row] = fmaf(lg2_approx(l_row), kLn2, m_fin * p.scale);
    }
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) mbar_arrive(&bars.st_full[0]);
    if (row_in_tile == 0) {
      if (mbar_wait(&bars.st_full[0], item_cnt & 1, ctx, kRoleEpilogue | kBarStFull)) {
        tma_store_4d(tm_o, stage, 0, item.hq, item.row0, item.b);
        tma_store_4d(tm_o, stage + kHalfBytes, 64, item.hq, item.row0, item.b);
        tma_store_commit();
        tma_store_wait_read0();
        mbar_arrive(&bars.q_empty[0]);
      }
    }
    ++item_cnt;
  }
}

__global__ void __launch_bounds__(kThreads, 1)
attn_fwd_sb3_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                    const FwdParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  uint64_t* bm = reinterpret_cast<uint64_t*>(smem + kSmemBars3);
  Bars3 bars;
  bars.q_full = bm;
  bars.q_empty = bars.q_full + 1;
  bars.kv_full = bars.q_empty + 1;
  bars.kv_empty = bars.kv_full + kSlots;
  bars.s_full = bars.kv_empty + kSlots;
  bars.p_half = bars.s_full + kSBufs;
  bars.p_full = bars.p_half + kSBufs;
  bars.pv_done = bars.p_full + kSBufs;
  bars.o_full = bars.pv_done + kSBufs;
  bars.o_empty = bars.o_full + 1;
  bars.l_full = bars.o_empty + 1;
  bars.l_empty = bars.l_full + 1;
  bars.st_full = bars.l_empty + 1;
  bars.m_ready = bars.st_full + 1;
  bars.sched_full = bars.m_ready + 8;
  bars.sched_empty = bars.sched_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kSmemMisc3);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kSmemMisc3 + 4);
  volatile int* sched_w = reinterpret_cast<volatile int*>(smem + kSmemMisc3 + 8);
  const WaitCtx ctx{abort_flag, p.status, kWaitLimitNs};

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;

  if ((smem_u32(smem) & 1023u) != 0) {  // the swizzled tiles need a 1024-byte aligned base
    if (tid == 0 && atomicCAS(p.status, 0, kBadSmemAlign) == 0) p.status[1] = static_cast<int>(blockIdx.x);
    return;
  }
  if (tid == 0) {
    mbar_init(&bars.q_full[0], 1);
    mbar_init(&bars.q_empty[0], 1);
    for (int i = 0; i < kSlots; ++i) {
      mbar_init(&bars.kv_full[i], 1);
      mbar_init(&bars.kv_empty[i], 1);
    }
    for (int i = 0; i < kSBufs; ++i) {
      mbar_init(&bars.s_full[i], 1);
      mbar_init(&bars.p_half[i], 4);
      mbar_init(&bars.p_full[i], 4);
      mbar_init(&bars.pv_done[i], 1);
    }
    mbar_init(&bars.o_full[0], 1);
    mbar_init(&bars.o_empty[0], 4);
    mbar_init(&bars.l_full[0], 2 * kTile);
    mbar_init(&bars.l_empty[0], kTile);
    mbar_init(&bars.st_full[0], 4);
    for (int i = 0; i < 8; ++i) mbar_init(&bars.m_ready[i], 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars.sched_full[i], 1);
      mbar_init(&bars.sched_empty[i], kSchedConsumers);
    }
    *abort_flag = 0;
    fence_mbar_init();
  }
  // no reference has been posted yet: shared memory keeps whatever an earlier kernel left there
  reinterpret_cast<volatile int*>(smem + kSmemPubTag)[tid] = 0;
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
    role_softmax3(p, bars, smem, sched_w, ctx, tmem, warp >> 2, tid & 127, lane);
  } else if (warp < 12) {
    reg_dealloc<ATTN_REGS_EPILOGUE>();
    role_epilogue3(p, bars, smem, sched_w, ctx, tmem, tid & 127, lane, &tm_o);
    tma_store_wait_all0();
  } else {
    reg_dealloc<ATTN_REGS_OTHER>();
    if (warp == 12) {
      role_mma3(p, bars, smem, sched_w, ctx, tmem, lane);
    } else if (warp == 13) {
      if (lane == 0) {
        role_loader3(p, bars, smem, sched_w, ctx, &tm_q, &tm_k, &tm_v);
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
}

}  // namespace sb3
}  // namespace attn

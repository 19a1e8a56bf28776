// Fused attention forward with TWO softmax threads per query row (option "kernel" = 3): the
// dual-query-stage kernel of attn_fwd_kernel.cuh (same loader, same MMA warp, same tensor- and
// shared-memory layout) with sixteen softmax warps instead of eight.
//
// A row's 128 scores of a K/V block are split between two threads of two different warps (the
// same lane of warps w and w + 4 of a stage: tensor memory lets a warp touch only the 32 lanes
// given by its index modulo 4, so both sit on the same sub-partition): thread h exponentiates keys
// 64 h .. 64 h + 63, which halves the latency of a block's softmax -- the longest link of the chain
// softmax -> P V -> next Q K^T -- and doubles the warps a sub-partition can choose from.  The two
// threads exchange their partial row maxima through shared memory once per block (an mbarrier the
// two warps arrive on and wait for with the same bounded wait as everywhere else, so that a warp
// whose partner has given up runs into the time limit instead of waiting for ever), so both take
// the exponentials against the same reference; each keeps its own
// partial row sum, rescales its own 64 columns of O when the reference moves, and hands over its
// own half of P: the first-half threads' arrival is the "first 64 keys" signal of the one-CTA
// kernel, the second-half threads' the "all of P" signal.  There are no epilogue warps: the
// softmax threads normalise and store their own 64 columns of O at the end of a work item.
#pragma once

#include "attn_fwd_kernel.cuh"

namespace attn {
namespace w16 {

constexpr int kThreads16 = 640;  // 16 softmax warps, MMA warp, loader warp, 2 idle
// setmaxnreg split of 640 x 96 registers: 16 softmax warps and 4 others
constexpr int kRegsSoftmax16 = 104;
constexpr int kRegsOther16 = 64;
static_assert(16 * kRegsSoftmax16 + 4 * kRegsOther16 <= 20 * 96, "register split");
constexpr int kSchedConsumers16 = 1 + 16;  // MMA lane and 16 softmax warps

enum : int { kBarToken = 23 };

// Barriers of the one-CTA kernel's layout that this kernel uses differently:
//   st_full[s]  : the 4 first-half warps of stage s have written their staging half
//   l_full[s]   : the 4 second-half warps of stage s have written theirs
//   l_empty[h]  : token of staging half h: use u (= 2 x work item + stage) has been read by its TMA store
//   stg_empty   : unused

__device__ __forceinline__ void role_softmax16(const FwdParams& p, const Barriers& bars, uint8_t* smem,
                                               const volatile int* sched_w, WaitCtx ctx, uint32_t tmem, int s,
                                               int h, int row_in_tile, int lane, const CUtensorMap* tm_o) {
  const uint32_t lane_sel = static_cast<uint32_t>(row_in_tile & ~31) << 16;
  const uint32_t t_s = tmem + lane_sel + s * kTile + h * 64;              // this thread's 64 score columns
  const uint32_t t_p = tmem + lane_sel + s * kTile + h * 32;              // its half of P (64 keys, BF16 pairs)
  const uint32_t t_o = tmem + lane_sel + 2 * kTile + s * kTile + h * 64;  // its 64 columns of O_s
  volatile float* ex = reinterpret_cast<volatile float*>(smem + kSmemStats);
  volatile float* mine = ex + (s * 2 + h) * kTile + row_in_tile;
  volatile float* partner = ex + (s * 2 + (1 - h)) * kTile + row_in_tile;
  // mbarrier of the two warps that share these rows (count 2: lane 0 of each); behind the barriers
  // of the one-CTA layout in the barrier array
  uint64_t* pair_bar = bars.q_full + (kNumBars - 8) + s * 4 + (row_in_tile >> 5);
  uint32_t x_cnt = 0;  // exchanges so far (phase of pair_bar)
  // Publishes this thread's value and returns when the partner's is readable; false on an expired wait.
  auto exchange = [&](float value) -> bool {
    *mine = value;
    __syncwarp();
    if (lane == 0) mbar_arrive(pair_bar);
    bool ok = mbar_wait(pair_bar, x_cnt & 1, ctx, kRoleSoftmax | kBarExchange);
    ok = __all_sync(0xffffffffu, ok);
    ++x_cnt;
    return ok;
  };
  uint64_t* my_p_bar = h == 0 ? &bars.p_half[s] : &bars.p_full[s];
  uint64_t* my_st_full = h == 0 ? &bars.st_full[s] : &bars.l_full[s];
  uint64_t* token = &bars.l_empty[h];
  const bool stores = (row_in_tile == 0);  // this thread issues the TMA store of (s, h)
  const float c = p.scale_log2;
  uint32_t s_cnt = 0;   // phase of s_full[s]
  uint32_t o_cnt = 0;   // work items of this stage so far (phase of o_full[s] and of the staging-full barrier)
  for (int it = 0;; ++it) {
    Work wk;
    const int w = consumer_next_work(p, bars, sched_w, it, ctx, kRoleSoftmax, lane == 0, true, wk);
    if (w < 0 || w >= p.n_work) return;
    const int n = wk.n[s];
    const uint32_t use_parity = static_cast<uint32_t>(2 * it + s + 1) & 1;  // parity of use u - 1
    if (n == 0) {  // the stage is idle in this item: pass the staging token on
      if (stores) {
        if (!mbar_wait(token, use_parity, ctx, kRoleSoftmax | kBarToken)) return;
        mbar_arrive(token);
      }
      continue;
    }
    const int row = wk.row0[s] + row_in_tile;
    const int row_limit = p.causal ? min(p.Sk, row + p.off + 1) : p.Sk;
    const int tile_clear = p.causal ? min(p.Sk, wk.row0[s] + p.off + 1) : p.Sk;
    float m_used = -INFINITY;
    float l = 0.f;  // this thread's part of the row sum
    for (int j = 0; j < n; ++j) {
      bool ok = mbar_wait(&bars.s_full[s], s_cnt & 1, ctx, kRoleSoftmax | kBarSFull);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return;
      ++s_cnt;
      tc_fence_after_sync();
      uint32_t xr[64];
      tmem_ld_x32(t_s + 0, xr + 0);
      tmem_ld_x32(t_s + 32, xr + 32);
      tmem_wait_ld();
#define X(i) __uint_as_float(xr[(i)])
      if ((j + 1) * kTile > tile_clear) {  // warp-uniform: some element of this block is masked
        const int vis = row_limit - j * kTile - h * 64;  // visible columns of this thread's half
#pragma unroll
        for (int i = 0; i < 64; ++i) {
          if (i >= vis) xr[i] = 0xff800000u;
        }
      }
      float m0 = X(0), m1 = X(1), m2 = X(2), m3 = X(3);
#pragma unroll
      for (int i = 4; i < 64; i += 8) {
        m0 = max3(m0, X(i), X(i + 1));
        m1 = max3(m1, X(i + 2), X(i + 3));
        if (i + 4 < 64) {
          m2 = max3(m2, X(i + 4), X(i + 5));
          m3 = max3(m3, X(i + 6), X(i + 7));
        }
      }
      const float m_half = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
      // The slot written here was last read by the partner before its previous hand-over of P, which
      // the scores just waited for were issued behind: the exchange needs no second barrier.
      if (!exchange(m_half)) return;
      const float m_blk = fmaxf(m_half, *partner);
      if (j == 0) {
        m_used = (m_blk == -INFINITY) ? 0.f : m_blk;
      } else {
        const float m_new = fmaxf(m_used, m_blk);
        const bool grow = (m_new - m_used) * c > p.rescale_threshold;
        if (__any_sync(0xffffffffu, grow)) {  // the partner warp holds the same rows and takes the same branch
          // P V of block j-1 has completed (S of block j was issued after it), so O_s is quiescent
          const float alpha = ex2_approx((m_used - m_new) * c);
          m_used = m_new;
          l *= alpha;
#pragma unroll
          for (int cc = 0; cc < 4; ++cc) {
            uint32_t o[16];
            tmem_ld_x16(t_o + cc * 16, o);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
            tmem_st_x16(t_o + cc * 16, o);
          }
        }
      }
      const float neg_mc = -m_used * c;
      const float2 c2 = make_float2(c, c);
      const float2 nm2 = make_float2(neg_mc, neg_mc);
      float2 la = make_float2(0.f, 0.f), lb = make_float2(0.f, 0.f);
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
        tmem_st_x16(t_p + cc * 16, pk);
      }
#undef X
      tmem_wait_st();
      tc_fence_before_sync();
      if (lane == 0) mbar_arrive(my_p_bar);
      la = add2(la, lb);
      l += la.x + la.y;
    }
    // ---- end of the work item: the row sum of both halves, then this thread's 64 columns of O ----
    if (!exchange(l)) return;
    float l_row = l + *partner;
    // both must have read before the slots carry maxima again
    __syncwarp();
    if (lane == 0) mbar_arrive(pair_bar);
    {
      bool ok2 = mbar_wait(pair_bar, x_cnt & 1, ctx, kRoleSoftmax | kBarExchange);
      ok2 = __all_sync(0xffffffffu, ok2);
      ++x_cnt;
      if (!ok2) return;
    }
    if (row_limit <= 0) l_row = 0.f;   // a row without any visible key has the sum 0 by definition
    bool ok = mbar_wait(&bars.o_full[s], o_cnt & 1, ctx, kRoleSoftmax | kBarOFull);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) return;
    tc_fence_after_sync();
    const float inv_l = l_row > 0.f ? __fdividef(1.0f, l_row) : 0.f;
    // staging half h is free once the store of its previous use has read it
    ok = mbar_wait(token, use_parity, ctx, kRoleSoftmax | kBarToken);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) return;
    uint8_t* stage = smem + kSmemStage + h * kHalfBytes;
#pragma unroll
    for (int cc = 0; cc < 2; ++cc) {
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
        const int chunk = cc * 4 + ch;  // 16-byte chunk of this half's 128-byte row
        *reinterpret_cast<uint4*>(stage + row_in_tile * 128 + ((chunk ^ (row_in_tile & 7)) << 4)) = val;
      }
    }
    tc_fence_before_sync();
    if (lane == 0) mbar_arrive(&bars.o_empty[s]);
    if (h == 0 && p.lse != nullptr && row < p.Sq) {
      p.lse[(static_cast<size_t>(wk.b) * p.Hq + wk.hq[s]) * p.Sq + row] = fmaf(lg2_approx(l_row), kLn2, m_used * p.scale);
    }
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) mbar_arrive(my_st_full);
    if (stores) {
      if (mbar_wait(my_st_full, o_cnt & 1, ctx, kRoleSoftmax | kBarStFull)) {
        tma_store_4d(tm_o, stage, h * 64, wk.hq[s], wk.row0[s], wk.b);
        tma_store_commit();
        tma_store_wait_read0();
        mbar_arrive(token);
      }
    }
    ++o_cnt;
  }
}

__global__ void __launch_bounds__(kThreads16, 1)
attn_fwd_w16_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
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
    if (blockIdx.x == 0 && p.clock_stamps != nullptr) {
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
      mbar_init(&bars.o_empty[i], 8);   // 8 softmax warps of the stage
      mbar_init(&bars.l_full[i], 4);    // staging half 1 of stage i written
      mbar_init(&bars.st_full[i], 4);   // staging half 0 of stage i written
      mbar_init(&bars.l_empty[i], 1);   // token of staging half i
      if (i == 0) mbar_init(&bars.stg_empty[0], 1);
      mbar_init(&bars.sched_full[i], 1);
      mbar_init(&bars.sched_empty[i], kSchedConsumers16);
    }
    for (int i = 0; i < 8; ++i) mbar_init(bar_mem + (kNumBars - 8) + i, 2);  // exchange barriers: two warps each
    for (int i = 0; i < kKvSlots; ++i) {
      mbar_init(&bars.kv_full[i], 1);
      mbar_init(&bars.kv_empty[i], 1);
    }
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 16) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  if (warp == 17 && lane == 0) {
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    tma_prefetch_desc(&tm_o);
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  if (warp < 16) {
    reg_alloc<kRegsSoftmax16>();
    role_softmax16(p, bars, smem, sched_w, ctx, tmem, warp >> 3, (warp >> 2) & 1, (warp & 3) * 32 + lane, lane, &tm_o);
    tma_store_wait_all0();
  } else {
    reg_dealloc<kRegsOther16>();
    if (warp == 16) {
      role_mma(p, bars, smem, sched_w, ctx, tmem, lane);
    } else if (warp == 17) {
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
  if (warp == 16) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, 512);
  }
  if (tid == 0 && blockIdx.x == 0 && p.clock_stamps != nullptr) {
    p.clock_stamps[2] = static_cast<unsigned long long>(clock64());
    p.clock_stamps[3] = global_timer_ns();
  }
}

}  // namespace w16
}  // namespace attn

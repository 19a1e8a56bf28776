// LSE-weighted merge of two partial attention results over disjoint key sets (HBM-bound,
// elementwise): O = w1 O1 + w2 O2 with w_i = exp(LSE_i - LSE), LSE = log(exp(LSE1) + exp(LSE2)).
// One thread handles one 16-byte chunk (8 BF16) of a [B, Sq, Hq, 128] row per grid-stride step, so
// consecutive threads touch consecutive 16-byte chunks: fully coalesced 128-bit loads and stores.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace attn {

constexpr int kMergeThreads = 256;
constexpr int kChunksPerRow = 128 * 2 / 16;  // 16-byte chunks in a 128-element BF16 row

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
// A part whose weight is 0 (an empty part) contributes nothing whatever its O holds -- also NaN or
// Inf from a buffer nobody wrote: 0 * NaN would poison the row, so its term is dropped, not multiplied.
__device__ __forceinline__ uint32_t merge_pair(uint32_t a, uint32_t b, float w1, float w2) {
  const float ta_lo = w1 != 0.f ? w1 * bf16_lo(a) : 0.f, ta_hi = w1 != 0.f ? w1 * bf16_hi(a) : 0.f;
  const float lo = w2 != 0.f ? fmaf(w2, bf16_lo(b), ta_lo) : ta_lo;
  const float hi = w2 != 0.f ? fmaf(w2, bf16_hi(b), ta_hi) : ta_hi;
  uint32_t y;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(y) : "f"(hi), "f"(lo));
  return y;
}

constexpr int kMergeUnroll = 1;  // 16-byte chunks per thread and step (more in flight measured slower)

// o may be the same buffer as o1 or o2 (every thread reads its chunk of both parts before it writes
// that chunk of o, and no other thread touches it), so the three O pointers are neither restrict-
// qualified nor read through the non-coherent path.
__global__ void __launch_bounds__(kMergeThreads)
attn_merge_kernel(const uint4* o1, const float* __restrict__ lse1, const uint4* o2,
                  const float* __restrict__ lse2, uint4* o, float* __restrict__ lse, int Hq, int Sq,
                  long long n_chunks) {
  const long long stride = static_cast<long long>(gridDim.x) * kMergeThreads;
  for (long long c0 = static_cast<long long>(blockIdx.x) * kMergeThreads + threadIdx.x; c0 < n_chunks;
       c0 += stride * kMergeUnroll) {
    uint4 x[kMergeUnroll], y[kMergeUnroll];
    float a[kMergeUnroll], bb[kMergeUnroll];
    long long li[kMergeUnroll];
#pragma unroll
    for (int u = 0; u < kMergeUnroll; ++u) {  // all loads first: kMergeUnroll x 2 x 16 bytes in flight
      const long long c = c0 + u * stride;
      if (c < n_chunks) {
        const long long row = c / kChunksPerRow;  // (b * Sq + i) * Hq + h
        const int h = static_cast<int>(row % Hq);
        const long long t = row / Hq;
        const int i = static_cast<int>(t % Sq);
        const long long b = t / Sq;
        li[u] = (b * Hq + h) * Sq + i;  // LSE is [B, Hq, Sq]
        x[u] = o1[c];
        y[u] = o2[c];
        a[u] = __ldg(lse1 + li[u]);
        bb[u] = __ldg(lse2 + li[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < kMergeUnroll; ++u) {
      const long long c = c0 + u * stride;
      if (c < n_chunks) {
        const float m = fmaxf(a[u], bb[u]);
        float w1 = 0.f, w2 = 0.f, tot = -INFINITY;
        if (m != -INFINITY) {
          tot = m + logf(expf(a[u] - m) + expf(bb[u] - m));
          w1 = expf(a[u] - tot);
          w2 = expf(bb[u] - tot);
        }
        uint4 r;
        r.x = merge_pair(x[u].x, y[u].x, w1, w2);
        r.y = merge_pair(x[u].y, y[u].y, w1, w2);
        r.z = merge_pair(x[u].z, y[u].z, w1, w2);
        r.w = merge_pair(x[u].w, y[u].w, w1, w2);
        o[c] = r;
        if ((c % kChunksPerRow) == 0) lse[li[u]] = tot;
      }
    }
  }
}

// The same merge for n parts stored back to back: o_parts [n][B, Sq, Hq, 128] BF16, lse_parts
// [n][B, Hq, Sq] fp32.  LSE = log(sum_i exp(LSE_i)), O = sum_i exp(LSE_i - LSE) O_i, accumulated in
// fp32 and rounded once.  The n LSE values of a row are read by the 16 threads that share the row
// (same addresses: one transaction each).
__global__ void __launch_bounds__(kMergeThreads)
attn_merge_n_kernel(const uint4* __restrict__ o_parts, const float* __restrict__ lse_parts, int n,
                    uint4* __restrict__ o, float* __restrict__ lse, int Hq, int Sq, long long n_chunks,
                    long long n_rows) {
  const long long stride = static_cast<long long>(gridDim.x) * kMergeThreads;
  for (long long c = static_cast<long long>(blockIdx.x) * kMergeThreads + threadIdx.x; c < n_chunks; c += stride) {
    const long long row = c / kChunksPerRow;  // (b * Sq + i) * Hq + h
    const int h = static_cast<int>(row % Hq);
    const long long t = row / Hq;
    const int i = static_cast<int>(t % Sq);
    const long long b = t / Sq;
    const long long li = (b * Hq + h) * Sq + i;  // LSE is [B, Hq, Sq]
    float m = -INFINITY;
    for (int p = 0; p < n; ++p) m = fmaxf(m, __ldg(lse_parts + p * n_rows + li));
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    float tot = -INFINITY;
    if (m != -INFINITY) {
      float sum = 0.f;
      for (int p = 0; p < n; ++p) sum += expf(__ldg(lse_parts + p * n_rows + li) - m);
      tot = m + logf(sum);
      for (int p = 0; p < n; ++p) {
        const float w = expf(__ldg(lse_parts + p * n_rows + li) - tot);
        if (w == 0.f) continue;  // an empty part may hold anything, also NaN from an untouched buffer
        const uint4 x = __ldg(o_parts + p * n_chunks + c);
        acc[0] = fmaf(w, bf16_lo(x.x), acc[0]); acc[1] = fmaf(w, bf16_hi(x.x), acc[1]);
        acc[2] = fmaf(w, bf16_lo(x.y), acc[2]); acc[3] = fmaf(w, bf16_hi(x.y), acc[3]);
        acc[4] = fmaf(w, bf16_lo(x.z), acc[4]); acc[5] = fmaf(w, bf16_hi(x.z), acc[5]);
        acc[6] = fmaf(w, bf16_lo(x.w), acc[6]); acc[7] = fmaf(w, bf16_hi(x.w), acc[7]);
      }
    }
    uint4 r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r.x) : "f"(acc[1]), "f"(acc[0]));
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r.y) : "f"(acc[3]), "f"(acc[2]));
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r.z) : "f"(acc[5]), "f"(acc[4]));
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r.w) : "f"(acc[7]), "f"(acc[6]));
    o[c] = r;
    if (lse != nullptr && (c % kChunksPerRow) == 0) lse[li] = tot;
  }
}

}  // namespace attn

// Conformal kernels: rank / p-value, threshold + stage label, calibration sort + merge-insert.
// All results are integers or raw bit moves, so they are exact and reproducible.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace atts {

// ---------------------------------------------------------------------------------------------
// Ordering of scores.  Candidates are compared with calibration scores as floats (a tie counts,
// -0 == +0).  The calibration buffer itself is ordered by a monotone 32-bit key of the
// canonicalised value, in which every NaN is one pattern that sorts after +inf.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t canonical_bits(float x) {
  uint32_t u = __float_as_uint(x);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FC00000u;  // any NaN
  if (u == 0x80000000u) return 0u;                            // -0 -> +0
  return u;
}
__device__ __forceinline__ uint32_t key_of_bits(uint32_t u) {
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ uint32_t bits_of_key(uint32_t k) {
  return (k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k;
}

// ---------------------------------------------------------------------------------------------
// K3  rank + p-value (Eq. p-value): numer = 1 + #{calib >= s} = 1 + n - lower_bound(calib, s).
//
// lower_bound = number of leading entries with calib[i] < s.  With NaNs sorted last the predicate
// calib[i] < s is true on a prefix and false after it, NaNs included, so NaN calibration entries
// count as ">= s".  The search is two-level: a block first copies `ns` evenly spaced splitters
// sp[t] = calib[t << L] into shared memory, a thread finds the splitter interval there and
// finishes in the (L2-resident) buffer over at most 2^L entries.  With L == 0 the whole buffer is
// in shared memory and the second level is skipped.
// ---------------------------------------------------------------------------------------------
constexpr int kRankThreads = 256;
constexpr int kRankPerThread = 4;

__device__ __forceinline__ uint32_t rank_one(float s, const float* __restrict__ sp, int ns, int L,
                                             const float* __restrict__ calib, int n) {
  if (s != s) return 0u;  // NaN candidate: no score
  // t = number of splitters < s
  int lo = 0, len = ns;
  while (len > 0) {
    int half = len >> 1;
    bool less = sp[lo + half] < s;
    lo = less ? lo + half + 1 : lo;
    len = less ? len - half - 1 : half;
  }
  int below;
  if (L == 0) {
    below = lo;
  } else if (lo == 0) {
    below = 0;
  } else {
    // calib[(lo-1) << L] < s and (if it exists) calib[lo << L] >= s
    int a = ((lo - 1) << L) + 1;
    int b = min(lo << L, n);
    int len2 = b - a;
    while (len2 > 0) {
      int half = len2 >> 1;
      bool less = __ldg(calib + a + half) < s;
      a = less ? a + half + 1 : a;
      len2 = less ? len2 - half - 1 : half;
    }
    below = a;
  }
  return (uint32_t)(n - below) + 1u;
}

__global__ void __launch_bounds__(kRankThreads)
rank_kernel(const float* __restrict__ scores, int64_t Nc, const float* __restrict__ calib, int n,
            int ns, int L, uint32_t* __restrict__ numer, float* __restrict__ pvalue) {
  extern __shared__ float sp[];
  for (int t = threadIdx.x; t < ns; t += kRankThreads) sp[t] = __ldg(calib + ((int64_t)t << L));
  __syncthreads();
  const float denom = (float)(n + 1);
  const int64_t per_block = (int64_t)kRankThreads * kRankPerThread;
  for (int64_t base = (int64_t)blockIdx.x * per_block; base < Nc; base += (int64_t)gridDim.x * per_block) {
    int64_t j = base + (int64_t)threadIdx.x * kRankPerThread;
    if (j + kRankPerThread <= Nc) {
      float4 s4 = *reinterpret_cast<const float4*>(scores + j);
      uint4 r;
      r.x = rank_one(s4.x, sp, ns, L, calib, n);
      r.y = rank_one(s4.y, sp, ns, L, calib, n);
      r.z = rank_one(s4.z, sp, ns, L, calib, n);
      r.w = rank_one(s4.w, sp, ns, L, calib, n);
      *reinterpret_cast<uint4*>(numer + j) = r;
      if (pvalue) {
        const float qnan = __uint_as_float(0x7FC00000u);
        float4 p;
        p.x = r.x ? __fdiv_rn((float)r.x, denom) : qnan;
        p.y = r.y ? __fdiv_rn((float)r.y, denom) : qnan;
        p.z = r.z ? __fdiv_rn((float)r.z, denom) : qnan;
        p.w = r.w ? __fdiv_rn((float)r.w, denom) : qnan;
        *reinterpret_cast<float4*>(pvalue + j) = p;
      }
    } else {
      for (int e = 0; e < kRankPerThread && j + e < Nc; ++e) {
        uint32_t r = rank_one(scores[j + e], sp, ns, L, calib, n);
        numer[j + e] = r;
        if (pvalue) pvalue[j + e] = r ? __fdiv_rn((float)r, denom) : __uint_as_float(0x7FC00000u);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// K4  threshold + ordinal stage (accept iff p > alpha  <=>  numer > k_alpha).
// ---------------------------------------------------------------------------------------------
constexpr int kClassifyThreads = 256;
constexpr int kClassifyPerThread = 16;

__device__ __forceinline__ uint32_t stage_of(uint32_t numer, uint32_t k_alpha) {
  return numer == 0u ? 1u : (numer <= k_alpha ? 3u : 2u);
}

__global__ void __launch_bounds__(kClassifyThreads)
classify_kernel(const uint32_t* __restrict__ numer, int64_t Nc, uint32_t k_alpha,
                uint8_t* __restrict__ stage, uint32_t* __restrict__ counts) {
  uint32_t c1 = 0, c3 = 0, cnt = 0;
  const int64_t per_block = (int64_t)kClassifyThreads * kClassifyPerThread;
  for (int64_t base = (int64_t)blockIdx.x * per_block; base < Nc; base += (int64_t)gridDim.x * per_block) {
    int64_t j = base + (int64_t)threadIdx.x * kClassifyPerThread;
    if (j + kClassifyPerThread <= Nc) {
      uint32_t packed[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint4 v = *reinterpret_cast<const uint4*>(numer + j + 4 * q);
        uint32_t s0 = stage_of(v.x, k_alpha), s1 = stage_of(v.y, k_alpha);
        uint32_t s2 = stage_of(v.z, k_alpha), s3 = stage_of(v.w, k_alpha);
        c1 += (s0 == 1u) + (s1 == 1u) + (s2 == 1u) + (s3 == 1u);
        c3 += (s0 == 3u) + (s1 == 3u) + (s2 == 3u) + (s3 == 3u);
        packed[q] = s0 | (s1 << 8) | (s2 << 16) | (s3 << 24);
      }
      cnt += kClassifyPerThread;
      *reinterpret_cast<uint4*>(stage + j) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
    } else {
      for (int e = 0; e < kClassifyPerThread && j + e < Nc; ++e) {
        uint32_t s = stage_of(numer[j + e], k_alpha);
        c1 += (s == 1u);
        c3 += (s == 3u);
        cnt += 1;
        stage[j + e] = (uint8_t)s;
      }
    }
  }
  if (counts == nullptr) return;
  uint32_t c2 = cnt - c1 - c3;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    c1 += __shfl_xor_sync(0xFFFFFFFFu, c1, o);
    c2 += __shfl_xor_sync(0xFFFFFFFFu, c2, o);
    c3 += __shfl_xor_sync(0xFFFFFFFFu, c3, o);
  }
  __shared__ uint32_t sh[3][kClassifyThreads / 32];
  int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  if (l == 0) { sh[0][w] = c1; sh[1][w] = c2; sh[2][w] = c3; }
  __syncthreads();
  if (threadIdx.x < 3) {
    uint32_t t = 0;
    for (int i = 0; i < kClassifyThreads / 32; ++i) t += sh[threadIdx.x][i];
    if (t) atomicAdd(counts + threadIdx.x, t);
  }
}

// ---------------------------------------------------------------------------------------------
// K5  sort of the new calibration scores by all-pairs ranking.  One warp per element: its lanes
// stride over all k keys (held in shared memory) and count those that precede it; equal keys keep
// their input order, so every element gets its own slot.  k is at most kSortMaxK per launch.
// ---------------------------------------------------------------------------------------------
constexpr int kSortMaxK = 16384;
constexpr int kSortThreads = 256;

__global__ void __launch_bounds__(kSortThreads)
sort_new_kernel(const float* __restrict__ new_scores, int k, uint32_t* __restrict__ sorted_keys) {
  extern __shared__ uint32_t keys[];
  for (int t = threadIdx.x; t < k; t += kSortThreads) keys[t] = key_of_bits(canonical_bits(new_scores[t]));
  __syncthreads();
  const int warps = kSortThreads / 32;
  const int lane = threadIdx.x & 31;
  for (int j = blockIdx.x * warps + (threadIdx.x >> 5); j < k; j += gridDim.x * warps) {
    const uint32_t kj = keys[j];
    int cnt = 0;
    for (int i = lane; i < k; i += 32) {
      uint32_t ki = keys[i];
      cnt += (ki < kj) || (ki == kj && i < j);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xFFFFFFFFu, cnt, o);
    if (lane == 0) sorted_keys[cnt] = kj;
  }
}

// ---------------------------------------------------------------------------------------------
// K6  merge-insert.  Stable merge of the old buffer (n entries) with the sorted new keys (k):
//   old[i]  -> slot i + #{new <  old[i]}
//   new[j]  -> slot j + #{old <= new[j]}
// written to `out` (n + k entries).  The new keys sit in shared memory for the first search; the
// second searches the old buffer in global memory.
// ---------------------------------------------------------------------------------------------
constexpr int kMergeThreads = 512;

__global__ void __launch_bounds__(kMergeThreads)
merge_kernel(const float* __restrict__ old_buf, int n, const uint32_t* __restrict__ new_keys, int k,
             float* __restrict__ out) {
  extern __shared__ uint32_t nk[];
  for (int t = threadIdx.x; t < k; t += kMergeThreads) nk[t] = new_keys[t];
  __syncthreads();
  const int total = n + k;
  for (int e = blockIdx.x * kMergeThreads + threadIdx.x; e < total; e += gridDim.x * kMergeThreads) {
    if (e < n) {
      uint32_t bits = canonical_bits(old_buf[e]);
      uint32_t key = key_of_bits(bits);
      int lo = 0, len = k;  // number of new keys < key
      while (len > 0) {
        int half = len >> 1;
        bool less = nk[lo + half] < key;
        lo = less ? lo + half + 1 : lo;
        len = less ? len - half - 1 : half;
      }
      out[e + lo] = __uint_as_float(bits);
    } else {
      int j = e - n;
      uint32_t key = nk[j];
      int lo = 0, len = n;  // number of old keys <= key
      while (len > 0) {
        int half = len >> 1;
        bool le = key_of_bits(canonical_bits(__ldg(old_buf + lo + half))) <= key;
        lo = le ? lo + half + 1 : lo;
        len = le ? len - half - 1 : half;
      }
      out[j + lo] = __uint_as_float(bits_of_key(key));
    }
  }
}

}  // namespace atts

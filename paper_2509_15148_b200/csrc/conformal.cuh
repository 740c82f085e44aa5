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
// count as ">= s".  The search is two-level and branch-free.  A block first copies the splitters
// sp[t] = calib[t << L], t < ns, into a shared table laid out as an implicit search tree in
// breadth-first order (2^P - 1 nodes; node b at depth l holds the splitter of sorted rank
// (2q + 1) * 2^(P-1-l) - 1, q = b - 2^l; ranks >= ns hold NaN, which never compares "less").
// Descending it takes exactly P steps, and nodes of one depth are contiguous, so the lanes of a
// warp spread over the banks (a sorted table probed at rank +- step puts every lane in one bank).
// The leaf reached gives the number of splitters below the score; the entries below it among the
// 2^L - 1 buffer entries that follow the last such splitter are counted in exactly L steps of
// (L2-resident) global loads.  With L == 0 the table is the whole buffer.  A thread carries four
// scores through every step together, so their loads overlap.
// ---------------------------------------------------------------------------------------------
constexpr int kRankThreads = 1024;
constexpr int kRankPerThread = 4;
constexpr int kRankMaxTableLog2 = 13;  // table of at most 8191 splitters (32 KB)

// Descent of the breadth-first table, P levels, four scores at a time.  `off` is 4 * (node number): the node's
// value sits at byte off - 4, its children at 2 * off and 2 * off + 4.  Returns the leaf number = number of
// splitters below each score.
template <int P>
__device__ __forceinline__ void tree_descend(const float (&s)[4], const float* __restrict__ sp, int (&cnt)[4]) {
  uint32_t off[4] = {4u, 4u, 4u, 4u};
  const char* base = reinterpret_cast<const char*>(sp) - 4;
#pragma unroll
  for (int depth = 0; depth < P; ++depth) {
    float v[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = *reinterpret_cast<const float*>(base + off[e]);
#pragma unroll
    for (int e = 0; e < 4; ++e) off[e] = 2u * off[e] + ((v[e] < s[e]) ? 4u : 0u);
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) cnt[e] = (int)(off[e] >> 2) - (1 << P);
}

__device__ __forceinline__ void rank_four(const float (&s)[4], const float* __restrict__ sp, int P, int L,
                                          const float* __restrict__ calib, int n, bool vec8, uint32_t (&numer)[4]) {
  int cnt[4];
  switch (P) {  // the descent is unrolled for every table depth
    case 1: tree_descend<1>(s, sp, cnt); break;
    case 2: tree_descend<2>(s, sp, cnt); break;
    case 3: tree_descend<3>(s, sp, cnt); break;
    case 4: tree_descend<4>(s, sp, cnt); break;
    case 5: tree_descend<5>(s, sp, cnt); break;
    case 6: tree_descend<6>(s, sp, cnt); break;
    case 7: tree_descend<7>(s, sp, cnt); break;
    case 8: tree_descend<8>(s, sp, cnt); break;
    case 9: tree_descend<9>(s, sp, cnt); break;
    case 10: tree_descend<10>(s, sp, cnt); break;
    case 11: tree_descend<11>(s, sp, cnt); break;
    case 12: tree_descend<12>(s, sp, cnt); break;
    default: tree_descend<13>(s, sp, cnt); break;
  }
  int below[4];
  if (L == 0) {
#pragma unroll
    for (int e = 0; e < 4; ++e) below[e] = cnt[e];
  } else {
    // calib[(cnt-1) << L] < s and, if it exists, calib[cnt << L] >= s: the answer is base + (number of
    // entries below s among calib[base .. base + 2^L - 2]) with base = ((cnt-1) << L) + 1.
    int base[4], pos[4] = {0, 0, 0, 0};
#pragma unroll
    for (int e = 0; e < 4; ++e) base[e] = cnt[e] ? ((cnt[e] - 1) << L) + 1 : n;
    // With vec8 (L >= 3 and a 32-byte aligned buffer) the binary steps stop at windows of 7 entries; those
    // 7 and the entry before them are one aligned 32-byte group, fetched with a single 256-bit load.
    const int last_step = vec8 ? 8 : 1;
    for (int step = 1 << (L - 1); step >= last_step; step >>= 1) {
      float v[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int idx = base[e] + pos[e] + step - 1;
        v[e] = idx < n ? __ldg(calib + idx) : __uint_as_float(0x7FC00000u);
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) pos[e] += (v[e] < s[e]) ? step : 0;
    }
    if (vec8) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int g0 = base[e] + pos[e] - 1;  // multiple of 8; entries g0 + 1 .. g0 + 7 are the window
        int c = 0;
        if (cnt[e] != 0) {
          if (g0 + 8 <= n) {
            float w[8];
            asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                         : "=f"(w[0]), "=f"(w[1]), "=f"(w[2]), "=f"(w[3]), "=f"(w[4]), "=f"(w[5]), "=f"(w[6]), "=f"(w[7])
                         : "l"(calib + g0));
#pragma unroll
            for (int i = 1; i < 8; ++i) c += (w[i] < s[e]) ? 1 : 0;
          } else {
            for (int i = 1; i < 8 && g0 + i < n; ++i) c += (__ldg(calib + g0 + i) < s[e]) ? 1 : 0;
          }
        }
        pos[e] += c;
      }
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) below[e] = cnt[e] ? base[e] + pos[e] : 0;
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) numer[e] = (s[e] != s[e]) ? 0u : (uint32_t)(n - below[e]) + 1u;  // NaN: no score
}

// Stage of a sample (accept iff p > alpha  <=>  numer > k_alpha): 1 no score, 2 accepted, 3 target takes over.
__device__ __forceinline__ uint32_t stage_of(uint32_t numer, uint32_t k_alpha) {
  return numer == 0u ? 1u : (numer <= k_alpha ? 3u : 2u);
}

constexpr int kMaxAlphas = 4;
// Optional thresholding fused into the rank kernel: for each of NA rejection rates the stage bytes and the
// three stage counts, exactly what classify_kernel would produce from the numerators.
struct FusedClassify {
  uint32_t k_alpha[kMaxAlphas];
  uint8_t* stage[kMaxAlphas];
  uint32_t* counts;  // [NA][3] or nullptr
};

// Per-thread tallies of the fused thresholding, and the code both rank kernels share: writing the numerators,
// p-values and stage bytes of four candidates, and the block's contribution to the stage counts.
template <int NA>
struct StageTally {
  uint32_t c1[NA > 0 ? NA : 1] = {}, c3[NA > 0 ? NA : 1] = {}, seen = 0;
};

template <int NA>
__device__ __forceinline__ void emit_four(int64_t j, int64_t Nc, bool full, const uint32_t (&r)[4], const float (&p)[4],
                                          uint32_t* __restrict__ numer, float* __restrict__ pvalue,
                                          const FusedClassify& fc, StageTally<NA>& tally) {
  if (full) {
    *reinterpret_cast<uint4*>(numer + j) = make_uint4(r[0], r[1], r[2], r[3]);
    if (pvalue) *reinterpret_cast<float4*>(pvalue + j) = make_float4(p[0], p[1], p[2], p[3]);
  } else {
    for (int e = 0; e < 4 && j + e < Nc; ++e) {
      numer[j + e] = r[e];
      if (pvalue) pvalue[j + e] = p[e];
    }
  }
  if (NA > 0) {
    const int valid = full ? 4 : (int)(Nc - j);
    tally.seen += (uint32_t)valid;
#pragma unroll
    for (int a = 0; a < NA; ++a) {
      uint32_t st[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        st[e] = stage_of(r[e], fc.k_alpha[a]);
        tally.c1[a] += (e < valid) && (st[e] == 1u);
        tally.c3[a] += (e < valid) && (st[e] == 3u);
      }
      if (full) {
        *reinterpret_cast<uint32_t*>(fc.stage[a] + j) = st[0] | (st[1] << 8) | (st[2] << 16) | (st[3] << 24);
      } else {
        for (int e = 0; e < valid; ++e) fc.stage[a][j + e] = (uint8_t)st[e];
      }
    }
  }
}

// Adds the block's stage counts to fc.counts ([NA][3]); every thread of the block calls it.
template <int NA>
__device__ __forceinline__ void flush_tally(const FusedClassify& fc, const StageTally<NA>& tally) {
  if (NA == 0 || fc.counts == nullptr) return;
  __shared__ uint32_t sh[kMaxAlphas][3][kRankThreads / 32];
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
#pragma unroll
  for (int a = 0; a < NA; ++a) {
    uint32_t v1 = tally.c1[a], v3 = tally.c3[a], v2 = tally.seen - tally.c1[a] - tally.c3[a];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      v1 += __shfl_xor_sync(0xFFFFFFFFu, v1, o);
      v2 += __shfl_xor_sync(0xFFFFFFFFu, v2, o);
      v3 += __shfl_xor_sync(0xFFFFFFFFu, v3, o);
    }
    if (l == 0) { sh[a][0][w] = v1; sh[a][1][w] = v2; sh[a][2][w] = v3; }
  }
  __syncthreads();
  if ((int)threadIdx.x < NA * 3) {
    const int a = threadIdx.x / 3, i = threadIdx.x % 3;
    uint32_t t = 0;
    for (int q = 0; q < kRankThreads / 32; ++q) t += sh[a][i][q];
    if (t) atomicAdd(fc.counts + threadIdx.x, t);
  }
}

template <int NA>
__global__ void __launch_bounds__(kRankThreads)
rank_kernel(const float* __restrict__ scores, int64_t Nc, const float* __restrict__ calib, int n,
            int ns, int P, int L, uint32_t* __restrict__ numer, float* __restrict__ pvalue,
            const FusedClassify fc) {
  extern __shared__ float sp[];
  StageTally<NA> tally;
  const int slots = (1 << P) - 1;
  // With the whole buffer in the table (L == 0) the p-values of all n + 2 possible numerators are tabulated
  // behind it once per block (the same correctly rounded division), so a candidate costs one load, not a divide.
  float* const ptab = sp + slots;
  const bool tabulated = (L == 0) && pvalue != nullptr;
  if (tabulated)
    for (int t = threadIdx.x; t <= n + 1; t += kRankThreads)
      ptab[t] = t ? __fdiv_rn((float)t, (float)(n + 1)) : __uint_as_float(0x7FC00000u);
  for (int t = threadIdx.x; t < slots; t += kRankThreads) {
    const int b = t + 1;                       // node number
    const int depth = 31 - __clz(b);
    const int q = b - (1 << depth);
    const int rank = ((2 * q + 1) << (P - 1 - depth)) - 1;
    sp[t] = rank < ns ? __ldg(calib + ((int64_t)rank << L)) : __uint_as_float(0x7FC00000u);
  }
  __syncthreads();
  const float denom = (float)(n + 1);
  const float qnan = __uint_as_float(0x7FC00000u);
  const bool vec8 = L >= 3 && (reinterpret_cast<uintptr_t>(calib) & 31u) == 0;
  const int64_t per_block = (int64_t)kRankThreads * kRankPerThread;
  for (int64_t base = (int64_t)blockIdx.x * per_block; base < Nc; base += (int64_t)gridDim.x * per_block) {
    const int64_t j = base + (int64_t)threadIdx.x * kRankPerThread;
    if (j >= Nc) continue;
    float s[4];
    uint32_t r[4];
    const bool full = j + kRankPerThread <= Nc;
    if (full) {
      const float4 s4 = *reinterpret_cast<const float4*>(scores + j);
      s[0] = s4.x; s[1] = s4.y; s[2] = s4.z; s[3] = s4.w;
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) s[e] = (j + e < Nc) ? scores[j + e] : qnan;
    }
    rank_four(s, sp, P, L, calib, n, vec8, r);
    float p[4] = {qnan, qnan, qnan, qnan};
    if (tabulated) {
#pragma unroll
      for (int e = 0; e < 4; ++e) p[e] = ptab[r[e]];
    } else if (pvalue) {
#pragma unroll
      for (int e = 0; e < 4; ++e) p[e] = r[e] ? __fdiv_rn((float)r[e], denom) : qnan;
    }
    emit_four<NA>(j, Nc, full, r, p, numer, pvalue, fc, tally);
  }
  flush_tally<NA>(fc, tally);
}

// ---------------------------------------------------------------------------------------------
// K3, bucket form: many candidates against a buffer that fits in shared memory (n <= kBucketMaxN).
//
// A search tree costs a candidate log2(n) dependent shared-memory loads, which bounds the kernel by the
// shared-memory pipe and by instruction issue long before HBM.  Here a candidate is first mapped to one of B
// buckets of equal width in the monotone key space between the smallest and largest buffer entry
// (bucket = ((key - key_lo) * mul) >> 32, clamped: a non-decreasing function of the key, applied alike to
// candidates and buffer entries).  start[b] = number of buffer entries in buckets below b, so entries before
// start[bucket(s)] are below s, entries from start[bucket(s) + 1] on are not, and only the entries of the
// candidate's own bucket are compared with it.  With B >= 4n a bucket seldom holds more than one entry: the
// start word carries min(entries in the bucket, 3) in its top bits; a candidate reads nothing from an empty
// bucket, one or two entries otherwise, and only in a bucket of three or more does it search the rest of the
// bucket.  Any distribution is handled exactly; a clustered one merely sends more candidates to that search.
// ---------------------------------------------------------------------------------------------
constexpr int kBucketMaxN = 8191;
constexpr int kBucketMaxLog2 = 15;   // at most 32768 buckets (128 KB)
constexpr int kBucketPad = 2;        // NaN entries behind the buffer copy (no probe can leave the array)
constexpr int64_t kBucketMinCandidates = 1 << 16;

struct BucketMap {
  uint32_t key_lo, mul, last;  // last = B - 1
};
// Buffer entries are canonicalised first (no -0, one NaN pattern that has the largest key).  Candidates are not:
// the key of -0 is the one just below that of +0, so a -0 candidate lands in the bucket of +0 or in the one
// before it, and in both cases exactly the entries below zero precede its bucket's entries that are not.
__device__ __forceinline__ uint32_t bucket_of(float value, const BucketMap& m) {
  const uint32_t u = __float_as_uint(value);
  const uint32_t key = u ^ ((uint32_t)((int32_t)u >> 31) | 0x80000000u);
  const uint32_t x = max(key, m.key_lo) - m.key_lo;
  return min(__umulhi(x, m.mul), m.last);
}

template <int NA>
__global__ void __launch_bounds__(kRankThreads, 1)
rank_bucket_kernel(const float* __restrict__ scores, int64_t Nc, const float* __restrict__ calib, int n, int Blog2,
                   uint32_t* __restrict__ numer, float* __restrict__ pvalue, const FusedClassify fc) {
  extern __shared__ uint32_t bsm[];
  const int B = 1 << Blog2;
  uint32_t* const start = bsm;                                         // [B + 1]
  float* const buf = reinterpret_cast<float*>(bsm + B + 1);           // [n + kBucketPad]
  float* const ptab = buf + n + kBucketPad;                            // [n + 2]
  __shared__ BucketMap map_sh;
  __shared__ uint32_t warp_max[kRankThreads / 32];
  const float qnan = __uint_as_float(0x7FC00000u);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  for (int t = threadIdx.x; t <= B; t += kRankThreads) start[t] = t == B ? (uint32_t)n : 0u;
  for (int t = threadIdx.x; t < n + kBucketPad; t += kRankThreads)
    buf[t] = t < n ? __uint_as_float(canonical_bits(__ldg(calib + t))) : qnan;
  if (pvalue)
    for (int t = threadIdx.x; t <= n + 1; t += kRankThreads)
      ptab[t] = t ? __fdiv_rn((float)t, (float)(n + 1)) : qnan;
  if (threadIdx.x == 0) {
    const uint32_t lo = key_of_bits(canonical_bits(__ldg(calib)));
    const uint32_t hi = key_of_bits(canonical_bits(__ldg(calib + n - 1)));
    const unsigned long long range = hi >= lo ? (unsigned long long)(hi - lo) + 1ull : 1ull;
    const unsigned long long mul = ((unsigned long long)B << 32) / range;
    map_sh.key_lo = lo;
    map_sh.mul = mul > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)mul;
    map_sh.last = (uint32_t)(B - 1);
  }
  __syncthreads();
  const BucketMap map = map_sh;
  // start[b + 1] <- 1 + (largest index of an entry in bucket b); a running maximum then gives every start[b].
  for (int t = threadIdx.x; t < n; t += kRankThreads) atomicMax(&start[bucket_of(buf[t], map) + 1u], (uint32_t)t + 1u);
  __syncthreads();
  {
    // warp w owns start[w * seg .. (w + 1) * seg), seg = B / 32, read 32 consecutive words at a time
    const int seg = B >> 5;
    uint32_t* const mine = start + warp * seg;
    uint32_t m = 0;
    for (int i = lane; i < seg; i += 32) m = max(m, mine[i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if (lane == 0) warp_max[warp] = m;
    __syncthreads();
    uint32_t carry = 0;
    for (int w = 0; w < warp; ++w) carry = max(carry, warp_max[w]);
    for (int i = 0; i < seg; i += 32) {
      uint32_t v = (i + lane < seg) ? mine[i + lane] : 0u;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, v, o);
        if (lane >= o) v = max(v, up);
      }
      v = max(v, carry);
      if (i + lane < seg) mine[i + lane] = v;
      carry = __shfl_sync(0xFFFFFFFFu, v, 31);
    }
  }
  __syncthreads();
  {
    // bits 31:30 of a start word: min(entries in the bucket, 3)
    uint64_t cls = 0;
    for (int i = 0, b = threadIdx.x; b < B; ++i, b += kRankThreads) {
      const uint32_t cnt = start[b + 1] - start[b];
      cls |= (uint64_t)(cnt < 3u ? cnt : 3u) << (2 * i);
    }
    __syncthreads();
    for (int i = 0, b = threadIdx.x; b < B; ++i, b += kRankThreads) start[b] |= (uint32_t)((cls >> (2 * i)) & 3u) << 30;
  }
  __syncthreads();

  StageTally<NA> tally;
  const int64_t per_block = (int64_t)kRankThreads * kRankPerThread;
  const int64_t stride = (int64_t)gridDim.x * per_block;
  int64_t j = (int64_t)blockIdx.x * per_block + (int64_t)threadIdx.x * kRankPerThread;
  float4 nxt = make_float4(qnan, qnan, qnan, qnan);
  if (j + 4 <= Nc) nxt = *reinterpret_cast<const float4*>(scores + j);
  for (; j < Nc; j += stride) {
    float s[4] = {nxt.x, nxt.y, nxt.z, nxt.w};
    const bool full = j + kRankPerThread <= Nc;
    if (!full) {
#pragma unroll
      for (int e = 0; e < 4; ++e) s[e] = (j + e < Nc) ? scores[j + e] : qnan;
    }
    if (j + stride + 4 <= Nc) nxt = *reinterpret_cast<const float4*>(scores + j + stride);  // next round's scores
    uint32_t word[4], below[4];
    float p0[4] = {qnan, qnan, qnan, qnan}, p1[4] = {qnan, qnan, qnan, qnan};
#pragma unroll
    for (int e = 0; e < 4; ++e) word[e] = start[bucket_of(s[e], map)];
    // Most buckets are empty: lanes whose bucket is read nothing, which also spares shared-memory bank conflicts.
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (word[e] >= (1u << 30)) p0[e] = buf[word[e] & 0x3FFFFFFFu];
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (word[e] >= (2u << 30)) p1[e] = buf[(word[e] & 0x3FFFFFFFu) + 1u];
#pragma unroll
    for (int e = 0; e < 4; ++e)
      below[e] = (word[e] & 0x3FFFFFFFu) + (p0[e] < s[e] ? 1u : 0u) + (p1[e] < s[e] ? 1u : 0u);
    if (max(max(word[0], word[1]), max(word[2], word[3])) >= (3u << 30)) {
      // a bucket of three or more: if its first two entries are below the score, lower bound among the rest of it
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if (word[e] >= (3u << 30) && p1[e] < s[e]) {
          int lo = (int)(word[e] & 0x3FFFFFFFu) + 2;
          int len = (int)(start[bucket_of(s[e], map) + 1u] & 0x3FFFFFFFu) - lo;
          while (len > 0) {
            const int half = len >> 1;
            const bool less = buf[lo + half] < s[e];
            lo = less ? lo + half + 1 : lo;
            len = less ? len - half - 1 : half;
          }
          below[e] = (uint32_t)lo;
        }
      }
    }
    uint32_t r[4];
    float p[4] = {qnan, qnan, qnan, qnan};
#pragma unroll
    for (int e = 0; e < 4; ++e) r[e] = (s[e] != s[e]) ? 0u : (uint32_t)n - below[e] + 1u;  // NaN: no score
    if (pvalue) {
#pragma unroll
      for (int e = 0; e < 4; ++e) p[e] = ptab[r[e]];
    }
    emit_four<NA>(j, Nc, full, r, p, numer, pvalue, fc, tally);
  }
  flush_tally<NA>(fc, tally);
}

// ---------------------------------------------------------------------------------------------
// K3, indexed form: many candidates against a buffer too large for shared memory.
//
// The plain kernel pays, per block, one strided load for each of up to 8191 splitters, and per candidate up to
// three dependent 4-byte loads plus one 32-byte load from the L2-resident buffer; divergent loads are served at
// one per cycle per SM, so they are what bounds it.  An index kept beside the buffer (rebuilt whenever the
// buffer changes, in the pass that writes the buffer anyway) removes most of them:
//   aux[i]  = calib[8 i + 7], the last entry of every aligned group of 8 (NaN where that lies beyond n);
//   tree    = the entries aux[8 r + 7] = calib[64 r + 63], r < ns = n / 64 + 1 (the last one always NaN), as an
//             implicit search tree in breadth-first order, ready to be copied into shared memory row by row.
// A candidate descends the tree (P shared-memory steps) to its group of 64, reads that group's 8 aux entries
// in one 32-byte load to find its group of 8, and reads that group in a second 32-byte load.
// Layout of the index (32-bit words): [0] n  [1] P  [2] ns  [3..7] 0  [8 ..) tree, kIndexTreeWords  [..) aux, 8 ns.
// ---------------------------------------------------------------------------------------------
constexpr int kIndexHeaderWords = 8;
constexpr int kIndexTreeWords = 1 << kRankMaxTableLog2;               // 8191 nodes + 1 pad
constexpr int64_t kIndexMaxN = 64ll * ((1 << kRankMaxTableLog2) - 1) - 1;   // ns = n / 64 + 1 <= 8191
constexpr int64_t kIndexMinCandidates = 1 << 14;

// Slot, in the breadth-first table of a P-level tree, of the splitter with sorted rank r (inverse of the fill rule
// of rank_kernel: node b at depth l holds rank (2q + 1) * 2^(P-1-l) - 1, q = b - 2^l).
__device__ __forceinline__ int index_slot_of_rank(int r, int P) {
  const int x = r + 1;
  const int tz = __ffs(x) - 1;
  const int depth = P - 1 - tz;
  return (1 << depth) + (x >> (tz + 1)) - 1;
}

// Writes the index of src[0, n); with COPY also dst[e] = src[e] (the copy-back of a merge), so a calibration
// update rebuilds the index in the pass that moves the merged buffer anyway.
template <bool COPY>
__global__ void __launch_bounds__(256)
index_build_kernel(const float* __restrict__ src, float* __restrict__ dst, int n, int P, int ns,
                   uint32_t* __restrict__ index) {
  float* const tree = reinterpret_cast<float*>(index + kIndexHeaderWords);
  float* const aux = tree + kIndexTreeWords;
  const float qnan = __uint_as_float(0x7FC00000u);
  const int tid = blockIdx.x * blockDim.x + threadIdx.x, nthreads = gridDim.x * blockDim.x;
  if (tid < kIndexHeaderWords) index[tid] = tid == 0 ? (uint32_t)n : tid == 1 ? (uint32_t)P : tid == 2 ? (uint32_t)ns : 0u;
  for (int e = tid; e < n; e += nthreads) {
    const float v = src[e];
    if (COPY) dst[e] = v;
    if ((e & 7) == 7) aux[e >> 3] = v;
    if ((e & 63) == 63) tree[index_slot_of_rank(e >> 6, P)] = v;
  }
  for (int i = (n >> 3) + tid; i < 8 * ns; i += nthreads) aux[i] = qnan;             // groups of 8 that end beyond n
  for (int r = (n >> 6) + tid; r < (1 << P) - 1; r += nthreads) tree[index_slot_of_rank(r, P)] = qnan;
}

template <int P>
__device__ __forceinline__ void rank_four_indexed(const float (&s)[4], const float* __restrict__ sp,
                                                  const float* __restrict__ aux, const float* __restrict__ calib, int n,
                                                  uint32_t (&numer)[4]) {
  int g[4];
  tree_descend<P>(s, sp, g);   // number of groups of 64 that lie entirely below the score
  float w[4][8];
#pragma unroll
  for (int e = 0; e < 4; ++e)
    asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(w[e][0]), "=f"(w[e][1]), "=f"(w[e][2]), "=f"(w[e][3]), "=f"(w[e][4]), "=f"(w[e][5]), "=f"(w[e][6]), "=f"(w[e][7])
                 : "l"(aux + 8 * g[e]));
  int h[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    int c = 0;
#pragma unroll
    for (int i = 0; i < 7; ++i) c += (w[e][i] < s[e]) ? 1 : 0;   // the eighth is the group's splitter: not below
    h[e] = 8 * g[e] + c;                                         // groups of 8 that lie entirely below the score
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    // the last group may be cut short by n: its 32 bytes are still inside the 32-byte aligned span only if whole
    if (8 * h[e] + 8 <= n) {
      asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                   : "=f"(w[e][0]), "=f"(w[e][1]), "=f"(w[e][2]), "=f"(w[e][3]), "=f"(w[e][4]), "=f"(w[e][5]), "=f"(w[e][6]), "=f"(w[e][7])
                   : "l"(calib + 8 * h[e]));
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) w[e][i] = (8 * h[e] + i < n) ? __ldg(calib + 8 * h[e] + i) : __uint_as_float(0x7FC00000u);
    }
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    int c = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) c += (w[e][i] < s[e]) ? 1 : 0;
    const int below = 8 * h[e] + c;
    numer[e] = (s[e] != s[e]) ? 0u : (uint32_t)(n - below) + 1u;   // NaN: no score
  }
}

template <int NA>
__global__ void __launch_bounds__(kRankThreads)
rank_indexed_kernel(const float* __restrict__ scores, int64_t Nc, const float* __restrict__ calib, int n, int P,
                    const uint32_t* __restrict__ index, uint32_t* __restrict__ numer, float* __restrict__ pvalue,
                    const FusedClassify fc, unsigned int* __restrict__ dev_status) {
  extern __shared__ float sp[];
  // an index built for another fill of the buffer would give wrong ranks silently: refuse it
  if (__ldg(index) != (uint32_t)n || __ldg(index + 1) != (uint32_t)P) {
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(dev_status, 8u);
    return;
  }
  const float* const tree = reinterpret_cast<const float*>(index + kIndexHeaderWords);
  const float* const aux = tree + kIndexTreeWords;
  for (int t = threadIdx.x; t < (1 << P) - 1; t += kRankThreads) sp[t] = __ldg(tree + t);
  __syncthreads();
  StageTally<NA> tally;
  const float denom = (float)(n + 1);
  const float qnan = __uint_as_float(0x7FC00000u);
  const int64_t per_block = (int64_t)kRankThreads * kRankPerThread;
  for (int64_t base = (int64_t)blockIdx.x * per_block; base < Nc; base += (int64_t)gridDim.x * per_block) {
    const int64_t j = base + (int64_t)threadIdx.x * kRankPerThread;
    if (j >= Nc) continue;
    float s[4];
    uint32_t r[4];
    const bool full = j + kRankPerThread <= Nc;
    if (full) {
      const float4 s4 = *reinterpret_cast<const float4*>(scores + j);
      s[0] = s4.x; s[1] = s4.y; s[2] = s4.z; s[3] = s4.w;
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) s[e] = (j + e < Nc) ? scores[j + e] : qnan;
    }
    switch (P) {
      case 1: rank_four_indexed<1>(s, sp, aux, calib, n, r); break;
      case 2: rank_four_indexed<2>(s, sp, aux, calib, n, r); break;
      case 3: rank_four_indexed<3>(s, sp, aux, calib, n, r); break;
      case 4: rank_four_indexed<4>(s, sp, aux, calib, n, r); break;
      case 5: rank_four_indexed<5>(s, sp, aux, calib, n, r); break;
      case 6: rank_four_indexed<6>(s, sp, aux, calib, n, r); break;
      case 7: rank_four_indexed<7>(s, sp, aux, calib, n, r); break;
      case 8: rank_four_indexed<8>(s, sp, aux, calib, n, r); break;
      case 9: rank_four_indexed<9>(s, sp, aux, calib, n, r); break;
      case 10: rank_four_indexed<10>(s, sp, aux, calib, n, r); break;
      case 11: rank_four_indexed<11>(s, sp, aux, calib, n, r); break;
      case 12: rank_four_indexed<12>(s, sp, aux, calib, n, r); break;
      default: rank_four_indexed<13>(s, sp, aux, calib, n, r); break;
    }
    float p[4] = {qnan, qnan, qnan, qnan};
    if (pvalue) {
#pragma unroll
      for (int e = 0; e < 4; ++e) p[e] = r[e] ? __fdiv_rn((float)r[e], denom) : qnan;
    }
    emit_four<NA>(j, Nc, full, r, p, numer, pvalue, fc, tally);
  }
  flush_tally<NA>(fc, tally);
}

// ---------------------------------------------------------------------------------------------
// K4  threshold + ordinal stage (accept iff p > alpha  <=>  numer > k_alpha).
// ---------------------------------------------------------------------------------------------
constexpr int kClassifyThreads = 256;
constexpr int kClassifyPerThread = 16;

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
// K5  sort of the new calibration scores by all-pairs ranking, spread over the whole GPU.  Every block
// holds all k keys in shared memory (padded to a multiple of 128 with a key above every canonical key).
// The slot of key j is the number of keys that sort before it: smaller keys, and equal keys that come earlier
// in the input - one comparison per pair, key_i < key_j + (i < j).  A warp ranks four consecutive keys at a
// time, so a 128-bit load of four other keys serves sixteen comparisons; those four others all come before or
// all come after the warp's four, except in the one group that holds them.  k is at most kSortMaxK per launch.
// ---------------------------------------------------------------------------------------------
constexpr int kSortMaxK = 16384;
constexpr int kSortThreads = 256;
constexpr int kSortKeysPerBlock = (kSortThreads / 32) * 4;

__global__ void __launch_bounds__(kSortThreads)
sort_new_kernel(const float* __restrict__ new_scores, int k, uint32_t* __restrict__ sorted_keys) {
  extern __shared__ __align__(16) uint32_t keys[];
  const int kpad = (k + 127) & ~127;
#pragma unroll 8
  for (int t = threadIdx.x; t < kpad; t += kSortThreads)
    keys[t] = t < k ? key_of_bits(canonical_bits(__ldg(new_scores + t))) : 0xFFFFFFFFu;
  __syncthreads();
  const int warps = kSortThreads / 32;
  const int lane = threadIdx.x & 31;
  for (int j0 = (blockIdx.x * warps + (threadIdx.x >> 5)) * 4; j0 < k; j0 += gridDim.x * warps * 4) {
    const uint4 mine = *reinterpret_cast<const uint4*>(keys + j0);   // keys j0 .. j0 + 3 (padding beyond k)
    const uint32_t kj[4] = {mine.x, mine.y, mine.z, mine.w};
    int cnt[4] = {0, 0, 0, 0};
    for (int i = lane * 4; i < kpad; i += 128) {
      const uint4 q = *reinterpret_cast<const uint4*>(keys + i);
      if (i != j0) {
        const uint32_t earlier = i < j0 ? 1u : 0u;   // canonical keys stay below 0xFFC00001: no overflow
#pragma unroll
        for (int y = 0; y < 4; ++y) {
          const uint32_t t = kj[y] + earlier;
          cnt[y] += (q.x < t) + (q.y < t) + (q.z < t) + (q.w < t);
        }
      } else {
        const uint32_t qv[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int y = 0; y < 4; ++y)
#pragma unroll
          for (int x = 0; x < 4; ++x) cnt[y] += qv[x] < kj[y] + (x < y ? 1u : 0u);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
      for (int y = 0; y < 4; ++y) cnt[y] += __shfl_xor_sync(0xFFFFFFFFu, cnt[y], o);
    if (lane < 4 && j0 + lane < k) {
      const int slot = lane == 0 ? cnt[0] : lane == 1 ? cnt[1] : lane == 2 ? cnt[2] : cnt[3];
      sorted_keys[slot] = keys[j0 + lane];
    }
  }
}

// ---------------------------------------------------------------------------------------------
// K6  merge-insert.  Stable merge of the old buffer (n entries) with the sorted new keys (k):
//   old[i]  -> slot i + #{new <  old[i]}
//   new[j]  -> slot j + #{old <= new[j]}
// written to `out` (n + k entries).  The new keys sit in shared memory for the first search; the
// second searches the old buffer in global memory, 32 probes at a time.
// ---------------------------------------------------------------------------------------------
constexpr int kMergeThreads = 512;

__global__ void __launch_bounds__(kMergeThreads)
merge_kernel(const float* __restrict__ old_buf, int n, const uint32_t* __restrict__ new_keys, int k,
             float* __restrict__ out) {
  extern __shared__ uint32_t nk[];
#pragma unroll 8
  for (int t = threadIdx.x; t < k; t += kMergeThreads) nk[t] = __ldg(new_keys + t);
  __syncthreads();
  // New keys first, one warp each: a 32-way search of the old buffer (every lane probes one of 32 evenly spaced
  // entries, a ballot keeps the interval between the last "<=" and the first ">"), so the chain of dependent
  // loads is log32(n) long instead of log2(n) and overlaps the bulk work below.
  const int lane = threadIdx.x & 31;
  const int warps_per_block = kMergeThreads / 32;
  for (int j = blockIdx.x * warps_per_block + (threadIdx.x >> 5); j < k; j += gridDim.x * warps_per_block) {
    const uint32_t key = nk[j];
    int lo = 0, hi = n;  // the number of old keys <= key lies in [lo, hi]
    while (hi > lo) {
      const int width = hi - lo;
      const int p = width >= 32 ? lo + (int)(((long long)width * (lane + 1)) >> 5) - 1 : lo + lane;
      const bool le = p < hi && key_of_bits(canonical_bits(__ldg(old_buf + p))) <= key;
      const int c = __popc(__ballot_sync(0xFFFFFFFFu, le));  // the predicate is true on a prefix of the lanes
      const int p_prev = __shfl_sync(0xFFFFFFFFu, p, c > 0 ? c - 1 : 0);
      const int p_next = __shfl_sync(0xFFFFFFFFu, p, c < 32 ? c : 31);
      const int probes = width >= 32 ? 32 : width;
      if (c > 0) lo = p_prev + 1;
      if (c < probes) hi = p_next;
    }
    if (lane == 0) out[j + lo] = __uint_as_float(bits_of_key(key));
  }
  // Old entries: each searches the sorted new keys in shared memory.
  for (int e = blockIdx.x * kMergeThreads + threadIdx.x; e < n; e += gridDim.x * kMergeThreads) {
    const uint32_t bits = canonical_bits(old_buf[e]);
    const uint32_t key = key_of_bits(bits);
    int lo = 0, len = k;  // number of new keys < key
    while (len > 0) {
      const int half = len >> 1;
      const bool less = nk[lo + half] < key;
      lo = less ? lo + half + 1 : lo;
      len = less ? len - half - 1 : half;
    }
    out[e + lo] = __uint_as_float(bits);
  }
}

// ---------------------------------------------------------------------------------------------
// Threshold form of the acceptance rule: tau = the k_alpha-th largest calibration score, and a sample is
// rejected iff s > tau (identical to numer <= k_alpha, ties included).  One comparison per sample.
// ---------------------------------------------------------------------------------------------
__global__ void threshold_kernel(const float* __restrict__ calib, int n, int k_alpha, float* __restrict__ tau) {
  if (threadIdx.x == 0 && blockIdx.x == 0) *tau = k_alpha >= 1 ? calib[n - k_alpha] : __uint_as_float(0x7F800000u);
}

__global__ void __launch_bounds__(kClassifyThreads)
classify_threshold_kernel(const float* __restrict__ scores, int64_t Nc, const float* __restrict__ tau_ptr,
                          uint8_t* __restrict__ stage, uint32_t* __restrict__ counts) {
  const float tau = __ldg(tau_ptr);
  uint32_t c1 = 0, c3 = 0, cnt = 0;
  auto st_of = [&](float s) { return s != s ? 1u : (s > tau ? 3u : 2u); };
  const int64_t per_block = (int64_t)kClassifyThreads * kClassifyPerThread;
  for (int64_t base = (int64_t)blockIdx.x * per_block; base < Nc; base += (int64_t)gridDim.x * per_block) {
    const int64_t j = base + (int64_t)threadIdx.x * kClassifyPerThread;
    if (j + kClassifyPerThread <= Nc) {
      uint32_t packed[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float4 v = *reinterpret_cast<const float4*>(scores + j + 4 * q);
        const uint32_t s0 = st_of(v.x), s1 = st_of(v.y), s2 = st_of(v.z), s3 = st_of(v.w);
        c1 += (s0 == 1u) + (s1 == 1u) + (s2 == 1u) + (s3 == 1u);
        c3 += (s0 == 3u) + (s1 == 3u) + (s2 == 3u) + (s3 == 3u);
        packed[q] = s0 | (s1 << 8) | (s2 << 16) | (s3 << 24);
      }
      cnt += kClassifyPerThread;
      *reinterpret_cast<uint4*>(stage + j) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
    } else {
      for (int e = 0; e < kClassifyPerThread && j + e < Nc; ++e) {
        const uint32_t s = st_of(scores[j + e]);
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
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  if (l == 0) { sh[0][w] = c1; sh[1][w] = c2; sh[2][w] = c3; }
  __syncthreads();
  if (threadIdx.x < 3) {
    uint32_t t = 0;
    for (int i = 0; i < kClassifyThreads / 32; ++i) t += sh[threadIdx.x][i];
    if (t) atomicAdd(counts + threadIdx.x, t);
  }
}

// ---------------------------------------------------------------------------------------------
// Budget report: the positions of the samples in stage 3 (the target takes over), in input order, and their
// number B.  Stream compaction in three launches: stage-3 count per tile of kIdsTile bytes; exclusive scan of the
// tile counts by one block (which also writes B); every tile then recounts its bytes, 64 per thread, and writes
// its positions from its offset on.  Everything is integer work in a fixed order: the result is unique.
// ---------------------------------------------------------------------------------------------
constexpr int kIdsThreads = 256;
constexpr int kIdsPerThread = 64;
constexpr int kIdsTile = kIdsThreads * kIdsPerThread;   // 16384 stage bytes per block

// Bit i of the result is set where byte i of the thread's 64 stage bytes is 3.
__device__ __forceinline__ uint64_t stage3_mask(const uint8_t* __restrict__ stage, int64_t j, int64_t Nc, bool vec) {
  uint64_t mask = 0;
  if (vec && j + kIdsPerThread <= Nc) {
    uint4 q[4];
#pragma unroll
    for (int v = 0; v < 4; ++v) q[v] = *reinterpret_cast<const uint4*>(stage + j + 16 * v);
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const uint32_t w[4] = {q[v].x, q[v].y, q[v].z, q[v].w};
      uint32_t m16 = 0;
#pragma unroll
      for (int i = 0; i < 16; ++i) m16 |= (((w[i >> 2] >> (8 * (i & 3))) & 0xFFu) == 3u ? 1u : 0u) << i;
      mask |= (uint64_t)m16 << (16 * v);
    }
  } else {
    for (int i = 0; i < kIdsPerThread && j + i < Nc; ++i) mask |= (uint64_t)(stage[j + i] == 3 ? 1u : 0u) << i;
  }
  return mask;
}

// Exclusive prefix sum of one value per thread over a block of kIdsThreads; *total gets the block's sum.
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* total) {
  __shared__ uint32_t warp_sum[kIdsThreads / 32];
  __shared__ uint32_t block_sum;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += up;
  }
  if (lane == 31) warp_sum[warp] = incl;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t run = 0;
    for (int w = 0; w < kIdsThreads / 32; ++w) {
      const uint32_t t = warp_sum[w];
      warp_sum[w] = run;
      run += t;
    }
    block_sum = run;
  }
  __syncthreads();
  const uint32_t excl = warp_sum[warp] + incl - v;
  *total = block_sum;
  __syncthreads();   // the shared words may be reused by the next call
  return excl;
}

__global__ void __launch_bounds__(kIdsThreads)
takeover_count_kernel(const uint8_t* __restrict__ stage, int64_t Nc, bool vec, uint32_t* __restrict__ tile_count) {
  const int64_t j = (int64_t)blockIdx.x * kIdsTile + (int64_t)threadIdx.x * kIdsPerThread;
  uint32_t c = j < Nc ? (uint32_t)__popcll(stage3_mask(stage, j, Nc, vec)) : 0u;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, o);
  __shared__ uint32_t sh[kIdsThreads / 32];
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = c;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t t = 0;
    for (int w = 0; w < kIdsThreads / 32; ++w) t += sh[w];
    tile_count[blockIdx.x] = t;
  }
}

// One block: tile_count[t] <- sum of the counts of the tiles before t; *count <- the sum of all (may be nullptr).
__global__ void __launch_bounds__(kIdsThreads)
takeover_scan_kernel(uint32_t* __restrict__ tile_count, int tiles, uint32_t* __restrict__ count) {
  uint32_t carry = 0;
  for (int base = 0; base < tiles; base += kIdsThreads) {
    const int t = base + threadIdx.x;
    const uint32_t v = t < tiles ? tile_count[t] : 0u;
    uint32_t total;
    const uint32_t excl = block_exclusive_scan(v, &total);
    if (t < tiles) tile_count[t] = carry + excl;
    carry += total;
  }
  if (threadIdx.x == 0 && count != nullptr) *count = carry;
}

__global__ void __launch_bounds__(kIdsThreads)
takeover_write_kernel(const uint8_t* __restrict__ stage, int64_t Nc, bool vec, const uint32_t* __restrict__ tile_offset,
                      int32_t* __restrict__ ids, int64_t ids_cap) {
  const int64_t j = (int64_t)blockIdx.x * kIdsTile + (int64_t)threadIdx.x * kIdsPerThread;
  const uint64_t mask = j < Nc ? stage3_mask(stage, j, Nc, vec) : 0ull;
  uint32_t total;
  const uint32_t excl = block_exclusive_scan((uint32_t)__popcll(mask), &total);
  int64_t pos = (int64_t)tile_offset[blockIdx.x] + excl;
  for (uint64_t m = mask; m != 0ull; m &= m - 1ull) {
    if (pos < ids_cap) ids[pos] = (int32_t)(j + (__ffsll((long long)m) - 1));
    ++pos;
  }
}

// ---------------------------------------------------------------------------------------------
// Conditional coverage (Proposition 2): a candidate is ranked against the calibration scores of its own
// input only.  The per-input buffers are ascending segments of one array; segments are short (the m samples
// of one input), so a thread searches its segment directly in (L2-resident) global memory.
//   numer = 1 + #{own segment >= s},  denom = |segment| + 1,  p = numer / denom;  reject iff
//   1 <= numer <= floor(alpha * denom)  (evaluated in IEEE double, as on the host for the marginal form).
// ---------------------------------------------------------------------------------------------
constexpr int kCondStage = 512;   // calibration entries a warp can stage in shared memory (2 KB)

// Lower bound of four scores in their own segments [lo, lo + len), advanced together so that the dependent loads
// overlap; `data` is indexed by the same positions as the segments (shared or global memory).
template <bool GLOBAL>
__device__ __forceinline__ void lower_bound_four(const float* data, const float (&s)[4], int (&lo)[4], int (&len)[4]) {
  const float qnan = __uint_as_float(0x7FC00000u);
  while (max(max(len[0], len[1]), max(len[2], len[3])) > 0) {
    float v[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = len[e] > 0 ? (GLOBAL ? __ldg(data + lo[e] + (len[e] >> 1)) : data[lo[e] + (len[e] >> 1)]) : qnan;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (len[e] > 0) {
        const int half = len[e] >> 1;
        const bool less = v[e] < s[e];
        lo[e] = less ? lo[e] + half + 1 : lo[e];
        len[e] = less ? len[e] - half - 1 : half;
      }
    }
  }
}

__global__ void __launch_bounds__(256)
rank_conditional_kernel(const float* __restrict__ scores, const int32_t* __restrict__ group_ids, int64_t Nc,
                        const float* __restrict__ calib, const int32_t* __restrict__ seg_offsets, int G,
                        uint32_t* __restrict__ numer, uint32_t* __restrict__ denom, float* __restrict__ pvalue,
                        bool vec4, unsigned int* __restrict__ dev_status) {
  // A warp takes 128 consecutive candidates, four per lane (128-bit loads and stores when every array is 16-byte
  // aligned: vec4).  The candidates of one input usually arrive together, so the segments a warp needs are few
  // and adjacent: if they span at most kCondStage entries the warp copies that span into shared memory with
  // coalesced loads and searches there; otherwise every lane searches its segments in global memory.
  __shared__ float stage_sh[8][kCondStage];
  const float qnan = __uint_as_float(0x7FC00000u);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* const stage = stage_sh[warp];
  const int64_t warps_total = (int64_t)gridDim.x * 8;
  for (int64_t w0 = ((int64_t)blockIdx.x * 8 + warp) * 128; w0 < Nc; w0 += warps_total * 128) {
    const int64_t j = w0 + 4 * lane;
    const bool full = vec4 && j + 4 <= Nc;
    float s[4];
    int g[4];
    if (full) {
      const float4 s4 = *reinterpret_cast<const float4*>(scores + j);
      const int4 g4 = *reinterpret_cast<const int4*>(group_ids + j);
      s[0] = s4.x; s[1] = s4.y; s[2] = s4.z; s[3] = s4.w;
      g[0] = g4.x; g[1] = g4.y; g[2] = g4.z; g[3] = g4.w;
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        s[e] = j + e < Nc ? scores[j + e] : qnan;
        g[e] = j + e < Nc ? group_ids[j + e] : -1;
      }
    }
    int lo[4], len[4], end[4];
    uint32_t den[4];
    bool bad = false;
    int span_lo = 0x7FFFFFFF, span_hi = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const bool ok = g[e] >= 0 && g[e] < G;
      bad = bad || (!ok && j + e < Nc);
      const int a = ok ? __ldg(seg_offsets + g[e]) : 0, b = ok ? __ldg(seg_offsets + g[e] + 1) : 0;
      lo[e] = a;
      end[e] = b;
      den[e] = ok ? (uint32_t)(b - a) + 1u : 1u;
      len[e] = (ok && s[e] == s[e]) ? b - a : -1;   // -1: no score (NaN, or no calibration set)
      if (len[e] > 0) {
        span_lo = min(span_lo, a);
        span_hi = max(span_hi, b);
      }
    }
    if (bad) atomicOr(dev_status, 4u);  // group id out of range: no calibration set, treated as "no score"
    const bool scored[4] = {len[0] >= 0, len[1] >= 0, len[2] >= 0, len[3] >= 0};
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      span_lo = min(span_lo, __shfl_xor_sync(0xFFFFFFFFu, span_lo, o));
      span_hi = max(span_hi, __shfl_xor_sync(0xFFFFFFFFu, span_hi, o));
    }
    // warp-uniform; no candidate of the warp with anything to search leaves span_lo above span_hi: nothing is staged
    if (span_hi > span_lo && span_hi - span_lo <= kCondStage) {
      __syncwarp();                          // the previous round's searches are done with the staging area
      for (int t = span_lo + lane; t < span_hi; t += 32) stage[t - span_lo] = __ldg(calib + t);
      __syncwarp();
      lower_bound_four<false>(stage - span_lo, s, lo, len);
    } else {
      lower_bound_four<true>(calib, s, lo, len);
    }
    uint32_t num[4];
    float p[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      num[e] = scored[e] ? (uint32_t)(end[e] - lo[e]) + 1u : 0u;
      p[e] = num[e] ? __fdiv_rn((float)num[e], (float)den[e]) : qnan;
    }
    if (full) {
      *reinterpret_cast<uint4*>(numer + j) = make_uint4(num[0], num[1], num[2], num[3]);
      *reinterpret_cast<uint4*>(denom + j) = make_uint4(den[0], den[1], den[2], den[3]);
      if (pvalue) *reinterpret_cast<float4*>(pvalue + j) = make_float4(p[0], p[1], p[2], p[3]);
    } else {
      for (int e = 0; e < 4 && j + e < Nc; ++e) {
        numer[j + e] = num[e];
        denom[j + e] = den[e];
        if (pvalue) pvalue[j + e] = p[e];
      }
    }
  }
}

__global__ void __launch_bounds__(256)
classify_conditional_kernel(const uint32_t* __restrict__ numer, const uint32_t* __restrict__ denom, int64_t Nc,
                            double alpha, uint8_t* __restrict__ stage, uint32_t* __restrict__ counts) {
  uint32_t c[3] = {0, 0, 0};
  for (int64_t j = (int64_t)blockIdx.x * 256 + threadIdx.x; j < Nc; j += (int64_t)gridDim.x * 256) {
    const uint32_t k_alpha = (uint32_t)floor(alpha * (double)denom[j]);
    const uint32_t s = stage_of(numer[j], k_alpha);
    stage[j] = (uint8_t)s;
    c[s - 1] += 1;
  }
  if (counts == nullptr) return;
#pragma unroll
  for (int i = 0; i < 3; ++i) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c[i] += __shfl_xor_sync(0xFFFFFFFFu, c[i], o);
    if ((threadIdx.x & 31) == 0 && c[i]) atomicAdd(counts + i, c[i]);
  }
}

// ---------------------------------------------------------------------------------------------
// K5+K6 for small problems (the model configurations: a few thousand calibration scores, tens of new ones):
// one block, one launch, truly in place, no workspace.  The block sorts the new keys in shared memory
// (bitonic network over k2 = k rounded up to a power of two, padded with a key above every canonical key),
// copies the old buffer into shared memory, and after a barrier - every read of the old buffer is done -
// writes each element to its merged slot (old[i] -> i + #{new < old[i]}, new[j] -> j + #{old <= new[j]}).
// ---------------------------------------------------------------------------------------------
constexpr int kSmallUpdThreads = 1024;
constexpr int kSmallUpdMaxOld = 28672;  // 112 KB of shared memory
constexpr int kSmallUpdMaxNew = 4096;   // 16 KB

__global__ void __launch_bounds__(kSmallUpdThreads, 1)
small_update_kernel(float* calib, int n, const float* __restrict__ new_scores, int k, int k2) {
  extern __shared__ uint32_t sm[];
  uint32_t* nk = sm;        // [k2] sorted new keys
  uint32_t* ok = sm + k2;   // [n] keys of the old buffer
  for (int t = threadIdx.x; t < k2; t += kSmallUpdThreads)
    nk[t] = t < k ? key_of_bits(canonical_bits(new_scores[t])) : 0xFFFFFFFFu;
#pragma unroll 8
  for (int t = threadIdx.x; t < n; t += kSmallUpdThreads) ok[t] = key_of_bits(canonical_bits(calib[t]));
  __syncthreads();
  for (int size = 2; size <= k2; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int t = threadIdx.x; t < (k2 >> 1); t += kSmallUpdThreads) {
        const int lo = 2 * t - (t & (stride - 1));
        const int hi = lo + stride;
        const uint32_t a = nk[lo], b = nk[hi];
        if ((a > b) == ((lo & size) == 0)) {
          nk[lo] = b;
          nk[hi] = a;
        }
      }
      __syncthreads();
    }
  }
  for (int e = threadIdx.x; e < n + k; e += kSmallUpdThreads) {
    if (e < n) {
      const uint32_t key = ok[e];
      int lo = 0, len = k;  // number of new keys < key
      while (len > 0) {
        const int half = len >> 1;
        const bool less = nk[lo + half] < key;
        lo = less ? lo + half + 1 : lo;
        len = less ? len - half - 1 : half;
      }
      calib[e + lo] = __uint_as_float(bits_of_key(key));
    } else {
      const int j = e - n;
      const uint32_t key = nk[j];
      int lo = 0, len = n;  // number of old keys <= key
      while (len > 0) {
        const int half = len >> 1;
        const bool le = ok[lo + half] <= key;
        lo = le ? lo + half + 1 : lo;
        len = le ? len - half - 1 : half;
      }
      calib[j + lo] = __uint_as_float(bits_of_key(key));
    }
  }
}

}  // namespace atts

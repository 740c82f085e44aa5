// Conformal kernels: rank / p-value, threshold + stage label, calibration sort + merge-insert.
// All results are integers or raw bit moves, so they are exact and reproducible.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace atts {

// Programmatic dependent launch.  A kernel launched with the programmatic-serialisation attribute may be set up
// on the SMs while the kernel before it in the stream is still running; pdl_wait() returns once that kernel has
// completed and its writes are visible, so nothing another kernel may have produced is read before it.
// pdl_launch_dependents() lets the kernel after this one be set up early in the same way.  Both are no-ops for a
// kernel launched the ordinary way.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

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

// Per-thread tallies of the fused thresholding, and the code the rank kernels share: writing the numerators,
// p-values and stage bytes of four candidates, and the block's contribution to the stage counts.
// Stage from the numerator with unsigned arithmetic: numer - 1 < k_alpha holds exactly for 1 <= numer <= k_alpha
// (numer = 0 wraps to the largest value), so stage = 2 + [numer - 1 < k_alpha] - [numer == 0].
template <int NA>
struct StageTally {
  uint32_t c3[NA > 0 ? NA : 1] = {}, c1 = 0, seen = 0;   // stage-1 samples (no score) are the same for every alpha
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
    uint32_t none[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      none[e] = (r[e] == 0u) ? 1u : 0u;
      tally.c1 += (e < valid) ? none[e] : 0u;
    }
#pragma unroll
    for (int a = 0; a < NA; ++a) {
      uint32_t st[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t rej = (r[e] - 1u < fc.k_alpha[a]) ? 1u : 0u;
        st[e] = 2u + rej - none[e];
        tally.c3[a] += (e < valid) ? rej : 0u;
      }
      if (full) {
        *reinterpret_cast<uint32_t*>(fc.stage[a] + j) = st[0] | (st[1] << 8) | (st[2] << 16) | (st[3] << 24);
      } else {
        for (int e = 0; e < valid; ++e) fc.stage[a][j + e] = (uint8_t)st[e];
      }
    }
  }
}

// The block's stage counts go to fc.counts ([NA][3]); every thread of the block calls it.  A grid of one block
// stores them; a larger grid adds them either to fc.counts itself (zeroed by the host before the launch:
// scratch == nullptr) or to 12 zeroed scratch words followed by a counter of finished blocks, in which case the
// last block to finish moves the totals to fc.counts and leaves the scratch zeroed for the next launch.
template <int NA>
__device__ __forceinline__ void flush_tally(const FusedClassify& fc, const StageTally<NA>& tally, uint32_t* scratch = nullptr) {
  if (NA == 0 || fc.counts == nullptr) return;
  __shared__ uint32_t sh[kMaxAlphas][3][kRankThreads / 32];
  __shared__ bool last_block;
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
#pragma unroll
  for (int a = 0; a < NA; ++a) {
    uint32_t v1 = tally.c1, v3 = tally.c3[a], v2 = tally.seen - tally.c1 - tally.c3[a];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      v1 += __shfl_xor_sync(0xFFFFFFFFu, v1, o);
      v2 += __shfl_xor_sync(0xFFFFFFFFu, v2, o);
      v3 += __shfl_xor_sync(0xFFFFFFFFu, v3, o);
    }
    if (l == 0) { sh[a][0][w] = v1; sh[a][1][w] = v2; sh[a][2][w] = v3; }
  }
  __syncthreads();
  uint32_t t = 0;
  if ((int)threadIdx.x < NA * 3) {
    const int a = threadIdx.x / 3, i = threadIdx.x % 3;
    for (int q = 0; q < kRankThreads / 32; ++q) t += sh[a][i][q];
    if (gridDim.x == 1) fc.counts[threadIdx.x] = t;
    else if (t) atomicAdd((scratch ? scratch : fc.counts) + threadIdx.x, t);
  }
  if (gridDim.x == 1 || scratch == nullptr) return;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) last_block = atomicAdd(scratch + 3 * kMaxAlphas, 1u) == gridDim.x - 1;
  __syncthreads();
  if (!last_block) return;
  __threadfence();
  if ((int)threadIdx.x < NA * 3) fc.counts[threadIdx.x] = atomicExch(scratch + threadIdx.x, 0u);
  if (threadIdx.x == 0) atomicExch(scratch + 3 * kMaxAlphas, 0u);
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
// The plain kernel pays, per block, one strided load for each of up to 8191 splitters, and per candidate several
// dependent loads from the L2-resident buffer; an SM serves divergent loads at one cache line per cycle, so they
// are what bounds it.  A calibration index kept beside the buffer removes most of them.  It holds, twice (two
// slots, see below):
//   buf     a copy of the sorted buffer, 32-byte aligned;
//   aux_a   a = 1 .. A: the last entry of every aligned group of 8^a entries, aux_a[i] = buf[8^a i + 8^a - 1]
//           (NaN where that lies beyond n);
//   tree    the last entries of the groups of G = 8^(A+1) entries, r < ns = n / G + 1 (the last one always NaN), as an
//           implicit search tree in breadth-first order, ready to be copied into shared memory.
// A candidate descends the tree (P shared-memory steps) to its group of G, then narrows by a factor of 8 per
// 32-byte load: A loads of aux entries and one of the buffer.  A is the smallest number of levels for which the
// tree has at most 32767 nodes (128 KB of shared memory; a level more costs every candidate one more load from L2, a
// deeper tree one more step in shared memory): 0 for n <= 262,143, 1 up to 2,097,151, 2 up to 16,776,703, 3 for the
// last few hundred sizes of the range.
//
// Two slots.  An update reads the buffer copy of the slot that describes the present fill n and writes the merged
// buffer to the other slot and to the caller's buffer, together with the other slot's aux entries and tree: no
// copy back, and nothing an update writes is read by a rank of the fill it started from, so the two may overlap.
// A kernel finds its slot by the fill it is given: slot descriptors hold the fill they describe.
//
// Layout (32-bit words): header [64]: [0] magic [1] capacity the layout was made for
//   [8 + 8 s ..] slot s: fill n (0xFFFFFFFF: none), P, A, ns;   [32 .. 45) zero between launches: scratch of the
//   rank kernel's stage counts;   then slot 0, slot 1, each: tree [32768],
//   aux_1, aux_2, aux_3, buf (every array a multiple of 8 words long).
// ---------------------------------------------------------------------------------------------
constexpr int kIndexHeaderWords = 64;
constexpr int kIndexMaxTreeLog2 = 15;                                 // the largest tree: 32767 nodes (128 KB of shared memory)
constexpr int kIndexTreeWords = 1 << kIndexMaxTreeLog2;
constexpr int kIndexMaxLevels = 3;
constexpr int kIndexCountScratch = 32;   // header words [32, 45): stage-count accumulators of the rank kernel, block counter
constexpr uint32_t kIndexMagic = 0x41545832u;
constexpr uint32_t kIndexNoFill = 0xFFFFFFFFu;
constexpr int64_t kIndexMinCandidates = 1 << 14;

struct IndexLayout {
  uint32_t aux_off[kIndexMaxLevels];   // word offsets inside a slot
  uint32_t buf_off;
  uint32_t slot_words;
};
__host__ __device__ inline IndexLayout index_layout(uint32_t cap) {
  IndexLayout L;
  uint32_t off = kIndexTreeWords;
  for (int a = 0; a < kIndexMaxLevels; ++a) {
    L.aux_off[a] = off;
    off += ((cap >> (3 * (a + 1))) + 16u) & ~7u;   // entries up to 8 * (n >> 3(a+1)) + 7 are read
  }
  L.buf_off = off;
  off += (cap + 15u) & ~7u;
  L.slot_words = (off + 63u) & ~63u;
  return L;
}
__host__ __device__ inline size_t index_words(uint32_t cap) {
  return (size_t)kIndexHeaderWords + 2 * (size_t)index_layout(cap).slot_words;
}
// Shape of the index of a fill n: aux levels A, tree depth P, tree entries ns.
struct IndexShape {
  int A, P, ns;
};
__host__ __device__ inline IndexShape index_shape(int64_t n) {
  IndexShape s;
  s.A = 0;
  while ((n >> (3 * (s.A + 1))) + 1 > (1 << kIndexMaxTreeLog2) - 1) ++s.A;
  s.ns = (int)(n >> (3 * (s.A + 1))) + 1;
  s.P = 1;
  while ((1 << s.P) - 1 < s.ns) ++s.P;
  return s;
}

// Slot, in the breadth-first table of a P-level tree, of the splitter with sorted rank r (inverse of the fill rule
// of rank_kernel: node b at depth l holds rank (2q + 1) * 2^(P-1-l) - 1, q = b - 2^l).
__device__ __forceinline__ int index_slot_of_rank(int r, int P) {
  const int x = r + 1;
  const int tz = __ffs(x) - 1;
  const int depth = P - 1 - tz;
  return (1 << depth) + (x >> (tz + 1)) - 1;
}

// The arrays of one slot, and the one operation that fills them: entry e of the sorted buffer has value v.
struct IndexSlot {
  float* tree;
  float* aux[kIndexMaxLevels];
  float* buf;
};
__device__ __forceinline__ IndexSlot index_slot(uint32_t* index, const IndexLayout& L, int s) {
  float* base = reinterpret_cast<float*>(index + kIndexHeaderWords + (size_t)s * L.slot_words);
  IndexSlot t;
  t.tree = base;
#pragma unroll
  for (int a = 0; a < kIndexMaxLevels; ++a) t.aux[a] = base + L.aux_off[a];
  t.buf = base + L.buf_off;
  return t;
}
__device__ __forceinline__ void index_put(const IndexSlot& t, const IndexShape& sh, int e, float v) {
  t.buf[e] = v;
  int m = 7;   // e ends an aligned group of 8^a entries iff its low 3a bits are all ones
#pragma unroll
  for (int a = 1; a <= kIndexMaxLevels; ++a) {
    if (a > sh.A) break;
    if ((e & m) != m) return;
    t.aux[a - 1][e >> (3 * a)] = v;
    m = (m << 3) | 7;
  }
  if ((e & m) == m) t.tree[index_slot_of_rank(e >> (3 * (sh.A + 1)), sh.P)] = v;   // ends a group of 8^(A+1)
}
// NaN for the aux entries and tree nodes whose group ends beyond n (spread over `nthreads` callers).
__device__ __forceinline__ void index_pad(const IndexSlot& t, const IndexShape& sh, int n, int tid, int nthreads) {
  const float qnan = __uint_as_float(0x7FC00000u);
#pragma unroll
  for (int a = 1; a <= kIndexMaxLevels; ++a) {
    if (a > sh.A) break;
    const int first = n >> (3 * a), last = 8 * (n >> (3 * (a + 1))) + 8;
    for (int i = first + tid; i < last; i += nthreads) t.aux[a - 1][i] = qnan;
  }
  for (int r = (n >> (3 * (sh.A + 1))) + tid; r < (1 << sh.P) - 1; r += nthreads) t.tree[index_slot_of_rank(r, sh.P)] = qnan;
}
// Header words of slot s.
__device__ __forceinline__ void index_describe(uint32_t* index, int s, uint32_t n, const IndexShape& sh) {
  uint32_t* d = index + 8 + 8 * s;
  d[0] = n; d[1] = (uint32_t)sh.P; d[2] = (uint32_t)sh.A; d[3] = (uint32_t)sh.ns;
}
// The slot that describes fill n of an index laid out for `cap` entries, or -1.
__device__ __forceinline__ int index_find(const uint32_t* __restrict__ index, uint32_t cap, uint32_t n) {
  if (index[0] != kIndexMagic || index[1] != cap) return -1;
  return index[8] == n ? 0 : (index[16] == n ? 1 : -1);
}

// Builds slot 0 of the index from src[0, n) (the caller's sorted buffer) and marks slot 1 empty.
__global__ void __launch_bounds__(256)
index_build_kernel(const float* __restrict__ src, int n, uint32_t cap, uint32_t* __restrict__ index) {
  const IndexLayout L = index_layout(cap);
  const IndexShape sh = index_shape(n);
  const IndexSlot t = index_slot(index, L, 0);
  const int tid = blockIdx.x * blockDim.x + threadIdx.x, nthreads = gridDim.x * blockDim.x;
  if (tid == 0) {
    index[0] = kIndexMagic;
    index[1] = cap;
    index_describe(index, 0, (uint32_t)n, sh);
    index[16] = kIndexNoFill;
  }
  if (tid >= kIndexCountScratch && tid < kIndexCountScratch + 3 * kMaxAlphas + 1) index[tid] = 0u;
  for (int e = tid; e < n; e += nthreads) index_put(t, sh, e, src[e]);
  index_pad(t, sh, n, tid, nthreads);
}

template <int P>
__device__ __forceinline__ void rank_four_indexed(const float (&s)[4], const float* __restrict__ sp, int A,
                                                  const float* const (&aux)[kIndexMaxLevels],
                                                  const float* __restrict__ calib, int n, uint32_t (&numer)[4]) {
  int g[4];
  tree_descend<P>(s, sp, g);   // number of groups of 8^(A+1) that lie entirely below the score
  float w[4][8];
#pragma unroll
  for (int a = kIndexMaxLevels; a >= 1; --a) {
    if (a > A) continue;
    const float* __restrict__ lvl = aux[a - 1];
#pragma unroll
    for (int e = 0; e < 4; ++e)
      asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                   : "=f"(w[e][0]), "=f"(w[e][1]), "=f"(w[e][2]), "=f"(w[e][3]), "=f"(w[e][4]), "=f"(w[e][5]), "=f"(w[e][6]), "=f"(w[e][7])
                   : "l"(lvl + 8 * g[e]));
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      int c = 0;
#pragma unroll
      for (int i = 0; i < 7; ++i) c += (w[e][i] < s[e]) ? 1 : 0;   // the eighth is the group's own splitter: not below
      g[e] = 8 * g[e] + c;                                         // groups of 8^a that lie entirely below the score
    }
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    // the last group may be cut short by n: its 32 bytes are read in one piece only if it is whole
    if (8 * g[e] + 8 <= n) {
      asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                   : "=f"(w[e][0]), "=f"(w[e][1]), "=f"(w[e][2]), "=f"(w[e][3]), "=f"(w[e][4]), "=f"(w[e][5]), "=f"(w[e][6]), "=f"(w[e][7])
                   : "l"(calib + 8 * g[e]));
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) w[e][i] = (8 * g[e] + i < n) ? __ldg(calib + 8 * g[e] + i) : __uint_as_float(0x7FC00000u);
    }
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    int c = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) c += (w[e][i] < s[e]) ? 1 : 0;
    const int below = 8 * g[e] + c;
    numer[e] = (s[e] != s[e]) ? 0u : (uint32_t)(n - below) + 1u;   // NaN: no score
  }
}

// Every block takes one contiguous, equal share of the candidates (in groups of four), so that all SMs finish
// together whatever the candidate count.
template <int NA>
__global__ void __launch_bounds__(kRankThreads)
rank_indexed_kernel(const float* __restrict__ scores, int64_t Nc, int n, uint32_t* __restrict__ index,
                    uint32_t* __restrict__ numer, float* __restrict__ pvalue, const FusedClassify fc,
                    unsigned int* __restrict__ dev_status) {
  extern __shared__ float sp[];
  const float qnan = __uint_as_float(0x7FC00000u);
  const int64_t quads = (Nc + 3) >> 2;
  const int64_t share = (quads + gridDim.x - 1) / gridDim.x;
  const int64_t q_end = min(quads, ((int64_t)blockIdx.x + 1) * share);
  const int64_t q_first = (int64_t)blockIdx.x * share + threadIdx.x;
  pdl_launch_dependents();
  pdl_wait();   // everything read below may come from the kernel before this one
  // the thread's first four scores are on their way while the index is looked at and the table filled
  float4 nxt = make_float4(qnan, qnan, qnan, qnan);
  if (q_first < q_end && 4 * q_first + 4 <= Nc) nxt = *reinterpret_cast<const float4*>(scores + 4 * q_first);
  // an index that does not describe this fill of the buffer would give wrong ranks silently: refuse it.  The header
  // words that matter (magic and capacity, the two slots' descriptions) are read together, in one round trip.
  const uint4 h0 = *reinterpret_cast<const uint4*>(index), d0 = *reinterpret_cast<const uint4*>(index + 8),
              d1 = *reinterpret_cast<const uint4*>(index + 16);
  const uint32_t cap = h0.y;   // the capacity the index was laid out for, as its builder recorded it
  const int slot = h0.x != kIndexMagic ? -1 : (d0.x == (uint32_t)n ? 0 : (d1.x == (uint32_t)n ? 1 : -1));
  if (slot < 0) {
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(dev_status, 8u);
    return;
  }
  const int P = (int)(slot ? d1.y : d0.y), A = (int)(slot ? d1.z : d0.z);
  const IndexLayout L = index_layout(cap);
  const float* const base = reinterpret_cast<const float*>(index + kIndexHeaderWords + (size_t)slot * L.slot_words);
  const float* const aux[kIndexMaxLevels] = {base + L.aux_off[0], base + L.aux_off[1], base + L.aux_off[2]};
  const float* const calib = base + L.buf_off;
  for (int t = threadIdx.x; t < (1 << P) - 1; t += kRankThreads) sp[t] = __ldg(base + t);
  __syncthreads();
  StageTally<NA> tally;
  const float denom = (float)(n + 1);
  for (int64_t q = q_first; q < q_end; q += kRankThreads) {
    const int64_t j = 4 * q;
    float s[4] = {nxt.x, nxt.y, nxt.z, nxt.w};
    uint32_t r[4];
    const bool full = j + kRankPerThread <= Nc;
    if (!full) {
#pragma unroll
      for (int e = 0; e < 4; ++e) s[e] = (j + e < Nc) ? scores[j + e] : qnan;
    }
    if (q + kRankThreads < q_end && j + 4 * kRankThreads + 4 <= Nc)   // the scores of the next round
      nxt = *reinterpret_cast<const float4*>(scores + j + 4 * kRankThreads);
    switch (P) {
      case 1: rank_four_indexed<1>(s, sp, A, aux, calib, n, r); break;
      case 2: rank_four_indexed<2>(s, sp, A, aux, calib, n, r); break;
      case 3: rank_four_indexed<3>(s, sp, A, aux, calib, n, r); break;
      case 4: rank_four_indexed<4>(s, sp, A, aux, calib, n, r); break;
      case 5: rank_four_indexed<5>(s, sp, A, aux, calib, n, r); break;
      case 6: rank_four_indexed<6>(s, sp, A, aux, calib, n, r); break;
      case 7: rank_four_indexed<7>(s, sp, A, aux, calib, n, r); break;
      case 8: rank_four_indexed<8>(s, sp, A, aux, calib, n, r); break;
      case 9: rank_four_indexed<9>(s, sp, A, aux, calib, n, r); break;
      case 10: rank_four_indexed<10>(s, sp, A, aux, calib, n, r); break;
      case 11: rank_four_indexed<11>(s, sp, A, aux, calib, n, r); break;
      case 12: rank_four_indexed<12>(s, sp, A, aux, calib, n, r); break;
      case 13: rank_four_indexed<13>(s, sp, A, aux, calib, n, r); break;
      case 14: rank_four_indexed<14>(s, sp, A, aux, calib, n, r); break;
      default: rank_four_indexed<15>(s, sp, A, aux, calib, n, r); break;
    }
    float p[4] = {qnan, qnan, qnan, qnan};
    if (pvalue) {
#pragma unroll
      for (int e = 0; e < 4; ++e) p[e] = r[e] ? __fdiv_rn((float)r[e], denom) : qnan;
    }
    emit_four<NA>(j, Nc, full, r, p, numer, pvalue, fc, tally);
  }
  flush_tally<NA>(fc, tally, index + kIndexCountScratch);
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
    if (gridDim.x == 1) counts[threadIdx.x] = t;   // a single block owns the counts: no zeroing beforehand
    else if (t) atomicAdd(counts + threadIdx.x, t);
  }
}

// ---------------------------------------------------------------------------------------------
// K5 + K6  calibration update: sort of the new scores and merge-insert, in one kernel.
//
// The merged buffer is the stable merge of the old buffer (n entries, ascending) with the k new keys:
//   old[e]  -> slot e + #{new <  old[e]}
//   new x   -> slot #{old <= x} + #{new before x in sorted order}
// No global sort of the new keys is needed for that.  The old buffer is cut into tiles of consecutive entries
// [e0, e1); a new key x belongs to the tile that holds its insertion point, #{old <= x} in [e0, e1), which two
// comparisons decide: old[e0 - 1] <= x < old[e1 - 1] (no lower test for the first tile, no upper test for the last).
// A block that owns a tile reads all k new keys once, counts those below its range (c_below: they precede
// everything the tile places), keeps its own (about k / tiles of them) in shared memory and sorts those few there;
// keys of other tiles lie above its range and shift nothing here.  Then
//   old[e], e in the tile  -> e + c_below + #{own keys <  old[e]}      (search among the few own keys)
//   own key x, i-th of the sorted own keys -> e0 + #{tile entries <= x} + c_below + i   (search in the tile, in shared memory)
// Equal keys are equal bit patterns after canonicalisation, so the order in which equal new keys are placed does
// not show in the result.  One launch, no scratch besides the output, every global load and store coalesced.
// A skewed batch (all new keys in one tile) only makes that block's sort longer, never wrong.
// ---------------------------------------------------------------------------------------------
constexpr int kSortMaxK = 16384;          // new keys per launch (larger batches are inserted slice by slice)
constexpr int kMergeThreads = 1024;
constexpr int kMergeTileMax = 8192;       // old entries per tile (32 KB of shared memory)
constexpr int kMergeRankSortMax = 384;    // own keys up to this many are sorted by all-pairs ranking, more by a bitonic network

// Block-wide bitonic sort, ascending, of the kMergeThreads * E keys in a[] (shared memory; the caller pads with a key
// above all others).  Thread t holds keys t E .. t E + E - 1 in registers: a compare-exchange whose partner lies in
// the same thread is done in registers, one whose partner lies in the same warp by a shuffle, and only the ones
// across warps go through shared memory - 15 of the 78 steps for 4096 keys.
template <int E>
__device__ __forceinline__ void block_bitonic_sort(uint32_t* a) {
  constexpr int kLogE = E == 1 ? 0 : E == 2 ? 1 : E == 4 ? 2 : E == 8 ? 3 : 4;
  const int base = threadIdx.x * E;
  uint32_t v[E];
#pragma unroll
  for (int i = 0; i < E; ++i) v[i] = a[base + i];
  for (int size = 2; size <= kMergeThreads * E; size <<= 1) {
    const bool asc = (base & size) == 0;   // for size > E every key of the thread lies in the same half
    for (int stride = size >> 1; stride >= E; stride >>= 1) {
      const bool keep_min = ((base & stride) == 0) == asc;
      if (stride >= 32 * E) {
        // the partner of key i of thread t is key i of thread t ^ (stride / E), same lane of another warp: exchanged
        // through shared memory laid out [i][thread], which neither the stores nor the loads conflict on
        __syncthreads();
#pragma unroll
        for (int i = 0; i < E; ++i) a[i * kMergeThreads + threadIdx.x] = v[i];
        __syncthreads();
        const int partner = threadIdx.x ^ (stride / E);
#pragma unroll
        for (int i = 0; i < E; ++i) {
          const uint32_t other = a[i * kMergeThreads + partner];
          v[i] = keep_min ? min(v[i], other) : max(v[i], other);
        }
      } else {
        const int lane_mask = stride / E;
#pragma unroll
        for (int i = 0; i < E; ++i) {
          const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, v[i], lane_mask);
          v[i] = keep_min ? min(v[i], other) : max(v[i], other);
        }
      }
    }
#pragma unroll
    for (int sb = kLogE - 1; sb >= 0; --sb) {
      const int st = 1 << sb;
      if (st < size) {
#pragma unroll
        for (int i = 0; i < E; ++i) {
          if ((i & st) == 0) {
            const bool up = ((base + i) & size) == 0;   // within a thread the direction can differ while size <= E
            const uint32_t lo = min(v[i], v[i | st]), hi = max(v[i], v[i | st]);
            v[i] = up ? lo : hi;
            v[i | st] = up ? hi : lo;
          }
        }
      }
    }
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < E; ++i) a[base + i] = v[i];
  __syncthreads();
}

// Launch shape of the merge for n old entries on `sms` SMs: entries per tile and number of tiles (>= 1).
__host__ __device__ inline void merge_tiling(int n, int sms, int& tile_len, int& tiles) {
  const int rounds = (int)(((long long)n + (long long)sms * kMergeTileMax - 1) / ((long long)sms * kMergeTileMax));
  const int want = sms * (rounds < 1 ? 1 : rounds);
  tile_len = (n + want - 1) / want;
  if (tile_len < 256) tile_len = 256;     // tiny buffers: a few tiles are enough
  tiles = (n + tile_len - 1) / tile_len;
  if (tiles < 1) tiles = 1;
}

// INDEXED == false: reads old_buf[0, n), writes the merged n + k entries to `out` (a scratch copy the host then
// copies back: a tile's slots overlap the entries of the tiles after it).  INDEXED == true: the old entries are
// read from the index slot that describes fill n, and every merged entry goes to the other slot (buffer copy, aux
// entries, tree) and to `out`, which is the caller's buffer itself - nothing read here is written here, so there is
// no copy back; `old_buf` is not used.
// Dynamic shared memory: 4 * (2 * k2 + tile_len) bytes, k2 = k rounded up to a power of two, at least kMergeThreads.
template <bool INDEXED>
__global__ void __launch_bounds__(kMergeThreads, 1)
merge_kernel(const float* __restrict__ old_buf, int n, const float* __restrict__ new_scores, int k, int k2, int tile_len,
             int tiles, float* __restrict__ out, uint32_t* __restrict__ index, uint32_t cap,
             unsigned int* __restrict__ dev_status) {
  extern __shared__ uint32_t msm[];
  uint32_t* const own = msm;             // [k2] this tile's new keys, as they come
  uint32_t* const own_sorted = msm + k2; // [k2] the same, ascending
  uint32_t* const tkeys = msm + 2 * k2;  // [tile_len] keys of the tile's old entries
  __shared__ int own_count, below_count;
  pdl_launch_dependents();
  pdl_wait();   // the new scores, the buffer and the index may come from the kernel before this one
  IndexSlot dst{};
  IndexShape sh{};
  if (INDEXED) {
    const int src = index_find(index, cap, (uint32_t)n);
    if (src < 0) {   // no description of this fill: nothing is changed, the condition is reported
      if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(dev_status, 8u);
      return;
    }
    const IndexLayout L = index_layout(cap);
    old_buf = index_slot(index, L, src).buf;
    dst = index_slot(index, L, src ^ 1);
    sh = index_shape(n + k);
    const int tid = blockIdx.x * kMergeThreads + threadIdx.x;
    if (tid == 0) index_describe(index, src ^ 1, (uint32_t)(n + k), sh);
    index_pad(dst, sh, n + k, tid, gridDim.x * kMergeThreads);
  }
  auto emit = [&](int slot, uint32_t key) {
    const float v = __uint_as_float(bits_of_key(key));
    out[slot] = v;
    if (INDEXED) index_put(dst, sh, slot, v);
  };
  for (int t = blockIdx.x; t < tiles; t += gridDim.x) {
    const int e0 = t * tile_len, e1 = min(n, e0 + tile_len), len = e1 - e0;
    const bool first = e0 == 0, last = t == tiles - 1;
    // every global load of the round is issued before anything waits on one: the tile's range, its entries
    // (at most 8 per thread) and the first 4096 new scores
    const float lo_f = first ? 0.f : old_buf[e0 - 1];
    const float hi_f = last ? 0.f : old_buf[e1 - 1];
    float tv[kMergeTileMax / kMergeThreads], nv[4];
#pragma unroll
    for (int u = 0; u < kMergeTileMax / kMergeThreads; ++u) {
      const int i = threadIdx.x + u * kMergeThreads;
      tv[u] = i < len ? old_buf[e0 + i] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int j = threadIdx.x + u * kMergeThreads;
      nv[u] = j < k ? __ldg(new_scores + j) : 0.f;
    }
    const uint32_t lo = key_of_bits(canonical_bits(lo_f)), hi = key_of_bits(canonical_bits(hi_f));
    if (threadIdx.x == 0) { own_count = 0; below_count = 0; }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < kMergeTileMax / kMergeThreads; ++u) {
      const int i = threadIdx.x + u * kMergeThreads;
      if (i < len) tkeys[i] = key_of_bits(canonical_bits(tv[u]));
    }
    int below = 0;
    for (int j0 = 0; j0 < k; j0 += kMergeThreads) {   // uniform trip count: the warp votes below
      const int j = j0 + threadIdx.x;
      float xf = 0.f;
      if (j0 < 4 * kMergeThreads) {
#pragma unroll
        for (int u = 0; u < 4; ++u) xf = (j0 == u * kMergeThreads) ? nv[u] : xf;
      } else if (j < k) {
        xf = __ldg(new_scores + j);
      }
      const uint32_t x = key_of_bits(canonical_bits(xf));
      const bool is_below = j < k && !first && x < lo;
      const bool is_own = j < k && !is_below && (last || x < hi);
      below += is_below ? 1 : 0;
      // one shared-memory atomic per warp, not per key: a skewed batch sends every key to the same counter
      const uint32_t votes = __ballot_sync(0xFFFFFFFFu, is_own);
      if (votes) {
        const int lane = threadIdx.x & 31, leader = __ffs((int)votes) - 1;
        int base = 0;
        if (lane == leader) base = atomicAdd(&own_count, __popc(votes));
        base = __shfl_sync(0xFFFFFFFFu, base, leader);
        if (is_own) own[base + __popc(votes & ((1u << lane) - 1u))] = x;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) below += __shfl_xor_sync(0xFFFFFFFFu, below, o);
    if ((threadIdx.x & 31) == 0 && below) atomicAdd(&below_count, below);
    __syncthreads();
    const int m = own_count, c_below = below_count;
    // ---- sort the tile's own keys into own_sorted ----
    if (m <= kMergeRankSortMax) {
      // all-pairs: the slot of key i is the number of keys that sort before it (equal keys by position)
      for (int i = threadIdx.x; i < m; i += kMergeThreads) {
        const uint32_t x = own[i];
        int r = 0;
        for (int j = 0; j < m; ++j) {
          const uint32_t y = own[j];
          r += (y < x) || (y == x && j < i);
        }
        own_sorted[r] = x;
      }
      __syncthreads();
    } else {
      // a skewed batch: this block owns hundreds or thousands of the new keys
      int m2 = kMergeThreads;
      while (m2 < m) m2 <<= 1;
      for (int i = threadIdx.x; i < m2; i += kMergeThreads) own_sorted[i] = i < m ? own[i] : 0xFFFFFFFFu;
      __syncthreads();
      switch (m2 / kMergeThreads) {
        case 1: block_bitonic_sort<1>(own_sorted); break;
        case 2: block_bitonic_sort<2>(own_sorted); break;
        case 4: block_bitonic_sort<4>(own_sorted); break;
        case 8: block_bitonic_sort<8>(own_sorted); break;
        default: block_bitonic_sort<16>(own_sorted); break;
      }
    }
    // ---- place the own keys: e0 + #{tile entries <= x} + c_below + i ----
    for (int i = threadIdx.x; i < m; i += kMergeThreads) {
      const uint32_t x = own_sorted[i];
      int p = 0, left = len;   // halving search: the first half goes if its last entry is not above x
      while (left > 1) {
        const int half = left >> 1;
        p += (tkeys[p + half - 1] <= x) ? half : 0;
        left -= half;
      }
      if (left == 1 && tkeys[p] <= x) ++p;
      emit(e0 + p + c_below + i, x);
    }
    // ---- place the tile's old entries: e + c_below + #{own keys < old[e]} ----
    for (int i = threadIdx.x; i < len; i += kMergeThreads) {
      const uint32_t key = tkeys[i];
      int p = 0, left = m;
      while (left > 1) {
        const int half = left >> 1;
        p += (own_sorted[p + half - 1] < key) ? half : 0;
        left -= half;
      }
      if (left == 1 && own_sorted[p] < key) ++p;
      emit(e0 + i + c_below + p, key);
    }
    __syncthreads();   // shared memory is reused by the next tile
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
    if (gridDim.x == 1) counts[threadIdx.x] = t;   // a single block owns the counts: no zeroing beforehand
    else if (t) atomicAdd(counts + threadIdx.x, t);
  }
}

// ---------------------------------------------------------------------------------------------
// Budget report: the positions of the samples in stage 3 (the target takes over), in input order, and their
// number B.  A stream compaction in one pass over the stage bytes.  Its arithmetic is light, so what decides the
// time is how few instructions a byte costs and whether the loads of the next piece of work are in flight while
// the present one is being expanded.
//
// The bytes, counted from the 16-byte boundary at or below the first one (`head` bytes earlier, never counted), are
// cut into ranges of 4096 Q bytes (Q even, <= 8: at most 32,768 bytes, so a position inside a range fits in 16
// bits); a block takes ranges in the order of a ticket counter, one ticket ahead of the range it works on.  For a range,
//  1. every thread has copied Q pieces of 16 bytes into shared memory with asynchronous copies issued while the
//     range before was being worked on (a warp's copy instruction covers 512 contiguous bytes; bytes past the end
//     arrive as zeros); it reads its own pieces back, turns each into 16 bits (bit set where the byte is 3) and
//     stores them in shared memory, where they form a bit map of the warp's 512 Q bytes in input order; then it
//     issues the copies of the next range into the slots it has just read;
//  2. every lane then owns 16 Q consecutive bits of that map, i.e. a contiguous piece of the input, so that one
//     prefix sum per warp (not one per row) gives the place of its first position, and its positions are consecutive;
//  3. the block publishes the range's count and sums the counts of all earlier ranges by looking back over their
//     published words (a word holds a range's own count or, once known, the count of everything up to and including
//     it) while the other warps already expand their bits into 16-bit positions in shared memory;
//  4. the staged positions are written out by the whole block, 32 consecutive words per warp instruction (a lane
//     writing its own short run straight to global memory would send eight partial sectors where one whole one does).
// A range with more stage-3 bytes than the staging area holds (more than a quarter of a full range) is written
// directly from the bit map, slower but the same result.
// Tickets are drawn in launch order and a block works through its tickets in increasing order, so the block that
// owns an earlier range is always running or done: the look-back cannot wait on a block that has not started.
// Every wait is bounded all the same.  Everything is integer work in a fixed order: the result is unique.
// ---------------------------------------------------------------------------------------------
constexpr int kIdsThreads = 256;
constexpr int kIdsMaxRows = 8;                           // 16-byte pieces per thread at most
constexpr int kIdsRowBytes = kIdsThreads * 16;           // 4096 stage bytes per row of pieces
constexpr int kIdsStageCap = 7680;                       // positions staged per range (four blocks fit an SM)
constexpr int kIdsSmemBytes = kIdsMaxRows * kIdsRowBytes + 2 * (kIdsThreads / 32) * kIdsMaxRows * 64 + 2 * kIdsStageCap;
constexpr unsigned long long kIdsOwnCount = 1ull << 32, kIdsPrefixKnown = 2ull << 32;
constexpr int kIdsSpinLimit = 1 << 22;

// Bit i of the result is set where byte i of the 16 bytes is 3.
__device__ __forceinline__ uint32_t stage3_mask16(const uint4& q) {
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
  uint32_t acc = 0;
#pragma unroll
  for (int i = 3; i >= 0; --i) {
    // A byte equals 3 iff (byte ^ 3) is zero: the zero-byte test on four bytes at once, exact (bit 7 of a byte of
    // t is set iff its low seven bits are not all zero; bit 7 of byte ^ 3 is bit 7 of the byte).  z has 0x80 in
    // every byte that was 3.  The multiplication moves bits 7, 15, 23, 31 to bits 28 .. 31 (no two partial
    // products meet, so nothing carries), and the funnel shift appends those four bits below the ones gathered
    // so far: the last word handled, word 0, ends in bits 0 .. 3.
    const uint32_t t = ((w[i] ^ 0x03030303u) & 0x7F7F7F7Fu) + 0x7F7F7F7Fu;
    const uint32_t z = ~(t | w[i] | 0x7F7F7F7Fu);
    acc = __funnelshift_l(z * 0x00204081u, acc, 4);
  }
  return acc;
}

// x >> n for n up to 32 (the hardware's shift gives zero for n = 32, which the language leaves undefined)
__device__ __forceinline__ uint32_t shr_clamped(uint32_t x, uint32_t n) {
  uint32_t y;
  asm("shr.b32 %0, %1, %2;" : "=r"(y) : "r"(x), "r"(n));
  return y;
}

__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}

// The Q asynchronous 16-byte copies of one thread for the range that starts `range_base` bytes after `base`
// (16-byte aligned); `len` bytes from `base` on exist, pieces beyond them arrive (partly) as zeros.
__device__ __forceinline__ void ids_prefetch(const uint8_t* __restrict__ base, int64_t len, int64_t range_base, int Q,
                                             uint4* raw) {
  const int64_t j0 = range_base + (int64_t)(threadIdx.x >> 5) * Q * 512 + (threadIdx.x & 31) * 16;
  const uint32_t dst = (uint32_t)__cvta_generic_to_shared(raw + threadIdx.x);
  if (range_base + (int64_t)Q * kIdsRowBytes <= len) {   // the whole range exists: nothing to test per piece
    const uint8_t* src = base + j0;
#pragma unroll
    for (int q = 0; q < kIdsMaxRows; ++q)
      if (q < Q)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + q * kIdsRowBytes), "l"(src + q * 512) : "memory");
  } else {
    for (int q = 0; q < Q; ++q) {
      const int64_t j = j0 + q * 512;
      const int64_t left = len - j;
      const uint32_t valid = left >= 16 ? 16u : (left > 0 ? (uint32_t)left : 0u);
      const uint8_t* src = base + (valid ? j : 0);
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + q * kIdsRowBytes), "l"(src), "r"(valid) : "memory");
    }
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
}

// state: one word per range (zero before the launch), ticket: one counter (zero before the launch); both unused
// (may be nullptr) when there is a single range.  base: the 16-byte boundary at or below the first stage byte, which
// is byte `head` from there; len = head + number of stage bytes.  Q: rows per range, even, 2 <= Q <= kIdsMaxRows.
//
// The loop is staggered by one turn: turn k reads range k and counts it, publishes that count, and then expands and
// writes out range k - 1, whose look-back (the only step that depends on other blocks) has had a whole turn for its
// predecessors' counts to appear; its loads are issued before the expansion and looked at after it.
__global__ void __launch_bounds__(kIdsThreads)
takeover_ids_kernel(const uint8_t* __restrict__ base, int64_t len, int head, int Q, int ranges,
                    unsigned long long* __restrict__ state, unsigned int* __restrict__ ticket,
                    int32_t* __restrict__ ids, int64_t ids_cap, uint32_t* __restrict__ count,
                    unsigned int* __restrict__ dev_status) {
  extern __shared__ uint4 ids_smem[];
  uint4* const raw = ids_smem;                                                                  // [Q][256] pieces
  uint32_t* const bitmap = reinterpret_cast<uint32_t*>(ids_smem + kIdsMaxRows * kIdsThreads);   // [2][warps][128]: one bit per byte
  uint16_t* const staged = reinterpret_cast<uint16_t*>(bitmap + 2 * (kIdsThreads / 32) * kIdsMaxRows * 16);
  __shared__ uint32_t warp_total[2][kIdsThreads / 32];
  __shared__ uint32_t range_sh[2], prefix_sh;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int words = Q >> 1;   // bit-map words per lane
  const int64_t range_bytes = (int64_t)Q * kIdsRowBytes;
  const uint32_t warp_first = (uint32_t)(warp * Q * 512);   // of the warp's bytes, inside the range

  // Thread 0 draws tickets two ranges ahead and keeps the newest in a register, so that the counter's round trip
  // is over long before the value is needed.
  uint32_t drawn = (uint32_t)ranges;
  if (threadIdx.x == 0) {
    range_sh[0] = ranges == 1 ? 0u : atomicAdd(ticket, 1u);
    if (ranges > 1) drawn = atomicAdd(ticket, 1u);
  }
  __syncthreads();
  int range = (int)range_sh[0];
  if (range < ranges) ids_prefetch(base, len, range * range_bytes, Q, raw);
  int prev = -1;                                  // the range counted in the turn before, to be written out in this one
  uint32_t prev_local = 0, prev_mine = 0, prev_turns = 0, prev_total = 0;
  for (int k = 0;; ++k) {
    const bool cur = range < ranges;
    if (!cur && prev < 0) break;
    uint32_t* const wmap = bitmap + ((k & 1) * (kIdsThreads / 32) + warp) * (kIdsMaxRows * 16);
    uint32_t mine = 0, incl = 0, turns = 0;
    if (cur) {
      // 1. lane l holds bytes [16 l, 16 l + 16) of each of the warp's Q rows of 512 bytes: its own copies have landed
      uint16_t* const rows16 = reinterpret_cast<uint16_t*>(wmap);
      asm volatile("cp.async.wait_all;" ::: "memory");
#pragma unroll
      for (int q = 0; q < kIdsMaxRows; ++q)
        if (q < Q) rows16[q * 32 + lane] = (uint16_t)stage3_mask16(raw[q * kIdsThreads + threadIdx.x]);
      if (range == 0 && threadIdx.x == 0) rows16[0] &= (uint16_t)(0xFFFFu << head);   // bytes before the first stage byte
      __syncwarp();
      // 2. lane l owns words [l Q/2, (l + 1) Q/2) of the warp's map = bytes [16 Q l, 16 Q (l + 1)) of the warp
      const uint32_t* const seg = wmap + lane * words;
      for (int i = 0; i < words; ++i) {
        const uint32_t c = (uint32_t)__popc(seg[i]);
        mine += c;
        turns += max(c, 1u);   // iterations of the expansion loop: one per bit and one per empty word
      }
      incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += up;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) turns = max(turns, __shfl_xor_sync(0xFFFFFFFFu, turns, o));
      if (lane == 31) warp_total[k & 1][warp] = incl;
    }
    if (threadIdx.x == 0) {
      range_sh[(k + 1) & 1] = drawn;   // the range after this one
      drawn = (ranges > 1 && drawn < (uint32_t)ranges) ? atomicAdd(ticket, 1u) : (uint32_t)ranges;
    }
    __syncthreads();
    const int next = cur ? (int)range_sh[(k + 1) & 1] : ranges;
    if (next < ranges) ids_prefetch(base, len, next * range_bytes, Q, raw);   // into the slots this thread has read
    uint32_t warp_off = 0, total = 0;
    if (cur) {
#pragma unroll
      for (int w = 0; w < kIdsThreads / 32; ++w) {
        const uint32_t t = warp_total[k & 1][w];
        warp_off += w < warp ? t : 0u;
        total += t;
      }
    }
    // 3. the count of this range is published; the look-back of the range before it is started
    unsigned long long win[8];
    if (warp == 0 && ranges > 1) {
      if (cur && lane == 0) atomicExch(state + range, (range == 0 ? kIdsPrefixKnown : kIdsOwnCount) | total);
      if (prev > 0) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int p = prev - 1 - 32 * u - lane;
          win[u] = p >= 0 ? ld_relaxed_u64(state + p) : kIdsPrefixKnown;
        }
      }
    }
    const uint32_t* const pseg = bitmap + (((k + 1) & 1) * (kIdsThreads / 32) + warp) * (kIdsMaxRows * 16) + lane * words;
    const bool fits = prev_total <= (uint32_t)kIdsStageCap;
    if (prev >= 0 && fits) {
      // One loop for all the lane's words, from its last bit down to its first: a lane whose word has run out fetches
      // the one before it while the others go on with theirs, so the lanes of a warp wait for one another once per
      // range, not once per word.  Every lane makes the same number of turns (the largest need among them), which
      // keeps the warp together; the body has no branch.
      uint16_t* dst = staged + prev_local + prev_mine;                         // one past the lane's last position
      uint32_t top = warp_first + (uint32_t)(lane * words + words) * 32u - 1u;   // position of bit 31 of the word in hand
      const uint32_t* wp = pseg + words - 1;
      uint32_t r = *wp;
      uint32_t ahead = wp > pseg ? wp[-1] : 0u;   // the word before the one in hand, loaded before it is needed
#pragma unroll 2
      for (uint32_t turn = 0; turn < prev_turns; ++turn) {
        const bool fetch = r == 0u && wp > pseg;
        wp -= fetch ? 1 : 0;
        top -= fetch ? 32u : 0u;
        r = fetch ? ahead : r;
        if (fetch && wp > pseg) ahead = wp[-1];
        const uint32_t z = (uint32_t)__clz((int)r);   // 32 for an empty word: nothing is written then
        const bool emit = r != 0u;
        dst -= emit ? 1 : 0;
        if (emit) *dst = (uint16_t)(top - z);
        r &= ~shr_clamped(0x80000000u, z);             // a shift by 32 gives zero: an empty word stays empty
      }
    }
    if (warp == 0 && prev >= 0) {
      // number of stage-3 bytes in all ranges before `prev`: windows of 256 predecessors, nearest first, the first
      // window loaded above
      uint32_t prefix = 0;
      if (prev > 0) {
        int spins = 0;
        bool found = false, loaded = true;
        for (int p0 = prev - 1; p0 >= 0 && !found; ) {
          if (!loaded) {
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const int p = p0 - 32 * u - lane;
              win[u] = p >= 0 ? ld_relaxed_u64(state + p) : kIdsPrefixKnown;
            }
          }
          loaded = false;
          bool ready = true;
#pragma unroll
          for (int u = 0; u < 8; ++u) ready = ready && (win[u] >> 32) != 0ull;
          if (!__all_sync(0xFFFFFFFFu, ready)) {
            if (++spins > kIdsSpinLimit) {   // cannot happen with tickets in launch order; give up rather than hang
              if (lane == 0) atomicOr(dev_status, 2u);
              break;
            }
            __nanosleep(20);
            continue;
          }
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            if (found) continue;
            const uint32_t known = __ballot_sync(0xFFFFFFFFu, (win[u] >> 32) == 2ull);
            const int stop = known ? __ffs((int)known) - 1 : 31;   // nearest predecessor whose prefix is known
            uint32_t v = lane <= stop ? (uint32_t)win[u] : 0u;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
            prefix += v;
            found = known != 0u;
          }
          p0 -= 256;
        }
        if (lane == 0) atomicExch(state + prev, kIdsPrefixKnown | (unsigned long long)(prefix + prev_total));
      }
      if (lane == 0) {
        prefix_sh = prefix;
        if (prev == ranges - 1 && count != nullptr) *count = prefix + prev_total;
      }
    }
    __syncthreads();
    if (prev >= 0) {
      const int64_t prefix = prefix_sh;
      const int64_t prev_base = prev * range_bytes - head;   // input position of the range's first byte
      if (fits) {
        // 4. a warp instruction writes 32 consecutive positions
        const int32_t id0 = (int32_t)prev_base;
        int32_t* const out = ids + prefix;
        if (prefix + (int64_t)prev_total <= ids_cap) {
#pragma unroll 4
          for (uint32_t t = threadIdx.x; t < prev_total; t += kIdsThreads) out[t] = id0 + (int32_t)staged[t];
        } else {
          for (uint32_t t = threadIdx.x; t < prev_total; t += kIdsThreads)
            if (prefix + t < ids_cap) out[t] = id0 + (int32_t)staged[t];
        }
      } else {
        int64_t at = prefix + prev_local;
        int64_t first = prev_base + warp_first + (int64_t)(lane * words) * 32;
        for (int i = 0; i < words; ++i, first += 32)
          for (uint32_t r = pseg[i]; r != 0u; r &= r - 1u, ++at)
            if (at < ids_cap) ids[at] = (int32_t)(first + __ffs((int)r) - 1);
      }
    }
    prev = cur ? range : -1;
    prev_local = warp_off + incl - mine;   // place of the lane's first position among the range's
    prev_mine = mine;
    prev_turns = turns;
    prev_total = total;
    range = next;
    // No barrier here: the next turn writes the other half of the bit map and meets a barrier before it touches the
    // staging area or the shared words that this turn has read.
    __syncwarp();
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
}

// ---------------------------------------------------------------------------------------------
// Conditional coverage (Proposition 2): a candidate is ranked against the calibration scores of its own
// input only.  The per-input buffers are ascending segments of one array.
//   numer = 1 + #{own segment >= s},  denom = |segment| + 1,  p = numer / denom;  reject iff
//   1 <= numer <= floor(alpha * denom)  (evaluated in IEEE double, as on the host for the marginal form).
// When the candidates of one input arrive together a warp stages the few segments it needs in shared memory.
// When they do not, every load of a search is a 32-byte sector of its own from L2, and those sectors are what
// bounds the kernel; the search is then made over the aligned groups of eight entries that overlap the segment
// (one probe per step, at a group's last entry) and finished with a single 32-byte load of the group found.
// ---------------------------------------------------------------------------------------------
constexpr int kCondStage = 512;   // calibration entries a warp can stage in shared memory (2 KB)

// Lower bound of four scores in their own segments [lo, lo + len) of `data` (shared memory), advanced together so
// that the dependent loads overlap.  The halving form: while more than one entry is left, the first half of them
// is dropped if its last entry is below the score; one comparison settles the last entry.  A step costs a load,
// a comparison and a select, and leaves no length to keep besides the one count.
__device__ __forceinline__ void lower_bound_four(const float* data, const float (&s)[4], int (&lo)[4], int (&len)[4]) {
  int left[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) left[e] = len[e] > 0 ? len[e] : 0;
  while (max(max(left[0], left[1]), max(left[2], left[3])) > 1) {
    float v[4];
    int half[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      half[e] = left[e] >> 1;   // 0 once at most one entry is left: nothing is read then
      v[e] = half[e] > 0 ? data[lo[e] + half[e] - 1] : __uint_as_float(0x7FC00000u);
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      lo[e] += v[e] < s[e] ? half[e] : 0;   // NaN compares false
      left[e] -= half[e];
    }
  }
#pragma unroll
  for (int e = 0; e < 4; ++e)
    if (left[e] == 1 && data[lo[e]] < s[e]) lo[e] += 1;
}

// The same in global memory, for segments [lo, end) with len = end - lo entries (len <= 0: nothing to search).
// Group g is calib[8 g, 8 g + 8).  All entries of a group whose last entry is below s are below s, and none of a
// group after one whose last entry is not: the first group of the segment whose last entry is not below s (the
// segment's last group if there is none) holds the boundary.  It is found by bisection over the groups, one probe a
// step, and read whole with one 32-byte load (`vec8`: calib is 32-byte aligned; `total` entries exist).
__device__ __forceinline__ void lower_bound_four_global(const float* __restrict__ calib, int total, bool vec8,
                                                        const float (&s)[4], int (&lo)[4], const int (&end)[4],
                                                        const int (&len)[4]) {
  const float qnan = __uint_as_float(0x7FC00000u);
  int g[4], gn[4];   // the boundary group is in [g, g + gn]
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    g[e] = lo[e] >> 3;
    gn[e] = len[e] > 0 ? ((end[e] - 1) >> 3) - g[e] : 0;
  }
  while (max(max(gn[0], gn[1]), max(gn[2], gn[3])) > 0) {
    float v[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = gn[e] > 0 ? __ldg(calib + 8 * (g[e] + (gn[e] >> 1)) + 7) : qnan;   // inside the segment
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (gn[e] > 0) {
        const int half = gn[e] >> 1;
        const bool less = v[e] < s[e];
        g[e] = less ? g[e] + half + 1 : g[e];
        gn[e] = less ? gn[e] - half - 1 : half;
      }
    }
  }
  // one candidate at a time: eight registers of loaded entries instead of thirty-two
#pragma unroll
  for (int h = 0; h < 4; h += 1) {
    float w[1][8];
#pragma unroll
    for (int e = h; e < h + 1; ++e) {
      const int g0 = 8 * g[e];
      if (len[e] > 0 && vec8 && g0 + 8 <= total) {
        asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=f"(w[e - h][0]), "=f"(w[e - h][1]), "=f"(w[e - h][2]), "=f"(w[e - h][3]), "=f"(w[e - h][4]),
                       "=f"(w[e - h][5]), "=f"(w[e - h][6]), "=f"(w[e - h][7])
                     : "l"(calib + g0));
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i)
          w[e - h][i] = (len[e] > 0 && g0 + i >= lo[e] && g0 + i < end[e]) ? __ldg(calib + g0 + i) : qnan;
      }
    }
#pragma unroll
    for (int e = h; e < h + 1; ++e) {
      if (len[e] > 0) {
        const int g0 = 8 * g[e];
        int c = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) c += (g0 + i >= lo[e] && g0 + i < end[e] && w[e - h][i] < s[e]) ? 1 : 0;
        lo[e] = max(g0, lo[e]) + c;
      }
    }
  }
}

// total: entries of calib that exist.  A group whose offsets do not describe a part of them (negative, beyond
// total, or decreasing) is treated like a group id out of range: flagged, and its candidates get no score.
__global__ void __launch_bounds__(256, 5)
rank_conditional_kernel(const float* __restrict__ scores, const int32_t* __restrict__ group_ids, int64_t Nc,
                        const float* __restrict__ calib, int total, const int32_t* __restrict__ seg_offsets, int G,
                        uint32_t* __restrict__ numer, uint32_t* __restrict__ denom, float* __restrict__ pvalue,
                        bool vec4, bool vec8, unsigned int* __restrict__ dev_status) {
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
      bool ok = g[e] >= 0 && g[e] < G;
      int a = ok ? __ldg(seg_offsets + g[e]) : 0, b = ok ? __ldg(seg_offsets + g[e] + 1) : 0;
      ok = ok && a >= 0 && a <= b && b <= total;
      if (!ok) a = b = 0;
      bad = bad || (!ok && j + e < Nc);
      lo[e] = a;
      end[e] = b;
      den[e] = ok ? (uint32_t)(b - a) + 1u : 1u;
      len[e] = (ok && s[e] == s[e]) ? b - a : -1;   // -1: no score (NaN, or no calibration set)
      if (len[e] > 0) {
        span_lo = min(span_lo, a);
        span_hi = max(span_hi, b);
      }
    }
    if (bad) atomicOr(dev_status, 4u);  // no such group, or not a part of the calibration array: no score
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
      lower_bound_four(stage - span_lo, s, lo, len);
    } else {
      lower_bound_four_global(calib, total, vec8, s, lo, end, len);
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
    if ((threadIdx.x & 31) == 0 && c[i]) atomicAdd(counts + i, c[i]);   // counts are zeroed by the host
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

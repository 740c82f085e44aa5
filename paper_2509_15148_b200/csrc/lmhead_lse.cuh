// Fused LM-head projection + online log-sum-exp + gather of the draft token's logit (sm_100a).
//
// logits[i, v] = sum_k H[i, k] * W[v, k] are produced in 128 x 256 tiles per CTA (256 x 256 per CTA pair)
// by tcgen05.mma (bf16 in, fp32 accumulators in tensor memory), read back with tcgen05.ld and reduced
// per row to a running (max, sum of exponentials); the logit of the row's own token is picked out on the
// way.  Logits never leave the SM.  A second, tiny kernel merges the per-chunk partials into token log-probs,
// a third reduces them per sample.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace atts {

constexpr int kBlockM = 128;   // rows of H per CTA tile (= TMEM lanes)
constexpr int kBlockN = 256;   // vocabulary entries per tile (= TMEM columns per accumulator)
constexpr int kBlockK = 64;    // bf16 elements per shared-memory stage row (128 bytes = swizzle span)
constexpr int kUmmaK = 16;     // K of one tcgen05.mma (kind::f16)
constexpr int kScoreThreads = 192;  // warp 0: TMA producer, warp 1: MMA issuer, warps 2-5: epilogue
constexpr int kTmemCols = 512;      // two 256-column accumulators
constexpr long long kWaitLimitCycles = 4000000000LL;  // default bound of a pipeline wait, ~2 s: far beyond any legitimate one

// Two forms of the kernel.  CTAS = 1: every CTA computes 128 x 256 tiles on its own.  CTAS = 2: the two CTAs
// of a cluster compute one 256 x 256 tile with tcgen05.mma.cta_group::2; each loads its own 128 rows of H and
// its own 128 of the 256 vocabulary rows, so a CTA moves a third less data through L2 and shared memory per
// flop, and the smaller stage leaves room for a deeper ring.
template <int CTAS>
struct ScoreCfg {
  static constexpr int kRowsPerUnit = kBlockM * CTAS;          // rows of H per unit (row block)
  static constexpr int kBRows = kBlockN / CTAS;                // vocabulary rows a CTA loads per stage
  static constexpr int kABytes = kBlockM * kBlockK * 2;
  static constexpr int kBBytes = kBRows * kBlockK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kStages = CTAS == 1 ? 4 : 6;
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
  // Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128 * CTAS, N = 256.
  static constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBlockN >> 3) << 17) |
                                     ((uint32_t)(kRowsPerUnit >> 4) << 24);
};

// Static schedule of one launch.  A unit is (row block rb, vocabulary chunk c); chunk c covers the
// tiles [c*NT/C, (c+1)*NT/C).  Units are numbered panel by panel (Gr row blocks each), chunk-major
// inside a panel, and dealt round-robin to the workers (CTAs, or CTA pairs), so that workers running at
// the same time share vocabulary tiles in L2 while their row blocks stay L2-resident.
struct ScorePlan {
  int M, V;
  int RB;      // row blocks  = ceil(M / rows per unit)
  int NT;      // vocab tiles = ceil(V / 256)
  int KB;      // k blocks    = d / 64
  int C;       // chunks per row block (partials per row)
  int Gr;      // row blocks per panel
  int units;   // RB * C
  int M_pad;   // RB * rows per unit
  int ctas;    // 1 or 2: CTAs per worker
  int vocab_offset;  // id of this W's first row (0 unless W is a slice of a sharded vocabulary)
  long long wait_limit;  // cycles after which a pipeline wait gives up (the host's setting; kWaitLimitCycles by default)
  int withhold_loads;    // diagnostic: the producer issues no loads, so the first wait for data must run out
};

__host__ __device__ inline void decode_unit(const ScorePlan& p, int u, int& rb, int& c, int& nt0, int& nt1) {
  const int per_panel = p.Gr * p.C;
  const int panel = u / per_panel;
  const int rem = u - panel * per_panel;
  const int r0 = panel * p.Gr;
  const int Rp = (p.RB - r0) < p.Gr ? (p.RB - r0) : p.Gr;
  c = rem / Rp;
  rb = r0 + (rem - c * Rp);
  nt0 = (int)(((long long)c * p.NT) / p.C);
  nt1 = (int)(((long long)(c + 1) * p.NT) / p.C);
}

// num_workers: CTAs (ctas == 1) or CTA pairs (ctas == 2) that run concurrently.
inline ScorePlan make_score_plan(int64_t M, int64_t d, int64_t V, int num_workers, int ctas) {
  ScorePlan p{};
  const int rows = kBlockM * ctas;
  p.ctas = ctas;
  p.M = (int)M;
  p.V = (int)V;
  p.RB = (int)((M + rows - 1) / rows);
  p.NT = (int)((V + kBlockN - 1) / kBlockN);
  p.KB = (int)(d / kBlockK);
  p.M_pad = p.RB * rows;
  int cmax = p.NT < num_workers ? p.NT : num_workers;
  if (p.RB > 0 && cmax > (1 << 30) / p.RB) cmax = (1 << 30) / p.RB;  // keep RB * C inside int
  if (cmax < 1) cmax = 1;
  long long best = -1;
  int bestC = 1;
  for (int C = 1; C <= cmax; ++C) {
    long long waves = ((long long)p.RB * C + num_workers - 1) / num_workers;
    long long span = waves * ((p.NT + C - 1) / C);
    if (best < 0 || span < best) { best = span; bestC = C; }
  }
  p.C = bestC;
  // Panel height: about 30 MB of H per panel stays L2-resident while W streams past it (measured: larger panels
  // thrash, DRAM reads grow 2x).  A multiple of 4, because workers whose index is congruent modulo Gr share a row
  // block and multiples of 4 measured 5-10 % faster than neighbouring heights.
  long long gr = ((30ll << 20) / ((long long)rows * d * 2) + 2) / 4 * 4;
  if (gr < 4) gr = 4;
  if (gr > p.RB) gr = p.RB;
  p.Gr = (int)(gr < 1 ? 1 : gr);
  p.units = p.RB * p.C;
  return p;
}

// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up when another thread of the CTA has raised `abort` or after `limit` cycles, in which
// case it raises `abort` itself - and, in a CTA pair, the flag of the other CTA too (`peer_abort`, an address in
// the cluster's shared window, 0 for a single CTA), so that both leave together.  Returns false when it gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort, long long limit,
                                          uint32_t peer_abort) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++spins & 7u) == 0u) {
      if (*abort) return false;
      if (clock64() - t0 > limit) {
        *abort = 1u;
        if (peer_abort) asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(peer_abort), "r"(1u) : "memory");
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t smem_dst, const CUtensorMap* tmap, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
// ---- cluster forms (CTA pair) ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address, in the cluster's shared window, of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load of a CTA pair: the data lands in this CTA's shared memory, the bytes are counted on the mbarrier
// `bar_cluster_addr`, which may live in the other CTA of the pair.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t smem_dst, const CUtensorMap* tmap, uint32_t bar_cluster_addr, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
      : "memory");
}
// D[tmem of both CTAs] (+)= A * B^T, 256 x 256 x 16 over the CTA pair (each CTA supplies 128 rows of A and 128 of B).
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// One arrival on the mbarrier at this offset in both CTAs of the pair once the MMAs issued so far have finished.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}

__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* tmap) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tmap)) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T, 128 x 256 x 16, bf16 inputs, fp32 accumulate, one CTA.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The mbarrier gets one arrival once every tcgen05.mma issued so far by this thread has finished.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Shared-memory matrix descriptor: K-major operand, rows of 128 bytes, 128-byte swizzle, groups of
// 8 rows 1024 bytes apart (the layout a 64-element-wide TMA box with SWIZZLE_128B produces).
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);   // start address, 16-byte units
  d |= (uint64_t)1u << 16;                        // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024u >> 4) << 32;              // stride byte offset between 8-row groups
  d |= (uint64_t)1u << 46;                        // descriptor version of sm_100
  d |= (uint64_t)2u << 61;                        // SWIZZLE_128B
  return d;
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

#define ATTS_TMEM_LD_32(taddr, v)                                                                         \
  asm volatile(                                                                                           \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                           \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "                           \
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"           \
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),   \
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),          \
        "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]),        \
        "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]),        \
        "=r"(v[29]), "=r"(v[30]), "=r"(v[31])                                                             \
      : "r"(taddr)                                                                                        \
      : "memory")

__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ------------------------------------------------------------------------------------------
// K1  the fused kernel.  Persistent: worker w (a CTA, or a CTA pair) runs units w, w + workers, ...
//   partial[c * M_pad + row] = (max_v z, sum_v exp(z - max)) over the vocabulary chunk c
//   gathered[row]            = z[row, token_ids[row]]   (written by the chunk that holds the id)
// Barriers.  full[s]: stage s of the ring holds data (one per worker: with two CTAs it lives in the leader,
// CTA 0 of the pair, and counts the bytes of both CTAs' loads).  empty[s]: the MMAs reading stage s are done
// (one per CTA; the leader's commit reaches both).  tmem_full[a] / tmem_empty[a]: accumulator a is complete /
// has been read by every epilogue warp of the worker (tmem_empty lives in the leader).
// ------------------------------------------------------------------------------------------
template <int CTAS>
__global__ void __launch_bounds__(kScoreThreads, 1)
lmhead_lse_kernel(const __grid_constant__ CUtensorMap tmap_h, const __grid_constant__ CUtensorMap tmap_w,
                  const int32_t* __restrict__ token_ids, const float* __restrict__ row_scale, const ScorePlan plan,
                  float2* __restrict__ partial, float* __restrict__ gathered, unsigned int* __restrict__ dev_status) {
  using Cfg = ScoreCfg<CTAS>;
  constexpr int kStages = Cfg::kStages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + kStages * Cfg::kStageBytes);
  const uint32_t bar0 = smem_base + kStages * Cfg::kStageBytes;
  // barrier slots: full[0..S), empty[S..2S), tmem_full[2S..2S+2), tmem_empty[2S+2..2S+4)
  auto full_bar = [&](int s) { return bar0 + 8u * (uint32_t)s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (uint32_t)(kStages + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (uint32_t)(2 * kStages + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (uint32_t)(2 * kStages + 2 + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + 2 * kStages + 4);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = CTAS == 2 ? cluster_ctarank() : 0u;   // 0 = leader
  const long long wait_limit = plan.wait_limit;
  const uint32_t peer_abort = CTAS == 2 ? map_to_cta(smem_u32((const void*)abort_flag), rank ^ 1u) : 0u;
  const int worker = blockIdx.x / CTAS;
  const int workers = gridDim.x / CTAS;

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmap_h);
    prefetch_tmap(&tmap_w);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), 4 * CTAS);
    }
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    if (CTAS == 1) {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)kTmemCols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)kTmemCols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  if (CTAS == 2) cluster_sync_all();   // the peer's barriers are initialised before anything signals them
  else __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer (every CTA loads its own operand halves) ----------------
    if (lane == 0 && !plan.withhold_loads) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = worker; u < plan.units && ok; u += workers) {
        int rb, c, nt0, nt1;
        decode_unit(plan, u, rb, c, nt0, nt1);
        const int row0 = rb * Cfg::kRowsPerUnit + (int)rank * kBlockM;
        for (int nt = nt0; nt < nt1 && ok; ++nt) {
          const int col0 = nt * kBlockN + (int)rank * Cfg::kBRows;
          for (int kb = 0; kb < plan.KB; ++kb) {
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, wait_limit, peer_abort)) { ok = false; break; }
            const uint32_t sa = smem_base + (uint32_t)stage * Cfg::kStageBytes;
            if (CTAS == 1) {
              mbar_expect_tx(full_bar(stage), Cfg::kStageBytes);
              tma_load_2d(sa, &tmap_h, full_bar(stage), kb * kBlockK, row0);
              tma_load_2d(sa + Cfg::kABytes, &tmap_w, full_bar(stage), kb * kBlockK, col0);
            } else {
              if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * Cfg::kStageBytes);
              const uint32_t leader_full = map_to_cta(full_bar(stage), 0);
              tma_load_2d_pair(sa, &tmap_h, leader_full, kb * kBlockK, row0);
              tma_load_2d_pair(sa + Cfg::kABytes, &tmap_w, leader_full, kb * kBlockK, col0);
            }
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------- MMA issuer (the leader CTA issues for the pair) ----------------
    if (lane == 0 && rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int u = worker; u < plan.units && ok; u += workers) {
        int rb, c, nt0, nt1;
        decode_unit(plan, u, rb, c, nt0, nt1);
        for (int nt = nt0; nt < nt1 && ok; ++nt) {
          if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, wait_limit, peer_abort)) { ok = false; break; }
          tc_fence_after();
          const uint32_t tmem_d = tmem_base + (uint32_t)acc * kBlockN;
          for (int kb = 0; kb < plan.KB; ++kb) {
            if (!mbar_wait(full_bar(stage), phase, abort_flag, wait_limit, peer_abort)) { ok = false; break; }
            tc_fence_after();
            const uint32_t sa = smem_base + (uint32_t)stage * Cfg::kStageBytes;
            const uint64_t da = umma_smem_desc(sa);
            const uint64_t db = umma_smem_desc(sa + Cfg::kABytes);
#pragma unroll
            for (int k = 0; k < kBlockK / kUmmaK; ++k) {
              // 16 bf16 = 32 bytes further along K inside the swizzled row: +2 in 16-byte units
              if (CTAS == 1) umma_bf16(tmem_d, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), Cfg::kIdesc, (uint32_t)((kb | k) != 0));
              else umma_bf16_pair(tmem_d, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), Cfg::kIdesc, (uint32_t)((kb | k) != 0));
            }
            if (CTAS == 1) umma_commit(empty_bar(stage));
            else umma_commit_pair(empty_bar(stage));
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          if (CTAS == 1) umma_commit(tfull_bar(acc));
          else umma_commit_pair(tfull_bar(acc));
          acc ^= 1;
          if (acc == 0) acc_phase ^= 1u;
        }
      }
    }
    __syncwarp();
  } else {
    // ---------------- epilogue: 4 warps, warp w reads TMEM lanes 32*(w%4) .. +31 of its own CTA ----------------
    const int quarter = warp & 3;
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const float kLog2e = 1.4426950408889634f;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int u = worker; u < plan.units && ok; u += workers) {
      int rb, c, nt0, nt1;
      decode_unit(plan, u, rb, c, nt0, nt1);
      const int row = rb * Cfg::kRowsPerUnit + (int)rank * kBlockM + quarter * 32 + lane;
      // the token's column in this W; ids outside [0, V) (another vocabulary slice, or invalid) never match
      int y = (row < plan.M) ? token_ids[row] - plan.vocab_offset : -1;
      if (y >= plan.V) y = -1;
      // optional per-row factor on the logits (finite, > 0): folded into the exponent's scale, so it costs nothing per
      // element; the running maximum is kept on the unscaled logits
      const float rs = (row_scale != nullptr && row < plan.M) ? row_scale[row] : 1.f;
      const float kScale = rs * kLog2e;
      float m = -INFINITY, l = 0.f;
      for (int nt = nt0; nt < nt1; ++nt) {
        if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, wait_limit, peer_abort)) { ok = false; break; }
        tc_fence_after();
        const int n0 = nt * kBlockN;
        const uint32_t taddr = tmem_base + lane_base + (uint32_t)(acc * kBlockN);
#pragma unroll 1
        for (int j = 0; j < kBlockN / 32; ++j) {
          const int col0 = n0 + j * 32;
          if (col0 >= plan.V) break;  // uniform: the rest of the tile is beyond the vocabulary
          uint32_t v[32];
          ATTS_TMEM_LD_32(taddr + (uint32_t)(j * 32), v);
          tmem_ld_wait();
          if (col0 + 32 > plan.V) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (col0 + i >= plan.V) v[i] = 0xFF800000u;  // -inf
          }
          if ((unsigned)(y - col0) < 32u) {
            const int yi = y - col0;
            float g = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (i == yi) g = __uint_as_float(v[i]);
            gathered[row] = g * rs;
          }
          float cmax = __uint_as_float(v[0]);
#pragma unroll
          for (int i = 1; i < 32; ++i) cmax = fmaxf(cmax, __uint_as_float(v[i]));
          const float m_new = fmaxf(m, cmax);
          const float ms = m_new * kScale;
          float s0 = 0.f, s1 = 0.f;
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            s0 += ex2_approx(fmaf(__uint_as_float(v[i]), kScale, -ms));
            s1 += ex2_approx(fmaf(__uint_as_float(v[i + 1]), kScale, -ms));
          }
          l = l * ex2_approx((m - m_new) * kScale) + (s0 + s1);
          m = m_new;
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (CTAS == 1) mbar_arrive(tempty_bar(acc));
          else mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));
        }
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
      if (ok && row < plan.M) partial[(size_t)c * plan.M_pad + row] = make_float2(m * rs, l);
    }
  }

  // ---------------- teardown ----------------
  tc_fence_before();
  if (CTAS == 2) cluster_sync_all();   // neither CTA leaves while the other may still touch its memory
  else __syncthreads();
  if (*abort_flag) {
    // A wait expired.  Record it, give copies and MMAs still in flight time to land, then free TMEM.
    if (threadIdx.x == 0) atomicOr(dev_status, 2u);
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    if (CTAS == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
  }
}

// ------------------------------------------------------------------------------------------
// Row factor of an RMS normalisation: out[i] = 1 / sqrt(mean_k h[i, k]^2 + eps).  One warp per row, 128-bit
// loads, fp32 accumulation in a fixed order.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
rms_inv_kernel(const uint4* __restrict__ hidden, int M, int d, float eps, float* __restrict__ out) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= M) return;
  const int lane = threadIdx.x & 31;
  const int vecs = d / 8;  // 8 bf16 per 16 bytes
  const uint4* p = hidden + (size_t)row * vecs;
  float acc = 0.f;
  for (int i = lane; i < vecs; i += 32) {
    const uint4 q = __ldg(p + i);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const float lo = __uint_as_float(w[t] << 16), hi = __uint_as_float(w[t] & 0xFFFF0000u);
      acc = fmaf(lo, lo, acc);
      acc = fmaf(hi, hi, acc);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
  if (lane == 0) out[row] = rsqrtf(acc / (float)d + eps);
}

// ------------------------------------------------------------------------------------------
// K2a  merge the per-chunk partials of a row: LSE = Mx + log(sum_c l_c * exp(m_c - Mx)),
//      token_logprob = gathered - LSE.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
lse_combine_kernel(const float2* __restrict__ partial, const float* __restrict__ gathered,
                   const int32_t* __restrict__ token_ids, int M, int M_pad, int C, int V,
                   float* __restrict__ logprob_ws, float* __restrict__ logprob_out,
                   unsigned int* __restrict__ dev_status) {
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= M) return;
  float mx = -INFINITY;
  for (int c = 0; c < C; ++c) mx = fmaxf(mx, partial[(size_t)c * M_pad + row].x);
  float sum = 0.f;
  for (int c = 0; c < C; ++c) {
    float2 p = partial[(size_t)c * M_pad + row];
    sum += p.y * expf(p.x - mx);
  }
  const int y = token_ids[row];
  float lp;
  if (y < 0 || y >= V) {
    lp = __uint_as_float(0x7FC00000u);
    atomicOr(dev_status, 1u);
  } else {
    lp = gathered[row] - (mx + logf(sum));
  }
  logprob_ws[row] = lp;
  if (logprob_out) logprob_out[row] = lp;
}

// ------------------------------------------------------------------------------------------
// Vocabulary sharding (W split by rows over GPUs).  A slice's chunk partials are reduced to one triple per
// row, stats[row] = (max z, sum exp(z - max), z[token] or -inf if the token lies in another slice); after the
// ranks have exchanged their triples, G triples per row are merged exactly as chunk partials are.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
slice_stats_kernel(const float2* __restrict__ partial, const float* __restrict__ gathered,
                   const int32_t* __restrict__ token_ids, int M, int M_pad, int C, int V, int vocab_offset,
                   float* __restrict__ stats) {
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= M) return;
  float mx = -INFINITY;
  for (int c = 0; c < C; ++c) mx = fmaxf(mx, partial[(size_t)c * M_pad + row].x);
  float sum = 0.f;
  for (int c = 0; c < C; ++c) {
    const float2 p = partial[(size_t)c * M_pad + row];
    sum += p.y * expf(p.x - mx);
  }
  const int y = token_ids[row] - vocab_offset;
  stats[3 * (size_t)row + 0] = mx;
  stats[3 * (size_t)row + 1] = sum;
  stats[3 * (size_t)row + 2] = (y >= 0 && y < V) ? gathered[row] : -INFINITY;
}

__global__ void __launch_bounds__(256)
stats_combine_kernel(const float* __restrict__ stats, int G, int M, float* __restrict__ logprob_ws,
                     float* __restrict__ logprob_out, unsigned int* __restrict__ dev_status) {
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= M) return;
  float mx = -INFINITY, g = -INFINITY;
  for (int s = 0; s < G; ++s) {
    const float* t = stats + 3 * ((size_t)s * M + row);
    mx = fmaxf(mx, t[0]);
    g = fmaxf(g, t[2]);
  }
  float sum = 0.f;
  for (int s = 0; s < G; ++s) {
    const float* t = stats + 3 * ((size_t)s * M + row);
    sum += t[1] * expf(t[0] - mx);
  }
  float lp;
  if (g == -INFINITY) {  // no slice held the token: id out of range
    lp = __uint_as_float(0x7FC00000u);
    atomicOr(dev_status, 1u);
  } else {
    lp = g - (mx + logf(sum));
  }
  logprob_ws[row] = lp;
  if (logprob_out) logprob_out[row] = lp;
}

// ------------------------------------------------------------------------------------------
// K2b  per-sample score: one block per sample, fixed summation order (thread t takes rows
//      a + t, a + t + 256, ...; then a fixed tree), fp64 accumulation.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
segment_score_kernel(const float* __restrict__ logprob, const int32_t* __restrict__ seg_offsets, int M,
                     int S, int mode, float* __restrict__ score) {
  const int k = blockIdx.x;
  if (k >= S) return;
  int a = seg_offsets[k], b = seg_offsets[k + 1];
  a = max(0, min(a, M));
  b = max(a, min(b, M));
  double acc = 0.0;
  for (int i = a + threadIdx.x; i < b; i += 256) acc += (double)logprob[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xFFFFFFFFu, acc, o);
  __shared__ double sh[8];
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w = 0; w < 8; ++w) t += sh[w];
    float out;
    if (b <= a) {
      out = __uint_as_float(0x7FC00000u);
    } else {
      if (mode == 0 || mode == 2) t /= (double)(b - a);
      out = (float)((mode == 0 || mode == 1) ? -t : t);
    }
    score[k] = out;
  }
}

}  // namespace atts

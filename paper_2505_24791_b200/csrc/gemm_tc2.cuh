// Two-CTA form of the tensor-core GEMM:  C[M,N] = A[M,K] * W[N,K]^T, bf16 operands, fp32 accumulation,
// one 256 x 256 output tile per pair of CTAs (a thread-block cluster of 2 on neighbouring SMs).
//
// Why: with one CTA per 128 x 256 tile every 64-wide k slab costs 48 KB of operand traffic from L2 per
// 512 tensor cycles, and the mainloop runs at the L2 fabric rate instead of the tensor rate.  In a pair,
// CTA r loads its own 128 rows of A and only its half (128 rows) of the 256 weight rows; the
// `tcgen05.mma.cta_group::2` instruction issued by the leader CTA lets both tensor cores read both halves
// of the weight tile, so each SM moves 32 KB per slab for the same math.
//
//   * both CTAs run a TMA producer for their own operand slices (plain per-CTA loads, no multicast); the
//     loads of both CTAs complete on the LEADER's "full" mbarrier (its address mapped with mapa);
//   * the leader's MMA thread waits on that barrier, issues the pair MMAs and commits with
//     `tcgen05.commit.cta_group::2 ... multicast::cluster` to the "empty" (stage free) and "accumulator
//     full" barriers of BOTH CTAs;
//   * each CTA's epilogue warps read their own CTA's tensor memory (128 rows x 256 columns, two buffers)
//     and release the accumulator on the leader's "accumulator empty" barrier (the peer arrives remotely);
//   * the epilogue itself is the bulk-store form of gemm_tc.cuh (functors with kTmaCols > 0).
// All mbarrier waits are bounded as in gemm_tc.cuh; the two cluster-wide barriers (after set-up, before
// the tensor memory is freed) are reached by every thread on every path.
#pragma once
#include "gemm_tc.cuh"

namespace tc2 {

using namespace tc;

constexpr int BN2 = 256;      // tile columns (each CTA loads 128 of the weight rows)
constexpr int STAGES2 = 6;    // 6 x (16 KB A + 16 KB W half)

struct Smem2 {
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = (BN2 / 2) * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGE_OUT_OFFSET = STAGES2 * STAGE_BYTES;
  static constexpr int STAGE_OUT_BYTES = NUM_EPI_WARPS * 4096;
  static constexpr int TILE_BIAS_OFFSET = STAGE_OUT_OFFSET + STAGE_OUT_BYTES;
  static constexpr int BAR_OFFSET = TILE_BIAS_OFFSET + BN2 * 4;
  static constexpr int NUM_BARS = 2 * STAGES2 + 4;
  static constexpr int TOTAL = BAR_OFFSET + NUM_BARS * 8 + 16 + 1024;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// per-CTA load of a pair kernel: the completion bytes go to the mbarrier at `bar_cluster_addr` (the leader's)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar_cluster_addr)
      : "memory");
}
__device__ __forceinline__ void umma_f16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  const uint32_t z = 0;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(z)
      : "memory");
}
// arrives on the mbarrier at this shared-memory offset in both CTAs of the pair once the MMAs issued so far are done
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
               "h"(mask)
               : "memory");
}
__host__ __device__ constexpr uint32_t make_idesc_pair(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

template <class Epi>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_a_lo,
                const __grid_constant__ CUtensorMap map_w, int M, int N, int K, int split, Epi epi, int* err, int ksplit,
                int part_rows) {
  static_assert(Epi::kTmaCols > 0, "the pair kernel has the bulk-store epilogue only");
  using SL = Smem2;
  extern __shared__ uint8_t smem_raw2[];
  pdl_launch_dependents();  // the next kernel of the stream may be scheduled; it waits for this one to complete
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw2) + 1023) & ~(uintptr_t)1023);
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_base + SL::BAR_OFFSET;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES2 + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES2 + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES2 + 2 + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + SL::BAR_OFFSET + SL::NUM_BARS * 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = leader
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int tiles_m = (M + 2 * BM - 1) / (2 * BM), tiles_n = (N + BN2 - 1) / BN2;
  // ksplit > 1: every output tile is computed ksplit times, each over its own range of k slabs; slice s stores its
  // partial tile part_rows * s rows further down and the consumer adds the slices in index order.  Tile index =
  // (m tile, n tile, slice) with the slice fastest.
  const int num_tiles = tiles_m * tiles_n * ksplit;
  // split != 0: A is an error-compensated pair (hi + lo).  A stage then holds [A_hi | A_lo | W] of one k slab
  // (48 KB, four stages in the same 192 KB), so the weight slab is fetched once for both products.
  const int kblocks_all = (K + BK - 1) / BK;
  auto slab_begin = [&](int slice) { return (int)((long long)kblocks_all * slice / ksplit); };
  const uint32_t stage_bytes = split ? (uint32_t)(2 * SL::A_BYTES + SL::B_BYTES) : (uint32_t)SL::STAGE_BYTES;
  const int nstages = split ? 4 : STAGES2;
  const uint32_t w_off = split ? 2u * SL::A_BYTES : (uint32_t)SL::A_BYTES;
  constexpr uint32_t TMEM_COLS = 2 * BN2;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES2; ++s) {
      mbar_init(full_bar(s), 1);   // leader's: its own arrive.expect_tx; both CTAs' bytes complete on it
      mbar_init(empty_bar(s), 1);  // one multicast commit of the leader's MMA thread
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), 2 * NUM_EPI_WARPS);  // leader's: epilogue warps of both CTAs
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // pair-wide allocation: the same warp in both CTAs, same destination
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tcgen05_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers exist before anything signals them
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // everything above (barriers, tensor memory, cluster handshake) overlaps the previous kernel's tail; its
  // activations and the error word are complete from here on
  pdl_wait();
  // an earlier kernel failed: both CTAs skip the work (the leader's view decides, so the pair agrees)
  const bool dead = *reinterpret_cast<volatile int*>(err) != 0;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0 && !dead) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
        const int mn = tile / ksplit, slice = tile - mn * ksplit;
        const int m0 = (mn / tiles_n) * (2 * BM) + (int)rank * BM, n0 = (mn % tiles_n) * BN2 + (int)rank * (BN2 / 2);
        const int kb0 = slab_begin(slice), kblocks = slab_begin(slice + 1) - kb0;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, err, TFERR_WAIT_EMPTY)) { ok = false; break; }
          if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), 2 * stage_bytes);
          const uint32_t lead_full = map_to_cta(full_bar(stage), 0);
          const uint32_t sa = smem_base + stage * stage_bytes;
          const int kk = (kb0 + kb) * BK;
          tma_load_2d_pair(sa, &map_a, kk, m0, lead_full);
          if (split) tma_load_2d_pair(sa + SL::A_BYTES, &map_a_lo, kk, m0, lead_full);
          tma_load_2d_pair(sa + w_off, &map_w, kk, n0, lead_full);
          if (++stage == nstages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && rank == 0 && !dead) {
      constexpr uint32_t idesc = make_idesc_pair(2 * BM, BN2);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int it = 0;
      for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1;
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, err, TFERR_WAIT_TMEM_EMPTY)) { ok = false; break; }
        tcgen05_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN2;
        const int slice = tile % ksplit;
        const int kblocks = slab_begin(slice + 1) - slab_begin(slice);
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, err, TFERR_WAIT_FULL)) { ok = false; break; }
          tcgen05_fence_after();
          const uint32_t sa = smem_base + stage * stage_bytes;
          const uint64_t adesc = make_smem_desc(sa), bdesc = make_smem_desc(sa + w_off);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) umma_f16_pair(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (kb | k) != 0);
          if (split) {  // the low halves against the same weight slab, into the same accumulator
            const uint64_t ldesc = make_smem_desc(sa + SL::A_BYTES);
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) umma_f16_pair(d_tmem, ldesc + 2u * k, bdesc + 2u * k, idesc, 1u);
          }
          umma_commit_pair(empty_bar(stage));  // frees the stage in both CTAs
          if (++stage == nstages) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit_pair(tfull_bar(acc));  // accumulator complete, in both CTAs
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (both CTAs, warps 2..9)
    const int quad = warp & 3;
    const int cgroup = (warp - 2) >> 2;
    constexpr int NCH = BN2 / 32 / (NUM_EPI_WARPS / 4);
    constexpr int CPG = Epi::kTmaCols / 32;
    const int etid = threadIdx.x - 64;
    uint8_t* box = smem + SL::STAGE_OUT_OFFSET + (warp - 2) * 4096;
    const uint32_t box_addr = smem_u32(box);
    float* tile_bias = reinterpret_cast<float*>(smem + SL::TILE_BIAS_OFFSET);
    bool ok = !dead;
    int it = 0;
    // this thread's bias of the next tile is fetched one tile ahead, so its latency is off the epilogue's path
    float next_bias = 0.f;
    if (pair < num_tiles && etid < BN2) {
      const int nn = ((pair / ksplit) % tiles_n) * BN2 + etid;
      next_bias = epi.col_const(nn, nn < N);
    }
    for (int tile = pair; tile < num_tiles; tile += num_pairs, ++it) {
      const int mn = tile / ksplit, slice = tile - mn * ksplit;
      const int m0 = (mn / tiles_n) * (2 * BM) + (int)rank * BM, n0 = (mn % tiles_n) * BN2;
      const int acc = it & 1;
      const uint32_t acc_phase = (it >> 1) & 1;
      named_bar_sync(1, 32 * NUM_EPI_WARPS);
      if (etid < BN2) tile_bias[etid] = next_bias;
      named_bar_sync(1, 32 * NUM_EPI_WARPS);
      if (tile + num_pairs < num_tiles && etid < BN2) {
        const int nn = (((tile + num_pairs) / ksplit) % tiles_n) * BN2 + etid;
        next_bias = epi.col_const(nn, nn < N);
      }
      if (ok && !mbar_wait(tfull_bar(acc), acc_phase, err, TFERR_WAIT_TMEM_FULL)) ok = false;
      if (!ok) continue;
      tcgen05_fence_after();
      const int row0 = m0 + quad * 32;
      float v[NCH][32];
#pragma unroll
      for (int ch = 0; ch < NCH; ++ch)
        tmem_ld_32x32b_x32_issue(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN2 + (cgroup * NCH + ch) * 32), v[ch]);
      tmem_ld_wait();
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));  // release on the leader's barrier
      if (row0 < M) {
#pragma unroll
        for (int g = 0; g < NCH / CPG; ++g) {
          const int cl = (cgroup * NCH + g * CPG) * 32;
          if (n0 + cl < N)
            epi.template tma_box<CPG>(v[g * CPG], v[g * CPG + CPG - 1], tile_bias + cl, n0 + cl, row0 + slice * part_rows, box, box_addr,
                                      lane);
        }
      }
    }
    if (lane == 0) tma_store_wait_all();
  }

  // teardown: both CTAs meet before the pair's tensor memory is released
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1 && *reinterpret_cast<volatile int*>(err) != 0) {
    unsigned long long t0 = globaltimer_ns();  // a role gave up: let copies and MMAs in flight drain
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  cluster_sync_all();
  if (warp == 1) {
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace tc2

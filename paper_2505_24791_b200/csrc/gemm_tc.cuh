// Tensor-core GEMM for sm_100a:  C[M,N] = A[M,K] * W[N,K]^T, bf16 operands, fp32 accumulation.
//
//   * operands are brought to shared memory by TMA (cp.async.bulk.tensor, 128-byte swizzle), one
//     64-element K slab per pipeline stage, completion signalled on mbarriers;
//   * tcgen05.mma (kind::f16, M=128, N=BN, K=16) is issued by one thread and accumulates in tensor
//     memory; two accumulator buffers let the epilogue of tile i overlap the main loop of tile i+1;
//   * optionally A is a two-term bf16 pair (hi + lo, about 16 significant bits): the same tile then
//     accumulates A_hi W^T + A_lo W^T;
//   * the kernel is persistent: gridDim.x CTAs walk the tile list with a fixed stride;
//   * warp roles: warp 0 = TMA producer, warp 1 = TMEM allocator + MMA issuer, warps 2..9 =
//     epilogue (tcgen05.ld -> registers -> 32x32 transpose in shared memory -> functor, so that a
//     warp's global accesses are contiguous row segments).
// Every wait is bounded by wall time; a wait that expires records a code in *err and every role
// leaves its loops, so the kernel always returns and frees its tensor memory.
// No cluster launch and no multicast is used: each CTA loads its own operands.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "epilogue.cuh"

namespace tc {

constexpr int BM = 128;
constexpr int BK = 64;  // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int NUM_EPI_WARPS = 8;  // two warps per TMEM lane quadrant, alternating 32-column chunks
constexpr int NUM_THREADS = 64 + 32 * NUM_EPI_WARPS;
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;  // 2 s

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
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
// Bounded wait.  Returns false (after recording `code`) when `limit_ns` of wall time pass or another role
// already reported a failure.
__device__ __forceinline__ bool mbar_wait_limit(uint32_t bar, uint32_t parity, int* err, int code, unsigned long long limit_ns) {
  if (mbar_try_wait(bar, parity)) return true;
  unsigned long long t0 = globaltimer_ns();
  for (uint32_t spin = 1;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 255u) == 0) {
      if (*reinterpret_cast<volatile int*>(err) != 0) return false;
      if (globaltimer_ns() - t0 > limit_ns) {
        atomicCAS(err, 0, code);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* err, int code) {
  return mbar_wait_limit(bar, parity, err, code, WAIT_LIMIT_NS);
}

// Self-test of the bounded wait: one thread waits on an mbarrier that nothing ever arrives on.  The wait runs out
// after limit_ns, records TFERR_WAIT_SELFTEST in *err and the kernel returns normally (nothing faults or hangs).
__global__ void wait_selftest_kernel(int* err, unsigned long long limit_ns) {
  __shared__ __align__(8) unsigned long long bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_wait_limit(smem_u32(&bar), 0u, err, TFERR_WAIT_SELFTEST, limit_ns);
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

// Bulk tensor stores from shared memory (the TMA engine writes whole row segments; the SM issues one
// instruction per box).  `tma_reduce_add_2d` adds the fp32 box into global memory instead of storing it.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(map), "r"(x), "r"(y), "r"(src)
               : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, int x, int y, uint32_t src) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];" ::"l"(map), "r"(x),
               "r"(y), "r"(src)
               : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// Byte offset of 16-byte chunk `k` (0..7) of row `r` inside a [rows][128 bytes] staging box with the
// 128-byte swizzle the tensor maps use (box base 1024-byte aligned).
__device__ __forceinline__ uint32_t swz128(int r, int k) { return (uint32_t)(r * 128 + ((k ^ (r & 7)) << 4)); }

__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major tile, rows of 128 bytes, 128-byte swizzle; 8-row groups
// are 1024 bytes apart (stride byte offset), the leading byte offset is unused for this layout.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
  uint64_t desc = 0;
  desc |= (uint64_t)((saddr & 0x3FFFFu) >> 4);   // start address, 16-byte units
  desc |= (uint64_t)1 << 16;                     // leading byte offset (ignored for swizzled K-major)
  desc |= (uint64_t)(1024 >> 4) << 32;           // stride byte offset
  desc |= (uint64_t)1 << 46;                     // descriptor version for this architecture
  desc |= (uint64_t)2 << 61;                     // 128-byte swizzle
  return desc;
}

// Instruction descriptor for kind::f16: bf16 x bf16 -> fp32, both operands K-major, M=128, N=BN.
__host__ __device__ constexpr uint32_t make_idesc(int bn) {
  return (1u << 4)                    // D format: fp32
         | (1u << 7)                  // A format: bf16
         | (1u << 10)                 // B format: bf16
         | ((uint32_t)(bn >> 3) << 17)  // N / 8
         | ((uint32_t)(BM >> 4) << 24); // M / 16
}

__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the mbarrier once every previously issued tcgen05.mma of this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Issue only: the registers are valid after tmem_ld_wait().
__device__ __forceinline__ void tmem_ld_32x32b_x32_issue(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

template <int BN, int STAGES>
struct SmemLayout {
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  // after the operand ring (a multiple of 1024 bytes): the epilogue staging area, per warp either a padded 32x33
  // fp32 transpose tile (4224 B stride) or a swizzled [32][128 B] box for bulk stores (4096 B stride) followed by
  // the tile's 256 biases; then the mbarriers and the TMEM slot
  static constexpr int STAGE_OUT_OFFSET = STAGES * STAGE_BYTES;
  static constexpr int STAGE_OUT_BYTES = NUM_EPI_WARPS * 32 * 33 * 4;
  static constexpr int TILE_BIAS_OFFSET = STAGE_OUT_OFFSET + NUM_EPI_WARPS * 4096;
  static constexpr int BAR_OFFSET = STAGE_OUT_OFFSET + STAGE_OUT_BYTES;
  static constexpr int NUM_BARS = 2 * STAGES + 4;
  static constexpr int TOTAL = BAR_OFFSET + NUM_BARS * 8 + 16 + 1024;  // + tmem slot + alignment slack
};

template <int BN, int STAGES, class Epi>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_a_lo,
               const __grid_constant__ CUtensorMap map_w, int M, int N, int K, int split, Epi epi, int* err,
               int ksplit, int part_rows) {
  static_assert(SmemLayout<BN, STAGES>::TILE_BIAS_OFFSET + 1024 <= SmemLayout<BN, STAGES>::STAGE_OUT_OFFSET +
                SmemLayout<BN, STAGES>::STAGE_OUT_BYTES, "bias tile must fit behind the store boxes");
  using SL = SmemLayout<BN, STAGES>;
  extern __shared__ uint8_t smem_raw[];
  pdl_launch_dependents();  // the next kernel of the stream may be scheduled; it waits for this one to complete

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_base + SL::BAR_OFFSET;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + SL::BAR_OFFSET + SL::NUM_BARS * 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_m = (M + BM - 1) / BM, tiles_n = (N + BN - 1) / BN;
  // ksplit > 1 (bulk-store epilogues only): every output tile is computed ksplit times, each over its own range of
  // k slabs, and slice s stores its partial tile part_rows * s rows further down; the consumer adds the slices in
  // index order.  Tile index = (m tile, n tile, slice) with the slice fastest.
  const int num_tiles_all = tiles_m * tiles_n * ksplit;
  // split != 0: A is an error-compensated pair (hi + lo); the K loop runs over [A_hi | A_lo] against
  // [W | W], i.e. both products accumulate into the same TMEM tile.
  const int kb_per_pass = (K + BK - 1) / BK;
  auto slab_begin = [&](int slice) { return (int)((long long)kb_per_pass * slice / ksplit); };
  constexpr uint32_t TMEM_COLS = 2 * BN;  // two accumulator buffers (power of two >= 32)

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), NUM_EPI_WARPS);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // everything above (barriers, tensor memory) overlaps the previous kernel's tail; its activations and the
  // error word are complete from here on.  After an earlier failure the CTA walks an empty tile list.
  pdl_wait();
  const int num_tiles = *reinterpret_cast<volatile int*>(err) != 0 ? 0 : num_tiles_all;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int mn = tile / ksplit, slice = tile - mn * ksplit;
        const int m0 = (mn / tiles_n) * BM, n0 = (mn % tiles_n) * BN;
        const int kb0 = slab_begin(slice), nkb = slab_begin(slice + 1) - kb0;
        const int kblocks = split ? 2 * nkb : nkb;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, err, TFERR_WAIT_EMPTY)) { ok = false; break; }
          mbar_arrive_expect_tx(full_bar(stage), SL::STAGE_BYTES);
          const uint32_t sa = smem_base + stage * SL::STAGE_BYTES;
          const int kk = (kb0 + (kb >= nkb ? kb - nkb : kb)) * BK;
          tma_load_2d(sa, kb >= nkb ? &map_a_lo : &map_a, kk, m0, full_bar(stage));
          tma_load_2d(sa + SL::A_BYTES, &map_w, kk, n0, full_bar(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(BN);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int it = 0;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1;
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, err, TFERR_WAIT_TMEM_EMPTY)) { ok = false; break; }
        tcgen05_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        const int slice = tile % ksplit;
        const int kblocks = (split ? 2 : 1) * (slab_begin(slice + 1) - slab_begin(slice));
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, err, TFERR_WAIT_FULL)) { ok = false; break; }
          tcgen05_fence_after();
          const uint32_t sa = smem_base + stage * SL::STAGE_BYTES;
          const uint64_t adesc = make_smem_desc(sa), bdesc = make_smem_desc(sa + SL::A_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advancing 16 bf16 = 32 bytes along K inside the swizzled row: +2 in 16-byte units
            umma_f16(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (kb | k) != 0);
          }
          umma_commit(empty_bar(stage));  // frees the stage once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(tfull_bar(acc));  // accumulator complete
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int quad = warp & 3;  // TMEM lane quadrant this warp may read
    const int cgroup = (warp - 2) >> 2;  // which of the NUM_EPI_WARPS/4 column groups of a quadrant
    float* stage_out = reinterpret_cast<float*>(smem + SL::STAGE_OUT_OFFSET) + (warp - 2) * (32 * 33);
    bool ok = true;
    int it = 0;
    if constexpr (Epi::kTmaCols > 0) {
      // Bulk-store epilogue: each warp owns NCH adjacent 32-column chunks of its 32 rows; values leave the
      // registers row-per-lane as 16-byte shared-memory writes into a swizzled [32][128 B] box, and one lane
      // hands the box to the TMA engine (store, or fp32 add into the residual stream).
      constexpr int NCH = BN / 32 / (NUM_EPI_WARPS / 4);
      constexpr int CPG = Epi::kTmaCols / 32;  // chunks per box: 2 (bf16, 64 columns) or 1 (fp32, 32 columns)
      static_assert(NCH % CPG == 0, "box width must divide the warp's columns");
      const int etid = threadIdx.x - 64;       // 0 .. 32 * NUM_EPI_WARPS - 1
      uint8_t* box = smem + SL::STAGE_OUT_OFFSET + (warp - 2) * 4096;
      const uint32_t box_addr = smem_u32(box);
      float* tile_bias = reinterpret_cast<float*>(smem + SL::TILE_BIAS_OFFSET);
      for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
        const int mn = tile / ksplit, slice = tile - mn * ksplit;
        const int m0 = (mn / tiles_n) * BM, n0 = (mn % tiles_n) * BN;
        const int acc = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1;
        // the tile's biases, once, while the mainloop still runs
        named_bar_sync(1, 32 * NUM_EPI_WARPS);
        if (etid < BN) tile_bias[etid] = epi.col_const(n0 + etid, n0 + etid < N);
        named_bar_sync(1, 32 * NUM_EPI_WARPS);
        // a warp whose wait gave up keeps walking the tile list (without work), so the named barrier above
        // is always reached by all epilogue warps
        if (ok && !mbar_wait(tfull_bar(acc), acc_phase, err, TFERR_WAIT_TMEM_FULL)) ok = false;
        if (!ok) continue;
        tcgen05_fence_after();
        const int row0 = m0 + quad * 32;
        float v[NCH][32];
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch)
          tmem_ld_32x32b_x32_issue(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN + (cgroup * NCH + ch) * 32),
                                   v[ch]);
        tmem_ld_wait();
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(acc));  // the accumulator is in registers: free it for the next tile
        if (row0 < M) {
#pragma unroll
          for (int g = 0; g < NCH / CPG; ++g) {
            const int cl = (cgroup * NCH + g * CPG) * 32;  // first column of the box inside the tile
            if (n0 + cl < N)
              epi.template tma_box<CPG>(v[g * CPG], v[g * CPG + CPG - 1], tile_bias + cl, n0 + cl, row0 + slice * part_rows, box,
                                        box_addr, lane);
          }
        }
      }
      if (lane == 0) tma_store_wait_all();
    } else {
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
      const int m0 = (tile / tiles_n) * BM, n0 = (tile % tiles_n) * BN;
      const int acc = it & 1;
      const uint32_t acc_phase = (it >> 1) & 1;
      if (!mbar_wait(tfull_bar(acc), acc_phase, err, TFERR_WAIT_TMEM_FULL)) { ok = false; break; }
      tcgen05_fence_after();
      const int row0 = m0 + quad * 32;
      const int nrows = (M - row0) < 32 ? (M - row0) : 32;  // rows of this warp inside the matrix (may be <= 0)
      float row_acc = 0.f;  // kRowReduce functors: a per-row value carried over the warp's chunks of this tile
#pragma unroll 1
      for (int c = cgroup; c < BN / 32; c += NUM_EPI_WARPS / 4) {
        const int col0 = n0 + c * 32;
        if (col0 >= N) break;  // uniform across the warp
        float v[32];
        tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN + c * 32), v);
        const int col = col0 + lane;
        const bool col_ok = col < N;
        const float cc = epi.col_const(col, col_ok);
        if constexpr (Epi::kRowwise) {
          // lane = row: the chunk's biases go through the warp's shared-memory slot (broadcast reads)
          stage_out[lane] = cc;
          __syncwarp();
          const int nv = (N - col0) < 32 ? (N - col0) : 32;
          if constexpr (Epi::kRowReduce) {
            if (lane < nrows) row_acc = epi.rowwise_reduce(row0 + lane, col0, v, nv, stage_out, row_acc);
          } else {
            if (lane < nrows) epi.rowwise(row0 + lane, col0, v, nv, stage_out);
          }
          __syncwarp();
        } else {
          // transpose through shared memory: lane = row on the way in, lane = column on the way out
#pragma unroll
          for (int j = 0; j < 32; ++j) stage_out[lane * 33 + j] = v[j];
          __syncwarp();
          if (nrows == 32) {
            constexpr int RB = Epi::kRowsBatch;  // rows a functor handles per call (its loads are issued together)
#pragma unroll
            for (int r0 = 0; r0 < 32; r0 += RB) {
              float a[RB];
#pragma unroll
              for (int r = 0; r < RB; ++r) a[r] = stage_out[(r0 + r) * 33 + lane];
              epi.template store_rows<RB>(row0 + r0, col, a, cc, col_ok, lane);
            }
          } else {
            for (int r = 0; r < nrows; ++r) epi.store(row0 + r, col, stage_out[r * 33 + lane], cc, col_ok, lane);
          }
          __syncwarp();
        }
      }
      if constexpr (Epi::kRowReduce) {
        if (lane < nrows) epi.row_done(row0 + lane, row_acc);
      }
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
    }
    }
  }

  // teardown: everybody arrives here because every wait above is bounded
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) {
    if (*reinterpret_cast<volatile int*>(err) != 0) {
      // a role gave up: let TMA copies and MMAs already in flight drain before the memory is released
      unsigned long long t0 = globaltimer_ns();
      while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace tc

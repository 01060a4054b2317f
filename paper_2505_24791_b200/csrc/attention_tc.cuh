// Causal self-attention on the 5th-generation tensor cores (head_dim 64, single bf16 operands).
//
// One CTA = one (slot, head, tile of 128 queries); key/value tiles of 64 keys from 0 up to the query tile (causal).
// Per key tile j:
//   S  = Q K_j^T                 tcgen05.mma M=128 N=64 K=64, both operands K-major from TMA tiles, S in TMEM
//   softmax                      4 warps, one query row per thread (TMEM lane = row, so row maximum and row sum
//                                need no shuffles): running maximum / sum in fp32, P_j = exp2(S - m) written as
//                                bf16 into a swizzled shared-memory tile (the A operand of the second MMA)
//   O_j = P_j V_j                tcgen05.mma M=128 N=64 K=64; V_j is used as it arrives from TMA ([key][channel],
//                                i.e. an MN-major B operand), no transposition anywhere
//   o += O_j (rescaled)          the running output stays in registers of the row's thread
// K and V each have one buffer: K_{j+1} is loaded as soon as the first MMA of tile j has completed, V_{j+1} after
// the second, so loads overlap the softmax; two CTAs fit on an SM and fill each other's bubbles.
// Rows are addressed through 3-D tensor maps [slot][position][column], so positions >= L read as zeros and are
// never written (ragged L).  Every mbarrier wait is bounded as in gemm_tc.cuh.
// qkv rows are [q | k | v] (3d wide); out is [slot, L, d] bf16.  map_qkv has a box of 128 positions (queries),
// map_kv one of 64 positions (keys / values), both 64 columns wide.
#pragma once
#include "gemm_tc.cuh"

namespace attn_tc {

using namespace tc;

constexpr int BQ = 128, BKV = 64, HD = 64;
constexpr int NUM_THREADS_ATTN = 192;  // warp 0 TMA, warp 1 MMA + TMEM, warps 2..5 softmax / epilogue
constexpr int Q_BYTES = BQ * HD * 2, K_BYTES = BKV * HD * 2, V_BYTES = BKV * HD * 2, P_BYTES = BQ * BKV * 2;
constexpr int SMEM_BYTES = Q_BYTES + K_BYTES + V_BYTES + P_BYTES + 128 + 1024;
constexpr uint32_t TMEM_COLS_ATTN = 128;  // S: columns 0..63, O_j: columns 64..127

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, int x, int y, int z, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];" ::"l"(map), "r"(x), "r"(y),
               "r"(z), "r"(src)
               : "memory");
}
// MN-major B operand tile [keys][64 channels] with 128-byte rows and 128-byte swizzle (what TMA delivers for V):
// 8 keys x 128 bytes per swizzle atom, atoms 1024 bytes apart along the key (K) direction.
__device__ __forceinline__ uint64_t make_smem_desc_mn(uint32_t saddr) {
  uint64_t desc = 0;
  desc |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  desc |= (uint64_t)((BKV * 128) >> 4) << 16;  // leading byte offset: next 64-channel atom (not used with N = 64)
  desc |= (uint64_t)(1024 >> 4) << 32;         // stride byte offset: next group of 8 keys
  desc |= (uint64_t)1 << 46;
  desc |= (uint64_t)2 << 61;
  return desc;
}
// kind::f16 instruction descriptor: bf16 x bf16 -> fp32, A K-major, B K-major (b_mn = 0) or MN-major (b_mn = 1)
__host__ __device__ constexpr uint32_t make_idesc_attn(int m, int n, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

__global__ void __launch_bounds__(NUM_THREADS_ATTN, 2)
attention_tc_kernel(const __grid_constant__ CUtensorMap map_qkv, const __grid_constant__ CUtensorMap map_kv,
                    const CUtensorMap* __restrict__ map_out, int L, int d,
                    float scale_log2e, int* err) {
  extern __shared__ uint8_t smem_attn_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_attn_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sQ = smem_u32(smem), sK = sQ + Q_BYTES, sV = sK + K_BYTES, sP = sV + V_BYTES;
  const uint32_t bar_base = sP + P_BYTES;
  // barriers: 0 q_full, 1 k_full, 2 k_empty, 3 v_full, 4 v_empty, 5 s_full, 6 p_ready, 7 o_done
  auto bar = [&](int i) { return bar_base + 8u * i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + Q_BYTES + K_BYTES + V_BYTES + P_BYTES + 64);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_qt = (L + BQ - 1) / BQ;
  const int qt = n_qt - 1 - (int)blockIdx.x;  // longest tiles first
  const int head = blockIdx.y, slot = blockIdx.z;
  const int q0 = qt * BQ;
  const int n_kv = ((q0 + BQ < L ? q0 + BQ : L) + BKV - 1) / BKV;  // key tiles that hold a visible key

  if (threadIdx.x == 0) {
    for (int i = 0; i < 8; ++i) mbar_init(bar(i), i == 6 ? 4 : 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)),
                 "r"(TMEM_COLS_ATTN)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const bool dead = *reinterpret_cast<volatile int*>(err) != 0;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && !dead) {
      mbar_arrive_expect_tx(bar(0), Q_BYTES);
      tma_load_3d(sQ, &map_qkv, head * HD, q0, slot, bar(0));
      bool ok = true;
      for (int j = 0; j < n_kv && ok; ++j) {
        const uint32_t ph = j & 1;
        if (!mbar_wait(bar(2), ph ^ 1u, err, TFERR_WAIT_EMPTY)) { ok = false; break; }
        mbar_arrive_expect_tx(bar(1), K_BYTES);
        tma_load_3d(sK, &map_kv, d + head * HD, j * BKV, slot, bar(1));
        if (!mbar_wait(bar(4), ph ^ 1u, err, TFERR_WAIT_EMPTY)) { ok = false; break; }
        mbar_arrive_expect_tx(bar(3), V_BYTES);
        tma_load_3d(sV, &map_kv, 2 * d + head * HD, j * BKV, slot, bar(3));
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && !dead) {
      constexpr uint32_t idesc_s = make_idesc_attn(BQ, BKV, 0), idesc_o = make_idesc_attn(BQ, HD, 1);
      bool ok = mbar_wait(bar(0), 0u, err, TFERR_WAIT_FULL);
      for (int j = 0; j < n_kv && ok; ++j) {
        const uint32_t ph = j & 1;
        if (!mbar_wait(bar(1), ph, err, TFERR_WAIT_FULL)) { ok = false; break; }
        tcgen05_fence_after();
        const uint64_t qdesc = make_smem_desc(sQ), kdesc = make_smem_desc(sK);
#pragma unroll
        for (int k = 0; k < HD / UMMA_K; ++k) umma_f16(tmem_base, qdesc + 2u * k, kdesc + 2u * k, idesc_s, k != 0);
        umma_commit(bar(2));  // K buffer free
        umma_commit(bar(5));  // S complete
        if (!mbar_wait(bar(6), ph, err, TFERR_WAIT_TMEM_EMPTY)) { ok = false; break; }  // P written, O_{j-1} consumed
        if (!mbar_wait(bar(3), ph, err, TFERR_WAIT_FULL)) { ok = false; break; }
        tcgen05_fence_after();
#pragma unroll
        for (int k = 0; k < BKV / UMMA_K; ++k) {
          // P: [128 rows][128 B] (64 keys), 16 keys = 32 bytes along a row.  V: 16 keys = 2048 bytes.
          const uint64_t pdesc = make_smem_desc(sP) + 2u * k;
          const uint64_t vdesc = make_smem_desc_mn(sV + k * (UMMA_K * 128));
          umma_f16(tmem_base + BKV, pdesc, vdesc, idesc_o, k != 0);
        }
        umma_commit(bar(4));  // V buffer (and P) free
        umma_commit(bar(7));  // O_j complete
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + output (warps 2..5)
    const int quad = warp & 3;
    const int r = quad * 32 + lane;            // row of this thread inside the query tile
    const int qpos = q0 + r;                   // position in the sequence
    const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16);
    uint8_t* sPg = smem + Q_BYTES + K_BYTES + V_BYTES;
    float o[HD];
#pragma unroll
    for (int i = 0; i < HD; ++i) o[i] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = !dead;
    for (int j = 0; j < n_kv && ok; ++j) {
      const uint32_t ph = j & 1;
      if (!mbar_wait(bar(5), ph, err, TFERR_WAIT_TMEM_FULL)) { ok = false; break; }
      tcgen05_fence_after();
      const int kv0 = j * BKV;
      const bool diag = kv0 + BKV - 1 > q0;  // some key of this tile lies after some query of the tile
      // the whole score row in one round of tensor-memory loads
      float s[BKV];
      tmem_ld_32x32b_x32_issue(t_row, *reinterpret_cast<float(*)[32]>(&s[0]));
      tmem_ld_32x32b_x32_issue(t_row + 32, *reinterpret_cast<float(*)[32]>(&s[32]));
      tmem_ld_wait();
      float mx = -INFINITY;
#pragma unroll
      for (int i = 0; i < BKV; ++i) {
        if (diag && kv0 + i > qpos) s[i] = -INFINITY;
        mx = fmaxf(mx, s[i]);
      }
      const float m_new = fmaxf(m_run, mx);  // finite from the first tile on: key 0 is visible to every row
      const float corr = exp2f((m_run - m_new) * scale_log2e);
      m_run = m_new;
      // the previous tile's P V product: add it (it is at the previous maximum), then move everything to the new one
      if (j > 0) {
        if (!mbar_wait(bar(7), ph ^ 1u, err, TFERR_WAIT_TMEM_FULL)) { ok = false; break; }
        tcgen05_fence_after();
        float t[HD];
        tmem_ld_32x32b_x32_issue(t_row + BKV, *reinterpret_cast<float(*)[32]>(&t[0]));
        tmem_ld_32x32b_x32_issue(t_row + BKV + 32, *reinterpret_cast<float(*)[32]>(&t[32]));
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < HD; ++i) o[i] = (o[i] + t[i]) * corr;
      }
      l_run *= corr;
      // probabilities -> bf16 P tile (swizzled rows of 128 bytes)
      const float mb = m_new * scale_log2e;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        uint32_t pk[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float p0 = exp2f(fmaf(s[8 * q + 2 * i], scale_log2e, -mb));      // exp2(-inf) = 0 for masked keys
          const float p1 = exp2f(fmaf(s[8 * q + 2 * i + 1], scale_log2e, -mb));
          const __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
          const float2 pf = __bfloat1622float2(pb);  // the sum uses the rounded probabilities the second MMA sees
          l_run += pf.x + pf.y;
          pk[i] = *reinterpret_cast<const uint32_t*>(&pb);
        }
        *reinterpret_cast<uint4*>(sPg + swz128(r, q)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
      }
      fence_proxy_async_smem();
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(6));
    }
    // last product, normalisation, store through a swizzled [32 rows][128 B] box per warp (inside the P tile,
    // which nobody reads any more)
    if (ok && mbar_wait(bar(7), (uint32_t)((n_kv - 1) & 1), err, TFERR_WAIT_TMEM_FULL)) {
      tcgen05_fence_after();
      float t[HD];
      tmem_ld_32x32b_x32_issue(t_row + BKV, *reinterpret_cast<float(*)[32]>(&t[0]));
      tmem_ld_32x32b_x32_issue(t_row + BKV + 32, *reinterpret_cast<float(*)[32]>(&t[32]));
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < HD; ++i) o[i] += t[i];
      const float inv = 1.f / l_run;
      uint8_t* box = sPg + quad * 4096;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const __nv_bfloat162 a = __floats2bfloat162_rn(o[8 * k] * inv, o[8 * k + 1] * inv);
        const __nv_bfloat162 b = __floats2bfloat162_rn(o[8 * k + 2] * inv, o[8 * k + 3] * inv);
        const __nv_bfloat162 c2 = __floats2bfloat162_rn(o[8 * k + 4] * inv, o[8 * k + 5] * inv);
        const __nv_bfloat162 d2 = __floats2bfloat162_rn(o[8 * k + 6] * inv, o[8 * k + 7] * inv);
        uint4 u;
        u.x = *reinterpret_cast<const uint32_t*>(&a); u.y = *reinterpret_cast<const uint32_t*>(&b);
        u.z = *reinterpret_cast<const uint32_t*>(&c2); u.w = *reinterpret_cast<const uint32_t*>(&d2);
        *reinterpret_cast<uint4*>(box + swz128(lane, k)) = u;
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0 && q0 + quad * 32 < L) {
        tma_store_3d(map_out, head * HD, q0 + quad * 32, slot, smem_u32(box));
        tma_store_commit();
        tma_store_wait_all();
      }
    }
  }

  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) {
    if (*reinterpret_cast<volatile int*>(err) != 0) {
      unsigned long long t0 = globaltimer_ns();
      while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS_ATTN) : "memory");
  }
}

}  // namespace attn_tc

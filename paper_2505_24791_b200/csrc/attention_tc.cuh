// Causal self-attention on the 5th-generation tensor cores (head_dim 64, single bf16 operands).
//
// One CTA = one (slot, head, tile of 128 queries); key/value tiles of 64 keys from 0 up to the query tile (causal).
// Per key tile j:
//   S  = Q K_j^T                 tcgen05.mma M=128 N=64 K=64, both operands K-major from TMA tiles, S in TMEM
//   softmax                      4 warps, one query row per thread (TMEM lane = row, so row maximum and row sum
//                                need no shuffles): running maximum / sum in fp32, P_j = exp2(S - m) written as
//                                bf16 into a swizzled shared-memory tile (the A operand of the second MMA)
//   O += P_j V_j                 tcgen05.mma M=128 N=64 K=64, accumulating in TMEM over the key tiles; V_j is used as
//                                it arrives from TMA ([key][channel], i.e. an MN-major B operand), no transposition
//   rescale (rare)               the reference maximum of a row moves only when the true maximum has grown by more
//                                than 2^8; only then is the accumulator read, scaled and written back
// S is released as soon as the softmax warps hold it in registers, so the first MMA of tile j+1 runs under the
// softmax of tile j; P is free again when the second MMA of the previous tile has completed, long before the
// next probabilities are ready.  K and V tiles travel through rings of two buffers each.  The CTA needs 128
// TMEM columns and about 65 KB of shared memory, so three CTAs (twelve softmax warps) share an SM and hide each
// other's latencies.
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
// SPLIT: every operand is an error-compensated bf16 pair (hi + lo) and every product keeps hi*hi + lo*hi + hi*lo;
// the low halves sit directly behind the high halves of Q, of each K / V ring slot and of P.
template <bool SPLIT>
struct Cfg {
  static constexpr int NT = SPLIT ? 2 : 1;           // tiles per operand
  static constexpr int KV_STAGES = SPLIT ? 1 : 2;    // K and V tiles in flight ahead of the tensor core
  static constexpr int Q_ALL = NT * Q_BYTES, K_SLOT = NT * K_BYTES, V_SLOT = NT * V_BYTES, P_ALL = NT * P_BYTES;
  static constexpr int KV_RING = KV_STAGES * (K_SLOT + V_SLOT);
  static constexpr int SMEM_BYTES = Q_ALL + KV_RING + P_ALL + 256 + 1024;
  static constexpr int CTAS_PER_SM = SPLIT ? 2 : 3;
};
constexpr uint32_t TMEM_COLS_ATTN = 128;  // S at column 0, the output accumulator at column 64

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
__device__ __forceinline__ void tmem_st_32x32b_x32(uint32_t taddr, const float (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
        "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
        "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15])), "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])),
        "r"(__float_as_uint(v[19])), "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])),
        "r"(__float_as_uint(v[23])), "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])),
        "r"(__float_as_uint(v[27])), "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])),
        "r"(__float_as_uint(v[31]))
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
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

template <bool SPLIT>
__global__ void __launch_bounds__(NUM_THREADS_ATTN, Cfg<SPLIT>::CTAS_PER_SM)
attention_tc_kernel(const __grid_constant__ CUtensorMap map_qkv, const __grid_constant__ CUtensorMap map_kv,
                    const __grid_constant__ CUtensorMap map_qkv_lo, const __grid_constant__ CUtensorMap map_kv_lo,
                    const CUtensorMap* __restrict__ map_out, const CUtensorMap* __restrict__ map_out_lo, int L, int d,
                    float scale_log2e, int* err) {
  using C = Cfg<SPLIT>;
  constexpr int KV_STAGES = C::KV_STAGES, KV_RING = C::KV_RING;
  extern __shared__ uint8_t smem_attn_raw[];
  pdl_launch_dependents();  // the next kernel of the stream may be scheduled; it waits for this one to complete
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_attn_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sQ = smem_u32(smem), sK = sQ + C::Q_ALL, sV = sK + KV_STAGES * C::K_SLOT, sP = sV + KV_STAGES * C::V_SLOT;
  const uint32_t bar_base = sP + C::P_ALL;
  // barriers: 0 q_full, then k_full[st], k_empty[st], v_full[st], v_empty[st], s_full, s_free, p_ready, o_done
  constexpr int B_KFULL = 1, B_KEMPTY = B_KFULL + KV_STAGES, B_VFULL = B_KEMPTY + KV_STAGES, B_VEMPTY = B_VFULL + KV_STAGES,
                B_SFULL = B_VEMPTY + KV_STAGES, B_SFREE = B_SFULL + 1, B_PREADY = B_SFREE + 1, B_ODONE = B_PREADY + 1,
                NUM_BARS = B_ODONE + 1;
  static_assert(NUM_BARS * 8 <= 192, "barrier area");
  auto bar = [&](int i) { return bar_base + 8u * i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + C::Q_ALL + KV_RING + C::P_ALL + 192);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_qt = (L + BQ - 1) / BQ;
  const int qt = n_qt - 1 - (int)blockIdx.x;  // longest tiles first
  const int head = blockIdx.y, slot = blockIdx.z;
  const int q0 = qt * BQ;
  const int n_kv = ((q0 + BQ < L ? q0 + BQ : L) + BKV - 1) / BKV;  // key tiles that hold a visible key

  if (threadIdx.x == 0) {
    for (int i = 0; i < NUM_BARS; ++i) mbar_init(bar(i), (i == B_PREADY || i == B_SFREE) ? 4 : 1);
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
  pdl_wait();  // set-up above overlaps the previous kernel's tail; q, k, v and the error word are complete from here on
  const bool dead = *reinterpret_cast<volatile int*>(err) != 0;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && !dead) {
      mbar_arrive_expect_tx(bar(0), C::Q_ALL);
      tma_load_3d(sQ, &map_qkv, head * HD, q0, slot, bar(0));
      if constexpr (SPLIT) tma_load_3d(sQ + Q_BYTES, &map_qkv_lo, head * HD, q0, slot, bar(0));
      bool ok = true;
      int st = 0;
      uint32_t ph = 0;
      for (int j = 0; j < n_kv && ok; ++j) {
        if (!mbar_wait(bar(B_KEMPTY + st), ph ^ 1u, err, TFERR_WAIT_EMPTY)) { ok = false; break; }
        mbar_arrive_expect_tx(bar(B_KFULL + st), C::K_SLOT);
        tma_load_3d(sK + st * C::K_SLOT, &map_kv, d + head * HD, j * BKV, slot, bar(B_KFULL + st));
        if constexpr (SPLIT) tma_load_3d(sK + st * C::K_SLOT + K_BYTES, &map_kv_lo, d + head * HD, j * BKV, slot, bar(B_KFULL + st));
        if (!mbar_wait(bar(B_VEMPTY + st), ph ^ 1u, err, TFERR_WAIT_EMPTY)) { ok = false; break; }
        mbar_arrive_expect_tx(bar(B_VFULL + st), C::V_SLOT);
        tma_load_3d(sV + st * C::V_SLOT, &map_kv, 2 * d + head * HD, j * BKV, slot, bar(B_VFULL + st));
        if constexpr (SPLIT) tma_load_3d(sV + st * C::V_SLOT + V_BYTES, &map_kv_lo, 2 * d + head * HD, j * BKV, slot, bar(B_VFULL + st));
        if (++st == KV_STAGES) { st = 0; ph ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && !dead) {
      constexpr uint32_t idesc_s = make_idesc_attn(BQ, BKV, 0), idesc_o = make_idesc_attn(BQ, HD, 1);
      bool ok = mbar_wait(bar(0), 0u, err, TFERR_WAIT_FULL);
      const uint64_t qdesc = make_smem_desc(sQ);
      auto scores = [&](int j) {  // S = Q K_j^T
        const int st = j % KV_STAGES;
        if (!mbar_wait(bar(B_KFULL + st), (uint32_t)((j / KV_STAGES) & 1), err, TFERR_WAIT_FULL)) return false;
        tcgen05_fence_after();
        const uint64_t kdesc = make_smem_desc(sK + st * C::K_SLOT);
#pragma unroll
        for (int k = 0; k < HD / UMMA_K; ++k) umma_f16(tmem_base, qdesc + 2u * k, kdesc + 2u * k, idesc_s, k != 0);
        if constexpr (SPLIT) {  // + Q_lo K_hi^T + Q_hi K_lo^T
          const uint64_t qldesc = make_smem_desc(sQ + Q_BYTES), kldesc = make_smem_desc(sK + st * C::K_SLOT + K_BYTES);
#pragma unroll
          for (int k = 0; k < HD / UMMA_K; ++k) umma_f16(tmem_base, qldesc + 2u * k, kdesc + 2u * k, idesc_s, 1u);
#pragma unroll
          for (int k = 0; k < HD / UMMA_K; ++k) umma_f16(tmem_base, qdesc + 2u * k, kldesc + 2u * k, idesc_s, 1u);
        }
        umma_commit(bar(B_KEMPTY + st));  // K buffer free
        umma_commit(bar(B_SFULL));        // S complete
        return true;
      };
      if (ok) ok = scores(0);
      for (int j = 0; j < n_kv && ok; ++j) {
        // the next tile's scores are issued as soon as the softmax warps hold this tile's scores in registers,
        // long before this tile's probabilities are ready
        if (j + 1 < n_kv) {
          if (!mbar_wait(bar(B_SFREE), (uint32_t)(j & 1), err, TFERR_WAIT_TMEM_EMPTY)) { ok = false; break; }
          if (!scores(j + 1)) { ok = false; break; }
        }
        const int st = j % KV_STAGES;
        if (!mbar_wait(bar(B_PREADY), (uint32_t)(j & 1), err, TFERR_WAIT_TMEM_EMPTY)) { ok = false; break; }
        if (!mbar_wait(bar(B_VFULL + st), (uint32_t)((j / KV_STAGES) & 1), err, TFERR_WAIT_FULL)) { ok = false; break; }
        tcgen05_fence_after();
#pragma unroll
        for (int k = 0; k < BKV / UMMA_K; ++k) {
          // P: [128 rows][128 B] (64 keys), 16 keys = 32 bytes along a row.  V: 16 keys = 2048 bytes.
          const uint64_t pdesc = make_smem_desc(sP) + 2u * k;
          const uint64_t vdesc = make_smem_desc_mn(sV + st * C::V_SLOT + k * (UMMA_K * 128));
          umma_f16(tmem_base + BKV, pdesc, vdesc, idesc_o, (j | k) != 0);
        }
        if constexpr (SPLIT) {  // + P_lo V_hi + P_hi V_lo
#pragma unroll
          for (int k = 0; k < BKV / UMMA_K; ++k) {
            const uint64_t pldesc = make_smem_desc(sP + P_BYTES) + 2u * k;
            const uint64_t vdesc = make_smem_desc_mn(sV + st * C::V_SLOT + k * (UMMA_K * 128));
            umma_f16(tmem_base + BKV, pldesc, vdesc, idesc_o, 1u);
          }
#pragma unroll
          for (int k = 0; k < BKV / UMMA_K; ++k) {
            const uint64_t pdesc = make_smem_desc(sP) + 2u * k;
            const uint64_t vldesc = make_smem_desc_mn(sV + st * C::V_SLOT + V_BYTES + k * (UMMA_K * 128));
            umma_f16(tmem_base + BKV, pdesc, vldesc, idesc_o, 1u);
          }
        }
        umma_commit(bar(B_VEMPTY + st));  // V buffer free
        umma_commit(bar(B_ODONE));        // products up to tile j complete (and P free)
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + output (warps 2..5)
    const int quad = warp & 3;
    const int r = quad * 32 + lane;            // row of this thread inside the query tile
    const int qpos = q0 + r;                   // position in the sequence
    const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16);
    const uint32_t t_o = t_row + BKV;          // this row's slice of the output accumulator
    uint8_t* sPg = smem + C::Q_ALL + KV_RING;
    // m_run is the reference maximum of the row (in raw score units); it trails the true running maximum by at
    // most kLazy / scale_log2e, so probabilities stay below 2^kLazy and the accumulator is rescaled only rarely
    constexpr float kLazy = 8.f;
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = !dead;
    for (int j = 0; j < n_kv && ok; ++j) {
      if (!mbar_wait(bar(B_SFULL), (uint32_t)(j & 1), err, TFERR_WAIT_TMEM_FULL)) { ok = false; break; }
      tcgen05_fence_after();
      const int kv0 = j * BKV;
      const bool diag = kv0 + BKV - 1 > q0;  // some key of this tile lies after some query of the tile
      // the whole score row in one round of tensor-memory loads
      float s[BKV];
      tmem_ld_32x32b_x32_issue(t_row, *reinterpret_cast<float(*)[32]>(&s[0]));
      tmem_ld_32x32b_x32_issue(t_row + 32, *reinterpret_cast<float(*)[32]>(&s[32]));
      tmem_ld_wait();
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_SFREE));  // the tensor core may overwrite S with the next tile's scores
      if (diag) {
#pragma unroll
        for (int i = 0; i < BKV; ++i)
          if (kv0 + i > qpos) s[i] = -INFINITY;
      }
      float mx0 = s[0], mx1 = s[1];
#pragma unroll
      for (int i = 2; i < BKV; i += 4) {
        mx0 = fmax3(mx0, s[i], s[i + 1]);
        if (i + 3 < BKV) mx1 = fmax3(mx1, s[i + 2], s[i + 3]);
      }
      const float mx = fmaxf(mx0, mx1);  // finite from the first tile on: key 0 is visible to every row
      float corr = 1.f;
      const bool bump = (mx - m_run) * scale_log2e > kLazy;  // also true on the first tile (m_run = -inf)
      if (bump) {
        corr = ex2_approx((m_run - mx) * scale_log2e);
        m_run = mx;
        l_run *= corr;
      }
      // P was the A operand of the previous tile's product, which also has to be in the accumulator before a rescale
      if (j > 0) {
        if (!mbar_wait(bar(B_ODONE), (uint32_t)((j - 1) & 1), err, TFERR_WAIT_TMEM_FULL)) { ok = false; break; }
        tcgen05_fence_after();
      }
      // probabilities -> bf16 P tile (swizzled rows of 128 bytes); two values per instruction where the
      // hardware has packed fp32 arithmetic
      const float mb = -m_run * scale_log2e;
      const float2 sc2 = make_float2(scale_log2e, scale_log2e), mb2 = make_float2(mb, mb);
      float2 lsum = make_float2(0.f, 0.f);
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        uint32_t pk[4], pl[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float2 e = ffma2(make_float2(s[8 * q + 2 * i], s[8 * q + 2 * i + 1]), sc2, mb2);
          e.x = ex2_approx(e.x);  // exp2(-inf) = 0 for masked keys
          e.y = ex2_approx(e.y);
          lsum = fadd2(lsum, e);
          const __nv_bfloat162 pb = __floats2bfloat162_rn(e.x, e.y);
          pk[i] = *reinterpret_cast<const uint32_t*>(&pb);
          if constexpr (SPLIT) {
            const float2 hi = __bfloat1622float2(pb);
            const __nv_bfloat162 pl2 = __floats2bfloat162_rn(e.x - hi.x, e.y - hi.y);
            pl[i] = *reinterpret_cast<const uint32_t*>(&pl2);
          }
        }
        *reinterpret_cast<uint4*>(sPg + swz128(r, q)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        if constexpr (SPLIT) *reinterpret_cast<uint4*>(sPg + P_BYTES + swz128(r, q)) = make_uint4(pl[0], pl[1], pl[2], pl[3]);
      }
      l_run += lsum.x + lsum.y;
      fence_proxy_async_smem();
      // the accumulator in tensor memory is at the old reference maximum: bring this warp's rows to the new one
      // before the tensor core adds this tile's product (rare after the first tile)
      if (j > 0 && __any_sync(0xffffffffu, bump)) {
        float t[HD];
        tmem_ld_32x32b_x32_issue(t_o, *reinterpret_cast<float(*)[32]>(&t[0]));
        tmem_ld_32x32b_x32_issue(t_o + 32, *reinterpret_cast<float(*)[32]>(&t[32]));
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < HD; ++i) t[i] *= corr;
        tmem_st_32x32b_x32(t_o, *reinterpret_cast<float(*)[32]>(&t[0]));
        tmem_st_32x32b_x32(t_o + 32, *reinterpret_cast<float(*)[32]>(&t[32]));
        tmem_st_wait();
      }
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_PREADY));
    }
    // normalisation and store through a swizzled [32 rows][128 B] box per warp (inside the P tile, which nobody
    // reads any more once the last product has completed)
    if (ok && mbar_wait(bar(B_ODONE), (uint32_t)((n_kv - 1) & 1), err, TFERR_WAIT_TMEM_FULL)) {
      tcgen05_fence_after();
      float o[HD];
      tmem_ld_32x32b_x32_issue(t_o, *reinterpret_cast<float(*)[32]>(&o[0]));
      tmem_ld_32x32b_x32_issue(t_o + 32, *reinterpret_cast<float(*)[32]>(&o[32]));
      tmem_ld_wait();
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
      if constexpr (SPLIT) {  // the low half of the output pair through the same box
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          uint32_t w[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float v0 = o[8 * k + 2 * i] * inv, v1 = o[8 * k + 2 * i + 1] * inv;
            const float2 hi = __bfloat1622float2(__floats2bfloat162_rn(v0, v1));
            const __nv_bfloat162 lo = __floats2bfloat162_rn(v0 - hi.x, v1 - hi.y);
            w[i] = *reinterpret_cast<const uint32_t*>(&lo);
          }
          *reinterpret_cast<uint4*>(box + swz128(lane, k)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0 && q0 + quad * 32 < L) {
          tma_store_3d(map_out_lo, head * HD, q0 + quad * 32, slot, smem_u32(box));
          tma_store_commit();
          tma_store_wait_all();
        }
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

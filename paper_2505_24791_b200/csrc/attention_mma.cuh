// Causal self-attention for the bf16 engine, head_dim = 64: flash-style streaming softmax with
// warp-level mma.sync (m16n8k16, bf16 in, fp32 accumulate).  One CTA = one (slot, head, 64-query
// tile); each of its 4 warps owns 16 query rows.  K/V tiles of 64 keys are double-buffered in shared
// memory with cp.async; softmax statistics live in registers (quad shuffles), in fp32.
// qkv rows are [q | k | v] (3d wide, row = slot*L + position); out is [rows, d].
#pragma once
#include "common.cuh"

namespace attn {

constexpr int HD = 64;
constexpr int BQ = 64;
constexpr int BKV = 64;

// 64x64 bf16 tile, rows of 128 bytes, 16-byte chunks XOR-swizzled by (row & 7): conflict-free ldmatrix
__device__ __forceinline__ int swz(int row, int col) { return row * 64 + ((((col >> 3) ^ (row & 7)) << 3) | (col & 7)); }

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem, bool pred) {
  uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
  int sz = pred ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(s), "l"(gmem), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const bf16* p) {
  uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], const bf16* p) {
  uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// load a 64-row x 64-col bf16 tile (rows row0.., clipped at L) from `src` (row stride ld elements)
__device__ __forceinline__ void load_tile(bf16* dst, const bf16* src, size_t ld, int row0, int L) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int e = threadIdx.x + i * 128;  // 512 chunks of 16 bytes
    int r = e >> 3, ch = e & 7;
    bool ok = (row0 + r) < L;
    const bf16* g = src + (size_t)(ok ? row0 + r : 0) * ld + ch * 8;
    cp_async16(dst + swz(r, ch * 8), g, ok);
  }
}

// SPLIT: every operand is an error-compensated bf16 pair (hi + lo).  Products keep the three
// leading terms (hi*hi + hi*lo + lo*hi), the softmax probabilities are split the same way, and the
// output is written as a pair, so the kernel carries about 16 significant bits end to end.
template <bool SPLIT>
__global__ void __launch_bounds__(128)
attention_mma_kernel(const bf16* __restrict__ qkv, const bf16* __restrict__ qkv_lo, bf16* __restrict__ out,
                     bf16* __restrict__ out_lo, int L, int d, float scale_log2e) {
  constexpr int NT = SPLIT ? 2 : 1;          // tiles per operand (hi, lo)
  constexpr int TILE = BQ * HD;              // elements
  extern __shared__ __align__(128) bf16 smem_attn[];
  bf16* sQ = smem_attn;                       // [NT][TILE]
  bf16* sK = sQ + NT * TILE;                  // [2][NT][TILE]
  bf16* sV = sK + 2 * NT * TILE;              // [2][NT][TILE]
  const int n_qt = (L + BQ - 1) / BQ;
  const int qt = n_qt - 1 - blockIdx.x;  // longest tiles first
  const int head = blockIdx.y, s = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const size_t ld = 3 * (size_t)d;
  const size_t off = (size_t)s * L * ld + (size_t)head * HD;
  const int q0 = qt * BQ;
  const int n_kv = qt + 1;  // causal: key tiles 0..qt

  auto load_kv = [&](int buf, int row0) {
    load_tile(sK + (buf * NT) * TILE, qkv + off + d, ld, row0, L);
    load_tile(sV + (buf * NT) * TILE, qkv + off + 2 * d, ld, row0, L);
    if constexpr (SPLIT) {
      load_tile(sK + (buf * NT + 1) * TILE, qkv_lo + off + d, ld, row0, L);
      load_tile(sV + (buf * NT + 1) * TILE, qkv_lo + off + 2 * d, ld, row0, L);
    }
  };
  load_tile(sQ, qkv + off, ld, q0, L);
  if constexpr (SPLIT) load_tile(sQ + TILE, qkv_lo + off, ld, q0, L);
  load_kv(0, 0);
  cp_async_commit();

  uint32_t qf[NT][4][4];
  float o[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) o[i][j] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

  for (int kt = 0; kt < n_kv; ++kt) {
    const int buf = kt & 1;
    if (kt + 1 < n_kv) {
      load_kv(buf ^ 1, (kt + 1) * BKV);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    if (kt == 0) {
#pragma unroll
      for (int h = 0; h < NT; ++h)
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          ldsm_x4(qf[h][kk], sQ + h * TILE + swz(warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, kk * 16 + (lane >> 4) * 8));
    }
    const bf16* cK = sK + (buf * NT) * TILE;
    const bf16* cV = sV + (buf * NT) * TILE;
    // S = Q K^T : 16 x 64 per warp
    float sc[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) sc[i][j] = 0.f;
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
      for (int np = 0; np < 4; ++np) {  // pairs of 8-key tiles
        const int so = swz(np * 16 + (lane & 7) + (lane >> 4) * 8, kk * 16 + ((lane >> 3) & 1) * 8);
        uint32_t kf[4];
        ldsm_x4(kf, cK + so);
        mma_bf16(sc[2 * np], qf[0][kk], kf[0], kf[1]);
        mma_bf16(sc[2 * np + 1], qf[0][kk], kf[2], kf[3]);
        if constexpr (SPLIT) {
          mma_bf16(sc[2 * np], qf[1][kk], kf[0], kf[1]);
          mma_bf16(sc[2 * np + 1], qf[1][kk], kf[2], kf[3]);
          uint32_t kl[4];
          ldsm_x4(kl, cK + TILE + so);
          mma_bf16(sc[2 * np], qf[0][kk], kl[0], kl[1]);
          mma_bf16(sc[2 * np + 1], qf[0][kk], kl[2], kl[3]);
        }
      }
    }
    // causal mask on the diagonal tile (keys beyond L are beyond every valid query row too)
    const int qrow0 = q0 + warp * 16 + g;  // rows qrow0 and qrow0 + 8
    if (kt == n_kv - 1) {
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        int key = kt * BKV + nt * 8 + 2 * t;
        if (key > qrow0) sc[nt][0] = -INFINITY;
        if (key + 1 > qrow0) sc[nt][1] = -INFINITY;
        if (key > qrow0 + 8) sc[nt][2] = -INFINITY;
        if (key + 1 > qrow0 + 8) sc[nt][3] = -INFINITY;
      }
    }
    // online softmax (base-2 exponent, scale folded in)
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      mx[0] = fmaxf(mx[0], fmaxf(sc[nt][0], sc[nt][1]));
      mx[1] = fmaxf(mx[1], fmaxf(sc[nt][2], sc[nt][3]));
    }
    float corr[2], mnew[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      mnew[r] = fmaxf(m_run[r], mx[r]);  // finite: key 0 is visible to every query row
      corr[r] = exp2f((m_run[r] - mnew[r]) * scale_log2e);
      m_run[r] = mnew[r];
      l_run[r] *= corr[r];
    }
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      o[nt][0] *= corr[0]; o[nt][1] *= corr[0];
      o[nt][2] *= corr[1]; o[nt][3] *= corr[1];
    }
    uint32_t pf[NT][4][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      float p0 = exp2f((sc[nt][0] - mnew[0]) * scale_log2e), p1 = exp2f((sc[nt][1] - mnew[0]) * scale_log2e);
      float p2 = exp2f((sc[nt][2] - mnew[1]) * scale_log2e), p3 = exp2f((sc[nt][3] - mnew[1]) * scale_log2e);
      l_run[0] += p0 + p1;
      l_run[1] += p2 + p3;
      // accumulator layout of two adjacent 8-key tiles = A-fragment layout of one 16-key slab
      const uint32_t h01 = pack_bf16(p0, p1), h23 = pack_bf16(p2, p3);
      pf[0][nt >> 1][(nt & 1) * 2 + 0] = h01;
      pf[0][nt >> 1][(nt & 1) * 2 + 1] = h23;
      if constexpr (SPLIT) {
        float2 f01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&h01));
        float2 f23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&h23));
        pf[1][nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0 - f01.x, p1 - f01.y);
        pf[1][nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2 - f23.x, p3 - f23.y);
      }
    }
    // O += P V
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {  // 16-key slabs
#pragma unroll
      for (int np = 0; np < 4; ++np) {  // pairs of 8-channel tiles
        const int so = swz(kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, np * 16 + (lane >> 4) * 8);
        uint32_t vf[4];
        ldsm_x4_t(vf, cV + so);
        mma_bf16(o[2 * np], pf[0][kk], vf[0], vf[1]);
        mma_bf16(o[2 * np + 1], pf[0][kk], vf[2], vf[3]);
        if constexpr (SPLIT) {
          mma_bf16(o[2 * np], pf[1][kk], vf[0], vf[1]);
          mma_bf16(o[2 * np + 1], pf[1][kk], vf[2], vf[3]);
          uint32_t vl[4];
          ldsm_x4_t(vl, cV + TILE + so);
          mma_bf16(o[2 * np], pf[0][kk], vl[0], vl[1]);
          mma_bf16(o[2 * np + 1], pf[0][kk], vl[2], vl[3]);
        }
      }
    }
    __syncthreads();  // everyone is done with buffer `buf` before it is refilled two iterations on
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }
  const float inv0 = 1.f / l_run[0], inv1 = 1.f / l_run[1];
  const int row0 = q0 + warp * 16 + g, row1 = row0 + 8;
  const size_t oo = (size_t)s * L * d + (size_t)head * HD;
#pragma unroll
  for (int nt = 0; nt < 8; ++nt) {
    int c = nt * 8 + 2 * t;
    const float a0 = o[nt][0] * inv0, a1 = o[nt][1] * inv0, b0 = o[nt][2] * inv1, b1 = o[nt][3] * inv1;
    const uint32_t ha = pack_bf16(a0, a1), hb = pack_bf16(b0, b1);
    if (row0 < L) *reinterpret_cast<uint32_t*>(out + oo + (size_t)row0 * d + c) = ha;
    if (row1 < L) *reinterpret_cast<uint32_t*>(out + oo + (size_t)row1 * d + c) = hb;
    if constexpr (SPLIT) {
      float2 fa = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&ha));
      float2 fb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&hb));
      if (row0 < L) *reinterpret_cast<uint32_t*>(out_lo + oo + (size_t)row0 * d + c) = pack_bf16(a0 - fa.x, a1 - fa.y);
      if (row1 < L) *reinterpret_cast<uint32_t*>(out_lo + oo + (size_t)row1 * d + c) = pack_bf16(b0 - fb.x, b1 - fb.y);
    }
  }
}

template <bool SPLIT>
constexpr int smem_bytes() { return (SPLIT ? 2 : 1) * 5 * BQ * HD * 2; }

}  // namespace attn

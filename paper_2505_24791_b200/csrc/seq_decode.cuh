// Sequential decoding with a key/value cache on the bf16 engine (Eq. 5; the sequential baseline and
// block 0 of the selective policy, Sec. 3.5).  One decoding step pushes ONE token per sample through
// the block's transformer, so every projection is a skinny GEMM  out[B, N] = A[B, K] W[N, K]^T  with
// B <= a few hundred rows: the cost is streaming W (from L2 or HBM) and launch latency, not FLOPs.
//
//   seq_gemm_kernel     one CTA per slice of NC output columns.  The activation rows (after an optional
//                       fused LayerNorm) are staged once in shared memory as bf16; each warp streams
//                       its 8 rows of W straight from global memory into registers with 16-byte loads
//                       (nothing of W is shared between warps, so it never touches shared memory) and
//                       multiplies with mma.sync m16n8k16; the K range is split over the warps of the
//                       CTA and reduced in shared memory in a fixed order (deterministic).
//   seq_attention_kernel one CTA per (sample, head): single query against cache rows 0..t.
//   seq_update_embed_kernel  affine update of token t+1 (Eq. 5) and its embedding for the next step.
// The step index is read from device memory (*step_base + step_off), so one captured CUDA graph of
// a few steps can be replayed for the whole block.
#pragma once
#include "common.cuh"

namespace seq {

constexpr int ROWS = 64;           // activation rows per CTA pass (4 m16 tiles)
constexpr int KC = 1024;           // K chunk staged in shared memory at a time
constexpr int A_PITCH = KC + 8;    // bf16 elements; +16 bytes per row keeps ldmatrix conflict-free
constexpr int THREADS = 256;
constexpr int WARPS = THREADS / 32;
constexpr int HD = 64;             // head_dim of the bf16 engine

__host__ __device__ constexpr int a_smem_bytes() { return ROWS * A_PITCH * 2; }
__host__ __device__ constexpr int red_smem_bytes() { return WARPS * ROWS * 8 * 4; }
__host__ __device__ constexpr int stat_smem_bytes() { return ROWS * 2 * 4; }
__host__ __device__ constexpr int gemm_smem_bytes() { return a_smem_bytes() + red_smem_bytes() + stat_smem_bytes(); }

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const bf16* p) {
  uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 ld_stream16(const void* p) {  // weights: read once per step, keep out of L1
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// Position inside a staged row of the element with (chunk-local) reduction index k.  A lane's 16-byte
// weight load covers 8 consecutive k; the two m16n8k16 steps of a 32-wide k group then take the
// lane's elements {0,1 | 2,3} and {4,5 | 6,7} as their B fragments.  The activation row is stored
// so that a plain ldmatrix of step (32c + 16j) delivers the matching elements:
//   k = 32c + 8t + 4j + 2h + e   ->   32c + 16j + 8h + 2t + e.
__device__ __forceinline__ int perm_k(int k) {
  const int c = k & ~31, r = k & 31;
  const int t = r >> 3, j = (r >> 2) & 1, h = (r >> 1) & 1, e = r & 1;
  return c + 16 * j + 8 * h + 2 * t + e;
}

// LayerNorm of RF rows at a time by one warp, rows held in registers (NV float4 per lane, K <= 128*NV):
// one round of global loads per RF rows, two-pass statistics from registers (eps 1e-5), result written
// as bf16 in the permuted order.  Rows >= nrows are written as zeros.
template <int RF, int NV>
__device__ __forceinline__ void ln_stage_rows(const float* __restrict__ h, const float* __restrict__ gamma,
                                              const float* __restrict__ beta, bf16* __restrict__ sA, int K, int row0,
                                              int nrows, int srows, int pitch) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nv4 = K >> 2;
  for (int rb = warp * RF; rb < srows; rb += WARPS * RF) {
    float4 v[RF][NV];
#pragma unroll
    for (int rr = 0; rr < RF; ++rr) {
      const bool rok = (rb + rr) < nrows;
      const float4* xr = reinterpret_cast<const float4*>(h + (size_t)(row0 + rb + rr) * K);
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const int idx = i * 32 + lane;
        v[rr][i] = (rok && idx < nv4) ? __ldcg(xr + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
#pragma unroll
    for (int rr = 0; rr < RF; ++rr) {
      if (rb + rr >= srows) break;
      float s = 0.f;
#pragma unroll
      for (int i = 0; i < NV; ++i) s += (v[rr][i].x + v[rr][i].y) + (v[rr][i].z + v[rr][i].w);
      const float mean = warp_sum(s) / K;
      float sq = 0.f;
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        if (i * 32 + lane < nv4) {
          const float a = v[rr][i].x - mean, b = v[rr][i].y - mean, c = v[rr][i].z - mean, e = v[rr][i].w - mean;
          sq += (a * a + b * b) + (c * c + e * e);
        }
      }
      const float rstd = rsqrtf(warp_sum(sq) / K + 1e-5f);
      const bool rok = (rb + rr) < nrows;
      bf16* dst = sA + (rb + rr) * pitch;
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const int idx = i * 32 + lane;
        if (idx < nv4) {
          float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
          if (rok) {
            const float4 gg = *reinterpret_cast<const float4*>(gamma + 4 * idx);
            const float4 bb = *reinterpret_cast<const float4*>(beta + 4 * idx);
            o.x = (v[rr][i].x - mean) * rstd * gg.x + bb.x; o.y = (v[rr][i].y - mean) * rstd * gg.y + bb.y;
            o.z = (v[rr][i].z - mean) * rstd * gg.z + bb.z; o.w = (v[rr][i].w - mean) * rstd * gg.w + bb.w;
          }
          *reinterpret_cast<__nv_bfloat162*>(dst + perm_k(4 * idx)) = __floats2bfloat162_rn(o.x, o.y);
          *reinterpret_cast<__nv_bfloat162*>(dst + perm_k(4 * idx + 2)) = __floats2bfloat162_rn(o.z, o.w);
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// epilogues: apply(row b, column n, value) for one finished output element (bias not yet added)
// ---------------------------------------------------------------------------------------------
struct EpiQKV {  // q -> q[b, :]; k, v -> cache row t of (b, head): cache layout [B][heads][L][64]
  bf16 *q, *kc, *vc;
  const float* bias;
  int d, L, heads;
  __device__ __forceinline__ void apply(int b, int n, float x, int t) const {
    const bf16 val = __float2bfloat16_rn(x + bias[n]);
    if (n < d) { q[(size_t)b * d + n] = val; return; }
    const int nn = n < 2 * d ? n - d : n - 2 * d;
    bf16* cache = n < 2 * d ? kc : vc;
    cache[(((size_t)b * heads + (nn >> 6)) * L + t) * HD + (nn & 63)] = val;
  }
};
struct EpiResidual {  // h[b, n] += x + bias[n]
  float* h;
  const float* bias;
  int ldh;
  __device__ __forceinline__ void apply(int b, int n, float x, int) const {
    float* p = h + (size_t)b * ldh + n;
    *p = *p + (x + bias[n]);
  }
};
struct EpiGelu {  // out[b, n] = bf16(gelu(x + bias[n]))
  bf16* out;
  const float* bias;
  int ld;
  __device__ __forceinline__ void apply(int b, int n, float x, int) const {
    out[(size_t)b * ld + n] = __float2bfloat16_rn(gelu_erf(x + bias[n]));
  }
};
struct EpiHead {  // o[b, n] = x + bias[n]  (fp32, interleaved mu~ / alpha~ columns)
  float* o;
  const float* bias;
  int ld;
  __device__ __forceinline__ void apply(int b, int n, float x, int) const { o[(size_t)b * ld + n] = x + bias[n]; }
};

// ---------------------------------------------------------------------------------------------
// out[B, N] = LN?(A)[B, K] * W[N, K]^T.   grid = (ceil(N / NC), ceil(B / 64)),  NC in {8, 16, 32}.
//   LN = true : A is the fp32 residual stream h [B, K] (K = width), normalised with gamma/beta.
//   LN = false: A is a bf16 matrix [B, K].
// Warp w owns the 8-column tile (w % (NC/8)) and the k-split (w / (NC/8)) of every staged K chunk.
// ---------------------------------------------------------------------------------------------
template <int NC, bool LN, class Epi>
__global__ void __launch_bounds__(THREADS, 1)
seq_gemm_kernel(const void* __restrict__ A_, const float* __restrict__ gamma, const float* __restrict__ beta,
                const bf16* __restrict__ W, int B, int N, int K, Epi epi, const int* __restrict__ step_base,
                int step_off, int n_steps) {
  const int t = *step_base + step_off;
  if (t >= n_steps) return;
  extern __shared__ __align__(128) uint8_t smem_seq[];
  bf16* sA = reinterpret_cast<bf16*>(smem_seq);
  float* sRed = reinterpret_cast<float*>(smem_seq + a_smem_bytes());
  float* sStat = reinterpret_cast<float*>(smem_seq + a_smem_bytes() + red_smem_bytes());
  constexpr int NT = NC / 8;       // 8-column tiles per CTA
  constexpr int KS = WARPS / NT;   // k-splits
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tq = lane & 3;
  const int nt = warp % NT, ks = warp / NT;
  const int n0 = blockIdx.x * NC + nt * 8;
  const int row0 = blockIdx.y * ROWS;
  const int nrows = (B - row0) < ROWS ? (B - row0) : ROWS;
  const int mtiles = (nrows + 15) >> 4;  // m16 tiles that hold real rows
  const int srows = mtiles * 16;         // rows staged in shared memory (rows past B are zero)

  const bool ln_fast = LN && K <= KC;  // whole rows fit the register-resident LayerNorm staging
  if (LN && !ln_fast) {  // general path: row statistics first (two-pass, eps 1e-5), one warp per row
    const float* h = reinterpret_cast<const float*>(A_);
    for (int r = warp; r < srows; r += WARPS) {
      float mean = 0.f, rstd = 0.f;
      if (r < nrows) {
        const float4* xr = reinterpret_cast<const float4*>(h + (size_t)(row0 + r) * K);
        float s = 0.f;
        for (int i = lane; i < (K >> 2); i += 32) { float4 v = xr[i]; s += (v.x + v.y) + (v.z + v.w); }
        mean = warp_sum(s) / K;
        float sq = 0.f;
        for (int i = lane; i < (K >> 2); i += 32) {
          float4 v = xr[i];
          float a = v.x - mean, b2 = v.y - mean, c = v.z - mean, e = v.w - mean;
          sq += (a * a + b2 * b2) + (c * c + e * e);
        }
        rstd = rsqrtf(warp_sum(sq) / K + 1e-5f);
      }
      if (lane == 0) { sStat[2 * r] = mean; sStat[2 * r + 1] = rstd; }
    }
    __syncthreads();
  }

  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  const int wrow = (n0 + g) < N ? (n0 + g) : (N - 1);  // clamp: columns past N are computed but never stored
  const bf16* wbase = W + (size_t)wrow * K;

  for (int k0 = 0; k0 < K; k0 += KC) {
    const int kc = (K - k0) < KC ? (K - k0) : KC;  // multiple of 32
    const int kper = kc / KS;                       // k range of one warp in this chunk (multiple of 32 by host check)
    uint4 wreg[8];
    const int ngroups = kper >> 5;
    const bf16* wp = wbase + k0 + ks * kper + 8 * tq;
    // stage A[row0 .. row0+63][k0 .. k0+kc) as bf16 with the k permutation, zero rows past B
    if (k0 > 0) __syncthreads();  // previous chunk fully consumed
    if (ln_fast) {
      const float* h = reinterpret_cast<const float*>(A_);
      if (K <= 512) ln_stage_rows<4, 4>(h, gamma, beta, sA, K, row0, nrows, srows, A_PITCH);
      else ln_stage_rows<2, 8>(h, gamma, beta, sA, K, row0, nrows, srows, A_PITCH);
    } else if constexpr (LN) {
      const float* h = reinterpret_cast<const float*>(A_);
      for (int i = threadIdx.x; i < srows * (kc >> 2); i += THREADS) {
        const int r = i / (kc >> 2), k4 = (i - r * (kc >> 2)) << 2;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r < nrows) {
          v = *reinterpret_cast<const float4*>(h + (size_t)(row0 + r) * K + k0 + k4);
          const float mean = sStat[2 * r], rstd = sStat[2 * r + 1];
          const float4 gg = *reinterpret_cast<const float4*>(gamma + k0 + k4);
          const float4 bb = *reinterpret_cast<const float4*>(beta + k0 + k4);
          v.x = (v.x - mean) * rstd * gg.x + bb.x; v.y = (v.y - mean) * rstd * gg.y + bb.y;
          v.z = (v.z - mean) * rstd * gg.z + bb.z; v.w = (v.w - mean) * rstd * gg.w + bb.w;
        }
        // k4 % 4 == 0: elements (k4, k4+1) and (k4+2, k4+3) are the two adjacent pairs h = 0, 1
        bf16* dst = sA + r * A_PITCH;
        *reinterpret_cast<__nv_bfloat162*>(dst + perm_k(k4)) = __floats2bfloat162_rn(v.x, v.y);
        *reinterpret_cast<__nv_bfloat162*>(dst + perm_k(k4 + 2)) = __floats2bfloat162_rn(v.z, v.w);
      }
    } else {
      const bf16* a = reinterpret_cast<const bf16*>(A_);
      const int per_row = kc >> 3, total = srows * per_row;
      for (int i0 = threadIdx.x; i0 < total; i0 += 8 * THREADS) {  // 8 loads in flight per thread
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int i = i0 + u * THREADS;
          const int r = i / per_row, k8 = (i - r * per_row) << 3;
          v[u] = (i < total && r < nrows) ? __ldcg(reinterpret_cast<const uint4*>(a + (size_t)(row0 + r) * K + k0 + k8))
                                          : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int i = i0 + u * THREADS;
          if (i < total) {
            const int r = i / per_row, k8 = (i - r * per_row) << 3;
            // 8 consecutive k = one lane's load (t = (k8 >> 3) & 3): pairs go to j*16 + h*8 + 2t
            bf16* dst = sA + r * A_PITCH + (k8 & ~31) + 2 * ((k8 >> 3) & 3);
            *reinterpret_cast<uint32_t*>(dst) = v[u].x;
            *reinterpret_cast<uint32_t*>(dst + 8) = v[u].y;
            *reinterpret_cast<uint32_t*>(dst + 16) = v[u].z;
            *reinterpret_cast<uint32_t*>(dst + 24) = v[u].w;
          }
        }
      }
    }
    __syncthreads();
    // stream the warp's weights in batches of up to 8 outstanding 16-byte loads per lane
    for (int g0 = 0; g0 < ngroups; g0 += 8) {
      const int nb = (ngroups - g0) < 8 ? (ngroups - g0) : 8;
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (i < nb) wreg[i] = ld_stream16(wp + (size_t)(g0 + i) * 32);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (i < nb) {
          const int kk = ks * kper + (g0 + i) * 32;  // chunk-local k of this 32-wide group
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const uint32_t b0 = j == 0 ? wreg[i].x : wreg[i].z, b1 = j == 0 ? wreg[i].y : wreg[i].w;
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
              if (mt >= mtiles) break;  // uniform across the CTA
              uint32_t af[4];
              ldsm_x4(af, sA + (mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * A_PITCH + kk + 16 * j + (lane >> 4) * 8);
              mma_bf16(acc[mt], af, b0, b1);
            }
          }
        }
      }
    }
  }

  // k-split reduction in shared memory (fixed order), then the epilogue: thread -> (row, column)
  float* my = sRed + warp * (ROWS * 8);
#pragma unroll
  for (int mt = 0; mt < 4; ++mt) {
    *reinterpret_cast<float2*>(my + (mt * 16 + g) * 8 + 2 * tq) = make_float2(acc[mt][0], acc[mt][1]);
    *reinterpret_cast<float2*>(my + (mt * 16 + g + 8) * 8 + 2 * tq) = make_float2(acc[mt][2], acc[mt][3]);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < ROWS * NC; i += THREADS) {
    const int r = i / NC, c = i - r * NC;
    const int tile = c >> 3, cc = c & 7;
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < KS; ++k) s += sRed[(k * NT + tile) * (ROWS * 8) + r * 8 + cc];
    const int n = blockIdx.x * NC + c;
    if (r < nrows && n < N) epi.apply(row0 + r, n, s, t);
  }
}

// ---------------------------------------------------------------------------------------------
// Single-query attention over cache rows 0..t of one (sample, head).  Cache layout [B][heads][L][64]
// bf16, so the rows of one (sample, head) are contiguous.  8 lanes share a key (16 bytes = 8 channels
// each); the 32 lane groups of the CTA take keys j = group (mod 32), four keys per round with the K
// and V rows of all four in flight together, and keep an online softmax (running max, sum, output)
// per group in fp32; the groups are merged through shared memory at the end.  q, out: [B, d].
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
seq_attention_kernel(const bf16* __restrict__ q, const bf16* __restrict__ kc, const bf16* __restrict__ vc,
                     bf16* __restrict__ out, int L, int d, int heads, float scale_log2e,
                     const int* __restrict__ step_base, int step_off, int n_steps) {
  const int t = *step_base + step_off;
  if (t >= n_steps) return;
  __shared__ float s_m[32], s_l[32], s_o[32][HD];
  const int head = blockIdx.x, b = blockIdx.y;
  const int nk = t + 1;
  const int sub = threadIdx.x & 7, grp = threadIdx.x >> 3;
  const bf16* kb = kc + ((size_t)b * heads + head) * L * HD + sub * 8;
  const bf16* vb = vc + ((size_t)b * heads + head) * L * HD + sub * 8;
  float qf[8];
  {
    const uint4 qv = *reinterpret_cast<const uint4*>(q + (size_t)b * d + head * HD + sub * 8);
    const __nv_bfloat162* q2 = reinterpret_cast<const __nv_bfloat162*>(&qv);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __bfloat1622float2(q2[i]);
      qf[2 * i] = f.x * scale_log2e;  // scores in base-2 units: softmax via exp2
      qf[2 * i + 1] = f.y * scale_log2e;
    }
  }
  float m_run = -INFINITY, l_run = 0.f, o[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) o[i] = 0.f;
  for (int j0 = 0; j0 < nk; j0 += 128) {
    uint4 kv[4], vv[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int j = j0 + u * 32 + grp;
      const bool ok = j < nk;
      kv[u] = ok ? __ldcg(reinterpret_cast<const uint4*>(kb + (size_t)j * HD)) : make_uint4(0u, 0u, 0u, 0u);
      vv[u] = ok ? __ldcg(reinterpret_cast<const uint4*>(vb + (size_t)j * HD)) : make_uint4(0u, 0u, 0u, 0u);
    }
    float sc[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&kv[u]);
      float s = 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(k2[i]);
        s = fmaf(qf[2 * i], f.x, s);
        s = fmaf(qf[2 * i + 1], f.y, s);
      }
      s += __shfl_xor_sync(0xffffffffu, s, 1);
      s += __shfl_xor_sync(0xffffffffu, s, 2);
      s += __shfl_xor_sync(0xffffffffu, s, 4);
      sc[u] = (j0 + u * 32 + grp) < nk ? s : -INFINITY;
    }
    const float m_new = fmaxf(fmaxf(m_run, fmaxf(sc[0], sc[1])), fmaxf(sc[2], sc[3]));
    if (m_new > -INFINITY) {  // this group has seen at least one key
      const float corr = exp2f(m_run - m_new);  // 0 when m_run = -inf
      l_run *= corr;
#pragma unroll
      for (int i = 0; i < 8; ++i) o[i] *= corr;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float pj = exp2f(sc[u] - m_new);  // 0 for a masked key
        l_run += pj;
        const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&vv[u]);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __bfloat1622float2(v2[i]);
          o[2 * i] = fmaf(pj, f.x, o[2 * i]);
          o[2 * i + 1] = fmaf(pj, f.y, o[2 * i + 1]);
        }
      }
      m_run = m_new;
    }
  }
  if (sub == 0) { s_m[grp] = m_run; s_l[grp] = l_run; }
#pragma unroll
  for (int i = 0; i < 8; ++i) s_o[grp][sub * 8 + i] = o[i];
  __syncthreads();
  if (threadIdx.x < HD) {
    float mx = s_m[0];  // group 0 always holds key 0
#pragma unroll 8
    for (int gI = 1; gI < 32; ++gI) mx = fmaxf(mx, s_m[gI]);
    float num = 0.f, den = 0.f;
#pragma unroll 8
    for (int gI = 0; gI < 32; ++gI) {
      const float w = exp2f(s_m[gI] - mx);  // 0 for a group without keys
      num = fmaf(w, s_o[gI][threadIdx.x], num);
      den = fmaf(w, s_l[gI], den);
    }
    out[(size_t)b * d + head * HD + threadIdx.x] = __float2bfloat16_rn(num / den);
  }
}

// ---------------------------------------------------------------------------------------------
// u[b, t+1, :] = v[b, t+1, :] * exp(alpha~) + mu~ from the head output o [B, 2D] (interleaved), then
// the embedding of that token for the next step: h[b, :] = u W_in^T + b_in + pos[t+1] (+ cls[y_b]).
// One CTA per sample.  With first != 0 the step is the block's start: u[b, 0, :] = v[b, 0, :] (Eq. 5,
// first row) and the embedding of token 0.
// ---------------------------------------------------------------------------------------------
__global__ void seq_update_embed_kernel(const float* __restrict__ o, const float* __restrict__ v, float* __restrict__ u,
                                        const int* __restrict__ labels, const float* __restrict__ w_in_t,
                                        const float* __restrict__ b_in, const float* __restrict__ pos,
                                        const float* __restrict__ cls, float* __restrict__ h, int L, int D, int d,
                                        int reversed, int first, const int* __restrict__ step_base, int step_off,
                                        int n_steps) {
  const int t = *step_base + step_off;
  if (!first && t >= n_steps) return;
  extern __shared__ float s_tok[];
  const int b = blockIdx.x;
  const int l_new = first ? 0 : t + 1;
  const size_t e0 = ((size_t)b * L + tok_index(l_new, L, reversed)) * D;
  for (int c = threadIdx.x; c < D; c += blockDim.x) {
    float val = v[e0 + c];
    if (!first) val = fmaf(val, expf(o[(size_t)b * 2 * D + 2 * c + 1]), o[(size_t)b * 2 * D + 2 * c]);
    u[e0 + c] = val;
    s_tok[c] = val;
  }
  __syncthreads();
  if (l_new >= L - 1) return;  // the last token is never fed back
  const float* cl = (cls != nullptr) ? cls + (size_t)labels[b] * d : nullptr;
  for (int j = threadIdx.x; j < d; j += blockDim.x) {
    float acc = 0.f;
    for (int c = 0; c < D; ++c) acc = fmaf(s_tok[c], w_in_t[(size_t)c * d + j], acc);
    acc += b_in[j] + pos[(size_t)l_new * d + j];
    if (cl) acc += cl[j];
    h[(size_t)b * d + j] = acc;
  }
}

__global__ void seq_advance_kernel(int* step_base, int by) {
  if (threadIdx.x == 0 && blockIdx.x == 0) *step_base += by;
}

}  // namespace seq

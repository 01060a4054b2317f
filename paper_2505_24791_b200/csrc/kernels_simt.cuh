// CUDA-core kernels: layout, embedding, LayerNorm, SIMT GEMM (fp32 engine and odd shapes), SIMT
// attention (fp32 engine), single-query attention over the KV cache, update / forward epilogues
// as stand-alone kernels, and Jacobi sweep control.
#pragma once
#include "common.cuh"
#include "epilogue.cuh"

// ------------------------------------------------------------------------------------------------
// image [B,C,H,W] <-> tokens [B,L,D]; raster patch order, (c,py,px) inside a token.
// ------------------------------------------------------------------------------------------------
__global__ void patchify_kernel(float* __restrict__ img, float* __restrict__ seq, int B, int C, int H,
                                int W, int p, int to_seq) {
  size_t n = (size_t)B * C * H * W;
  int gw = W / p, D = C * p * p, L = (H / p) * gw;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    int x = i % W, y = (i / W) % H, c = (i / ((size_t)W * H)) % C, b = i / ((size_t)W * H * C);
    int l = (y / p) * gw + (x / p);
    int e = (c * p + (y % p)) * p + (x % p);
    size_t j = ((size_t)b * L + l) * D + e;
    if (to_seq) seq[j] = img[i]; else img[i] = seq[j];
  }
}

// ------------------------------------------------------------------------------------------------
// token embedding: h[s,l,:] = u[b,pos(l),:] W_in^T + b_in + pos_emb[l] (+ cls[y_b]), b = idx[s].
// w_in_t is W_in transposed to [D, d] so consecutive threads read consecutive addresses.
// One CTA per output row.  `l_fixed` >= 0: rows are samples and every row uses position l_fixed
// (sequential decoding step).
// ------------------------------------------------------------------------------------------------
__global__ void embed_kernel(const float* __restrict__ u, const int* __restrict__ idx, const int* __restrict__ labels,
                             const float* __restrict__ w_in_t, const float* __restrict__ b_in,
                             const float* __restrict__ pos, const float* __restrict__ cls, float* __restrict__ h,
                             int L, int D, int d, int reversed, int l_fixed) {
  extern __shared__ float s_u[];
  int row = blockIdx.x;
  int s = (l_fixed >= 0) ? row : row / L;
  int l = (l_fixed >= 0) ? l_fixed : row - s * L;
  int b = idx ? idx[s] : s;
  const float* up = u + ((size_t)b * L + tok_index(l, L, reversed)) * D;
  for (int c = threadIdx.x; c < D; c += blockDim.x) s_u[c] = up[c];
  __syncthreads();
  const float* cl = (cls != nullptr) ? cls + (size_t)labels[b] * d : nullptr;
  for (int j = threadIdx.x; j < d; j += blockDim.x) {
    float acc = 0.f;
    for (int c = 0; c < D; ++c) acc = fmaf(s_u[c], w_in_t[(size_t)c * d + j], acc);
    acc += b_in[j] + pos[(size_t)l * d + j];
    if (cl) acc += cl[j];
    h[(size_t)row * d + j] = acc;
  }
}

// The same embedding for the rows of a full pass, R rows per CTA: every weight element a thread loads is
// used for R rows (the one-row kernel re-reads the whole [D, d] matrix per row).  The R tokens sit in
// shared memory transposed, [D][R], so that four rows come with one broadcast 16-byte read.
template <int R>
__global__ void __launch_bounds__(256)
embed_rows_kernel(const float* __restrict__ u, const int* __restrict__ idx, const int* __restrict__ labels,
                  const float* __restrict__ w_in_t, const float* __restrict__ b_in, const float* __restrict__ pos,
                  const float* __restrict__ cls, float* __restrict__ h, int L, int D, int d, int reversed, int n_rows) {
  extern __shared__ __align__(16) float s_ut[];  // [D][R]
  pdl_launch_dependents();
  pdl_wait();
  const int row0 = blockIdx.x * R;
  for (int e = threadIdx.x; e < R * D; e += blockDim.x) {
    const int r = e / D, c = e - r * D, row = row0 + r;
    float val = 0.f;
    if (row < n_rows) {
      const int s = row / L, l = row - s * L;
      const int b = idx ? idx[s] : s;
      val = u[((size_t)b * L + tok_index(l, L, reversed)) * D + c];
    }
    s_ut[c * R + r] = val;
  }
  __syncthreads();
  for (int j = threadIdx.x; j < d; j += blockDim.x) {
    float acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = 0.f;
    for (int c = 0; c < D; ++c) {
      const float w = w_in_t[(size_t)c * d + j];
#pragma unroll
      for (int r4 = 0; r4 < R; r4 += 4) {
        const float4 x = *reinterpret_cast<const float4*>(s_ut + c * R + r4);
        acc[r4] = fmaf(x.x, w, acc[r4]);
        acc[r4 + 1] = fmaf(x.y, w, acc[r4 + 1]);
        acc[r4 + 2] = fmaf(x.z, w, acc[r4 + 2]);
        acc[r4 + 3] = fmaf(x.w, w, acc[r4 + 3]);
      }
    }
    const float bj = b_in[j];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int row = row0 + r;
      if (row < n_rows) {
        const int s = row / L, l = row - s * L;
        float a = acc[r] + (bj + pos[(size_t)l * d + j]);
        if (cls != nullptr) a += cls[(size_t)labels[idx ? idx[s] : s] * d + j];
        h[(size_t)row * d + j] = a;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Embedding of R rows per CTA fused with the first LayerNorm of the block:
//   h[row, :]  = u[token] W_in^T + b_in + pos[l] (+ cls[y])          (fp32 residual stream)
//   xn[row, :] = LayerNorm(h[row, :]) * gamma + beta                  (T; plus the "lo" half of a two-term pair)
// Thread k owns columns 4k..4k+3 of all R rows (blockDim.x = d / 4 rounded up to whole warps, d % 4 == 0): per
// token value one 16-byte weight load feeds 4 R FMAs, the R tokens sit in shared memory transposed ([D][R]) so
// four rows come with one broadcast 16-byte read.  The row statistics (two-pass, eps 1e-5) are reduced over the
// CTA's warps through shared memory.  h is bit-identical to embed_rows_kernel's.
// ------------------------------------------------------------------------------------------------
template <class T, int R>
__global__ void __launch_bounds__(256)
embed_ln_rows_kernel(const float* __restrict__ u, const int* __restrict__ idx, const int* __restrict__ labels,
                     const float* __restrict__ w_in_t, const float* __restrict__ b_in, const float* __restrict__ pos,
                     const float* __restrict__ cls, float* __restrict__ h, const float* __restrict__ gamma,
                     const float* __restrict__ beta, T* __restrict__ xn, T* __restrict__ xn_lo, int L, int D, int d,
                     int reversed, int n_rows) {
  extern __shared__ __align__(16) float s_ut[];  // [D][R]
  __shared__ float s_red[2][8][R];
  __shared__ int s_l[R], s_b[R];
  pdl_launch_dependents();
  pdl_wait();
  const int row0 = blockIdx.x * R;
  if (threadIdx.x < R) {
    const int row = row0 + threadIdx.x;
    int l = 0, b = -1;
    if (row < n_rows) {
      const int s = row / L;
      l = row - s * L;
      b = idx ? idx[s] : s;
    }
    s_l[threadIdx.x] = l;
    s_b[threadIdx.x] = b;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < R * D; e += blockDim.x) {
    const int r = e / D, c = e - r * D, b = s_b[r];
    s_ut[c * R + r] = b >= 0 ? u[((size_t)b * L + tok_index(s_l[r], L, reversed)) * D + c] : 0.f;
  }
  __syncthreads();
  const int k = threadIdx.x, dv = d >> 2;
  const bool act = k < dv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = (blockDim.x + 31) >> 5;
  float4 acc[R];
#pragma unroll
  for (int r = 0; r < R; ++r) acc[r] = make_float4(0.f, 0.f, 0.f, 0.f);
  if (act) {
    const float4* w4 = reinterpret_cast<const float4*>(w_in_t) + k;
#pragma unroll (R <= 4 ? 16 : 4)
    for (int c = 0; c < D; ++c) {
      const float4 w = __ldg(w4 + (size_t)c * dv);
#pragma unroll
      for (int r4 = 0; r4 < R; r4 += 4) {
        const float4 x = *reinterpret_cast<const float4*>(s_ut + c * R + r4);
        const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          acc[r4 + q].x = fmaf(xs[q], w.x, acc[r4 + q].x);
          acc[r4 + q].y = fmaf(xs[q], w.y, acc[r4 + q].y);
          acc[r4 + q].z = fmaf(xs[q], w.z, acc[r4 + q].z);
          acc[r4 + q].w = fmaf(xs[q], w.w, acc[r4 + q].w);
        }
      }
    }
  }
  // residual stream row, first statistic
  float4 bj = make_float4(0.f, 0.f, 0.f, 0.f);
  if (act) bj = reinterpret_cast<const float4*>(b_in)[k];
  float part[R];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int row = row0 + r;
    part[r] = 0.f;
    if (act && row < n_rows) {
      const float4 p = __ldg(reinterpret_cast<const float4*>(pos) + (size_t)s_l[r] * dv + k);
      float4 a = acc[r];
      a.x += bj.x + p.x; a.y += bj.y + p.y; a.z += bj.z + p.z; a.w += bj.w + p.w;
      if (cls != nullptr) {
        const float4 cl = __ldg(reinterpret_cast<const float4*>(cls) + (size_t)labels[s_b[r]] * dv + k);
        a.x += cl.x; a.y += cl.y; a.z += cl.z; a.w += cl.w;
      }
      acc[r] = a;
      reinterpret_cast<float4*>(h)[(size_t)row * dv + k] = a;
      part[r] = (a.x + a.y) + (a.z + a.w);
    }
  }
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const float v = warp_sum(part[r]);
    if (lane == 0) s_red[0][warp][r] = v;
  }
  __syncthreads();
  const float inv_d = 1.f / (float)d;
#pragma unroll
  for (int r = 0; r < R; ++r) {
    float tot = 0.f;
    for (int w = 0; w < nwarps; ++w) tot += s_red[0][w][r];
    const float mean = tot * inv_d;
    float sq = 0.f;
    if (act) {
      acc[r].x -= mean; acc[r].y -= mean; acc[r].z -= mean; acc[r].w -= mean;
      sq = (acc[r].x * acc[r].x + acc[r].y * acc[r].y) + (acc[r].z * acc[r].z + acc[r].w * acc[r].w);
    }
    part[r] = warp_sum(sq);
    if (lane == 0) s_red[1][warp][r] = part[r];
  }
  __syncthreads();
  if (!act) return;
  const float4 g = reinterpret_cast<const float4*>(gamma)[k], bb = reinterpret_cast<const float4*>(beta)[k];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int row = row0 + r;
    if (row >= n_rows) continue;
    float tot = 0.f;
    for (int w = 0; w < nwarps; ++w) tot += s_red[1][w][r];
    const float rstd = rsqrtf(tot * inv_d + 1e-5f);
    const float o0 = acc[r].x * rstd * g.x + bb.x, o1 = acc[r].y * rstd * g.y + bb.y;
    const float o2 = acc[r].z * rstd * g.z + bb.z, o3 = acc[r].w * rstd * g.w + bb.w;
    if constexpr (sizeof(T) == 4) {
      reinterpret_cast<float4*>(xn)[(size_t)row * dv + k] = make_float4(o0, o1, o2, o3);
    } else {
      __nv_bfloat162 p0 = __floats2bfloat162_rn(o0, o1), p1 = __floats2bfloat162_rn(o2, o3);
      uint2 w2;
      w2.x = *reinterpret_cast<uint32_t*>(&p0); w2.y = *reinterpret_cast<uint32_t*>(&p1);
      reinterpret_cast<uint2*>(xn)[(size_t)row * dv + k] = w2;
      if (xn_lo != nullptr) {  // second term of the error-compensated pair
        const float2 f0 = __bfloat1622float2(p0), f1 = __bfloat1622float2(p1);
        __nv_bfloat162 q0 = __floats2bfloat162_rn(o0 - f0.x, o1 - f0.y), q1 = __floats2bfloat162_rn(o2 - f1.x, o3 - f1.y);
        w2.x = *reinterpret_cast<uint32_t*>(&q0); w2.y = *reinterpret_cast<uint32_t*>(&q1);
        reinterpret_cast<uint2*>(xn_lo)[(size_t)row * dv + k] = w2;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// LayerNorm over the last dimension (eps 1e-5), fp32 in, T out.  One warp per row, the row is
// held in registers (d <= 32*4*MAXV).
// ------------------------------------------------------------------------------------------------
template <class T, int MAXV>
__global__ void layernorm_kernel(const float* __restrict__ x, const float* __restrict__ gamma,
                                 const float* __restrict__ beta, T* __restrict__ y, T* __restrict__ y_lo, int rows,
                                 int d) {
  pdl_launch_dependents();
  pdl_wait();
  int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= rows) return;
  const float4* xr = reinterpret_cast<const float4*>(x + (size_t)warp * d);
  int nv = d >> 2;  // float4 per row
  float4 v[MAXV];
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    int k = lane + i * 32;
    if (k < nv) { v[i] = xr[k]; sum += v[i].x + v[i].y + v[i].z + v[i].w; }
  }
  float mean = warp_sum(sum) / d;
  float sq = 0.f;
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    int k = lane + i * 32;
    if (k < nv) {
      float a = v[i].x - mean, b = v[i].y - mean, c = v[i].z - mean, e = v[i].w - mean;
      sq += a * a + b * b + c * c + e * e;
    }
  }
  float rstd = rsqrtf(warp_sum(sq) / d + 1e-5f);
  T* yr = y + (size_t)warp * d;
#pragma unroll
  for (int i = 0; i < MAXV; ++i) {
    int k = lane + i * 32;
    if (k < nv) {
      float4 g = reinterpret_cast<const float4*>(gamma)[k], bb = reinterpret_cast<const float4*>(beta)[k];
      float o0 = (v[i].x - mean) * rstd * g.x + bb.x, o1 = (v[i].y - mean) * rstd * g.y + bb.y;
      float o2 = (v[i].z - mean) * rstd * g.z + bb.z, o3 = (v[i].w - mean) * rstd * g.w + bb.w;
      if constexpr (sizeof(T) == 4) {
        reinterpret_cast<float4*>(yr)[k] = make_float4(o0, o1, o2, o3);
      } else {
        __nv_bfloat162 p0 = __floats2bfloat162_rn(o0, o1), p1 = __floats2bfloat162_rn(o2, o3);
        uint2 w;
        w.x = *reinterpret_cast<uint32_t*>(&p0); w.y = *reinterpret_cast<uint32_t*>(&p1);
        reinterpret_cast<uint2*>(yr)[k] = w;
        if (y_lo != nullptr) {  // second term of the error-compensated pair
          float2 f0 = __bfloat1622float2(p0), f1 = __bfloat1622float2(p1);
          __nv_bfloat162 q0 = __floats2bfloat162_rn(o0 - f0.x, o1 - f0.y), q1 = __floats2bfloat162_rn(o2 - f1.x, o3 - f1.y);
          w.x = *reinterpret_cast<uint32_t*>(&q0); w.y = *reinterpret_cast<uint32_t*>(&q1);
          reinterpret_cast<uint2*>(y_lo + (size_t)warp * d)[k] = w;
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Residual add + LayerNorm for sweeps over few rows, where the projection before it left its result as `ksplit`
// K-slice partial products (slice s of row r at part[(s * part_rows + r) * d]).  One CTA per row, one thread per
// four columns (blockDim.x = d / 4, a multiple of 32), so that every load of a row is in flight at once:
//   x[row] <- x[row] + bias + slice 0 + slice 1 + ...   (this order: the sum does not depend on which slice finished first)
//   y[row] <- LayerNorm(x[row]) (two-pass statistics, eps 1e-5), as T (plus the second term of the pair in y_lo).
// ------------------------------------------------------------------------------------------------
template <class T>
__global__ void __launch_bounds__(1024)
resid_sum_ln_kernel(float* x, const float* __restrict__ part, int ksplit, int part_rows, const float* __restrict__ rbias,
                    const float* __restrict__ gamma, const float* __restrict__ beta, T* __restrict__ y,
                    T* __restrict__ y_lo, int d) {
  constexpr int MAXS = 8;
  __shared__ float s_red[2][32];
  pdl_launch_dependents();
  const int row = blockIdx.x, k = threadIdx.x, dv = d >> 2;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  const float4 g = reinterpret_cast<const float4*>(gamma)[k], bb = reinterpret_cast<const float4*>(beta)[k];
  const float4 rb = reinterpret_cast<const float4*>(rbias)[k];
  pdl_wait();
  float4 a = reinterpret_cast<const float4*>(x)[(size_t)row * dv + k];
  float4 p[MAXS];
#pragma unroll
  for (int s = 0; s < MAXS; ++s)
    if (s < ksplit) p[s] = reinterpret_cast<const float4*>(part)[((size_t)s * part_rows + row) * dv + k];
  a.x += rb.x; a.y += rb.y; a.z += rb.z; a.w += rb.w;
#pragma unroll
  for (int s = 0; s < MAXS; ++s)
    if (s < ksplit) { a.x += p[s].x; a.y += p[s].y; a.z += p[s].z; a.w += p[s].w; }
  reinterpret_cast<float4*>(x)[(size_t)row * dv + k] = a;
  float v = warp_sum((a.x + a.y) + (a.z + a.w));
  if (lane == 0) s_red[0][warp] = v;
  __syncthreads();
  float tot = 0.f;
  for (int w = 0; w < nwarps; ++w) tot += s_red[0][w];
  const float mean = tot / d;
  const float e0 = a.x - mean, e1 = a.y - mean, e2 = a.z - mean, e3 = a.w - mean;
  v = warp_sum((e0 * e0 + e1 * e1) + (e2 * e2 + e3 * e3));
  if (lane == 0) s_red[1][warp] = v;
  __syncthreads();
  tot = 0.f;
  for (int w = 0; w < nwarps; ++w) tot += s_red[1][w];
  const float rstd = rsqrtf(tot / d + 1e-5f);
  const float o0 = e0 * rstd * g.x + bb.x, o1 = e1 * rstd * g.y + bb.y, o2 = e2 * rstd * g.z + bb.z, o3 = e3 * rstd * g.w + bb.w;
  if constexpr (sizeof(T) == 4) {
    reinterpret_cast<float4*>(y)[(size_t)row * dv + k] = make_float4(o0, o1, o2, o3);
  } else {
    __nv_bfloat162 p0 = __floats2bfloat162_rn(o0, o1), p1 = __floats2bfloat162_rn(o2, o3);
    uint2 w;
    w.x = *reinterpret_cast<uint32_t*>(&p0); w.y = *reinterpret_cast<uint32_t*>(&p1);
    reinterpret_cast<uint2*>(y)[(size_t)row * dv + k] = w;
    if (y_lo != nullptr) {
      float2 f0 = __bfloat1622float2(p0), f1 = __bfloat1622float2(p1);
      __nv_bfloat162 q0 = __floats2bfloat162_rn(o0 - f0.x, o1 - f0.y), q1 = __floats2bfloat162_rn(o2 - f1.x, o3 - f1.y);
      w.x = *reinterpret_cast<uint32_t*>(&q0); w.y = *reinterpret_cast<uint32_t*>(&q1);
      reinterpret_cast<uint2*>(y_lo)[(size_t)row * dv + k] = w;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// SIMT GEMM: C[M,N] = A[M,K] W[N,K]^T, fp32 FMA accumulate, 64x64 tile, 16-wide K slab, 256 threads,
// 4x4 outputs per thread.  Used by the fp32 engine everywhere and by the bf16 engine for shapes
// the tensor-core kernels do not take.
// ------------------------------------------------------------------------------------------------
template <class TA, class Epi>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const TA* __restrict__ A, const TA* __restrict__ Wt, int M,
                                                        int N, int K, Epi epi) {
  __shared__ float sA[16][64 + 4];
  __shared__ float sB[16][64 + 4];
  int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  for (int k0 = 0; k0 < K; k0 += 16) {
    // 64 rows x 16 k per operand = 1024 elements, 4 per thread
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int e = threadIdx.x + i * 256;
      int r = e >> 4, k = e & 15;
      int gm = m0 + r, gn = n0 + r, gk = k0 + k;
      sA[k][r] = (gm < M && gk < K) ? to_f32(A[(size_t)gm * K + gk]) : 0.f;
      sB[k][r] = (gn < N && gk < K) ? to_f32(Wt[(size_t)gn * K + gk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = sA[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = sB[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int row = m0 + ty * 4 + i, col0 = n0 + tx * 4;
    if (row < M && col0 < N) {
      int nv = N - col0 < 4 ? N - col0 : 4;
      epi.template apply<4>(row, col0, acc[i], nv);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Causal attention, SIMT: one warp per (slot, head, query position).  qkv rows are [q | k | v],
// 3d wide.  Scores for keys j <= i in shared memory, fp32 softmax, output a[row, head*hd + c].
// ------------------------------------------------------------------------------------------------
template <class T>
__global__ void attention_simt_kernel(const T* __restrict__ qkv, T* __restrict__ out, int L, int d, int hd,
                                      float scale) {
  extern __shared__ float s_p[];  // [warps][L] scores, then [warps][hd] query
  int warps = blockDim.x >> 5, w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int i = blockIdx.x * warps + w;  // query position
  int head = blockIdx.y, s = blockIdx.z;
  float* p = s_p + (size_t)w * L;
  float* sq = s_p + (size_t)warps * L + (size_t)w * hd;
  if (i >= L) return;
  size_t ld = 3 * (size_t)d;
  const T* base = qkv + (size_t)s * L * ld + (size_t)head * hd;
  for (int c = lane; c < hd; c += 32) sq[c] = to_f32(base[(size_t)i * ld + c]);
  __syncwarp();
  float mx = -INFINITY;
  for (int j = lane; j <= i; j += 32) {
    const T* kr = base + (size_t)j * ld + d;
    float acc = 0.f;
    for (int c = 0; c < hd; ++c) acc = fmaf(sq[c], to_f32(kr[c]), acc);
    acc *= scale;
    p[j] = acc;
    mx = fmaxf(mx, acc);
  }
  mx = warp_max(mx);
  float sum = 0.f;
  for (int j = lane; j <= i; j += 32) {
    float e = expf(p[j] - mx);
    p[j] = e;
    sum += e;
  }
  sum = warp_sum(sum);
  __syncwarp();
  float inv = 1.f / sum;
  for (int c = lane; c < hd; c += 32) {
    float acc = 0.f;
    for (int j = 0; j <= i; ++j) acc = fmaf(p[j], to_f32(base[(size_t)j * ld + 2 * d + c]), acc);
    out[((size_t)s * L + i) * d + (size_t)head * hd + c] = from_f32<T>(acc * inv);
  }
}

// ------------------------------------------------------------------------------------------------
// Sequential decoding: one query per (sample, head) over cache rows 0..t.  4 warps split the keys.
// kc, vc: [B, L, d]; q, out: [B, d].
// ------------------------------------------------------------------------------------------------
template <class T>
__global__ void __launch_bounds__(128) attention_step_kernel(const T* __restrict__ q, const T* __restrict__ kc,
                                                             const T* __restrict__ vc, T* __restrict__ out, int L,
                                                             int d, int hd, int t, float scale) {
  extern __shared__ float sm[];  // p[t+1] | q[hd] | red[8] | acc[4][hd]
  int head = blockIdx.x, b = blockIdx.y;
  int nk = t + 1;
  float* p = sm;
  float* sq = p + L;
  float* red = sq + hd;
  float* sacc = red + 8;
  int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const T* kb = kc + (size_t)b * L * d + (size_t)head * hd;
  const T* vb = vc + (size_t)b * L * d + (size_t)head * hd;
  for (int c = threadIdx.x; c < hd; c += 128) sq[c] = to_f32(q[(size_t)b * d + head * hd + c]);
  __syncthreads();
  float mx = -INFINITY;
  for (int j = threadIdx.x; j < nk; j += 128) {
    const T* kr = kb + (size_t)j * d;
    float acc = 0.f;
    for (int c = 0; c < hd; ++c) acc = fmaf(sq[c], to_f32(kr[c]), acc);
    acc *= scale;
    p[j] = acc;
    mx = fmaxf(mx, acc);
  }
  mx = warp_max(mx);
  if (lane == 0) red[w] = mx;
  __syncthreads();
  mx = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
  float sum = 0.f;
  for (int j = threadIdx.x; j < nk; j += 128) {
    float e = expf(p[j] - mx);
    p[j] = e;
    sum += e;
  }
  sum = warp_sum(sum);
  if (lane == 0) red[4 + w] = sum;
  __syncthreads();
  float inv = 1.f / (red[4] + red[5] + red[6] + red[7]);
  // warp w accumulates keys j = w, w+4, ...; lanes over channels
  for (int c = lane; c < hd; c += 32) {
    float acc = 0.f;
    for (int j = w; j < nk; j += 4) acc = fmaf(p[j], to_f32(vb[(size_t)j * d + c]), acc);
    sacc[w * hd + c] = acc;
  }
  __syncthreads();
  for (int c = threadIdx.x; c < hd; c += 128) {
    float acc = (sacc[c] + sacc[hd + c]) + (sacc[2 * hd + c] + sacc[3 * hd + c]);
    out[(size_t)b * d + head * hd + c] = from_f32<T>(acc * inv);
  }
}

// ------------------------------------------------------------------------------------------------
// Stand-alone Jacobi update (Algorithm 1's inner line + norm) from a stored head output.
// o: [rows, 2D]; interleaved != 0: columns (2c,2c+1) = (mu~_c, alpha~_c), else [mu~ | alpha~].
// One thread per (row, c).  u updated in place; maxdiff via order-independent atomic max.
// ------------------------------------------------------------------------------------------------
__global__ void jacobi_update_kernel(const float* __restrict__ o, const float* __restrict__ v, float* __restrict__ u,
                                     float* __restrict__ maxdiff, const int* __restrict__ idx, int n_rows, int L,
                                     int D, int reversed, int interleaved) {
  size_t n = (size_t)n_rows * D;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    int c = i % D;
    int row = i / D;
    int s = row / L, l = row - s * L;
    int b = idx ? idx[s] : s;
    float nw, old;
    if (l < L - 1) {
      size_t e = ((size_t)b * L + tok_index(l + 1, L, reversed)) * D + c;
      const float* orow = o + (size_t)row * 2 * D;
      float mu = interleaved ? orow[2 * c] : orow[c];
      float al = interleaved ? orow[2 * c + 1] : orow[D + c];
      old = u[e];
      nw = fmaf(v[e], expf(al), mu);
      u[e] = nw;
    } else {
      size_t e = ((size_t)b * L + tok_index(0, L, reversed)) * D + c;
      old = u[e];
      nw = v[e];
      u[e] = nw;
    }
    atomic_max_nonneg(maxdiff + b, fabsf(nw - old));
  }
}

// Jacobi update of sweeps over few rows, where the head projection left its result as `ksplit` K-slice partial
// products (slice s of row r at part[(s * part_rows + r) * npad], columns interleaved (mu~_c, alpha~_c), npad >= 2D):
// head = bias + slice 0 + slice 1 + ... (this order), then Algorithm 1's update line as in the fused epilogue: row
// (slot s, position l) updates token l + 1 of sample idx[s], the last position's row copies token 0.  One warp per
// row; per-row max|du| merged with the order-independent atomic max (NaN propagates).
__global__ void __launch_bounds__(256)
jacobi_update_split_kernel(const float* __restrict__ part, int ksplit, int part_rows, int npad, const float* __restrict__ bias,
                           const float* __restrict__ v, float* __restrict__ u, float* __restrict__ maxdiff,
                           const int* __restrict__ idx, int n_rows, int L, int D, int reversed) {
  pdl_launch_dependents();
  pdl_wait();
  const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (row >= n_rows) return;
  const int s = row / L, l = row - s * L;
  const int b = idx ? idx[s] : s;
  const bool upd = l < L - 1;
  const size_t e0 = ((size_t)b * L + tok_index(upd ? l + 1 : 0, L, reversed)) * D;
  float df = 0.f;
  for (int c = lane; c < D; c += 32) {
    float2 o = *reinterpret_cast<const float2*>(bias + 2 * c);
    for (int k = 0; k < ksplit; ++k) {
      const float2 p = __ldcg(reinterpret_cast<const float2*>(part + ((size_t)k * part_rows + row) * npad + 2 * c));
      o.x += p.x;
      o.y += p.y;
    }
    const float old = u[e0 + c], vv = v[e0 + c];
    const float nw = upd ? fmaf(vv, expf(o.y), o.x) : vv;
    u[e0 + c] = nw;
    const float dd = fabsf(nw - old);
    df = (dd > df || dd != dd) ? dd : df;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float other = __shfl_xor_sync(0xffffffffu, df, o);
    df = (other > df || other != other) ? other : df;
  }
  if (lane == 0) atomic_max_nonneg(maxdiff + b, df);
}

// Sequential decoding: token t+1 of every sample from the head output of token t (Eq. 5).
// o: [B, 2D] interleaved.
__global__ void seq_update_kernel(const float* __restrict__ o, const float* __restrict__ v, float* __restrict__ u,
                                  int B, int L, int D, int reversed, int t) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B * D) return;
  int b = i / D, c = i - b * D;
  size_t e = ((size_t)b * L + tok_index(t + 1, L, reversed)) * D + c;
  u[e] = fmaf(v[e], expf(o[(size_t)b * 2 * D + 2 * c + 1]), o[(size_t)b * 2 * D + 2 * c]);
}

// First token of a block passes through unchanged (Eq. 4 / Eq. 5 first row).
__global__ void copy_first_token_kernel(const float* __restrict__ v, float* __restrict__ u, int B, int L, int D,
                                        int reversed) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B * D) return;
  int b = i / D, c = i - b * D;
  size_t e = ((size_t)b * L + tok_index(0, L, reversed)) * D + c;
  u[e] = v[e];
}

// Forward direction (Eq. 4): v_l = (u_l - mu_l) exp(-alpha_l), logdet[b] -= sum alpha.  One CTA per
// sample so the per-sample sum is a fixed-order tree (deterministic).  o: [B*L, 2D] interleaved.
__global__ void __launch_bounds__(256) forward_affine_kernel(const float* __restrict__ o, const float* __restrict__ u,
                                                             float* __restrict__ v, float* __restrict__ logdet, int L,
                                                             int D, int reversed) {
  __shared__ float red[8];
  int b = blockIdx.x;
  float part = 0.f;
  for (int i = threadIdx.x; i < L * D; i += 256) {
    int l = i / D, c = i - l * D;
    size_t e = ((size_t)b * L + tok_index(l, L, reversed)) * D + c;
    float mu = 0.f, al = 0.f;
    if (l > 0) {
      const float* orow = o + ((size_t)b * L + (l - 1)) * 2 * D;
      mu = orow[2 * c];
      al = orow[2 * c + 1];
    }
    v[e] = (u[e] - mu) * expf(-al);
    part += al;
  }
  part = warp_sum(part);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = part;
  __syncthreads();
  if (threadIdx.x == 0 && logdet != nullptr) {
    float s = 0.f;
    for (int i = 0; i < 8; ++i) s += red[i];
    logdet[b] -= s;
  }
}

// ------------------------------------------------------------------------------------------------
// Sweep control.  After sweep `t`: record the sweep
// count of every active sample, drop the samples that passed the test, move a sample to the
// two-term ("hp") phase once its own max|du| <= switch_thresh, and rebuild the slot list as
// [single-precision samples..., hp samples...] with a stable partition, so the slot order never
// depends on timing and a sample's schedule depends on that sample alone.
// ctrl[0] = n_active, ctrl[1] = non-finite flag, ctrl[2] = bits of max over active samples of
// maxdiff, ctrl[3] = number of active samples in the hp phase (the tail of idx); ctrl[CTRL_SWEEP] = sweeps finished in
// this block, ctrl[CTRL_TAU] / ctrl[CTRL_SWITCH] = bits of tau and of the escalation threshold.
// ------------------------------------------------------------------------------------------------
constexpr int CTRL_WORDS = 16, CTRL_LABEL_FLAG = 5, CTRL_SWEEP = 8, CTRL_TAU = 9, CTRL_SWITCH = 10;
// One CTA of 256 threads; the order of the surviving samples is kept (stable compaction), single-term samples first.
__global__ void __launch_bounds__(256)
jacobi_finalize_kernel(float* __restrict__ maxdiff, int* __restrict__ idx, int* __restrict__ idx_tmp,
                       int* __restrict__ phase, int* __restrict__ ctrl, int* __restrict__ iters_sample) {
  __shared__ int s_cnt[2][8];
  __shared__ float s_top[8];
  __shared__ int s_flag[2][8];
  pdl_launch_dependents();
  pdl_wait();
  if (blockIdx.x != 0) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned below = (1u << lane) - 1u;
  const int n = ctrl[0];
  // the sweep number and the two thresholds live in device memory (set by jacobi_begin_kernel), so one captured
  // launch sequence serves every sweep of a block
  const int t = ctrl[CTRL_SWEEP] + 1;
  const float tau = __int_as_float(ctrl[CTRL_TAU]), switch_thresh = __int_as_float(ctrl[CTRL_SWITCH]);
  int base0 = 0, base1 = 0;  // survivors so far: single-term phase, two-term phase
  float top = 0.f;
  int bad = 0, nan = 0;
  for (int c0 = 0; c0 < n; c0 += 256) {
    const int s = c0 + threadIdx.x;
    int b = 0;
    bool f0 = false, f1 = false;
    if (s < n) {
      b = idx[s];
      const float m = maxdiff[b];
      maxdiff[b] = 0.f;
      if (m != m) nan = 1; else top = fmaxf(top, m);
      if (iters_sample) iters_sample[b] = t;
      if (!(m <= 3.0e38f)) bad = 1;
      if (tau < 0.f || !(m <= tau)) {
        int ph = phase[b];
        if (m <= switch_thresh) { phase[b] = 1; ph = 1; }
        f0 = ph == 0;
        f1 = !f0;
      }
    }
    const unsigned b0 = __ballot_sync(0xffffffffu, f0), b1 = __ballot_sync(0xffffffffu, f1);
    if (lane == 0) { s_cnt[0][warp] = __popc(b0); s_cnt[1][warp] = __popc(b1); }
    __syncthreads();  // every idx[s] of this chunk has been read before any slot of the chunk is overwritten
    int off0 = base0, off1 = base1;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      if (w < warp) { off0 += s_cnt[0][w]; off1 += s_cnt[1][w]; }
      base0 += s_cnt[0][w];
      base1 += s_cnt[1][w];
    }
    if (f0) idx[off0 + __popc(b0 & below)] = b;      // slot <= s: already read
    if (f1) idx_tmp[off1 + __popc(b1 & below)] = b;
    __syncthreads();
  }
  for (int j = threadIdx.x; j < base1; j += 256) idx[base0 + j] = idx_tmp[j];
  top = warp_max(top);
  bad = __any_sync(0xffffffffu, bad != 0);
  nan = __any_sync(0xffffffffu, nan != 0);
  if (lane == 0) { s_top[warp] = top; s_flag[0][warp] = bad; s_flag[1][warp] = nan; }
  __syncthreads();
  if (threadIdx.x == 0) {
    int anybad = ctrl[1], anynan = 0;
    for (int w = 0; w < 8; ++w) {
      top = fmaxf(top, s_top[w]);
      anybad |= s_flag[0][w];
      anynan |= s_flag[1][w];
    }
    ctrl[0] = base0 + base1;
    ctrl[1] = anybad;
    ctrl[2] = anynan ? 0x7fc00000 : __float_as_int(top);
    ctrl[3] = base1;
    ctrl[CTRL_SWEEP] = t;
  }
}

// The same sweep control for large batches (thousands of samples, the MLP-based flow): three launches instead of one
// CTA walking the list.  Stable order, identical results.
//   count:   CTA j looks at slots [1024 j, 1024 j + 1024): per-slot decision into code[] (0 = leaves, 1 = stays with
//            single-term operands, 2 = stays with two-term operands), per-CTA survivor counts, maximum and flags;
//   scan:    one CTA turns the counts into exclusive offsets and writes ctrl[];
//   scatter: CTA j writes its survivors to idx_out at offset + rank (single-term samples first, then two-term).
constexpr int FIN_CHUNK = 1024;

__global__ void __launch_bounds__(FIN_CHUNK)
jacobi_finalize_count_kernel(float* __restrict__ maxdiff, const int* __restrict__ idx, int* __restrict__ phase,
                             const int* __restrict__ ctrl, int* __restrict__ iters_sample, unsigned char* __restrict__ code,
                             int* __restrict__ blk_cnt /*[2][nblk]*/, float* __restrict__ blk_top, int* __restrict__ blk_flag,
                             int nblk) {
  const int n = ctrl[0];
  const int t = ctrl[CTRL_SWEEP] + 1;
  const float tau = __int_as_float(ctrl[CTRL_TAU]), switch_thresh = __int_as_float(ctrl[CTRL_SWITCH]);
  const int s = blockIdx.x * FIN_CHUNK + threadIdx.x;
  bool f0 = false, f1 = false;
  float top = 0.f;
  int bad = 0, nan = 0;
  if (s < n) {
    const int b = idx[s];
    const float m = maxdiff[b];
    maxdiff[b] = 0.f;
    if (m != m) nan = 1; else top = m;
    if (iters_sample) iters_sample[b] = t;
    if (!(m <= 3.0e38f)) bad = 1;
    if (tau < 0.f || !(m <= tau)) {
      int ph = phase[b];
      if (m <= switch_thresh) { phase[b] = 1; ph = 1; }
      f0 = ph == 0;
      f1 = !f0;
    }
    code[s] = f0 ? 1 : (f1 ? 2 : 0);
  }
  const int c0 = __syncthreads_count(f0), c1 = __syncthreads_count(f1);
  const int anybad = __syncthreads_or(bad), anynan = __syncthreads_or(nan);
  __shared__ float s_top[32];
  top = warp_max(top);
  if ((threadIdx.x & 31) == 0) s_top[threadIdx.x >> 5] = top;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tt = 0.f;
    for (int w = 0; w < FIN_CHUNK / 32; ++w) tt = fmaxf(tt, s_top[w]);
    blk_cnt[blockIdx.x] = c0;
    blk_cnt[nblk + blockIdx.x] = c1;
    blk_top[blockIdx.x] = tt;
    blk_flag[blockIdx.x] = (anybad ? 1 : 0) | (anynan ? 2 : 0);
  }
}

__global__ void __launch_bounds__(256)
jacobi_finalize_scan_kernel(int* __restrict__ blk_cnt, const float* __restrict__ blk_top, const int* __restrict__ blk_flag,
                            int* __restrict__ ctrl, int nblk) {
  __shared__ int s_w[2][8];
  __shared__ float s_top[8];
  __shared__ int s_flag[8];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int base0 = 0, base1 = 0, flags = 0;
  float top = 0.f;
  for (int c0 = 0; c0 < nblk; c0 += 256) {
    const int j = c0 + threadIdx.x;
    const int a = j < nblk ? blk_cnt[j] : 0, b = j < nblk ? blk_cnt[nblk + j] : 0;
    if (j < nblk) { top = fmaxf(top, blk_top[j]); flags |= blk_flag[j]; }
    int xa = a, xb = b;  // inclusive scan inside the warp
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int ya = __shfl_up_sync(0xffffffffu, xa, o), yb = __shfl_up_sync(0xffffffffu, xb, o);
      if (lane >= o) { xa += ya; xb += yb; }
    }
    if (lane == 31) { s_w[0][warp] = xa; s_w[1][warp] = xb; }
    __syncthreads();
    int wa = 0, wb = 0, ta = 0, tb = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      if (w < warp) { wa += s_w[0][w]; wb += s_w[1][w]; }
      ta += s_w[0][w];
      tb += s_w[1][w];
    }
    if (j < nblk) {
      blk_cnt[j] = base0 + wa + xa - a;         // exclusive offsets
      blk_cnt[nblk + j] = base1 + wb + xb - b;
    }
    base0 += ta;
    base1 += tb;
    __syncthreads();
  }
  top = warp_max(top);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) flags |= __shfl_xor_sync(0xffffffffu, flags, o);
  if (lane == 0) { s_top[warp] = top; s_flag[warp] = flags; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 0; w < 8; ++w) { top = fmaxf(top, s_top[w]); flags |= s_flag[w]; }
    ctrl[6] = ctrl[0];                 // slots of the sweep just finished (the scatter kernel's bound)
    ctrl[0] = base0 + base1;
    ctrl[1] = ctrl[1] | (flags & 1);
    ctrl[2] = (flags & 2) ? 0x7fc00000 : __float_as_int(top);
    ctrl[3] = base1;
    ctrl[7] = base0;                   // two-term survivors start here
    ctrl[CTRL_SWEEP] = ctrl[CTRL_SWEEP] + 1;
  }
}

__global__ void __launch_bounds__(FIN_CHUNK)
jacobi_finalize_scatter_kernel(const int* __restrict__ idx, int* __restrict__ idx_out, const unsigned char* __restrict__ code,
                               const int* __restrict__ blk_off, const int* __restrict__ ctrl, int nblk) {
  __shared__ int s_w[2][FIN_CHUNK / 32];
  const int n = ctrl[6], base1 = ctrl[7];
  const int s = blockIdx.x * FIN_CHUNK + threadIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned below = (1u << lane) - 1u;
  int b = 0, cd = 0;
  if (s < n) { b = idx[s]; cd = code[s]; }
  const unsigned b0 = __ballot_sync(0xffffffffu, cd == 1), b1 = __ballot_sync(0xffffffffu, cd == 2);
  if (lane == 0) { s_w[0][warp] = __popc(b0); s_w[1][warp] = __popc(b1); }
  __syncthreads();
  int o0 = blk_off[blockIdx.x], o1 = base1 + blk_off[nblk + blockIdx.x];
  for (int w = 0; w < warp; ++w) { o0 += s_w[0][w]; o1 += s_w[1][w]; }
  if (cd == 1) idx_out[o0 + __popc(b0 & below)] = b;
  if (cd == 2) idx_out[o1 + __popc(b1 & below)] = b;
}

__global__ void jacobi_begin_kernel(float* __restrict__ maxdiff, int* __restrict__ idx, int* __restrict__ phase,
                                    int* __restrict__ ctrl, int B, int start_phase, float tau, float switch_thresh) {
  for (int b = blockIdx.x * blockDim.x + threadIdx.x; b < B; b += gridDim.x * blockDim.x) {
    maxdiff[b] = 0.f;
    idx[b] = b;
    phase[b] = start_phase;
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    ctrl[0] = B; ctrl[1] = 0; ctrl[2] = 0; ctrl[3] = start_phase ? B : 0;
    ctrl[CTRL_SWEEP] = 0;
    ctrl[CTRL_TAU] = __float_as_int(tau);
    ctrl[CTRL_SWITCH] = __float_as_int(switch_thresh);
  }
}

// Rows of nf floats each: dst[s] = src[idx[s]] (to_compact != 0) or dst[idx[s]] = src[s] (to_compact == 0), s < n.
// Used to decode a subset of a batch (the samples still active in a Jacobi block) as a dense batch of its own.
__global__ void gather_rows_kernel(const float* __restrict__ src, float* __restrict__ dst, const int* __restrict__ idx,
                                   int n, int nf, int to_compact) {
  const size_t total = (size_t)n * nf;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int s = (int)(i / nf), k = (int)(i - (size_t)s * nf), b = idx[s];
    if (to_compact) dst[(size_t)s * nf + k] = src[(size_t)b * nf + k];
    else dst[(size_t)b * nf + k] = src[(size_t)s * nf + k];
  }
}
__global__ void gather_int_kernel(const int* __restrict__ src, int* __restrict__ dst, const int* __restrict__ idx, int n) {
  int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s < n) dst[s] = src[idx[s]];
}
// iters[idx[s]] += add for the s < n listed samples
__global__ void add_int_rows_kernel(int* __restrict__ iters, const int* __restrict__ idx, int n, int add) {
  int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s < n) iters[idx[s]] += add;
}

// out[b] = || u[b] - ref[b] ||_2 over the n values of sample b (one CTA per sample, fixed-order tree).
__global__ void __launch_bounds__(256) l2_distance_kernel(const float* __restrict__ u, const float* __restrict__ ref,
                                                          float* __restrict__ out, int n) {
  __shared__ float red[8];
  const int b = blockIdx.x;
  float acc = 0.f;
  for (int i = threadIdx.x; i < n; i += 256) {
    const float dlt = u[(size_t)b * n + i] - ref[(size_t)b * n + i];
    acc = fmaf(dlt, dlt, acc);
  }
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int i = 0; i < 8; ++i) t += red[i];
    out[b] = sqrtf(t);
  }
}

// MLP-based flow: input of the first layer, a[s, :] = T(u[idx[s], :]) (+ the second bf16 term when a_lo != null).
// Four values per thread when D % 4 == 0 (16-byte loads, 8- or 16-byte stores), else one.
template <class T>
__global__ void maf_cast_rows_kernel(const float* __restrict__ u, const int* __restrict__ idx, T* __restrict__ a,
                                     T* __restrict__ a_lo, int n_slots, int D) {
  if ((D & 3) == 0) {
    const int d4 = D >> 2;
    const size_t total = (size_t)n_slots * d4;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
      const int s = (int)(i / d4), c4 = (int)(i - (size_t)s * d4);
      const float4 x = *(reinterpret_cast<const float4*>(u + (size_t)(idx ? idx[s] : s) * D) + c4);
      const float xs[4] = {x.x, x.y, x.z, x.w};
      T hi[4], lo[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        hi[k] = from_f32<T>(xs[k]);
        lo[k] = from_f32<T>(xs[k] - to_f32(hi[k]));
      }
      T* dst = a + (size_t)s * D + 4 * c4;
      if constexpr (sizeof(T) == 2) {
        *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(hi);
        if (a_lo != nullptr) *reinterpret_cast<uint2*>(a_lo + (size_t)s * D + 4 * c4) = *reinterpret_cast<const uint2*>(lo);
      } else {
        *reinterpret_cast<float4*>(dst) = *reinterpret_cast<const float4*>(hi);
        if (a_lo != nullptr) *reinterpret_cast<float4*>(a_lo + (size_t)s * D + 4 * c4) = *reinterpret_cast<const float4*>(lo);
      }
    }
    return;
  }
  const size_t total = (size_t)n_slots * D;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int s = (int)(i / D), c = (int)(i - (size_t)s * D);
    const float x = u[(size_t)(idx ? idx[s] : s) * D + c];
    const T hi = from_f32<T>(x);
    a[i] = hi;
    if (a_lo != nullptr) a_lo[i] = from_f32<T>(x - to_f32(hi));
  }
}

// MLP-based flow, the update of Algorithm 1 from a stored output o [n_slots, 2D] (interleaved mu_i, alpha_i): one warp
// per slot, u[b, i] <- v[b, i] exp(alpha_i) + mu_i for sample b = idx[slot], maxdiff[b] = max_i |u_new - u_old| (the warp
// owns the row: plain store).  only_col >= 0: only that dimension changes (one step of sequential decoding, Eq. 5).
__global__ void __launch_bounds__(256) maf_update_kernel(const float* __restrict__ o, const float* __restrict__ v,
                                                         float* __restrict__ u, float* __restrict__ maxdiff,
                                                         const int* __restrict__ idx, int n_slots, int D, int only_col) {
  const int lane = threadIdx.x & 31;
  const int s = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (s >= n_slots) return;
  const int b = idx ? idx[s] : s;
  const float2* orow = reinterpret_cast<const float2*>(o + (size_t)s * 2 * D);
  const float* vrow = v + (size_t)b * D;
  float* urow = u + (size_t)b * D;
  float m = 0.f;
  if (only_col >= 0) {
    if (lane == 0) {
      const float2 p = orow[only_col];
      const float old = urow[only_col], nw = fmaf(vrow[only_col], expf(p.y), p.x);
      urow[only_col] = nw;
      m = fabsf(nw - old);
      maxdiff[b] = m;
    }
    return;
  }
  for (int i0 = 0; i0 < D; i0 += 128) {  // four dimensions in flight per lane
    float2 p[4];
    float vv[4], old[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = i0 + k * 32 + lane;
      if (i < D) { p[k] = orow[i]; vv[k] = vrow[i]; old[k] = urow[i]; }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = i0 + k * 32 + lane;
      if (i < D) {
        const float nw = fmaf(vv[k], expf(p[k].y), p[k].x);
        urow[i] = nw;
        const float df = fabsf(nw - old[k]);
        m = (df > m || df != df) ? df : m;
      }
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {  // NaN-propagating max
    const float other = __shfl_xor_sync(0xffffffffu, m, off);
    m = (other > m || other != other) ? other : m;
  }
  if (lane == 0) maxdiff[b] = m;
}

// MLP-based flow, forward direction (Eq. 4): v = (u - mu) exp(-alpha), logdet[b] -= sum alpha.  One CTA per sample
// (fixed-order tree: deterministic).  o: [B, 2D] interleaved (mu_i, alpha_i).
__global__ void __launch_bounds__(256) maf_forward_affine_kernel(const float* __restrict__ o, const float* __restrict__ u,
                                                                 float* __restrict__ v, float* __restrict__ logdet, int D) {
  __shared__ float red[8];
  const int b = blockIdx.x;
  float part = 0.f;
  for (int i = threadIdx.x; i < D; i += 256) {
    const float mu = o[(size_t)b * 2 * D + 2 * i], al = o[(size_t)b * 2 * D + 2 * i + 1];
    v[(size_t)b * D + i] = (u[(size_t)b * D + i] - mu) * expf(-al);
    part += al;
  }
  part = warp_sum(part);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = part;
  __syncthreads();
  if (threadIdx.x == 0 && logdet != nullptr) {
    float sum = 0.f;
    for (int i = 0; i < 8; ++i) sum += red[i];
    logdet[b] -= sum;
  }
}

// out[b] = labels[b] clamped to [0, n_classes); *flag is set when a label had to be clamped.
__global__ void labels_check_kernel(const int* __restrict__ labels, int* __restrict__ out, int B, int n_classes,
                                    int* __restrict__ flag) {
  int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  int y = labels[b];
  if (y < 0 || y >= n_classes) {
    *flag = 1;
    y = y < 0 ? 0 : n_classes - 1;
  }
  out[b] = y;
}

// One CTA per guard region (blockDim.x words): counts the words that no longer hold the fill pattern.
__global__ void guard_check_kernel(unsigned char* const* __restrict__ guards, int* __restrict__ count, unsigned pattern) {
  const unsigned w = reinterpret_cast<const unsigned*>(guards[blockIdx.x])[threadIdx.x];
  if (w != pattern) atomicAdd(count, 1);
}

__global__ void fill_int_kernel(int* p, int n, int v) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}

__global__ void f32_to_bf16_kernel(const float* __restrict__ in, bf16* __restrict__ out, size_t n) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    out[i] = __float2bfloat16_rn(in[i]);
}

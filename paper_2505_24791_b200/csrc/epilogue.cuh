// GEMM epilogue functors, with two calling conventions.
//   * apply<NC>(row, col0, v, n_valid): the thread owns NC consecutive accumulator columns of one
//     output row (col0 % NC == 0, n_valid = min(NC, N - col0)).  Used by the SIMT GEMM (NC = 4).
//   * col_const(col) / store(row, col, acc, cc, lane): the tcgen05 GEMM transposes each 32x32
//     accumulator chunk through shared memory, so that the 32 lanes of a warp hold 32 consecutive
//     columns of ONE row and every global access of a warp is a contiguous row segment.
//     col_const is evaluated once per chunk (the bias of the lane's column), store once per row.
//     All 32 lanes call store together (it may shuffle); lanes with col >= N pass col_ok = false.
//   * kRowwise functors (bf16 outputs) skip the transpose: rowwise(row, col0, v, nv, sbias) gets the 32
//     accumulator columns of the lane's own row and the chunk's bias in shared memory, and writes the
//     row segment with 16-byte stores (64 contiguous bytes per lane: whole sectors).
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace tc {  // defined in gemm_tc.cuh
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, uint32_t src);
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, int x, int y, uint32_t src);
__device__ __forceinline__ void tma_store_commit();
__device__ __forceinline__ void tma_store_wait_read();
__device__ __forceinline__ void fence_proxy_async_smem();
__device__ __forceinline__ uint32_t swz128(int r, int k);
}  // namespace tc

// Activation selector of the store epilogues: 0 = none, 1 = erf-GELU, 2 = ReLU (false / true select none / GELU).
constexpr int ACT_NONE = 0, ACT_GELU = 1, ACT_RELU = 2;

// out[row, col] = act(acc + bias[col]).  With `out_lo` set (bf16 only) the value is stored as an
// error-compensated pair: out = bf16(x), out_lo = bf16(x - out), so that out + out_lo carries about
// 16 significant bits; the next GEMM/attention consumes both terms.
template <class OutT, int ACT>
struct EpiStore {
  OutT* out;
  const float* bias;  // may be null
  int ldc;
  OutT* out_lo = nullptr;
  static constexpr bool kRowwise = sizeof(OutT) == 2;
  static constexpr bool kRowReduce = false;
  static constexpr int kRowsBatch = 8;
  static constexpr int kTmaCols = 0;
  // sbias: the 32 biases of columns col0.. (zeros without a bias), warp-private shared memory
  __device__ __forceinline__ void rowwise(int row, int col0, float (&v)[32], int nv, const float* sbias) const {
#pragma unroll
    for (int j = 0; j < 32; j += 4) {
      const float4 b = *reinterpret_cast<const float4*>(sbias + j);
      v[j] += b.x; v[j + 1] += b.y; v[j + 2] += b.z; v[j + 3] += b.w;
    }
    if (ACT == ACT_GELU) {
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = gelu_erf_fast(v[j]);
    }
    if (ACT == ACT_RELU) {
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], 0.f);
    }
    store_bf16<32>(out + (size_t)row * ldc + col0, v, nv);
    if (out_lo != nullptr) {
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] -= __bfloat162float(__float2bfloat16_rn(v[j]));
      store_bf16<32>(out_lo + (size_t)row * ldc + col0, v, nv);
    }
  }
  template <int NC>
  __device__ __forceinline__ void apply(int row, int col0, const float (&v)[NC], int nv) const {
    OutT* p = out + (size_t)row * ldc + col0;
    float r[NC];
#pragma unroll
    for (int j = 0; j < NC; ++j) {
      float x = v[j] + ((bias != nullptr && j < nv) ? bias[col0 + j] : 0.f);
      r[j] = ACT == ACT_GELU ? gelu_erf(x) : (ACT == ACT_RELU ? fmaxf(x, 0.f) : x);
    }
    if constexpr (sizeof(OutT) == 4) {
      if (nv == NC && (ldc % 4) == 0) {
#pragma unroll
        for (int j = 0; j < NC; j += 4)
          *reinterpret_cast<float4*>(reinterpret_cast<float*>(p) + j) = make_float4(r[j], r[j + 1], r[j + 2], r[j + 3]);
      } else {
#pragma unroll
        for (int j = 0; j < NC; ++j)
          if (j < nv) p[j] = from_f32<OutT>(r[j]);
      }
    } else {
      store_bf16<NC>(p, r, nv);
      if (out_lo != nullptr) {
#pragma unroll
        for (int j = 0; j < NC; ++j) r[j] -= __bfloat162float(__float2bfloat16_rn(r[j]));
        store_bf16<NC>(out_lo + (size_t)row * ldc + col0, r, nv);
      }
    }
  }
  __device__ __forceinline__ float col_const(int col, bool col_ok) const {
    return (bias != nullptr && col_ok) ? bias[col] : 0.f;
  }
  __device__ __forceinline__ void store(int row, int col, float acc, float cc, bool col_ok, int) const {
    float x = acc + cc;
    if (ACT == ACT_GELU) x = (sizeof(OutT) == 2) ? gelu_erf_fast(x) : gelu_erf(x);
    if (ACT == ACT_RELU) x = fmaxf(x, 0.f);
    if (!col_ok) return;
    const size_t e = (size_t)row * ldc + col;
    if constexpr (sizeof(OutT) == 4) {
      out[e] = from_f32<OutT>(x);
    } else {
      const bf16 hi = __float2bfloat16_rn(x);
      out[e] = hi;
      if (out_lo != nullptr) out_lo[e] = __float2bfloat16_rn(x - __bfloat162float(hi));
    }
  }
  template <int R>
  __device__ __forceinline__ void store_rows(int row0, int col, const float (&acc)[R], float cc, bool col_ok, int lane) const {
#pragma unroll
    for (int r = 0; r < R; ++r) store(row0 + r, col, acc[r], cc, col_ok, lane);
  }
  template <int NC>
  __device__ __forceinline__ void store_bf16(OutT* p, const float (&r)[NC], int nv) const {
    if (nv == NC && (ldc % 8) == 0) {
      if constexpr (NC >= 8) {
#pragma unroll
        for (int j = 0; j < NC; j += 8) {
          __nv_bfloat162 a = __floats2bfloat162_rn(r[j], r[j + 1]), b = __floats2bfloat162_rn(r[j + 2], r[j + 3]);
          __nv_bfloat162 c = __floats2bfloat162_rn(r[j + 4], r[j + 5]), d = __floats2bfloat162_rn(r[j + 6], r[j + 7]);
          uint4 u;
          u.x = *reinterpret_cast<uint32_t*>(&a); u.y = *reinterpret_cast<uint32_t*>(&b);
          u.z = *reinterpret_cast<uint32_t*>(&c); u.w = *reinterpret_cast<uint32_t*>(&d);
          *reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(p) + j) = u;
        }
      } else {
        __nv_bfloat162 a = __floats2bfloat162_rn(r[0], r[1]), b = __floats2bfloat162_rn(r[2], r[3]);
        uint2 u;
        u.x = *reinterpret_cast<uint32_t*>(&a); u.y = *reinterpret_cast<uint32_t*>(&b);
        *reinterpret_cast<uint2*>(p) = u;
      }
    } else {
#pragma unroll
      for (int j = 0; j < NC; ++j)
        if (j < nv) p[j] = from_f32<OutT>(r[j]);
    }
  }
};

struct EpiResid {  // h[row, col] += acc + bias[col]   (fp32 residual stream, in place)
  float* h;
  const float* bias;
  int ldc;
  static constexpr bool kRowwise = false;
  static constexpr bool kRowReduce = false;
  static constexpr int kRowsBatch = 8;
  static constexpr int kTmaCols = 0;
  __device__ __forceinline__ float col_const(int col, bool col_ok) const { return col_ok ? bias[col] : 0.f; }
  __device__ __forceinline__ void store(int row, int col, float acc, float cc, bool col_ok, int) const {
    if (col_ok) {
      float* p = h + (size_t)row * ldc + col;
      *p = *p + (acc + cc);
    }
  }
  // all loads of the residual stream are issued before the first store, so their latencies overlap
  template <int R>
  __device__ __forceinline__ void store_rows(int row0, int col, const float (&acc)[R], float cc, bool col_ok, int) const {
    if (!col_ok) return;
    float* p = h + (size_t)row0 * ldc + col;
    float old[R];
#pragma unroll
    for (int r = 0; r < R; ++r) old[r] = __ldcg(p + (size_t)r * ldc);
#pragma unroll
    for (int r = 0; r < R; ++r) p[(size_t)r * ldc] = old[r] + (acc[r] + cc);
  }
  template <int NC>
  __device__ __forceinline__ void apply(int row, int col0, const float (&v)[NC], int nv) const {
    float* p = h + (size_t)row * ldc + col0;
    if (nv == NC && (ldc % 4) == 0) {
#pragma unroll
      for (int j = 0; j < NC; j += 4) {
        float4 o = *reinterpret_cast<float4*>(p + j);
        float4 b = *reinterpret_cast<const float4*>(bias + col0 + j);
        o.x += v[j] + b.x; o.y += v[j + 1] + b.y; o.z += v[j + 2] + b.z; o.w += v[j + 3] + b.w;
        *reinterpret_cast<float4*>(p + j) = o;
      }
    } else {
#pragma unroll
      for (int j = 0; j < NC; ++j)
        if (j < nv) p[j] += v[j] + bias[col0 + j];
    }
  }
};

// Sequential decoding step: the QKV projection of the one new token per sample.  Column ranges
// [0,d) -> query buffer q[b, :], [d,2d) -> key cache row t, [2d,3d) -> value cache row t.
template <class T>
struct EpiQKVCache {
  T* q;          // [B, d]
  T* kc;         // [B, L, d]  this layer's key cache
  T* vc;         // [B, L, d]
  const float* bias;
  int d, L, t;
  template <int NC>
  __device__ __forceinline__ void apply(int row, int col0, const float (&v)[NC], int nv) const {
#pragma unroll
    for (int j = 0; j < NC; ++j) {
      if (j >= nv) break;
      int col = col0 + j;
      T val = from_f32<T>(v[j] + bias[col]);
      if (col < d) q[(size_t)row * d + col] = val;
      else if (col < 2 * d) kc[((size_t)row * L + t) * d + (col - d)] = val;
      else vc[((size_t)row * L + t) * d + (col - 2 * d)] = val;
    }
  }
};

// The fused step of Algorithm 1 in the head projection's epilogue.  The head matrix is stored with
// interleaved rows, so accumulator columns (2c, 2c+1) are (mu~_c, alpha~_c) of output row (slot s,
// core position l).  That row updates token l+1 of sample b = idx[s]:
//     u[b, l+1, c] <- v[b, l+1, c] * exp(alpha~) + mu~          (Eq. 5 / Alg. 1 inner line)
// and the row of the last position, whose head output is unused, performs u[b, 0, :] <- v[b, 0, :]
// (Alg. 1: the first sub-variable is copied).  u is updated in place (every element is read and
// written by exactly one thread of this launch); per-sample max |u_new - u_old| is accumulated
// into maxdiff[b] with an order-independent integer atomic max.
struct EpiHeadUpdate {
  const float* v;      // [B, L, D] block input, raster order
  float* u;            // [B, L, D] iterate, raster order, updated in place
  float* maxdiff;      // [B]
  const int* idx;      // [n_slots] slot -> sample (null = identity)
  const float* bias;   // [2D] interleaved
  int L, D, reversed;
  static constexpr bool kRowwise = false;
  static constexpr bool kRowReduce = false;
  static constexpr int kRowsBatch = 8;
  static constexpr int kTmaCols = 0;
  __device__ __forceinline__ float col_const(int col, bool col_ok) const { return col_ok ? bias[col] : 0.f; }
  // lane-per-column form: even lanes hold mu~_c, the next lane alpha~_c
  __device__ __forceinline__ void store(int row, int col, float acc, float cc, bool col_ok, int lane) const {
    const float mine = acc + cc;
    const float al = __shfl_down_sync(0xffffffffu, mine, 1);
    const int s = row / L, l = row - s * L;
    const int b = idx ? idx[s] : s;
    float df = 0.f;
    if (col_ok && (lane & 1) == 0) {
      const int c = col >> 1;
      const bool upd = l < L - 1;  // the last position's head output is unused: that row copies token 0
      const size_t e = ((size_t)b * L + tok_index(upd ? l + 1 : 0, L, reversed)) * D + c;
      const float old = u[e], vv = v[e];
      const float nw = upd ? fmaf(vv, expf(al), mine) : vv;
      u[e] = nw;
      df = fabsf(nw - old);
    }
    // NaN-propagating max over the warp, then one atomic per row
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float other = __shfl_xor_sync(0xffffffffu, df, o);
      df = (other > df || other != other) ? other : df;
    }
    if (lane == 0) atomic_max_nonneg(maxdiff + b, df);
  }
  // R consecutive rows at once: all loads of the old iterate and of v are issued before the first store (the rows
  // of a batch touch distinct tokens), so a warp pays one memory round trip per batch instead of one per row;
  // rows of the same sample share one reduction and one atomic.
  template <int R>
  __device__ __forceinline__ void store_rows(int row0, int col, const float (&acc)[R], float cc, bool col_ok, int lane) const {
    const bool active = col_ok && (lane & 1) == 0;
    const int c = col >> 1;
    float mine[R], al[R], old[R], vv[R], df[R];
    size_t e[R];
    int bs[R], ss[R];
    bool upd[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      mine[r] = acc[r] + cc;
      al[r] = __shfl_down_sync(0xffffffffu, mine[r], 1);
      const int row = row0 + r;
      const int s = row / L, l = row - s * L;
      ss[r] = s;
      bs[r] = idx ? idx[s] : s;
      upd[r] = l < L - 1;  // the last position's head output is unused: that row copies token 0
      e[r] = ((size_t)bs[r] * L + tok_index(upd[r] ? l + 1 : 0, L, reversed)) * D + c;
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      old[r] = 0.f;
      vv[r] = 0.f;
      if (active) {
        old[r] = u[e[r]];
        vv[r] = v[e[r]];
      }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      df[r] = 0.f;
      if (active) {
        const float nw = upd[r] ? fmaf(vv[r], expf(al[r]), mine[r]) : vv[r];
        u[e[r]] = nw;
        df[r] = fabsf(nw - old[r]);
      }
    }
    // NaN-propagating max; the slot index is the same in every lane, so the branch is uniform
    if (ss[0] == ss[R - 1]) {
      float m = df[0];
#pragma unroll
      for (int r = 1; r < R; ++r) m = (df[r] > m || df[r] != df[r]) ? df[r] : m;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float other = __shfl_xor_sync(0xffffffffu, m, o);
        m = (other > m || other != other) ? other : m;
      }
      if (lane == 0) atomic_max_nonneg(maxdiff + bs[0], m);
    } else {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float m = df[r];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float other = __shfl_xor_sync(0xffffffffu, m, o);
          m = (other > m || other != other) ? other : m;
        }
        if (lane == 0) atomic_max_nonneg(maxdiff + bs[r], m);
      }
    }
  }
  template <int NC>
  __device__ __forceinline__ void apply(int row, int col0, const float (&acc)[NC], int nv) const {
    int s = row / L, l = row - s * L;
    int b = idx ? idx[s] : s;
    float m = 0.f;
    if (l < L - 1) {
      size_t base = ((size_t)b * L + tok_index(l + 1, L, reversed)) * D;
#pragma unroll
      for (int j = 0; j < NC; j += 2) {
        if (j < nv) {
          int c = (col0 + j) >> 1;
          float mu = acc[j] + bias[col0 + j], al = acc[j + 1] + bias[col0 + j + 1];
          float old = u[base + c];
          float nw = fmaf(v[base + c], expf(al), mu);
          u[base + c] = nw;
          float df = fabsf(nw - old);
          m = (df > m || df != df) ? df : m;
        }
      }
    } else {
      size_t base = ((size_t)b * L + tok_index(0, L, reversed)) * D;
#pragma unroll
      for (int j = 0; j < NC; j += 2) {
        if (j < nv) {
          int c = (col0 + j) >> 1;
          float old = u[base + c], nw = v[base + c];
          u[base + c] = nw;
          float df = fabsf(nw - old);
          m = (df > m || df != df) ? df : m;
        }
      }
    }
    atomic_max_nonneg(maxdiff + b, m);
  }
};

// The fused step of Algorithm 1 for the MLP-based flow (App. E.3): one output row holds (mu_i, alpha_i), i < D, of
// one sample (columns interleaved, already in the sample's own dimension order), so row s updates sample b = idx[s]:
//     u[b, i] <- v[b, i] * exp(alpha_i) + mu_i,   maxdiff[b] = max_i |u_new - u_old|.
// With only_col >= 0 only dimension only_col is updated (one step of sequential decoding, Eq. 5).
struct EpiMafUpdate {
  const float* v;      // [B, D]
  float* u;            // [B, D], updated in place
  float* maxdiff;      // [B]
  const int* idx;      // [n_slots] slot -> sample (null = identity)
  const float* bias;   // [2D] interleaved
  int D, only_col;
  static constexpr bool kRowwise = false;
  static constexpr bool kRowReduce = false;
  static constexpr int kTmaCols = 0;
  // lane = column: a warp's accesses to u and v are contiguous row segments.  All 32 rows of a chunk are handled in
  // one batch, so the warp pays one memory round trip per chunk for the old iterate and the layer input.
  static constexpr int kRowsBatch = 32;
  __device__ __forceinline__ float col_const(int col, bool col_ok) const { return col_ok ? bias[col] : 0.f; }
  __device__ __forceinline__ void store(int row, int col, float acc, float cc, bool col_ok, int lane) const {
    const float a1[1] = {acc};
    store_rows<1>(row, col, a1, cc, col_ok, lane);
  }
  template <int R>
  __device__ __forceinline__ void store_rows(int row0, int col, const float (&acc)[R], float cc, bool col_ok, int lane) const {
    const int c = col >> 1;
    if (only_col >= 0 && __all_sync(0xffffffffu, c != only_col)) return;  // this chunk does not hold the one dimension
    const bool active = col_ok && (lane & 1) == 0 && (only_col < 0 || c == only_col);
    float al[R], old[R], vv[R];
    int bs[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      al[r] = __shfl_down_sync(0xffffffffu, acc[r] + cc, 1);
      bs[r] = idx ? idx[row0 + r] : row0 + r;
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      old[r] = 0.f;
      vv[r] = 0.f;
      if (active) {
        old[r] = u[(size_t)bs[r] * D + c];
        vv[r] = v[(size_t)bs[r] * D + c];
      }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float df = 0.f;
      if (active) {
        const float nw = fmaf(vv[r], expf(al[r]), acc[r] + cc);
        u[(size_t)bs[r] * D + c] = nw;
        df = fabsf(nw - old[r]);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {  // NaN-propagating max over the row segment
        const float other = __shfl_xor_sync(0xffffffffu, df, o);
        df = (other > df || other != other) ? other : df;
      }
      if (lane == 0 && df != 0.f) atomic_max_nonneg(maxdiff + bs[r], df);  // maxdiff starts at 0: a zero adds nothing
    }
  }
  template <int NC>
  __device__ __forceinline__ void apply(int row, int col0, const float (&acc)[NC], int nv) const {
    const int b = idx ? idx[row] : row;
    float m = 0.f;
#pragma unroll
    for (int j = 0; j < NC; j += 2) {
      if (j < nv) {
        const int c = (col0 + j) >> 1;
        if (only_col < 0 || c == only_col) {
          const float mu = acc[j] + bias[col0 + j], al = acc[j + 1] + bias[col0 + j + 1];
          const size_t e = (size_t)b * D + c;
          const float old = u[e];
          const float nw = fmaf(v[e], expf(al), mu);
          u[e] = nw;
          const float df = fabsf(nw - old);
          m = (df > m || df != df) ? df : m;
        }
      }
    }
    if (m != 0.f) atomic_max_nonneg(maxdiff + b, m);
  }
};

// ---- bulk-store forms for the tcgen05 GEMM (kTmaCols > 0): tma_box<CPG>(first chunk, last chunk, biases of the box's
// columns in shared memory, first column, first row, staging box, its shared address, lane).  The lane owns row
// `row0 + lane`; it writes its 128 bytes of the box as eight 16-byte pieces in the swizzled order of the tensor map.

// bf16 activations: out[row, col..col+63] = bf16(act(acc + bias)), optionally with the second (error) term.
template <int ACT>
struct EpiStoreTma {
  const float* bias;  // may be null
  const CUtensorMap* tmap;
  const CUtensorMap* tmap_lo;  // null = single term
  static constexpr bool kRowwise = false;
  static constexpr bool kRowReduce = false;
  static constexpr int kTmaCols = 64;
  __device__ __forceinline__ float col_const(int col, bool col_ok) const { return (bias != nullptr && col_ok) ? bias[col] : 0.f; }
  template <int CPG>
  __device__ __forceinline__ void tma_box(float (&v0)[32], float (&v1)[32], const float* sbias, int col0, int row0, uint8_t* box,
                                          uint32_t box_addr, int lane) const {
    static_assert(CPG == 2, "a bf16 box is two 32-column chunks");
#pragma unroll
    for (int j = 0; j < 32; j += 4) {  // bias (+ GELU) two values per instruction
      const float4 b0 = *reinterpret_cast<const float4*>(sbias + j), b1 = *reinterpret_cast<const float4*>(sbias + 32 + j);
      float2 a0 = fadd2(make_float2(v0[j], v0[j + 1]), make_float2(b0.x, b0.y));
      float2 a1 = fadd2(make_float2(v0[j + 2], v0[j + 3]), make_float2(b0.z, b0.w));
      float2 c0 = fadd2(make_float2(v1[j], v1[j + 1]), make_float2(b1.x, b1.y));
      float2 c1 = fadd2(make_float2(v1[j + 2], v1[j + 3]), make_float2(b1.z, b1.w));
      if (ACT == ACT_GELU) {
        a0 = gelu_erf_fast2(a0); a1 = gelu_erf_fast2(a1);
        c0 = gelu_erf_fast2(c0); c1 = gelu_erf_fast2(c1);
      }
      if (ACT == ACT_RELU) {
        a0.x = fmaxf(a0.x, 0.f); a0.y = fmaxf(a0.y, 0.f); a1.x = fmaxf(a1.x, 0.f); a1.y = fmaxf(a1.y, 0.f);
        c0.x = fmaxf(c0.x, 0.f); c0.y = fmaxf(c0.y, 0.f); c1.x = fmaxf(c1.x, 0.f); c1.y = fmaxf(c1.y, 0.f);
      }
      v0[j] = a0.x; v0[j + 1] = a0.y; v0[j + 2] = a1.x; v0[j + 3] = a1.y;
      v1[j] = c0.x; v1[j + 1] = c0.y; v1[j + 2] = c1.x; v1[j + 3] = c1.y;
    }
    // the engine reads the warp's previous box while the values above are computed; only now must it be done
    if (lane == 0) tc::tma_store_wait_read();
    __syncwarp();
    write_box(v0, v1, box, lane);
    tc::fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) { tc::tma_store_2d(tmap, col0, row0, box_addr); tc::tma_store_commit(); }
    if (tmap_lo != nullptr) {
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        v0[j] -= __bfloat162float(__float2bfloat16_rn(v0[j]));
        v1[j] -= __bfloat162float(__float2bfloat16_rn(v1[j]));
      }
      if (lane == 0) tc::tma_store_wait_read();  // the engine has read the first box
      __syncwarp();
      write_box(v0, v1, box, lane);
      tc::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) { tc::tma_store_2d(tmap_lo, col0, row0, box_addr); tc::tma_store_commit(); }
    }
  }
  __device__ __forceinline__ void write_box(const float (&v0)[32], const float (&v1)[32], uint8_t* box, int lane) const {
#pragma unroll
    for (int k = 0; k < 8; ++k) {  // 16-byte piece k = columns 8k .. 8k+7 of the box
      const float* src = k < 4 ? &v0[8 * k] : &v1[8 * (k - 4)];
      const __nv_bfloat162 a = __floats2bfloat162_rn(src[0], src[1]), b = __floats2bfloat162_rn(src[2], src[3]);
      const __nv_bfloat162 c = __floats2bfloat162_rn(src[4], src[5]), d = __floats2bfloat162_rn(src[6], src[7]);
      uint4 u;
      u.x = *reinterpret_cast<const uint32_t*>(&a); u.y = *reinterpret_cast<const uint32_t*>(&b);
      u.z = *reinterpret_cast<const uint32_t*>(&c); u.w = *reinterpret_cast<const uint32_t*>(&d);
      *reinterpret_cast<uint4*>(box + tc::swz128(lane, k)) = u;
    }
  }
};

// fp32 residual stream: h[row, col..col+31] += acc + bias, added in memory by the TMA engine (no read by the SM).
struct EpiResidTma {
  const float* bias;
  const CUtensorMap* tmap;  // fp32 [rows, d], box 32 columns x 32 rows, 128-byte swizzle
  static constexpr bool kRowwise = false;
  static constexpr bool kRowReduce = false;
  static constexpr int kTmaCols = 32;
  __device__ __forceinline__ float col_const(int col, bool col_ok) const { return col_ok ? bias[col] : 0.f; }
  template <int CPG>
  __device__ __forceinline__ void tma_box(float (&v)[32], float (&)[32], const float* sbias, int col0, int row0, uint8_t* box,
                                          uint32_t box_addr, int lane) const {
    static_assert(CPG == 1, "an fp32 box is one 32-column chunk");
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float4 b = *reinterpret_cast<const float4*>(sbias + 4 * k);
      v[4 * k] += b.x; v[4 * k + 1] += b.y; v[4 * k + 2] += b.z; v[4 * k + 3] += b.w;
    }
    if (lane == 0) tc::tma_store_wait_read();  // the engine has read the warp's previous box
    __syncwarp();
#pragma unroll
    for (int k = 0; k < 8; ++k)
      *reinterpret_cast<float4*>(box + tc::swz128(lane, k)) = make_float4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
    tc::fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) { tc::tma_reduce_add_2d(tmap, col0, row0, box_addr); tc::tma_store_commit(); }
  }
};

// fp32 output through the TMA engine: out[row, col..col+31] = acc + bias (box 32 columns x 32 rows, 128-byte swizzle).
struct EpiStoreF32Tma {
  const float* bias;
  const CUtensorMap* tmap;
  static constexpr bool kRowwise = false;
  static constexpr bool kRowReduce = false;
  static constexpr int kTmaCols = 32;
  __device__ __forceinline__ float col_const(int col, bool col_ok) const { return (bias != nullptr && col_ok) ? bias[col] : 0.f; }
  template <int CPG>
  __device__ __forceinline__ void tma_box(float (&v)[32], float (&)[32], const float* sbias, int col0, int row0, uint8_t* box,
                                          uint32_t box_addr, int lane) const {
    static_assert(CPG == 1, "an fp32 box is one 32-column chunk");
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float4 b = *reinterpret_cast<const float4*>(sbias + 4 * k);
      v[4 * k] += b.x; v[4 * k + 1] += b.y; v[4 * k + 2] += b.z; v[4 * k + 3] += b.w;
    }
    if (lane == 0) tc::tma_store_wait_read();  // the engine has read the warp's previous box
    __syncwarp();
#pragma unroll
    for (int k = 0; k < 8; ++k)
      *reinterpret_cast<float4*>(box + tc::swz128(lane, k)) = make_float4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
    tc::fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) { tc::tma_store_2d(tmap, col0, row0, box_addr); tc::tma_store_commit(); }
  }
};

// Sequential decoding with a key/value cache on the bf16 engine (Eq. 5; the sequential baseline and
// block 0 of the selective policy, Sec. 3.5).  One decoding step pushes ONE token per sample through
// the block's transformer, so every projection is a skinny GEMM  out[B, N] = A[B, K] W[N, K]^T  with
// B <= a few hundred rows: the cost is streaming W (from L2 or HBM) and the latency of a chain of
// small dependent kernels, not FLOPs.  Every projection is split along N and K over the grid and writes
// fp32 partial tiles; the (cheap, per-sample) consumer that follows sums them in a fixed order, so the
// result does not depend on scheduling.  The chain per layer is
//   resid_ln -> gemm(QKV) -> attention (sums q, k, v; appends the cache) -> gemm(out)
//   resid_ln -> gemm(MLP up) -> bias_gelu -> gemm(MLP down)
// and per step  ... -> resid_ln -> gemm(head) -> update_embed,  where
//   seq_gemm_kernel      one CTA per (64 output columns, 256-wide slice of K): it multiplies a [64, klen]
//                        activation slice with a [klen, 64] weight slice, so it reads as many activation
//                        bytes as weight bytes.  The activation slice is staged in shared memory with
//                        asynchronous copies; each warp streams its 8 rows of W straight from global
//                        memory into registers with 16-byte loads (nothing of W is shared between warps,
//                        so it never touches shared memory) and multiplies with mma.sync m16n8k16;
//   seq_resid_ln_kernel  h += sum of partial tiles + bias, then the LayerNorm of the next projection's
//                        input, written as bf16;
//   seq_attention_kernel one CTA per (sample, head): sums the partial q, k, v of the new token, appends k, v
//                        to the cache and attends over cache rows 0..t;
//   seq_bias_gelu_kernel GELU(sum of partial tiles + bias) as bf16;
//   seq_update_embed_kernel  affine update of token t+1 (Eq. 5) from the head's partial tiles and its
//                        embedding for the next step.
// Consecutive kernels are chained with programmatic dependent launch, and the step index is read from
// device memory (*step_base + step_off), so one captured CUDA graph of a few steps can be replayed
// for the whole block.
#pragma once
#include "common.cuh"
#include "gemm_tc.cuh"

namespace seq {

constexpr int ROWS = 64;           // activation rows per CTA pass (4 m16 tiles)
constexpr int KC = 1024;           // largest K slice staged in shared memory
constexpr int THREADS = 256;
constexpr int WARPS = THREADS / 32;
constexpr int HD = 64;             // head_dim of the bf16 engine

// staged activation slice (row pitch klen + 8 bf16: the 16 extra bytes keep ldmatrix conflict-free)
// + one [64, 8] fp32 tile per warp for the in-CTA reduction
__host__ __device__ constexpr int gemm_smem_bytes(int klen) { return ROWS * (klen + 8) * 2 + WARPS * ROWS * 8 * 4; }

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const bf16* p) {
  uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 ld_stream16(const void* p) {  // weights: read once per step, keep out of L1
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  const uint32_t sa = (uint32_t)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sa), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

// Programmatic dependent launch (pdl_launch_dependents / pdl_wait of common.cuh): a kernel lets its successor in
// the stream start early (its CTAs are scheduled, fetch weights, and then block in pdl_wait) and itself waits for
// its predecessor's results only where it first needs them.  Every kernel of the chain calls pdl_wait before it
// ends, so "kernel k finished" always implies "kernels < k finished".

// B fragments from 16-byte weight loads.  Lane (g, t) of a warp loads W[n0 + g][k0 + 8t .. k0 + 8t + 7],
// i.e. the four lanes of a quad hold the four 16-byte chunks of one 32-wide k group of row g, as pairs
// in[0..3].  The m16n8k16 B fragment of k step s (s = 0, 1) wants, in lane t, the pairs
// (k = 16s + 2t, +1) and (k = 16s + 8 + 2t, +1): pair t of chunk 2s and pair t of chunk 2s + 1.
// A 4x4 transpose across the quad delivers out[c] = pair t of chunk c with three shuffles.
__device__ __forceinline__ uint32_t pick4(const uint32_t (&v)[4], int i) {
  return i == 0 ? v[0] : i == 1 ? v[1] : i == 2 ? v[2] : v[3];
}
__device__ __forceinline__ void quad_transpose(const uint4& w, int lane, uint32_t (&out)[4]) {
  const uint32_t in[4] = {w.x, w.y, w.z, w.w};
  const int t = lane & 3;
  uint32_t got[4];
  got[0] = pick4(in, t);  // round 0: own chunk
#pragma unroll
  for (int r = 1; r < 4; ++r)  // round r: lane t reads lane (t + r) & 3, which offers its pair (own index - r) & 3
    got[r] = __shfl_sync(0xffffffffu, pick4(in, (t - r) & 3), (lane & ~3) | ((t + r) & 3));
  // got[r] is pair t of chunk (t + r) & 3
#pragma unroll
  for (int c = 0; c < 4; ++c) out[c] = pick4(got, (c - t) & 3);
}

// ---------------------------------------------------------------------------------------------
// part[ks][B, N] = A[B, k-slice ks] * W[N, k-slice ks]^T,  A bf16 [B, K] row-major, part fp32.
//   grid = (ceil(N / NC), K / klen, ceil(B / 64)),  NC in {8, 16, 32, 64},  klen % (32 * 64 / NC) == 0.
// Warp w owns the 8-column tile (w % (NC/8)) and the part (w / (NC/8)) of the CTA's K slice.
// ---------------------------------------------------------------------------------------------
template <int NC>
__global__ void __launch_bounds__(THREADS)
seq_gemm_kernel(const bf16* __restrict__ A, const bf16* __restrict__ W, int B, int N, int K, int klen,
                float* __restrict__ part, const int* __restrict__ step_base, int step_off, int n_steps,
                int check_steps) {
  pdl_launch_dependents();
  extern __shared__ __align__(128) uint8_t smem_seq[];
  const int pitch = klen + 8;
  bf16* sA = reinterpret_cast<bf16*>(smem_seq);
  float* sRed = reinterpret_cast<float*>(smem_seq + ROWS * pitch * 2);
  constexpr int NT = NC / 8;       // 8-column tiles per CTA
  constexpr int KS = WARPS / NT;   // warps splitting the CTA's K slice
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tq = lane & 3;
  const int nt = warp % NT, ks = warp / NT;
  const int n0 = blockIdx.x * NC + nt * 8;
  const int kbase = blockIdx.y * klen;
  const int row0 = blockIdx.z * ROWS;
  const int nrows = (B - row0) < ROWS ? (B - row0) : ROWS;
  const int mtiles = (nrows + 15) >> 4;  // m16 tiles that hold real rows
  const int srows = mtiles * 16;         // rows staged in shared memory (rows past B are zero)
  const int kper = klen / KS, ngroups = kper >> 5;  // 32-wide k groups of this warp

  // weights are constants: the first batch is requested before waiting for the previous kernel
  const int wrow = (n0 + g) < N ? (n0 + g) : (N - 1);  // columns past N are computed but never stored
  const bf16* wp = W + (size_t)wrow * K + kbase + ks * kper + 8 * tq;
  uint4 wreg[8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
    if (i < ngroups) wreg[i] = ld_stream16(wp + i * 32);

  pdl_wait();  // activations and the step counter are complete from here on
  if (check_steps && *step_base + step_off >= n_steps) return;

  // stage A[row0 .. row0+63][kbase .. kbase+klen) row-major with asynchronous 16-byte copies (one L2 round
  // trip for the whole slice, no registers held); rows past B inside the last m16 tile are zero
  const int per_row = klen >> 3, total = srows * per_row;
  for (int i = threadIdx.x; i < total; i += THREADS) {
    const int r = i / per_row, k8 = (i - r * per_row) << 3;
    if (r < nrows) cp_async16(sA + r * pitch + k8, A + (size_t)(row0 + r) * K + kbase + k8);
    else *reinterpret_cast<uint4*>(sA + r * pitch + k8) = make_uint4(0u, 0u, 0u, 0u);
  }
  cp_async_wait_all();
  __syncthreads();

  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  const bf16* a_lane = sA + ((lane & 7) + ((lane >> 3) & 1) * 8) * pitch + ks * kper + (lane >> 4) * 8;
  for (int g0 = 0; g0 < ngroups; g0 += 8) {
    if (g0 > 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (g0 + i < ngroups) wreg[i] = ld_stream16(wp + (g0 + i) * 32);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (g0 + i < ngroups) {
        uint32_t bq[4];
        quad_transpose(wreg[i], lane, bq);
        // all A fragments of the group first (independent loads), then the MMAs
        uint32_t af[2][4][4];
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
          for (int mt = 0; mt < 4; ++mt)
            if (mt < mtiles) ldsm_x4(af[j][mt], a_lane + mt * 16 * pitch + (g0 + i) * 32 + 16 * j);
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
          for (int mt = 0; mt < 4; ++mt)
            if (mt < mtiles) mma_bf16(acc[mt], af[j][mt], bq[2 * j], bq[2 * j + 1]);  // mtiles is uniform across the CTA
      }
    }
  }

  float* out = part + ((size_t)blockIdx.y * B + row0) * N;
  if constexpr (KS == 1) {  // every warp holds finished columns: 8-byte stores straight from the fragments
    const int n = n0 + 2 * tq;
    if (n < N) {
#pragma unroll
      for (int mt = 0; mt < 4; ++mt) {
        const int r = mt * 16 + g;
        if (r < nrows) *reinterpret_cast<float2*>(out + (size_t)r * N + n) = make_float2(acc[mt][0], acc[mt][1]);
        if (r + 8 < nrows) *reinterpret_cast<float2*>(out + (size_t)(r + 8) * N + n) = make_float2(acc[mt][2], acc[mt][3]);
      }
    }
  } else {  // reduction over the CTA's warps in shared memory (fixed order): thread -> (row, column)
    float* my = sRed + warp * (ROWS * 8);
#pragma unroll
    for (int mt = 0; mt < 4; ++mt) {
      *reinterpret_cast<float2*>(my + (mt * 16 + g) * 8 + 2 * tq) = make_float2(acc[mt][0], acc[mt][1]);
      *reinterpret_cast<float2*>(my + (mt * 16 + g + 8) * 8 + 2 * tq) = make_float2(acc[mt][2], acc[mt][3]);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < nrows * NC; i += THREADS) {
      const int r = i / NC, c = i - r * NC;
      const int tile = c >> 3, cc = c & 7;
      float sum = 0.f;
#pragma unroll
      for (int k = 0; k < KS; ++k) sum += sRed[(k * NT + tile) * (ROWS * 8) + r * 8 + cc];
      const int n = blockIdx.x * NC + c;
      if (n < N) out[(size_t)r * N + n] = sum;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// The same partial product on the 5th-generation tensor cores (legacy mma.sync runs at a fraction of the
// tcgen05 rate on this architecture).  The roles are swapped so that the weight slice supplies the M = 128
// dimension of the instruction: D^T[128 columns n, RT batch rows] = W[n0.., k-slice] * A[row0.., k-slice]^T.
//   * TMA brings kbn (<= 4) slabs of 64 k into shared memory, weights [128 x 64] and activations [RT x 64],
//     128-byte swizzled, one mbarrier per slab; the weight loads are issued before the wait on the
//     previous kernel (weights are constants), the activation loads after it;
//   * one thread issues 4 tcgen05.mma (M=128, N=RT, K=16) per slab into RT columns of tensor memory;
//   * the four warps read their 32 TMEM lanes (lane = output column n), transpose through shared memory
//     and store part[ks][b][n] with 16-byte stores, 512 contiguous bytes per warp.
//   grid = (ceil(N / 128), (K / 64) / kbn, ceil(B / RT)), 128 threads, RT in {16, 32, 64}.
// The launch covers the B samples row_base .. row_base + B - 1 of the activation buffer the tensor map describes
// (several such launches, each on its own group of samples, may run side by side); part and gelu_out are indexed
// by the sample's position inside the group.
// When the whole reduction fits the CTA's slab buffers (K <= 64 NS, one K slice) the kernel can finish the output
// itself: bf16(GELU(sum + bias)) for the MLP hidden layer, so no partial tiles and no consumer kernel are needed.
// Every wait is bounded (see gemm_tc.cuh); a wait that expires records a code in *err and the CTA
// leaves without storing.
// ---------------------------------------------------------------------------------------------
// Fixed-order sum of the K-slice partials of 4 consecutive outputs of row b, plus their bias.
__device__ __forceinline__ float4 sum_partials4(const float* __restrict__ part, const float* __restrict__ bias, int nsplit,
                                                int B, int N, int b, int n4) {
  float4 acc = *reinterpret_cast<const float4*>(bias + 4 * n4);
  float4 p[8];
  for (int s0 = 0; s0 < nsplit; s0 += 8) {
#pragma unroll
    for (int sl = 0; sl < 8; ++sl)
      if (s0 + sl < nsplit) p[sl] = __ldcg(reinterpret_cast<const float4*>(part + ((size_t)(s0 + sl) * B + b) * N) + n4);
#pragma unroll
    for (int sl = 0; sl < 8; ++sl)
      if (s0 + sl < nsplit) { acc.x += p[sl].x; acc.y += p[sl].y; acc.z += p[sl].z; acc.w += p[sl].w; }
  }
  return acc;
}

// What the LAST K slice of a column tile to finish does with the complete sums (the CTAs of a tile take a ticket after
// their partial tile is visible; no CTA waits for another):
//   mode 1: out_bf16[row, n] = bf16(GELU(bias[n] + sum of partials))          (the MLP hidden layer)
//   mode 2: h[row, n] += bias[n] + sum of partials, and stats[tile][row] = (sum, sum of squares) of the new h over
//           the tile's 128 columns                                            (a residual projection; the statistics
//           are what the LayerNorm of the next projection's input needs)
// The sums run over the K slices in index order whoever arrives last, so results do not depend on scheduling.
struct SeqFin {
  int mode = 0;
  int* tickets = nullptr;     // [row tiles][column tiles], zero between launches (the last arriver resets its own)
  const float* bias = nullptr;
  bf16* out_bf16 = nullptr;   // mode 1: [B, N]
  float* h = nullptr;         // mode 2: [B, N]
  float2* stats = nullptr;    // mode 2: [column tiles][B]
};
// Non-null h: the activation operand is bf16(LayerNorm(h) * gamma + beta), computed by the CTA for its own K slice
// from the fp32 rows and the per-tile statistics a SeqFin mode-2 launch left, instead of a TMA load of a stored copy.
struct SeqLnA {
  const float* h = nullptr;       // [B, K]
  const float2* stats = nullptr;  // [K / 128][B]
  const float* gamma = nullptr;
  const float* beta = nullptr;
};

// NS = slab buffers (kbn <= NS).  With gelu_out != null (one K slice only: gridDim.y == 1) the CTA holds finished
// sums and writes bf16(GELU(sum + bias)) itself instead of a partial tile, which saves the consumer kernel.
template <int RT, int NS = 4>
__host__ __device__ constexpr int gemm_tc_smem_bytes() { return NS * (128 * 64 * 2 + RT * 64 * 2) + 128 + 1024; }

template <int RT, int NS = 4>
__global__ void __launch_bounds__(128)
seq_gemm_tc_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_a, int row_base, int B,
                   int N, int kbn, float* __restrict__ part, const int* __restrict__ step_base, int step_off, int n_steps,
                   int check_steps, int* err, const float* __restrict__ gelu_bias, bf16* __restrict__ gelu_out, SeqFin fin,
                   SeqLnA lna) {
  using namespace tc;
  pdl_launch_dependents();
  __shared__ float s_mean[RT], s_rstd[RT];
  __shared__ int s_last;
  constexpr int W_BYTES = 128 * 64 * 2, A_BYTES = RT * 64 * 2, STAGE = W_BYTES + A_BYTES;
  constexpr uint32_t TMEM_COLS = RT < 32 ? 32 : RT;
  extern __shared__ uint8_t smem_seq_tc[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_seq_tc) + 1023) & ~(uintptr_t)1023);
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_base + NS * STAGE;  // full[0..NS-1], done
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + NS * STAGE + 96);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * 128, ks = blockIdx.y, row0 = blockIdx.z * RT;
  const int k0 = ks * kbn * 64;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NS + 1; ++i) mbar_init(bar_base + 8u * i, 1);
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

  if (threadIdx.x == 0) {  // weight slabs: constants, requested before the previous kernel has finished
    for (int kb = 0; kb < kbn; ++kb) {
      mbar_arrive_expect_tx(bar_base + 8u * kb, lna.h != nullptr ? W_BYTES : STAGE);
      tma_load_2d(smem_base + kb * STAGE, &map_w, k0 + kb * 64, n0, bar_base + 8u * kb);
    }
  }
  pdl_wait();  // activations and the step counter are complete from here on
  const bool skip = check_steps && (*step_base + step_off >= n_steps);
  bool ok = true;
  if (lna.h != nullptr) {
    // the activation slabs: LayerNorm of this CTA's K slice of the fp32 rows, written in the 128-byte-swizzled
    // K-major layout the tensor core reads (what the TMA load of a stored copy would have produced)
    const int K = kbn * 64 * (int)gridDim.y, stat_tiles = K >> 7;
    const int nrows_a = (B - row0) < RT ? (B - row0) : RT;
    if (threadIdx.x < RT) {
      float sum = 0.f, sq = 0.f;
      if ((int)threadIdx.x < nrows_a)
        for (int tl = 0; tl < stat_tiles; ++tl) {
          const float2 st = __ldcg(lna.stats + (size_t)tl * B + row0 + threadIdx.x);
          sum += st.x;
          sq += st.y;
        }
      const float mean = sum / K;
      s_mean[threadIdx.x] = mean;
      s_rstd[threadIdx.x] = rsqrtf(fmaxf(sq / K - mean * mean, 0.f) + 1e-5f);
    }
    __syncthreads();
    const int chunks_per_row = kbn * 8;  // 16-byte chunks (8 bf16) of a row of this K slice
    for (int c = threadIdx.x; c < RT * chunks_per_row; c += 128) {
      const int r = c / chunks_per_row, q = c - r * chunks_per_row, kb = q >> 3, kk = q & 7;
      uint4 pk = make_uint4(0u, 0u, 0u, 0u);
      if (r < nrows_a) {
        const int col = k0 + kb * 64 + kk * 8;
        const float4 x0 = __ldcg(reinterpret_cast<const float4*>(lna.h + (size_t)(row0 + r) * K + col));
        const float4 x1 = __ldcg(reinterpret_cast<const float4*>(lna.h + (size_t)(row0 + r) * K + col) + 1);
        const float4 g0 = *reinterpret_cast<const float4*>(lna.gamma + col), g1 = *reinterpret_cast<const float4*>(lna.gamma + col + 4);
        const float4 b0 = *reinterpret_cast<const float4*>(lna.beta + col), b1 = *reinterpret_cast<const float4*>(lna.beta + col + 4);
        const float mean = s_mean[r], rstd = s_rstd[r];
        const __nv_bfloat162 o0 = __floats2bfloat162_rn((x0.x - mean) * rstd * g0.x + b0.x, (x0.y - mean) * rstd * g0.y + b0.y);
        const __nv_bfloat162 o1 = __floats2bfloat162_rn((x0.z - mean) * rstd * g0.z + b0.z, (x0.w - mean) * rstd * g0.w + b0.w);
        const __nv_bfloat162 o2 = __floats2bfloat162_rn((x1.x - mean) * rstd * g1.x + b1.x, (x1.y - mean) * rstd * g1.y + b1.y);
        const __nv_bfloat162 o3 = __floats2bfloat162_rn((x1.z - mean) * rstd * g1.z + b1.z, (x1.w - mean) * rstd * g1.w + b1.w);
        pk.x = *reinterpret_cast<const uint32_t*>(&o0); pk.y = *reinterpret_cast<const uint32_t*>(&o1);
        pk.z = *reinterpret_cast<const uint32_t*>(&o2); pk.w = *reinterpret_cast<const uint32_t*>(&o3);
      }
      *reinterpret_cast<uint4*>(smem + kb * STAGE + W_BYTES + swz128(r, kk)) = pk;
    }
    fence_proxy_async_smem();  // generic-proxy writes above are read by the tensor core through the async proxy
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    if (lna.h == nullptr)
      for (int kb = 0; kb < kbn; ++kb)
        tma_load_2d(smem_base + kb * STAGE + W_BYTES, &map_a, k0 + kb * 64, row_base + row0, bar_base + 8u * kb);
    constexpr uint32_t idesc = make_idesc(RT);
    for (int kb = 0; kb < kbn && ok; ++kb) {
      ok = mbar_wait(bar_base + 8u * kb, 0u, err, TFERR_WAIT_FULL);
      if (!ok) break;
      tcgen05_fence_after();
      const uint64_t wdesc = make_smem_desc(smem_base + kb * STAGE), adesc = make_smem_desc(smem_base + kb * STAGE + W_BYTES);
#pragma unroll
      for (int k = 0; k < 4; ++k) umma_f16(tmem_base, wdesc + 2u * k, adesc + 2u * k, idesc, (kb | k) != 0);
    }
    if (ok) umma_commit(bar_base + 8u * NS);
  }
  ok = mbar_wait(bar_base + 8u * NS, 0u, err, TFERR_WAIT_TMEM_FULL);
  tcgen05_fence_after();
  // TMEM (lane = output column) -> shared memory tile [RT rows][128 columns] in the operand stages, which are
  // free once the MMAs have completed -> 16-byte stores, 512 contiguous bytes per warp
  constexpr int TP = 128 + 4;  // tile pitch in floats
  float* tile = reinterpret_cast<float*>(smem);
  if (ok) {
#pragma unroll 1
    for (int c = 0; c < (RT + 31) / 32; ++c) {
      float v[32];
      tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(c * 32), v);
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (c * 32 + j < RT) tile[(c * 32 + j) * TP + warp * 32 + lane] = v[j];
    }
  }
  const bool good = __syncthreads_and(ok && !skip) != 0;  // the same for every thread of the CTA
  if (good) {
    const int nrows = (B - row0) < RT ? (B - row0) : RT;
    const int n = n0 + 4 * lane;
    float* out = part + ((size_t)ks * B + row0) * N + n;
    if (gelu_out != nullptr) {  // N % 4 == 0 here
      if (n < N) {
        const float4 bj = *reinterpret_cast<const float4*>(gelu_bias + n);
        for (int r = warp; r < nrows; r += 4) {
          const float4 x = *reinterpret_cast<const float4*>(tile + r * TP + 4 * lane);
          const __nv_bfloat162 o0 = __floats2bfloat162_rn(gelu_erf(bj.x + x.x), gelu_erf(bj.y + x.y));
          const __nv_bfloat162 o1 = __floats2bfloat162_rn(gelu_erf(bj.z + x.z), gelu_erf(bj.w + x.w));
          uint2 w2;
          w2.x = *reinterpret_cast<const uint32_t*>(&o0);
          w2.y = *reinterpret_cast<const uint32_t*>(&o1);
          *reinterpret_cast<uint2*>(gelu_out + (size_t)(row0 + r) * N + n) = w2;
        }
      }
    } else {
      for (int r = warp; r < nrows; r += 4) {
        const float4 x = *reinterpret_cast<const float4*>(tile + r * TP + 4 * lane);
        if (n + 3 < N) {
          *reinterpret_cast<float4*>(out + (size_t)r * N) = x;
        } else {
          if (n < N) out[(size_t)r * N] = x.x;
          if (n + 1 < N) out[(size_t)r * N + 1] = x.y;
          if (n + 2 < N) out[(size_t)r * N + 2] = x.z;
        }
      }
    }
  }
  if (fin.mode != 0 && good) {
    __threadfence();  // this CTA's partial tile is visible device-wide before its ticket is taken
    __syncthreads();
    if (threadIdx.x == 0) {
      int* tk = fin.tickets + blockIdx.z * gridDim.x + blockIdx.x;
      const int got = atomicAdd(tk, 1);
      s_last = got == (int)gridDim.y - 1;
      if (s_last) *tk = 0;  // nobody else touches the ticket of this tile any more: ready for the next launch
    }
    __syncthreads();
    if (s_last) {
      __threadfence();
      const int nrows = (B - row0) < RT ? (B - row0) : RT;
      const int n = n0 + 4 * lane, nsplit = (int)gridDim.y;  // N % 4 == 0 (checked by the host)
      for (int r = warp; r < nrows; r += 4) {
        float sum = 0.f, sq = 0.f;
        if (n < N) {
          float4 x = sum_partials4(part, fin.bias, nsplit, B, N, row0 + r, n >> 2);
          if (fin.mode == 1) {
            const __nv_bfloat162 o0 = __floats2bfloat162_rn(gelu_erf(x.x), gelu_erf(x.y));
            const __nv_bfloat162 o1 = __floats2bfloat162_rn(gelu_erf(x.z), gelu_erf(x.w));
            uint2 w2;
            w2.x = *reinterpret_cast<const uint32_t*>(&o0);
            w2.y = *reinterpret_cast<const uint32_t*>(&o1);
            *reinterpret_cast<uint2*>(fin.out_bf16 + (size_t)(row0 + r) * N + n) = w2;
          } else {
            float4* hp = reinterpret_cast<float4*>(fin.h + (size_t)(row0 + r) * N + n);
            const float4 old = __ldcg(hp);
            x.x += old.x; x.y += old.y; x.z += old.z; x.w += old.w;
            *hp = x;
            sum = (x.x + x.y) + (x.z + x.w);
            sq = (x.x * x.x + x.y * x.y) + (x.z * x.z + x.w * x.w);
          }
        }
        if (fin.mode == 2) {  // the warp holds the 128 columns of row r of this tile
          sum = warp_sum(sum);
          sq = warp_sum(sq);
          if (lane == 0) fin.stats[(size_t)blockIdx.x * B + row0 + r] = make_float2(sum, sq);
        }
      }
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) {
    if (*reinterpret_cast<volatile int*>(err) != 0) {  // a wait gave up: let copies and MMAs in flight drain
      unsigned long long t0 = globaltimer_ns();
      while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tcgen05_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------
// out[b, n] = bf16(GELU(bias[n] + sum of partials)) for the MLP hidden layer.  One thread per 4 outputs.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
seq_bias_gelu_kernel(const float* __restrict__ part, int nsplit, const float* __restrict__ bias, bf16* __restrict__ out,
                     int B, int N, const int* __restrict__ step_base, int step_off, int n_steps, int check_steps) {
  pdl_launch_dependents();
  pdl_wait();
  if (check_steps && *step_base + step_off >= n_steps) return;
  const int n4s = N >> 2;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B * n4s) return;
  const int b = i / n4s, n4 = i - b * n4s;
  const float4 x = sum_partials4(part, bias, nsplit, B, N, b, n4);
  const __nv_bfloat162 o0 = __floats2bfloat162_rn(gelu_erf(x.x), gelu_erf(x.y));
  const __nv_bfloat162 o1 = __floats2bfloat162_rn(gelu_erf(x.z), gelu_erf(x.w));
  uint2 w2;
  w2.x = *reinterpret_cast<const uint32_t*>(&o0);
  w2.y = *reinterpret_cast<const uint32_t*>(&o1);
  reinterpret_cast<uint2*>(out + (size_t)b * N)[n4] = w2;
}

// ---------------------------------------------------------------------------------------------
// Residual update and LayerNorm of one row per CTA (blockDim.x = d / 4, one float4 per thread):
//   h[b, :] += bias + sum_{s < nsplit} part[s][b][:]      (skipped when nsplit == 0)
//   xn[b, :] = bf16( LayerNorm(h[b, :]) * gamma + beta )   (two-pass statistics, eps 1e-5)
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(512)
seq_resid_ln_kernel(float* __restrict__ h, const float* __restrict__ part, const float* __restrict__ bias, int nsplit,
                    const float* __restrict__ gamma, const float* __restrict__ beta, bf16* __restrict__ xn, int B, int d,
                    const int* __restrict__ step_base, int step_off, int n_steps, int check_steps) {
  pdl_launch_dependents();
  __shared__ float red[2][16];
  const int b = blockIdx.x, i = threadIdx.x;  // i < d / 4
  const float4 gg = reinterpret_cast<const float4*>(gamma)[i];
  const float4 bb = reinterpret_cast<const float4*>(beta)[i];
  pdl_wait();
  if (check_steps && *step_base + step_off >= n_steps) return;
  float4 x = __ldcg(reinterpret_cast<const float4*>(h + (size_t)b * d) + i);
  if (nsplit > 0) {
    const float4 add = sum_partials4(part, bias, nsplit, B, d, b, i);
    x.x += add.x; x.y += add.y; x.z += add.z; x.w += add.w;
    reinterpret_cast<float4*>(h + (size_t)b * d)[i] = x;
  }
  const int warp = i >> 5, lane = i & 31, nwarps = (blockDim.x + 31) >> 5;
  float s = warp_sum((x.x + x.y) + (x.z + x.w));
  if (lane == 0) red[0][warp] = s;
  __syncthreads();
  float tot = 0.f;
  for (int w = 0; w < nwarps; ++w) tot += red[0][w];
  const float mean = tot / d;
  const float a0 = x.x - mean, a1 = x.y - mean, a2 = x.z - mean, a3 = x.w - mean;
  float sq = warp_sum((a0 * a0 + a1 * a1) + (a2 * a2 + a3 * a3));
  if (lane == 0) red[1][warp] = sq;
  __syncthreads();
  tot = 0.f;
  for (int w = 0; w < nwarps; ++w) tot += red[1][w];
  const float rstd = rsqrtf(tot / d + 1e-5f);
  const __nv_bfloat162 o0 = __floats2bfloat162_rn(a0 * rstd * gg.x + bb.x, a1 * rstd * gg.y + bb.y);
  const __nv_bfloat162 o1 = __floats2bfloat162_rn(a2 * rstd * gg.z + bb.z, a3 * rstd * gg.w + bb.w);
  uint2 w2;
  w2.x = *reinterpret_cast<const uint32_t*>(&o0);
  w2.y = *reinterpret_cast<const uint32_t*>(&o1);
  reinterpret_cast<uint2*>(xn + (size_t)b * d)[i] = w2;
}

// ---------------------------------------------------------------------------------------------
// Attention of the new token of one (sample, head).  The CTA first finishes that token's q, k, v (64
// channels each) from the QKV projection's partial tiles (+ bias), appends k and v to the cache
// (layout [B][heads][L][64] bf16: the rows of one (sample, head) are contiguous) and keeps q in fp32.
// Then a single query against rows 0..t: 8 lanes share a key (16 bytes = 8 channels each); the NT / 8 lane
// groups of the CTA take keys j = group (mod NT / 8), four keys per round with the K and V rows of all four in
// flight together, and keep an online softmax (running max, sum, output) per group in fp32; the groups
// are merged through shared memory at the end.  Row t itself is taken from shared memory.  out: [B, d].
// ---------------------------------------------------------------------------------------------
// NT threads per CTA = NT / 8 lane groups: 256 for few (sample, head) pairs with long caches, 128 (at most 64
// registers, eight CTAs per SM) when there are more pairs than three 256-thread CTAs per SM can hold at once, so that
// the launch is one wave instead of three.
template <int NT>
__global__ void __launch_bounds__(NT, NT == 128 ? 8 : 3)
seq_attention_kernel(const float* __restrict__ part, int nsplit, const float* __restrict__ bias, bf16* __restrict__ kc,
                     bf16* __restrict__ vc, bf16* __restrict__ out, int B, int L, int d, int heads, float scale_log2e,
                     const int* __restrict__ step_base, int step_off, int n_steps) {
  pdl_launch_dependents();
  pdl_wait();
  const int t = *step_base + step_off;
  if (t >= n_steps) return;
  constexpr int NG = NT / 8;  // lane groups
  __shared__ float s_m[NG], s_l[NG], s_o[NG][HD];
  __shared__ __align__(16) float s_q[HD];
  __shared__ __align__(16) bf16 s_k[HD], s_v[HD];
  const int head = blockIdx.x, b = blockIdx.y;
  const int nk = t + 1;
  const int sub = threadIdx.x & 7, grp = threadIdx.x >> 3;
  bf16* kb = kc + ((size_t)b * heads + head) * L * HD;
  bf16* vb = vc + ((size_t)b * heads + head) * L * HD;
  if (threadIdx.x < 48) {  // 3 x 64 channels, 4 per thread
    const int which = threadIdx.x >> 4, c4 = threadIdx.x & 15;  // 0 = q, 1 = k, 2 = v
    const float4 x = sum_partials4(part, bias, nsplit, B, 3 * d, b, (which * d + head * HD) / 4 + c4);
    if (which == 0) {
      *reinterpret_cast<float4*>(s_q + 4 * c4) = x;
    } else {
      const __nv_bfloat162 lo = __floats2bfloat162_rn(x.x, x.y), hi = __floats2bfloat162_rn(x.z, x.w);
      uint2 w2;
      w2.x = *reinterpret_cast<const uint32_t*>(&lo);
      w2.y = *reinterpret_cast<const uint32_t*>(&hi);
      *reinterpret_cast<uint2*>((which == 1 ? s_k : s_v) + 4 * c4) = w2;
      *reinterpret_cast<uint2*>((which == 1 ? kb : vb) + (size_t)t * HD + 4 * c4) = w2;
    }
  }
  __syncthreads();
  float qf[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) qf[i] = s_q[sub * 8 + i] * scale_log2e;  // scores in base-2 units: softmax via exp2
  const bf16* kr = kb + sub * 8;
  const bf16* vr = vb + sub * 8;
  float m_run = -INFINITY, l_run = 0.f, o[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) o[i] = 0.f;
  for (int j0 = 0; j0 < nk; j0 += 4 * NG) {
    uint4 kv[4], vv[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int j = j0 + u * NG + grp;
      if (j < t) {
        kv[u] = __ldcg(reinterpret_cast<const uint4*>(kr + (size_t)j * HD));
        vv[u] = __ldcg(reinterpret_cast<const uint4*>(vr + (size_t)j * HD));
      } else if (j == t) {  // the row this CTA has just produced
        kv[u] = *reinterpret_cast<const uint4*>(s_k + sub * 8);
        vv[u] = *reinterpret_cast<const uint4*>(s_v + sub * 8);
      } else {
        kv[u] = make_uint4(0u, 0u, 0u, 0u);
        vv[u] = make_uint4(0u, 0u, 0u, 0u);
      }
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
      sc[u] = (j0 + u * NG + grp) < nk ? s : -INFINITY;
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
    for (int gI = 1; gI < NG; ++gI) mx = fmaxf(mx, s_m[gI]);
    float num = 0.f, den = 0.f;
#pragma unroll 8
    for (int gI = 0; gI < NG; ++gI) {
      const float w = exp2f(s_m[gI] - mx);  // 0 for a group without keys
      num = fmaf(w, s_o[gI][threadIdx.x], num);
      den = fmaf(w, s_l[gI], den);
    }
    out[(size_t)b * d + head * HD + threadIdx.x] = __float2bfloat16_rn(num / den);
  }
}

// ---------------------------------------------------------------------------------------------
// u[b, t+1, :] = v[b, t+1, :] * exp(alpha~) + mu~ from the head projection's partial tiles [.][B, 2D]
// (+ bias; columns interleaved mu~_c, alpha~_c), then
// the embedding of that token for the next step: h[b, :] = u W_in^T + b_in + pos[t+1] (+ cls[y_b]).
// grid = (B, ceil(d / blockDim.x)): every CTA of a sample recomputes the D values of the token (cheap) and
// embeds blockDim.x channels, one per thread; the CTA with blockIdx.y == 0 stores the token.  With
// first != 0 the step is the block's start: u[b, 0, :] = v[b, 0, :] (Eq. 5, first row) and the
// embedding of token 0.  stats != null (128 threads per CTA, d % 128 == 0): also (sum, sum of squares) of the CTA's 128
// channels per sample, the statistics layer 0's projection needs to normalise the row itself.
// ---------------------------------------------------------------------------------------------
__global__ void seq_update_embed_kernel(const float* __restrict__ part, int nsplit, const float* __restrict__ bias,
                                        int B, const float* __restrict__ v, float* __restrict__ u,
                                        const int* __restrict__ labels, const float* __restrict__ w_in_t,
                                        const float* __restrict__ b_in, const float* __restrict__ pos,
                                        const float* __restrict__ cls, float* __restrict__ h, int L, int D, int d,
                                        int reversed, int first, const int* __restrict__ step_base, int step_off,
                                        int n_steps, float2* __restrict__ stats) {
  pdl_launch_dependents();
  pdl_wait();
  const int t = *step_base + step_off;
  if (!first && t >= n_steps) return;
  extern __shared__ float s_tok[];
  const int b = blockIdx.x;
  const int l_new = first ? 0 : t + 1;
  const size_t e0 = ((size_t)b * L + tok_index(l_new, L, reversed)) * D;
  for (int c = threadIdx.x; c < D; c += blockDim.x) {
    float val = v[e0 + c];
    if (!first) {
      float mu = bias[2 * c], al = bias[2 * c + 1];
      for (int sl = 0; sl < nsplit; ++sl) {
        const float2 p = __ldcg(reinterpret_cast<const float2*>(part + ((size_t)sl * B + b) * 2 * D) + c);
        mu += p.x;
        al += p.y;
      }
      val = fmaf(val, expf(al), mu);
    }
    if (blockIdx.y == 0) u[e0 + c] = val;
    s_tok[c] = val;
  }
  __syncthreads();
  if (l_new >= L - 1) return;  // the last token is never fed back
  const int j = blockIdx.y * blockDim.x + threadIdx.x;
  if (j >= d) return;
  float acc = b_in[j] + pos[(size_t)l_new * d + j];
  if (cls != nullptr) acc += cls[(size_t)labels[b] * d + j];
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;  // four independent chains over the token's values
  int c = 0;
  for (; c + 4 <= D; c += 4) {
    a0 = fmaf(s_tok[c], w_in_t[(size_t)c * d + j], a0);
    a1 = fmaf(s_tok[c + 1], w_in_t[(size_t)(c + 1) * d + j], a1);
    a2 = fmaf(s_tok[c + 2], w_in_t[(size_t)(c + 2) * d + j], a2);
    a3 = fmaf(s_tok[c + 3], w_in_t[(size_t)(c + 3) * d + j], a3);
  }
  for (; c < D; ++c) a0 = fmaf(s_tok[c], w_in_t[(size_t)c * d + j], a0);
  const float hv = acc + ((a0 + a1) + (a2 + a3));
  h[(size_t)b * d + j] = hv;
  if (stats != nullptr) {  // blockDim.x == 128 and d % 128 == 0 here: the CTA holds one 128-column tile of the row
    __shared__ float s_red[2][4];
    const float sm = warp_sum(hv), sq = warp_sum(hv * hv);
    if ((threadIdx.x & 31) == 0) { s_red[0][threadIdx.x >> 5] = sm; s_red[1][threadIdx.x >> 5] = sq; }
    __syncthreads();
    if (threadIdx.x == 0)
      stats[(size_t)blockIdx.y * B + b] = make_float2((s_red[0][0] + s_red[0][1]) + (s_red[0][2] + s_red[0][3]),
                                                      (s_red[1][0] + s_red[1][1]) + (s_red[1][2] + s_red[1][3]));
  }
}

// ---------------------------------------------------------------------------------------------
// Tail of a decoding step in one kernel, for heads small enough that one CTA per sample can stream the head
// matrix (2 D d bf16) itself.  CTA b does, for sample b and step t = *step_base + step_off:
//   x    = h[b] + bias + partial tiles of the last MLP-down projection        (as seq_resid_ln_kernel)
//   y    = bf16(LayerNorm_f(x))                                               (the head's input, rounded as xn is)
//   o[n] = y . w_out[n, :] + b_out[n],  n < 2 D                               (warp per output, fp32 accumulation)
//   u[b, t+1, c] = v[b, t+1, c] * exp(o[2c+1]) + o[2c]                         (Eq. 5)
//   h[b] = embedding of that token;  xn[b] = bf16(LayerNorm_1(h[b]))          (layer 0's input of the next step)
// With first != 0 it is the block's start instead: token 0 is copied (u = v), embedded and normalised.
// It replaces resid_ln -> head GEMM -> update_embed -> resid_ln(layer 0), i.e. three kernel boundaries per step.
// blockDim.x = 256, d % 4 == 0, d <= 1024; dynamic shared memory: (d + 2 D + D) floats.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float block_sum_256(float v, float* red /* [8] */, int warp, int lane) {
  v = warp_sum(v);
  __syncthreads();  // red free again
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];
  return tot;
}

__global__ void __launch_bounds__(256)
seq_tail_kernel(float* __restrict__ h, const float* __restrict__ part, const float* __restrict__ bias, int nsplit,
                const float* __restrict__ lnf_g, const float* __restrict__ lnf_b, const bf16* __restrict__ w_out,
                const float* __restrict__ b_out, int B, const float* __restrict__ v, float* __restrict__ u,
                const int* __restrict__ labels, const float* __restrict__ w_in_t, const float* __restrict__ b_in,
                const float* __restrict__ pos, const float* __restrict__ cls, const float* __restrict__ ln1_g,
                const float* __restrict__ ln1_b, bf16* __restrict__ xn, int L, int D, int d, int reversed, int first,
                const int* __restrict__ step_base, int step_off, int n_steps) {
  pdl_launch_dependents();
  extern __shared__ __align__(16) float s_tail[];
  float* s_y = s_tail;          // [d]  head input
  float* s_o = s_tail + d;      // [2D] head output
  float* s_tok = s_o + 2 * D;   // [D]  new token
  __shared__ float red[8];
  const int b = blockIdx.x, i = threadIdx.x, warp = i >> 5, lane = i & 31;
  const int dv = d >> 2;
  const bool act = i < dv;
  // constants first: they are requested before the previous kernel has finished
  constexpr int WPRE = 12;  // rows of W_in kept in registers
  const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
  float4 gf = zero4, bf = zero4, g1 = zero4, b1 = zero4, bi = zero4, wpre[WPRE];
  const float4* w4 = reinterpret_cast<const float4*>(w_in_t) + i;
  if (act) {
    gf = reinterpret_cast<const float4*>(lnf_g)[i];
    bf = reinterpret_cast<const float4*>(lnf_b)[i];
    g1 = reinterpret_cast<const float4*>(ln1_g)[i];
    b1 = reinterpret_cast<const float4*>(ln1_b)[i];
    bi = reinterpret_cast<const float4*>(b_in)[i];
#pragma unroll
    for (int c = 0; c < WPRE; ++c)
      if (c < D) wpre[c] = w4[(size_t)c * dv];
  }
  // this warp's head outputs are n = warp, warp + 8, ...; the first HPRE 16-byte weight pieces of its lanes too
  constexpr int HPRE = 8;
  const int chunks = (d + 255) >> 8;  // 256-wide k chunks per output
  uint4 hpre[HPRE];
  if (!first) {
#pragma unroll
    for (int q = 0; q < HPRE; ++q) {
      const int n = warp + 8 * (q / chunks), k0 = lane * 8 + 256 * (q % chunks);
      hpre[q] = make_uint4(0u, 0u, 0u, 0u);
      if (n < 2 * D && k0 < d) hpre[q] = ld_stream16(w_out + (size_t)n * d + k0);
    }
  }
  pdl_wait();
  const int t = *step_base + step_off;
  if (!first && t >= n_steps) return;
  const int l_new = first ? 0 : t + 1;
  const size_t e0 = ((size_t)b * L + tok_index(l_new, L, reversed)) * D;
  // everything that depends on the step index only
  float vtok = 0.f;
  if (i < D) vtok = v[e0 + i];
  float4 base = zero4;
  if (act && l_new < L - 1) {
    const float4 po = reinterpret_cast<const float4*>(pos)[(size_t)l_new * dv + i];
    base = make_float4(bi.x + po.x, bi.y + po.y, bi.z + po.z, bi.w + po.w);
    if (cls != nullptr) {
      const float4 cl = reinterpret_cast<const float4*>(cls)[(size_t)labels[b] * dv + i];
      base.x += cl.x; base.y += cl.y; base.z += cl.z; base.w += cl.w;
    }
  }
  if (!first) {
    // residual + final LayerNorm (two-pass statistics, eps 1e-5)
    float4 x = zero4;
    if (act) {
      x = __ldcg(reinterpret_cast<const float4*>(h + (size_t)b * d) + i);
      if (nsplit > 0) {
        const float4 add = sum_partials4(part, bias, nsplit, B, d, b, i);
        x.x += add.x; x.y += add.y; x.z += add.z; x.w += add.w;
      }
    }
    const float mean = block_sum_256((x.x + x.y) + (x.z + x.w), red, warp, lane) / d;
    const float a0 = x.x - mean, a1 = x.y - mean, a2 = x.z - mean, a3 = x.w - mean;
    const float sq = act ? (a0 * a0 + a1 * a1) + (a2 * a2 + a3 * a3) : 0.f;
    const float rstd = rsqrtf(block_sum_256(sq, red, warp, lane) / d + 1e-5f);
    if (act) {
      const __nv_bfloat162 o0 = __floats2bfloat162_rn(a0 * rstd * gf.x + bf.x, a1 * rstd * gf.y + bf.y);
      const __nv_bfloat162 o1 = __floats2bfloat162_rn(a2 * rstd * gf.z + bf.z, a3 * rstd * gf.w + bf.w);
      const float2 f0 = __bfloat1622float2(o0), f1 = __bfloat1622float2(o1);
      *reinterpret_cast<float4*>(s_y + 4 * i) = make_float4(f0.x, f0.y, f1.x, f1.y);
    }
    __syncthreads();
    // head: a lane takes 8 consecutive k per 256-wide chunk of an output row
    int q = 0;
    for (int n = warp; n < 2 * D; n += 8) {
      float acc = 0.f;
      for (int ch = 0; ch < chunks; ++ch, ++q) {
        const int k0 = lane * 8 + 256 * ch;
        if (k0 >= d) continue;
        uint4 wv;
        if (q < HPRE) {
          wv = hpre[0];
#pragma unroll
          for (int z = 1; z < HPRE; ++z)
            if (q == z) wv = hpre[z];
        } else {
          wv = ld_stream16(w_out + (size_t)n * d + k0);
        }
        const __nv_bfloat162* w2 = reinterpret_cast<const __nv_bfloat162*>(&wv);
        const float4 y0 = *reinterpret_cast<const float4*>(s_y + k0), y1 = *reinterpret_cast<const float4*>(s_y + k0 + 4);
        const float2 c0 = __bfloat1622float2(w2[0]), c1 = __bfloat1622float2(w2[1]);
        const float2 c2 = __bfloat1622float2(w2[2]), c3 = __bfloat1622float2(w2[3]);
        acc = fmaf(y0.x, c0.x, acc); acc = fmaf(y0.y, c0.y, acc); acc = fmaf(y0.z, c1.x, acc); acc = fmaf(y0.w, c1.y, acc);
        acc = fmaf(y1.x, c2.x, acc); acc = fmaf(y1.y, c2.y, acc); acc = fmaf(y1.z, c3.x, acc); acc = fmaf(y1.w, c3.y, acc);
      }
      acc = warp_sum(acc);
      if (lane == 0) s_o[n] = acc + b_out[n];
    }
    __syncthreads();
  }
  // new token (Eq. 5; the first token of a block is copied)
  for (int c = i; c < D; c += 256) {
    float val = c == i ? vtok : v[e0 + c];
    if (!first) val = fmaf(val, expf(s_o[2 * c + 1]), s_o[2 * c]);
    u[e0 + c] = val;
    s_tok[c] = val;
  }
  __syncthreads();
  if (l_new >= L - 1) return;  // the last token is never fed back
  // embedding of the token (same accumulation order as seq_update_embed_kernel) and layer 0's LayerNorm
  float4 e = zero4;
  if (act) {
    float4 q0 = zero4, q1 = zero4, q2 = zero4, q3 = zero4;  // four independent chains over the token's values
    auto add = [&](float4& acc, float tv, const float4& w) {
      acc.x = fmaf(tv, w.x, acc.x); acc.y = fmaf(tv, w.y, acc.y); acc.z = fmaf(tv, w.z, acc.z); acc.w = fmaf(tv, w.w, acc.w);
    };
    const int d4 = D & ~3;
#pragma unroll
    for (int c = 0; c < WPRE; c += 4) {
      if (c < d4) {
        add(q0, s_tok[c], wpre[c]); add(q1, s_tok[c + 1], wpre[c + 1]);
        add(q2, s_tok[c + 2], wpre[c + 2]); add(q3, s_tok[c + 3], wpre[c + 3]);
      }
    }
    for (int c = WPRE; c < d4; c += 4) {
      add(q0, s_tok[c], w4[(size_t)c * dv]); add(q1, s_tok[c + 1], w4[(size_t)(c + 1) * dv]);
      add(q2, s_tok[c + 2], w4[(size_t)(c + 2) * dv]); add(q3, s_tok[c + 3], w4[(size_t)(c + 3) * dv]);
    }
    for (int c = d4; c < D; ++c) add(q0, s_tok[c], w4[(size_t)c * dv]);
    e.x = base.x + ((q0.x + q1.x) + (q2.x + q3.x));
    e.y = base.y + ((q0.y + q1.y) + (q2.y + q3.y));
    e.z = base.z + ((q0.z + q1.z) + (q2.z + q3.z));
    e.w = base.w + ((q0.w + q1.w) + (q2.w + q3.w));
    reinterpret_cast<float4*>(h + (size_t)b * d)[i] = e;
  }
  const float mean = block_sum_256((e.x + e.y) + (e.z + e.w), red, warp, lane) / d;
  const float a0 = e.x - mean, a1 = e.y - mean, a2 = e.z - mean, a3 = e.w - mean;
  const float sq = act ? (a0 * a0 + a1 * a1) + (a2 * a2 + a3 * a3) : 0.f;
  const float rstd = rsqrtf(block_sum_256(sq, red, warp, lane) / d + 1e-5f);
  if (act) {
    const __nv_bfloat162 o0 = __floats2bfloat162_rn(a0 * rstd * g1.x + b1.x, a1 * rstd * g1.y + b1.y);
    const __nv_bfloat162 o1 = __floats2bfloat162_rn(a2 * rstd * g1.z + b1.z, a3 * rstd * g1.w + b1.w);
    uint2 w2;
    w2.x = *reinterpret_cast<const uint32_t*>(&o0);
    w2.y = *reinterpret_cast<const uint32_t*>(&o1);
    reinterpret_cast<uint2*>(xn + (size_t)b * d)[i] = w2;
  }
}

__global__ void seq_advance_kernel(int* step_base, int by) {
  pdl_wait();  // every kernel of the replayed steps has finished reading the counter
  if (threadIdx.x == 0 && blockIdx.x == 0) *step_base += by;
}

}  // namespace seq

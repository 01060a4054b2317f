// libtarflow: host side of the selective-Jacobi TarFlow engine and its C ABI (see include/tarflow.h).
//
// One tf_model owns: the weights of K flow blocks (fp32, or bf16 matrices + fp32 vectors), two
// token-sequence buffers that ping-pong between blocks, the activation workspace of one causal pass
// over up to max_batch * L rows, the per-layer key/value cache of the sequential path, and the
// sweep-control words.  All sequences stay in raster token order; the block permutation (reversal
// on odd blocks) is folded into the index arithmetic of the embedding and update kernels.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <string>
#include <tuple>
#include <vector>

#include "../../include/tarflow.h"
#include "attention_mma.cuh"
#include "attention_tc.cuh"
#include "common.cuh"
#include "epilogue.cuh"
#include "gemm_tc.cuh"
#include "gemm_tc2.cuh"
#include "kernels_simt.cuh"
#include "seq_decode.cuh"

// ------------------------------------------------------------------------------------------------
// errors
// ------------------------------------------------------------------------------------------------
static thread_local char g_err[512] = "";
static int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}
#define CU_OK(expr)                                                                       \
  do {                                                                                    \
    cudaError_t e__ = (expr);                                                             \
    if (e__ != cudaSuccess) return fail(TF_ECUDA, "%s: %s", #expr, cudaGetErrorString(e__)); \
  } while (0)
#define TF_TRY(expr)            \
  do {                          \
    int r__ = (expr);           \
    if (r__ < 0) return r__;    \
  } while (0)

// ------------------------------------------------------------------------------------------------
// TMA tensor maps (driver entry point fetched at run time; libcuda is not linked)
// ------------------------------------------------------------------------------------------------
typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static encode_tiled_fn get_encode_fn() {
  static encode_tiled_fn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<encode_tiled_fn>(p);
  }
  return fn;
}
// bf16 matrix [rows, K] row-major; box = 64 (K) x box_rows, 128-byte swizzle, zero fill outside.
static int make_map_bf16(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t K, uint32_t box_rows) {
  encode_tiled_fn fn = get_encode_fn();
  if (!fn) return fail(TF_ECUDA, "cuTensorMapEncodeTiled entry point not available");
  if ((reinterpret_cast<uintptr_t>(ptr) & 15) || (K * 2) % 16) return fail(TF_EINVAL, "TMA operand not 16-byte aligned");
  cuuint64_t dims[2] = {K, rows};
  cuuint64_t strides[1] = {K * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(TF_ECUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
  return TF_OK;
}

// Store map for the bulk-store epilogues: matrix [rows, cols] row-major of 2-byte (bf16) or 4-byte (fp32) elements,
// box = 128 bytes of a row x 32 rows, 128-byte swizzle.
static int make_map_store(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, int elem_bytes) {
  encode_tiled_fn fn = get_encode_fn();
  if (!fn) return fail(TF_ECUDA, "cuTensorMapEncodeTiled entry point not available");
  if ((reinterpret_cast<uintptr_t>(ptr) & 15) || (cols * elem_bytes) % 16) return fail(TF_EINVAL, "TMA operand not 16-byte aligned");
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * (uint64_t)elem_bytes};
  cuuint32_t box[2] = {(cuuint32_t)(128 / elem_bytes), 32};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                  const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(TF_ECUDA, "cuTensorMapEncodeTiled (store map) failed (%d)", (int)r);
  return TF_OK;
}

// bf16 tensor [slots][L][cols] seen as 3-D, box = 64 columns x box_rows positions of one slot, 128-byte swizzle:
// positions >= L read as zeros and are not written, whatever L is.
static int make_map_3d(CUtensorMap* map, const void* ptr, uint64_t slots, uint64_t L, uint64_t cols, uint32_t box_rows) {
  encode_tiled_fn fn = get_encode_fn();
  if (!fn) return fail(TF_ECUDA, "cuTensorMapEncodeTiled entry point not available");
  if ((reinterpret_cast<uintptr_t>(ptr) & 15) || (cols * 2) % 16) return fail(TF_EINVAL, "TMA operand not 16-byte aligned");
  cuuint64_t dims[3] = {cols, L, slots};
  cuuint64_t strides[2] = {cols * 2, L * cols * 2};
  cuuint32_t box[3] = {64, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(TF_ECUDA, "cuTensorMapEncodeTiled (3-D map) failed (%d)", (int)r);
  return TF_OK;
}

// ------------------------------------------------------------------------------------------------
// model
// ------------------------------------------------------------------------------------------------
enum KernelClass {
  KC_LAYOUT, KC_EMBED, KC_LN, KC_GEMM_QKV, KC_ATTN, KC_GEMM_O, KC_GEMM_MLP1, KC_GEMM_MLP2, KC_GEMM_HEAD_UPDATE,
  KC_GEMM_HEAD, KC_AFFINE, KC_CTRL, KC_SEQ_EMBED, KC_SEQ_LN, KC_SEQ_GEMM, KC_SEQ_ATTN, KC_SEQ_UPDATE, KC_SEQ_BLOCK, KC_COUNT
};
static const char* kKernelClassNames[KC_COUNT] = {
    "layout", "embed", "layernorm", "gemm_qkv", "attention", "gemm_out", "gemm_mlp_up", "gemm_mlp_down",
    "gemm_head_update", "gemm_head", "forward_affine", "sweep_control", "seq_embed", "seq_layernorm", "seq_gemm",
    "seq_attention", "seq_update", "seq_block"};

struct Matrix {       // a linear layer's weight [N, K]
  void* w = nullptr;  // float* or bf16*
  int N = 0, K = 0;
  CUtensorMap map;    // bf16 engine: box 64 x bn
  int bn = 0;
  CUtensorMap map_seq;  // bf16 engine: box 64 x 128 for the sequential-step GEMM
};
struct LayerW {
  float *ln1_g, *ln1_b, *b_qkv, *b_o, *ln2_g, *ln2_b, *b_1, *b_2;
  Matrix w_qkv, w_o, w_1, w_2;
};
struct BlockW {
  float *w_in_t, *b_in, *pos, *cls, *lnf_g, *lnf_b, *b_out;  // b_out interleaved (mu_c, alpha_c)
  Matrix w_out;                                                // rows interleaved the same way
  std::vector<LayerW> layers;
};

struct tf_model {
  tf_config cfg;
  int L, D, d, hid, hd;
  int num_sms = 148;
  std::vector<BlockW> blocks;
  std::vector<void*> allocs;
  std::vector<unsigned char*> guards;   // start of every guard region (two per allocation)
  unsigned char** guards_dev = nullptr; // the same list on the device, built by the first check
  int* guard_count = nullptr;
  int64_t device_bytes = 0;
  // workspace
  float *seq_a = nullptr, *seq_b = nullptr, *h = nullptr, *o = nullptr, *maxdiff = nullptr;
  void *xn = nullptr, *qkv = nullptr, *att = nullptr, *mlp = nullptr, *kcache = nullptr, *vcache = nullptr;
  void *xn_lo = nullptr, *qkv_lo = nullptr, *att_lo = nullptr, *mlp_lo = nullptr;  // second terms (bf16 engine)
  CUtensorMap map_xn, map_att, map_mlp, map_xn_lo, map_att_lo, map_mlp_lo;
  enum { SM_QKV, SM_QKV_LO, SM_MLP, SM_MLP_LO, SM_H, SM_ATT3, SM_ATT3_LO, SM_PART, SM_PART_HEAD, SM_COUNT };
  CUtensorMap map_qkv3, map_kv3, map_qkv3_lo, map_kv3_lo;  // qkv as [slot][position][3d] for the tensor-core attention (query / key boxes)
  bool use_tc_attention = true;   // single-operand attention on tcgen05 (TARFLOW_ATTN_TC=0: the mma.sync kernel)
  bool use_tc_attention_split = true;  // two-term attention on tcgen05 too (TARFLOW_ATTN_TC_SPLIT=0: mma.sync)
  CUtensorMap* store_maps = nullptr;  // device copy of the bulk-store maps of qkv, qkv_lo, mlp, mlp_lo, h
  CUtensorMap map_seq_a[3][3];  // sequential-step GEMM operands {xn, att, mlp} x row tile {16, 32, 64}
  bool use_pair_gemm = true;    // sweep GEMMs on 2-CTA tile pairs (false: one CTA per tile)
  bool seq_use_tc = true;       // sequential-step GEMMs on tcgen05 (false: the mma.sync kernel)
  int seq_fuse_tail = -1;       // step tail (final LN, head, update, embed, next LN) in one kernel: -1 = when the head
                                // matrix is at most 64 KB, 0 = never, 1 = always
  bool seq_fuse_gelu = false;   // MLP-up step GEMM with K <= 512 applies bias + GELU itself (no K split): one kernel
                                // less per layer, but 16 CTAs instead of 64 stream the weights; measured slower
  int *idx = nullptr, *idx_tmp = nullptr, *phase = nullptr, *ctrl = nullptr, *iters_sample = nullptr, *err = nullptr;
  // sweep control of large batches (more than FIN_CHUNK samples): per-slot decisions and per-CTA counts
  unsigned char* fin_code = nullptr;
  int *fin_cnt = nullptr, *fin_flag = nullptr;
  float* fin_top = nullptr;
  // precision policy of Jacobi blocks on the bf16 engine: 0 = escalate per sample, 1 = single bf16
  // operands only, 2 = two-term operands for every sweep
  int precision_mode = 0;
  float switch_threshold = 0.03125f;   // a sample's sweeps use two-term operands once its max|du| <= this
  float single_ok_tau = 0.015625f;     // tau at or above this never escalates
  int* ctrl_host = nullptr;  // pinned: n_active, nonfinite, device error
  // sequential decoding on the bf16 engine: step counter on the device, model-owned copy of the labels
  // (fixed address for captured graphs), one instantiated graph of `unroll` steps per (block, batch)
  int* step_ctr = nullptr;
  int* labels_own = nullptr;
  cudaStream_t cap_stream = nullptr;
  struct SeqGraph { cudaGraphExec_t exec = nullptr; int unroll = 0; int nodes = 0; };
  std::map<std::tuple<int, int, int, int>, SeqGraph> seq_graphs;  // (block g, first sample, samples, buffer set) of a chain
  enum { MAX_CHAINS = 4 };
  cudaStream_t seq_streams[MAX_CHAINS] = {nullptr};  // one stream per chain of a sequential block
  cudaEvent_t seq_fork = nullptr, seq_join[MAX_CHAINS] = {nullptr};
  int seq_chains_force = 0;  // TARFLOW_SEQ_CHAINS=1|2|4: chains per sequential block (0 = by the size of the weights)
  enum { SEQ_TICKETS = 1024 };
  int* seq_tickets = nullptr;      // [MAX_CHAINS][SEQ_TICKETS]
  float2* seq_stats = nullptr;     // [MAX_CHAINS][16 column tiles][max_batch]
  bool seq_kbn8 = true;            // TARFLOW_SEQ_KBN8=0: finishing launches never take eight k slabs per CTA
  // TARFLOW_SEQ_FIN=1: five kernels per layer instead of eight (the last K slice of a projection finishes its tile, the
  // next projection normalises its own operand slice).  Off by default: measured 55.8 / 144.7 / 416 ms per block against
  // 28.3 / 84.1 / 283 ms for the eight-kernel chain (256 tokens width 512, 256 tokens width 1024, 1024 tokens): the
  // fence + ticket + fence of the last arriver and its one-CTA reduction cost more than the kernel boundary and the
  // many-CTA consumer kernel they replace.
  bool seq_fin = false;
  int seq_attn_threads = 0;  // TARFLOW_SEQ_ATTN_THREADS=128|256: CTA size of the step attention (0 = by the number of CTAs)
  int seq_kbn_force = 0;     // TARFLOW_SEQ_KBN
  // Jacobi sweeps over few rows are replayed from graphs: one per (block, single-term slots, two-term slots, buffers)
  std::map<std::tuple<int, int, int, const void*, const void*, const void*, const void*>, SeqGraph> sweep_graphs;
  int small_m_rows = 1024;      // TARFLOW_SMALL_M_ROWS: sweeps of at most this many rows use 128 x 128 single-CTA tiles
  int split_m_rows = 4096;      // TARFLOW_SPLIT_M_ROWS: up to this many rows the residual projections on pair tiles are cut in K too
  bool small_m_split = true;    // TARFLOW_SMALL_M_SPLIT=0: the residual projections of such sweeps keep whole-K tiles
  float* sweep_part = nullptr;  // K-slice partial products of the residual projections of such sweeps [part_cap_rows, d]
  int part_cap_rows = 0;
  int part_head_npad = 0, part_head_rows = 0;  // the same buffer seen as [part_head_rows, part_head_npad] for the head's slices
  int64_t sweep_graph_rows = 4096;  // TARFLOW_SWEEP_GRAPH_ROWS: largest slots x tokens replayed from a graph (0 = never)
  int seq_variant = 0;       // 0: the block's own token buffers, 1: the compact buffers of the sequential fall-back
  size_t seq_part_row_floats = 0;  // floats of partial tiles available per sample
  bool use_graphs = true;
  int seq_check_steps = 0;    // 1 when a replayed graph can run past the last step (kernels then test the counter)
  float* seq_part = nullptr;  // fp32 partial tiles [K slices][B][N] of the projection in flight
  size_t seq_part_floats = 0;
  float *cmp_v = nullptr, *cmp_u = nullptr, *ref_seq = nullptr;  // compact token buffers (fall-back), reference state
  int* cmp_labels = nullptr;
  float* trace_l2 = nullptr;            // [n_blocks][trace_l2_sweeps][max_batch] when the trace is on
  int trace_l2_sweeps = 0;
  std::vector<int> trace_l2_count;      // sweeps recorded per block in the last call
  // second workload: MLP-based autoregressive flow (MADE networks, App. E.3).  Such a model reuses the token buffers
  // (L = D values of token dimension 1), the sweep control and the GEMM machinery; the TarFlow calls refuse it.
  bool is_maf = false;
  struct MafBlock { Matrix w1, w2, w3; float *b1 = nullptr, *b2 = nullptr, *b3 = nullptr; };
  std::vector<MafBlock> maf_blocks;
  int maf_H = 0;
  void *maf_a0 = nullptr, *maf_a0_lo = nullptr, *maf_h1 = nullptr, *maf_h1_lo = nullptr, *maf_h2 = nullptr, *maf_h2_lo = nullptr;
  CUtensorMap maf_map[3][2];               // A-operand maps of {a0, h1, h2} x {hi, lo}
  CUtensorMap* maf_store_maps = nullptr;   // device copy: bulk-store maps of h1, h1_lo, h2, h2_lo, o (fp32)
  float *io_z = nullptr, *io_x = nullptr;  // staging for the host-buffer entry point
  int* io_labels = nullptr;
  cudaStream_t stream = nullptr;
  int64_t launches = 0;
  // profiling
  bool prof_on = false;
  int prof_mode = 0;       // 1: every launch; 2: sweep kernels per launch, a sequential block as one timed unit (from its graph)
  bool prof_suspend = false;
  std::vector<cudaEvent_t> ev_pool;
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> ev_pending[KC_COUNT];
  double prof_ms[KC_COUNT] = {0};
  int64_t prof_n[KC_COUNT] = {0};
  double prof_rows[KC_COUNT] = {0};  // activation rows the timed launches of a class processed
  int64_t cur_rows = 0;              // rows of the launches being issued (set by the pass drivers)
  cudaEvent_t cur_start = nullptr;
  // convergence trace (one record per sweep of the last inverse call)
  struct TraceRec { int block, sweep, active; float maxdiff; };
  bool trace_on = false;
  std::vector<TraceRec> trace;
  std::vector<cudaEvent_t> block_ev;  // n_blocks + 1 events bracketing the blocks of the last inverse call
  bool block_ev_valid = false;

  cudaEvent_t get_event() {
    if (!ev_pool.empty()) {
      cudaEvent_t e = ev_pool.back();
      ev_pool.pop_back();
      return e;
    }
    cudaEvent_t e;
    cudaEventCreate(&e);
    return e;
  }
  void pre(int) {
    if (prof_on && !prof_suspend) {
      cur_start = get_event();
      cudaEventRecord(cur_start, stream);
    }
  }
  void post(int cls) {
    ++launches;
    if (prof_on && !prof_suspend) {
      cudaEvent_t e = get_event();
      cudaEventRecord(e, stream);
      ev_pending[cls].push_back({cur_start, e});
      prof_rows[cls] += (double)cur_rows;
    }
  }
  void prof_collect() {
    for (int c = 0; c < KC_COUNT; ++c) {
      for (auto& pr : ev_pending[c]) {
        float ms = 0.f;
        cudaEventSynchronize(pr.second);
        cudaEventElapsedTime(&ms, pr.first, pr.second);
        prof_ms[c] += ms;
        prof_n[c] += 1;
        ev_pool.push_back(pr.first);
        ev_pool.push_back(pr.second);
      }
      ev_pending[c].clear();
    }
  }
};

#define LAUNCH(m, cls, kern, grid, block, smem, ...)           \
  do {                                                         \
    (m)->pre(cls);                                             \
    kern<<<(grid), (block), (smem), (m)->stream>>>(__VA_ARGS__); \
    (m)->post(cls);                                            \
  } while (0)

// Launch with programmatic stream serialization: only for kernels that call pdl_wait() before they touch global
// memory, so their CTAs may be scheduled while the previous kernel of the stream drains.
template <class... KArgs, class... Args>
static void launch_pdl_raw(cudaStream_t stream, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, Args... args) {
  cudaLaunchConfig_t lc = {};
  lc.gridDim = grid;
  lc.blockDim = block;
  lc.dynamicSmemBytes = smem;
  lc.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = 1;
  cudaLaunchKernelEx(&lc, kern, static_cast<KArgs>(args)...);  // errors surface in check_launch()
}
#define LAUNCH_PDL(m, cls, kern, grid, block, smem, ...)                                        \
  do {                                                                                          \
    (m)->pre(cls);                                                                              \
    launch_pdl_raw((m)->stream, kern, dim3(grid), dim3(block), (size_t)(smem), __VA_ARGS__);    \
    (m)->post(cls);                                                                             \
  } while (0)

static int check_launch(const char* what) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(TF_ECUDA, "%s: %s", what, cudaGetErrorString(e));
  return TF_OK;
}

// Per-device host state (kernel attributes set, error words, symbol addresses) is indexed by device ordinal.
constexpr int kMaxDevices = 64;
static int current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}

// Every device buffer of a model sits between two guard regions of GUARD_BYTES filled with a fixed pattern.  A kernel
// that writes outside its buffer (the kind of fault a memory checker would report) damages a guard instead of a
// neighbouring buffer, and tf_debug_check_guards counts the damaged words after any call.
constexpr size_t GUARD_BYTES = 256;
constexpr unsigned char GUARD_BYTE = 0xA5;

template <class T>
static int dev_alloc(tf_model* m, T** p, size_t count) {
  size_t bytes = ((count * sizeof(T)) + 255) & ~(size_t)255;
  if (bytes == 0) bytes = 256;
  void* q = nullptr;
  cudaError_t e = cudaMalloc(&q, bytes + 2 * GUARD_BYTES);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return fail(TF_ENOMEM, "cudaMalloc(%zu bytes) failed: %s", bytes, cudaGetErrorString(e));
  }
  m->allocs.push_back(q);
  unsigned char* base = reinterpret_cast<unsigned char*>(q);
  CU_OK(cudaMemset(base, GUARD_BYTE, GUARD_BYTES));
  CU_OK(cudaMemset(base + GUARD_BYTES + bytes, GUARD_BYTE, GUARD_BYTES));
  m->guards.push_back(base);
  m->guards.push_back(base + GUARD_BYTES + bytes);
  m->device_bytes += (int64_t)(bytes + 2 * GUARD_BYTES);
  *p = reinterpret_cast<T*>(base + GUARD_BYTES);
  return TF_OK;
}

// ------------------------------------------------------------------------------------------------
// GEMM dispatch
// ------------------------------------------------------------------------------------------------
template <int BN, int STAGES, class Epi>
static int launch_gemm_tc(tf_model* m, int cls, cudaStream_t stream, const CUtensorMap& ma, const CUtensorMap* ma_lo,
                          const CUtensorMap& mw, int M, int N, int K, const Epi& epi, int* err, int num_sms,
                          int64_t* launches, int ksplit = 1, int part_rows = 0) {
  using SL = tc::SmemLayout<BN, STAGES>;
  if (ksplit < 1 || ksplit > (K + tc::BK - 1) / tc::BK || (ksplit > 1 && Epi::kTmaCols == 0))
    return fail(TF_EINVAL, "gemm_tc_kernel: bad K split %d", ksplit);
  auto kern = tc::gemm_tc_kernel<BN, STAGES, Epi>;
  static bool configured[kMaxDevices] = {false};  // per instantiation and device
  const int dev = current_device();
  if (dev < 0) return fail(TF_ECUDA, "no usable current device");
  if (!configured[dev]) {
    CU_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SL::TOTAL));
    configured[dev] = true;
  }
  int tiles = ((M + tc::BM - 1) / tc::BM) * ((N + BN - 1) / BN) * ksplit;
  int grid = tiles < num_sms ? tiles : num_sms;
  if (m) m->pre(cls);
  launch_pdl_raw(stream, kern, dim3(grid), dim3(tc::NUM_THREADS), (size_t)SL::TOTAL, ma, ma_lo ? *ma_lo : ma, mw, M, N, K,
                 ma_lo ? 1 : 0, epi, err, ksplit, part_rows);
  if (m) m->post(cls); else if (launches) ++*launches;
  return check_launch("gemm_tc_kernel");
}

// pair kernel: 256 x 256 tiles on clusters of two CTAs (N % 256 == 0, bulk-store epilogues)
template <class Epi>
static int launch_gemm_tc2(tf_model* m, int cls, const CUtensorMap& ma, const CUtensorMap* ma_lo, const CUtensorMap& mw, int M,
                           int N, int K, const Epi& epi, int ksplit = 1, int part_rows = 0) {
  if (ksplit < 1 || ksplit > (K + tc::BK - 1) / tc::BK) return fail(TF_EINVAL, "gemm_tc2_kernel: bad K split %d", ksplit);
  auto kern = tc2::gemm_tc2_kernel<Epi>;
  static bool configured[kMaxDevices] = {false};  // per instantiation and device
  const int dev = current_device();
  if (dev < 0) return fail(TF_ECUDA, "no usable current device");
  if (!configured[dev]) {
    CU_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, tc2::Smem2::TOTAL));
    configured[dev] = true;
  }
  const int tiles = ((M + 2 * tc::BM - 1) / (2 * tc::BM)) * (N / tc2::BN2) * ksplit;
  int pairs = m->num_sms / 2;
  if (tiles < pairs) pairs = tiles;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(2 * pairs);
  lc.blockDim = dim3(tc::NUM_THREADS);
  lc.dynamicSmemBytes = tc2::Smem2::TOTAL;
  lc.stream = m->stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 2;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = 2;
  m->pre(cls);
  cudaError_t e = cudaLaunchKernelEx(&lc, kern, ma, ma_lo ? *ma_lo : ma, mw, M, N, K, ma_lo ? 1 : 0, epi, m->err, ksplit, part_rows);
  m->post(cls);
  if (e != cudaSuccess) return fail(TF_ECUDA, "gemm_tc2_kernel launch failed: %s", cudaGetErrorString(e));
  return TF_OK;
}

template <class T, class Epi>
static int launch_gemm_simt(tf_model* m, int cls, const T* A, const Matrix& W, int M, const Epi& epi) {
  dim3 grid((W.N + 63) / 64, (M + 63) / 64);
  LAUNCH(m, cls, (gemm_simt_kernel<T, Epi>), grid, 256, 0, A, reinterpret_cast<const T*>(W.w), M, W.N, W.K, epi);
  return check_launch("gemm_simt_kernel");
}

// A [M, K] activations (type T) times W^T.  bf16 engine: tensor-core kernel (map_a_lo != null: A is a
// two-term pair); fp32 engine: SIMT kernel.
template <class T, class Epi>
static int gemm(tf_model* m, int cls, const T* A, const CUtensorMap* map_a, const CUtensorMap* map_a_lo,
                const Matrix& W, int M, const Epi& epi, int ksplit = 1, int part_rows = 0) {
  if constexpr (sizeof(T) == 2) {
    if constexpr (Epi::kTmaCols > 0) {
      // few rows: 128 x 128 tiles on single CTAs put four times as many SMs on the weights as 256 x 256 pair tiles,
      // and K slices (ksplit > 1: partial products, added by the consumer) fill the rest of the GPU
      if (M <= m->small_m_rows && W.N % 128 == 0)
        return launch_gemm_tc<128, 6, Epi>(m, cls, m->stream, *map_a, map_a_lo, W.map_seq, M, W.N, W.K, epi, m->err,
                                           m->num_sms, nullptr, ksplit, part_rows);
      if (m->use_pair_gemm && W.N % 256 == 0 && M >= 256)
        return launch_gemm_tc2<Epi>(m, cls, *map_a, map_a_lo, W.map_seq, M, W.N, W.K, epi, ksplit, part_rows);
    }
    if (ksplit > 1) return fail(TF_EINVAL, "no K-split kernel for this shape");
    if (W.bn == 256)
      return launch_gemm_tc<256, 4, Epi>(m, cls, m->stream, *map_a, map_a_lo, W.map, M, W.N, W.K, epi, m->err,
                                         m->num_sms, nullptr);
    return launch_gemm_tc<128, 6, Epi>(m, cls, m->stream, *map_a, map_a_lo, W.map, M, W.N, W.K, epi, m->err,
                                       m->num_sms, nullptr);
  } else {
    return launch_gemm_simt<T, Epi>(m, cls, A, W, M, epi);
  }
}

// ------------------------------------------------------------------------------------------------
// one causal pass over n_slots * L rows (a Jacobi sweep, or the forward direction)
// ------------------------------------------------------------------------------------------------
// A projection into the residual stream that was left as K-slice partial products: the LayerNorm after it adds them.
struct SplitSum {
  const float* part;
  int ksplit, part_rows;
  const float* bias;
};

template <class T>
static int layernorm(tf_model* m, int cls, const float* x, const float* g, const float* b, T* y, T* y_lo, int rows,
                     const SplitSum* ss = nullptr) {
  int d = m->d;
  if (ss != nullptr) {  // d % 128 == 0 and d <= 4096 on this path
    LAUNCH_PDL(m, cls, resid_sum_ln_kernel<T>, rows, d / 4, 0, const_cast<float*>(x), ss->part, ss->ksplit, ss->part_rows, ss->bias,
               g, b, y, y_lo, d);
    return check_launch("resid_sum_ln_kernel");
  }
  int blocks = (rows * 32 + 255) / 256;
  if (d <= 128 * 1) LAUNCH_PDL(m, cls, (layernorm_kernel<T, 1>), blocks, 256, 0, x, g, b, y, y_lo, rows, d);
  else if (d <= 128 * 4) LAUNCH_PDL(m, cls, (layernorm_kernel<T, 4>), blocks, 256, 0, x, g, b, y, y_lo, rows, d);
  else if (d <= 128 * 8) LAUNCH_PDL(m, cls, (layernorm_kernel<T, 8>), blocks, 256, 0, x, g, b, y, y_lo, rows, d);
  else LAUNCH_PDL(m, cls, (layernorm_kernel<T, 16>), blocks, 256, 0, x, g, b, y, y_lo, rows, d);
  return check_launch("layernorm_kernel");
}

enum PassMode { PASS_JACOBI, PASS_FORWARD };

// hp: every bf16 operand travels as a two-term pair (bf16 engine only).
template <class T>
static int run_pass(tf_model* m, int g, int n_slots, const float* u_src, const int* idx, const int* labels,
                    PassMode mode, const float* v, float* u_upd, bool hp) {
  const BlockW& bw = m->blocks[g];
  const int L = m->L, D = m->D, d = m->d, M = n_slots * L, rev = g & 1;
  T* xn = reinterpret_cast<T*>(m->xn);
  T* qkv = reinterpret_cast<T*>(m->qkv);
  T* att = reinterpret_cast<T*>(m->att);
  T* mlp = reinterpret_cast<T*>(m->mlp);
  T* xn_lo = hp ? reinterpret_cast<T*>(m->xn_lo) : nullptr;
  T* qkv_lo = hp ? reinterpret_cast<T*>(m->qkv_lo) : nullptr;
  T* att_lo = hp ? reinterpret_cast<T*>(m->att_lo) : nullptr;
  T* mlp_lo = hp ? reinterpret_cast<T*>(m->mlp_lo) : nullptr;
  const CUtensorMap* mxl = hp ? &m->map_xn_lo : nullptr;
  const CUtensorMap* mal = hp ? &m->map_att_lo : nullptr;
  const CUtensorMap* mml = hp ? &m->map_mlp_lo : nullptr;
  int ethreads = d < 256 ? d : 256;
  m->cur_rows = M;
  // embedding fused with the first LayerNorm when a thread can own four columns of a row
  const bool fused_embed = d % 4 == 0 && d <= 1024 && (size_t)16 * D * sizeof(float) <= 40 * 1024;
  if (fused_embed) {
    const LayerW& l0 = bw.layers[0];
    if (M <= m->small_m_rows)  // few rows: four per CTA instead of sixteen, for four times the CTAs
      LAUNCH_PDL(m, KC_EMBED, (embed_ln_rows_kernel<T, 4>), (M + 3) / 4, ((d / 4 + 31) / 32) * 32, 4 * D * sizeof(float), u_src,
                 idx, labels, bw.w_in_t, bw.b_in, bw.pos, bw.cls, m->h, l0.ln1_g, l0.ln1_b, xn, xn_lo, L, D, d, rev, M);
    else
      LAUNCH_PDL(m, KC_EMBED, (embed_ln_rows_kernel<T, 16>), (M + 15) / 16, ((d / 4 + 31) / 32) * 32, 16 * D * sizeof(float), u_src,
                 idx, labels, bw.w_in_t, bw.b_in, bw.pos, bw.cls, m->h, l0.ln1_g, l0.ln1_b, xn, xn_lo, L, D, d, rev, M);
  } else {
    LAUNCH_PDL(m, KC_EMBED, embed_rows_kernel<16>, (M + 15) / 16, ethreads, 16 * D * sizeof(float), u_src, idx, labels,
               bw.w_in_t, bw.b_in, bw.pos, bw.cls, m->h, L, D, d, rev, M);
  }
  TF_TRY(check_launch("embed_kernel"));
  // Few rows (bf16 engine): the two projections into the residual stream have d / 128 column tiles per 128 rows, too few
  // CTAs to stream their weights, so they are cut into K slices that leave partial products; the LayerNorm that follows
  // (this layer's second, the next layer's first, or the block's last) adds them to the stream in slice order.
  const int m_pad = (M + 127) / 128 * 128;
  auto slices_for = [&](int K) -> int {
    if (sizeof(T) != 2 || m->sweep_part == nullptr || !m->small_m_split || d > 4096) return 1;
    int ks;
    if (M <= m->small_m_rows) ks = m->num_sms / ((m_pad / 128) * (d / 128));  // 128 x 128 tiles
    else if (M <= m->split_m_rows && m->use_pair_gemm && d % 256 == 0 && M >= 256)
      ks = (m->num_sms / 2) / (((M + 255) / 256) * (d / 256));                // pair tiles
    else return 1;
    if (ks > K / (2 * tc::BK)) ks = K / (2 * tc::BK);  // at least two k slabs per slice
    if (ks > 8) ks = 8;
    if (ks > m->part_cap_rows / m_pad) ks = m->part_cap_rows / m_pad;
    return ks < 1 ? 1 : ks;
  };
  SplitSum pend{nullptr, 0, 0, nullptr};
  bool has_pend = false;
  bool first_layer = true;
  for (const LayerW& lw : bw.layers) {
    if (!(first_layer && fused_embed)) TF_TRY(layernorm<T>(m, KC_LN, m->h, lw.ln1_g, lw.ln1_b, xn, xn_lo, M, has_pend ? &pend : nullptr));
    has_pend = false;
    first_layer = false;
    if constexpr (sizeof(T) == 2) {
      const CUtensorMap* sm = m->store_maps;
      TF_TRY(gemm<T>(m, KC_GEMM_QKV, xn, &m->map_xn, mxl, lw.w_qkv, M,
                     EpiStoreTma<false>{lw.b_qkv, sm + tf_model::SM_QKV, hp ? sm + tf_model::SM_QKV_LO : nullptr}));
    } else {
      TF_TRY(gemm<T>(m, KC_GEMM_QKV, xn, &m->map_xn, mxl, lw.w_qkv, M, EpiStore<T, false>{qkv, lw.b_qkv, 3 * d, qkv_lo}));
    }
    if constexpr (sizeof(T) == 2) {
      dim3 grid((L + attn::BQ - 1) / attn::BQ, m->cfg.n_heads, n_slots);
      const float sl2 = 1.4426950408889634f / sqrtf((float)m->hd);
      const dim3 grid_tc((L + attn_tc::BQ - 1) / attn_tc::BQ, m->cfg.n_heads, n_slots);
      if (hp && m->use_tc_attention && m->use_tc_attention_split)
        LAUNCH_PDL(m, KC_ATTN, attn_tc::attention_tc_kernel<true>, grid_tc, attn_tc::NUM_THREADS_ATTN, attn_tc::Cfg<true>::SMEM_BYTES,
                   m->map_qkv3, m->map_kv3, m->map_qkv3_lo, m->map_kv3_lo, m->store_maps + tf_model::SM_ATT3,
                   m->store_maps + tf_model::SM_ATT3_LO, L, d, sl2, m->err);
      else if (hp)
        LAUNCH(m, KC_ATTN, attn::attention_mma_kernel<true>, grid, 128, attn::smem_bytes<true>(), qkv, qkv_lo, att,
               att_lo, L, d, sl2);
      else if (m->use_tc_attention)
        LAUNCH_PDL(m, KC_ATTN, attn_tc::attention_tc_kernel<false>, grid_tc, attn_tc::NUM_THREADS_ATTN, attn_tc::Cfg<false>::SMEM_BYTES,
                   m->map_qkv3, m->map_kv3, m->map_qkv3, m->map_kv3, m->store_maps + tf_model::SM_ATT3,
                   m->store_maps + tf_model::SM_ATT3, L, d, sl2, m->err);
      else
        LAUNCH(m, KC_ATTN, attn::attention_mma_kernel<false>, grid, 128, attn::smem_bytes<false>(), qkv, qkv_lo, att,
               att_lo, L, d, sl2);
    } else {
      const int warps = 4;
      dim3 grid((L + warps - 1) / warps, m->cfg.n_heads, n_slots);
      size_t smem = (size_t)warps * (L + m->hd) * sizeof(float);
      LAUNCH(m, KC_ATTN, (attention_simt_kernel<T>), grid, warps * 32, smem, qkv, att, L, d, m->hd,
             1.0f / sqrtf((float)m->hd));
    }
    TF_TRY(check_launch("attention kernel"));
    if constexpr (sizeof(T) == 2) {
      const int ks = slices_for(d);
      if (ks > 1) {
        TF_TRY(gemm<T>(m, KC_GEMM_O, att, &m->map_att, mal, lw.w_o, M, EpiStoreF32Tma{nullptr, m->store_maps + tf_model::SM_PART},
                       ks, m_pad));
        pend = SplitSum{m->sweep_part, ks, m_pad, lw.b_o};
        has_pend = true;
      } else {
        TF_TRY(gemm<T>(m, KC_GEMM_O, att, &m->map_att, mal, lw.w_o, M, EpiResidTma{lw.b_o, m->store_maps + tf_model::SM_H}));
      }
    } else {
      TF_TRY(gemm<T>(m, KC_GEMM_O, att, &m->map_att, mal, lw.w_o, M, EpiResid{m->h, lw.b_o, d}));
    }
    TF_TRY(layernorm<T>(m, KC_LN, m->h, lw.ln2_g, lw.ln2_b, xn, xn_lo, M, has_pend ? &pend : nullptr));
    has_pend = false;
    if constexpr (sizeof(T) == 2) {
      const CUtensorMap* sm = m->store_maps;
      TF_TRY(gemm<T>(m, KC_GEMM_MLP1, xn, &m->map_xn, mxl, lw.w_1, M,
                     EpiStoreTma<true>{lw.b_1, sm + tf_model::SM_MLP, hp ? sm + tf_model::SM_MLP_LO : nullptr}));
      const int ks = slices_for(m->hid);
      if (ks > 1) {
        TF_TRY(gemm<T>(m, KC_GEMM_MLP2, mlp, &m->map_mlp, mml, lw.w_2, M, EpiStoreF32Tma{nullptr, sm + tf_model::SM_PART}, ks, m_pad));
        pend = SplitSum{m->sweep_part, ks, m_pad, lw.b_2};
        has_pend = true;
      } else {
        TF_TRY(gemm<T>(m, KC_GEMM_MLP2, mlp, &m->map_mlp, mml, lw.w_2, M, EpiResidTma{lw.b_2, sm + tf_model::SM_H}));
      }
    } else {
      TF_TRY(gemm<T>(m, KC_GEMM_MLP1, xn, &m->map_xn, mxl, lw.w_1, M, EpiStore<T, true>{mlp, lw.b_1, m->hid, mlp_lo}));
      TF_TRY(gemm<T>(m, KC_GEMM_MLP2, mlp, &m->map_mlp, mml, lw.w_2, M, EpiResid{m->h, lw.b_2, d}));
    }
  }
  TF_TRY(layernorm<T>(m, KC_LN, m->h, bw.lnf_g, bw.lnf_b, xn, xn_lo, M, has_pend ? &pend : nullptr));
  if (mode == PASS_JACOBI) {
    // few rows: the head projection has one or two CTAs that walk K alone, so it is cut into K slices too and a small
    // kernel adds them and applies the update (otherwise the update is the projection's epilogue)
    int ks_head = 1;
    if constexpr (sizeof(T) == 2) {
      if (M <= m->small_m_rows && m->sweep_part != nullptr && m->small_m_split && bw.w_out.bn == 128 && D % 2 == 0 && d % 128 == 0) {
        ks_head = m->num_sms / ((m_pad / 128) * ((2 * D + 127) / 128));
        if (ks_head > d / (2 * tc::BK)) ks_head = d / (2 * tc::BK);
        if (ks_head > 8) ks_head = 8;
        if (ks_head > m->part_head_rows / m_pad) ks_head = m->part_head_rows / m_pad;
        if (ks_head < 1) ks_head = 1;
      }
    }
    if (ks_head > 1) {
      if constexpr (sizeof(T) == 2) {
        TF_TRY((launch_gemm_tc<128, 6, EpiStoreF32Tma>(m, KC_GEMM_HEAD_UPDATE, m->stream, m->map_xn, mxl, bw.w_out.map, M, 2 * D, d,
                                                       EpiStoreF32Tma{nullptr, m->store_maps + tf_model::SM_PART_HEAD}, m->err,
                                                       m->num_sms, nullptr, ks_head, m_pad)));
        LAUNCH_PDL(m, KC_GEMM_HEAD_UPDATE, jacobi_update_split_kernel, (M * 32 + 255) / 256, 256, 0, m->sweep_part, ks_head, m_pad,
                   m->part_head_npad, bw.b_out, v, u_upd, m->maxdiff, idx, M, L, D, rev);
        TF_TRY(check_launch("jacobi_update_split_kernel"));
      }
    } else {
      EpiHeadUpdate epi{v, u_upd, m->maxdiff, idx, bw.b_out, L, D, rev};
      TF_TRY(gemm<T>(m, KC_GEMM_HEAD_UPDATE, xn, &m->map_xn, mxl, bw.w_out, M, epi));
    }
  } else {
    TF_TRY(gemm<T>(m, KC_GEMM_HEAD, xn, &m->map_xn, mxl, bw.w_out, M, EpiStore<float, false>{m->o, bw.b_out, 2 * D}));
  }
  return TF_OK;
}

// ------------------------------------------------------------------------------------------------
// sequential block with KV cache (Eq. 5): L-1 single-token passes
// ------------------------------------------------------------------------------------------------
template <class T>
static int run_sequential_block(tf_model* m, int g, int B, const int* labels, const float* v, float* u) {
  const BlockW& bw = m->blocks[g];
  const int L = m->L, D = m->D, d = m->d, rev = g & 1, nl = m->cfg.n_layers;
  T* xn = reinterpret_cast<T*>(m->xn);
  T* q = reinterpret_cast<T*>(m->qkv);
  T* att = reinterpret_cast<T*>(m->att);
  T* mlp = reinterpret_cast<T*>(m->mlp);
  const size_t layer_stride = (size_t)m->cfg.max_batch * L * d;
  const float scale = 1.0f / sqrtf((float)m->hd);
  int ethreads = d < 256 ? d : 256;
  m->cur_rows = B;
  LAUNCH(m, KC_SEQ_UPDATE, copy_first_token_kernel, (B * D + 127) / 128, 128, 0, v, u, B, L, D, rev);
  for (int t = 0; t + 1 < L; ++t) {
    LAUNCH(m, KC_SEQ_EMBED, embed_kernel, B, ethreads, D * sizeof(float), u, (const int*)nullptr, labels, bw.w_in_t,
           bw.b_in, bw.pos, bw.cls, m->h, L, D, d, rev, t);
    for (int i = 0; i < nl; ++i) {
      const LayerW& lw = bw.layers[i];
      T* kc = reinterpret_cast<T*>(m->kcache) + i * layer_stride;
      T* vc = reinterpret_cast<T*>(m->vcache) + i * layer_stride;
      TF_TRY(layernorm<T>(m, KC_SEQ_LN, m->h, lw.ln1_g, lw.ln1_b, xn, (T*)nullptr, B));
      TF_TRY(launch_gemm_simt<T>(m, KC_SEQ_GEMM, xn, lw.w_qkv, B, EpiQKVCache<T>{q, kc, vc, lw.b_qkv, d, L, t}));
      size_t smem = (size_t)(L + m->hd + 8 + 4 * m->hd) * sizeof(float);
      LAUNCH(m, KC_SEQ_ATTN, (attention_step_kernel<T>), dim3(m->cfg.n_heads, B), 128, smem, q, kc, vc, att, L, d,
             m->hd, t, scale);
      TF_TRY(launch_gemm_simt<T>(m, KC_SEQ_GEMM, att, lw.w_o, B, EpiResid{m->h, lw.b_o, d}));
      TF_TRY(layernorm<T>(m, KC_SEQ_LN, m->h, lw.ln2_g, lw.ln2_b, xn, (T*)nullptr, B));
      TF_TRY(launch_gemm_simt<T>(m, KC_SEQ_GEMM, xn, lw.w_1, B, EpiStore<T, true>{mlp, lw.b_1, m->hid}));
      TF_TRY(launch_gemm_simt<T>(m, KC_SEQ_GEMM, mlp, lw.w_2, B, EpiResid{m->h, lw.b_2, d}));
    }
    TF_TRY(layernorm<T>(m, KC_SEQ_LN, m->h, bw.lnf_g, bw.lnf_b, xn, (T*)nullptr, B));
    TF_TRY(launch_gemm_simt<T>(m, KC_SEQ_GEMM, xn, bw.w_out, B, EpiStore<float, false>{m->o, bw.b_out, 2 * D}));
    LAUNCH(m, KC_SEQ_UPDATE, seq_update_kernel, (B * D + 127) / 128, 128, 0, m->o, v, u, B, L, D, rev, t);
  }
  return check_launch("sequential block");
}

// ---- bf16 engine: fused-LayerNorm skinny GEMMs on tensor cores, replayed from a CUDA graph -------
// Launch of a sequential-step kernel with programmatic dependent launch, so that consecutive kernels of
// the chain overlap their launch latency and weight prefetch (see seq_decode.cuh).
template <class... KArgs, class... Args>
static int launch_seq(tf_model* m, int cls, void (*kern)(KArgs...), dim3 grid, int threads, int smem, Args... args) {
  cudaLaunchConfig_t lc = {};
  lc.gridDim = grid;
  lc.blockDim = dim3(threads);
  lc.dynamicSmemBytes = smem;
  lc.stream = m->stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = 1;
  m->pre(cls);
  cudaError_t e = cudaLaunchKernelEx(&lc, kern, static_cast<KArgs>(args)...);
  m->post(cls);
  if (e != cudaSuccess) return fail(TF_ECUDA, "sequential-step kernel launch failed: %s", cudaGetErrorString(e));
  return TF_OK;
}

// A chain decodes the samples b0 .. b0 + B - 1 of a sequential block on its own stream, with its own step counter
// and its own region of the partial-tile buffer.  Samples are independent, so a block's batch may be split over a few
// chains that run side by side: every kernel of a decoding step is bound by the latency of its dependent chain, not
// by throughput, and the chains fill each other's idle time.  A sample's arithmetic does not depend on the split.
struct SeqCtx {
  int b0 = 0, B = 0;
  int* step_ctr = nullptr;
  float* part = nullptr;
  int* tickets = nullptr;    // last-arriver tickets of the step GEMMs' column tiles (zero between launches)
  float2* stats = nullptr;   // per column tile and sample: (sum, sum of squares) of the residual row, for the next LayerNorm
};

// One skinny GEMM of a decoding step: part[ks][B, N] = A[B, K slice ks] W[N, K slice ks]^T.  Returns the number of
// K slices in *nsplit; the kernel that consumes the tiles adds them up.  CTAs of 64 columns x 256 of K read as many
// activation bytes as weight bytes and give a grid of (N / 64) * (K / 256) CTAs.
// gelu_bias / gelu_out non-null: the caller wants bf16(GELU(product + bias)) in gelu_out.  When the whole reduction
// fits one CTA (K <= 512) the GEMM writes that itself and *nsplit = 0; otherwise it writes partial tiles as usual
// and the caller runs the bias + GELU kernel.
static int seq_gemm(tf_model* m, const SeqCtx& cx, int cls, int abuf, const Matrix& W, int step_off, int* nsplit,
                    const float* gelu_bias = nullptr, bf16* gelu_out = nullptr, const seq::SeqFin* fin = nullptr,
                    const seq::SeqLnA* lna = nullptr) {
  const int N = W.N, K = W.K, n_steps = m->L - 1, B = cx.B;
  const bf16* A = reinterpret_cast<const bf16*>(abuf == 0 ? m->xn : abuf == 1 ? m->att : m->mlp) + (size_t)cx.b0 * K;
  const bf16* w = reinterpret_cast<const bf16*>(W.w);
  const size_t part_cap = (size_t)B * m->seq_part_row_floats;
  if (m->seq_use_tc && gelu_out != nullptr && m->seq_fuse_gelu && K % 64 == 0 && K / 64 <= 8 && N % 4 == 0) {
    *nsplit = 0;
    dim3 grid((N + 127) / 128, 1, (B + 63) / 64);
    return launch_seq(m, cls, seq::seq_gemm_tc_kernel<64, 8>, grid, 128, seq::gemm_tc_smem_bytes<64, 8>(), W.map_seq,
                      m->map_seq_a[abuf][2], cx.b0, B, N, K / 64, cx.part, cx.step_ctr, step_off, n_steps, m->seq_check_steps,
                      m->err, gelu_bias, gelu_out + (size_t)cx.b0 * N, seq::SeqFin{}, seq::SeqLnA{});
  }
  if (m->seq_use_tc) {  // tcgen05 kernel: CTAs of 128 columns x kbn slabs of 64 k
    const int slabs = K / 64;
    int kbn = slabs % 4 == 0 ? 4 : slabs % 2 == 0 ? 2 : 1;
    // two slabs per CTA (more CTAs) while the grid is below one wave and the partial tiles stay <= 16
    if (kbn == 4 && ((N + 127) / 128) * (slabs / 4) < m->num_sms && slabs / 2 <= 16) kbn = 2;
    // a launch whose last K slice finishes the tile reads all partials of it: keep them to eight where that is possible
    if (fin != nullptr && slabs / kbn > 8 && slabs % 4 == 0) kbn = 4;
    if (fin != nullptr && slabs / kbn > 8 && slabs % 8 == 0 && m->seq_kbn8) kbn = 8;  // eight slab buffers per CTA
    if (m->seq_kbn_force > 0 && slabs % m->seq_kbn_force == 0 && slabs / m->seq_kbn_force <= 16) kbn = m->seq_kbn_force;
    const int ksplit = slabs / kbn;
    if (ksplit > 16) return fail(TF_EINVAL, "sequential decoding: reduction length %d not supported", K);
    *nsplit = fin != nullptr ? 0 : ksplit;  // with a finishing launch nothing is left for the consumer to add up
    if ((size_t)ksplit * B * N > part_cap) return fail(TF_EINVAL, "sequential decoding: partial-tile buffer too small");
    const int ri = B <= 16 ? 0 : B <= 32 ? 1 : 2, rt = 16 << ri;
    dim3 grid((N + 127) / 128, ksplit, (B + rt - 1) / rt);
    if (fin != nullptr && (int)(grid.x * grid.z) > tf_model::SEQ_TICKETS) return fail(TF_EINVAL, "sequential decoding: too many column tiles");
    const seq::SeqFin fin_v = fin ? *fin : seq::SeqFin{};
    const seq::SeqLnA lna_v = lna ? *lna : seq::SeqLnA{};
#define TF_SEQ_TC_CASE(RTV)                                                                                              \
  if (rt == RTV)                                                                                                         \
    return launch_seq(m, cls, seq::seq_gemm_tc_kernel<RTV>, grid, 128, seq::gemm_tc_smem_bytes<RTV>(), W.map_seq,         \
                      m->map_seq_a[abuf][ri], cx.b0, B, N, kbn, cx.part, cx.step_ctr, step_off, n_steps,                 \
                      m->seq_check_steps, m->err, (const float*)nullptr, (bf16*)nullptr, fin_v, lna_v);
#define TF_SEQ_TC_CASE8(RTV)                                                                                             \
  if (rt == RTV && kbn == 8)                                                                                             \
    return launch_seq(m, cls, seq::seq_gemm_tc_kernel<RTV, 8>, grid, 128, seq::gemm_tc_smem_bytes<RTV, 8>(), W.map_seq,   \
                      m->map_seq_a[abuf][ri], cx.b0, B, N, kbn, cx.part, cx.step_ctr, step_off, n_steps,                 \
                      m->seq_check_steps, m->err, (const float*)nullptr, (bf16*)nullptr, fin_v, lna_v);
    TF_SEQ_TC_CASE8(16)
    TF_SEQ_TC_CASE8(32)
    TF_SEQ_TC_CASE8(64)
#undef TF_SEQ_TC_CASE8
    TF_SEQ_TC_CASE(16)
    TF_SEQ_TC_CASE(32)
    TF_SEQ_TC_CASE(64)
#undef TF_SEQ_TC_CASE
  }
  if (fin != nullptr || lna != nullptr) return fail(TF_EINVAL, "fused step kernels need the tcgen05 step GEMM");
  const int row_tiles = (B + seq::ROWS - 1) / seq::ROWS;
  int klen = (K % 256 == 0) ? 256 : K;
  while (K / klen > 16 && K % (klen * 2) == 0) klen *= 2;  // at most 16 partial tiles
  if (klen > seq::KC || K / klen > 16) return fail(TF_EINVAL, "sequential decoding: reduction length %d not supported", K);
  const int ksplit = K / klen;
  *nsplit = ksplit;
  if ((size_t)ksplit * B * N > part_cap) return fail(TF_EINVAL, "sequential decoding: partial-tile buffer too small");
  // column slices: the narrowest (most CTAs, shortest per-warp MMA chain) that keeps the grid within two waves; the
  // warps of a CTA split its K slice, which needs klen % (32 * 64 / NC) == 0
  int nc = 64;
  if (klen % 256 == 0 && ((N + 7) / 8) * ksplit <= 2 * m->num_sms) nc = 8;
  else if (klen % 128 == 0 && ((N + 15) / 16) * ksplit <= 2 * m->num_sms) nc = 16;
  else if (klen % 64 == 0 && ((N + 31) / 32) * ksplit <= 2 * m->num_sms) nc = 32;
  if (const char* e = getenv("TARFLOW_SEQ_NC")) {  // tuning aid: force the slice width where it is valid
    const int f = atoi(e);
    if ((f == 8 && klen % 256 == 0) || (f == 16 && klen % 128 == 0) || (f == 32 && klen % 64 == 0) || f == 64) nc = f;
  }
  dim3 grid((N + nc - 1) / nc, ksplit, row_tiles);
  const int smem = seq::gemm_smem_bytes(klen);
#define TF_SEQ_GEMM_CASE(NCV)                                                                                            \
  if (nc == NCV)                                                                                                         \
    return launch_seq(m, cls, seq::seq_gemm_kernel<NCV>, grid, seq::THREADS, smem, A, w, B, N, K, klen, cx.part,         \
                      cx.step_ctr, step_off, n_steps, m->seq_check_steps);
  TF_SEQ_GEMM_CASE(8)
  TF_SEQ_GEMM_CASE(16)
  TF_SEQ_GEMM_CASE(32)
  TF_SEQ_GEMM_CASE(64)
#undef TF_SEQ_GEMM_CASE
  return fail(TF_EINVAL, "no sequential GEMM variant for this shape");
}

static int seq_resid_ln(tf_model* m, const SeqCtx& cx, const float* bias, int nsplit, const float* gamma, const float* beta,
                        int step_off) {
  return launch_seq(m, KC_SEQ_LN, seq::seq_resid_ln_kernel, dim3(cx.B), m->d / 4, 0, m->h + (size_t)cx.b0 * m->d, cx.part, bias,
                    nsplit, gamma, beta, reinterpret_cast<bf16*>(m->xn) + (size_t)cx.b0 * m->d, cx.B, m->d, cx.step_ctr, step_off,
                    m->L - 1, m->seq_check_steps);
}

static bool seq_tail_fused(const tf_model* m) {
  if (m->d % 8 != 0 || m->d > 1024) return false;
  if (m->seq_fuse_tail >= 0) return m->seq_fuse_tail != 0;
  return (size_t)2 * m->D * m->d * sizeof(bf16) <= 64 * 1024;
}

// the fused tail of step step_off (first = 0) or the block's start (first = 1)
static int seq_tail(tf_model* m, const SeqCtx& cx, int g, const int* labels, const float* v, float* u,
                    const float* pending_bias, int pending, int first, int step_off) {
  const BlockW& bw = m->blocks[g];
  const LayerW& l0 = bw.layers[0];
  const int smem = (m->d + 3 * m->D) * (int)sizeof(float);
  const size_t tok0 = (size_t)cx.b0 * m->L * m->D;
  return launch_seq(m, KC_SEQ_UPDATE, seq::seq_tail_kernel, dim3(cx.B), 256, smem, m->h + (size_t)cx.b0 * m->d, cx.part,
                    pending_bias, pending, bw.lnf_g, bw.lnf_b, reinterpret_cast<const bf16*>(bw.w_out.w), bw.b_out, cx.B,
                    v + tok0, u + tok0, labels ? labels + cx.b0 : nullptr, bw.w_in_t, bw.b_in, bw.pos, bw.cls, l0.ln1_g, l0.ln1_b,
                    reinterpret_cast<bf16*>(m->xn) + (size_t)cx.b0 * m->d, m->L, m->D, m->d, g & 1, first, cx.step_ctr, step_off,
                    m->L - 1);
}

static bool seq_chain_fused(const tf_model* m) {
  return m->seq_fin && m->seq_use_tc && !m->seq_fuse_gelu && m->d % 128 == 0 && m->hid % 4 == 0 && m->d / 128 <= 16;
}

static int seq_update_embed(tf_model* m, const SeqCtx& cx, int g, const int* labels, const float* v, float* u, int ns,
                            int first, int step_off) {
  const BlockW& bw = m->blocks[g];
  const int d = m->d, D = m->D, ethreads = d < 128 ? d : 128;
  const size_t tok0 = (size_t)cx.b0 * m->L * D;
  return launch_seq(m, KC_SEQ_UPDATE, seq::seq_update_embed_kernel, dim3(cx.B, (d + ethreads - 1) / ethreads), ethreads,
                    (int)(D * sizeof(float)), cx.part, ns, bw.b_out, cx.B, v + tok0, u + tok0, labels ? labels + cx.b0 : nullptr,
                    bw.w_in_t, bw.b_in, bw.pos, bw.cls, m->h + (size_t)cx.b0 * d, m->L, D, d, g & 1, first, cx.step_ctr, step_off,
                    m->L - 1, (seq_chain_fused(m) && ethreads == 128) ? cx.stats : (float2*)nullptr);
}

// attention of the new token of every (sample, head) of the chain over its cache rows
static int seq_attention(tf_model* m, const SeqCtx& cx, int ns, const float* b_qkv, bf16* kc, bf16* vc, bf16* att, int step_off) {
  const int heads = m->cfg.n_heads, L = m->L;
  const float sl2 = 1.4426950408889634f / sqrtf((float)m->hd);
  // more (sample, head) pairs than three 256-thread CTAs per SM hold at once: the 128-thread form runs as one wave
  const bool small = m->seq_attn_threads == 128 || (m->seq_attn_threads == 0 && heads * cx.B > 3 * m->num_sms);
  if (small)
    return launch_seq(m, KC_SEQ_ATTN, seq::seq_attention_kernel<128>, dim3(heads, cx.B), 128, 0, cx.part, ns, b_qkv, kc, vc, att,
                      cx.B, L, m->d, heads, sl2, cx.step_ctr, step_off, L - 1);
  return launch_seq(m, KC_SEQ_ATTN, seq::seq_attention_kernel<256>, dim3(heads, cx.B), 256, 0, cx.part, ns, b_qkv, kc, vc, att,
                    cx.B, L, m->d, heads, sl2, cx.step_ctr, step_off, L - 1);
}

// kernels of decoding steps step_off .. step_off+count-1 relative to the chain's device step counter
static int seq_enqueue_steps(tf_model* m, const SeqCtx& cx, int g, const int* labels, const float* v, float* u, int count) {
  const BlockW& bw = m->blocks[g];
  const int L = m->L, d = m->d, nl = m->cfg.n_layers, B = cx.B;
  bf16* att = reinterpret_cast<bf16*>(m->att) + (size_t)cx.b0 * d;
  bf16* mlp = reinterpret_cast<bf16*>(m->mlp) + (size_t)cx.b0 * m->hid;
  const size_t layer_stride = (size_t)m->cfg.max_batch * L * d, kv0 = (size_t)cx.b0 * L * d;
  m->cur_rows = B;
  const bool tail = seq_tail_fused(m);
  // Fused form (opt-in, measured slower): the last K slice of a residual projection adds the finished sums to h and
  // leaves the row statistics, the next projection normalises its own K slice of h while staging it, the MLP-up
  // projection applies bias + GELU itself: five kernels per layer instead of eight.
  const bool fused = seq_chain_fused(m);
  float* hrow = m->h + (size_t)cx.b0 * d;
  for (int s = 0; s < count; ++s) {
    const float* pending_bias = nullptr;  // bias of the projection whose partial tiles are not yet in h
    int pending = 0, ns = 0;
    for (int i = 0; i < nl; ++i) {
      const LayerW& lw = bw.layers[i];
      bf16* kc = reinterpret_cast<bf16*>(m->kcache) + i * layer_stride + kv0;
      bf16* vc = reinterpret_cast<bf16*>(m->vcache) + i * layer_stride + kv0;
      if (fused) {
        const seq::SeqLnA ln1{hrow, cx.stats, lw.ln1_g, lw.ln1_b}, ln2{hrow, cx.stats, lw.ln2_g, lw.ln2_b};
        const seq::SeqFin fin_o{2, cx.tickets, lw.b_o, nullptr, hrow, cx.stats};
        const seq::SeqFin fin_1{1, cx.tickets, lw.b_1, mlp, nullptr, nullptr};
        const seq::SeqFin fin_2{2, cx.tickets, lw.b_2, nullptr, hrow, cx.stats};
        if (i == 0 && tail) {  // layer 0's input was normalised by the fused tail of the previous step
          TF_TRY(seq_gemm(m, cx, KC_SEQ_GEMM, 0, lw.w_qkv, s, &ns));
        } else {  // (for layer 0 the statistics come from the embedding kernel)
          TF_TRY(seq_gemm(m, cx, KC_SEQ_GEMM, 0, lw.w_qkv, s, &ns, nullptr, nullptr, nullptr, &ln1));
        }
        TF_TRY(seq_attention(m, cx, ns, lw.b_qkv, kc, vc, att, s));
        int none = 0;
        TF_TRY(seq_gemm(m, cx, KC_SEQ_GEMM, 1, lw.w_o, s, &none, nullptr, nullptr, &fin_o));
        TF_TRY(seq_gemm(m, cx, KC_SEQ_GEMM, 0, lw.w_1, s, &none, nullptr, nullptr, &fin_1, &ln2));
        TF_TRY(seq_gemm(m, cx, KC_SEQ_GEMM, 2, lw.w_2, s, &none, nullptr, nullptr, &fin_2));
        pending_bias = nullptr;
        pending = 0;
        continue;
      }
      // layer 0's input comes from the fused tail of the previous step (or of the block's start) when that is on
      if (!(tail && i == 0)) TF_TRY(seq_resid_ln(m, cx, pending_bias, pending, lw.ln1_g, lw.ln1_b, s));
      TF_TRY(seq_gemm(m, cx, KC_SEQ_GEMM, 0, lw.w_qkv, s, &ns));
      TF_TRY(seq_attention(m, cx, ns, lw.b_qkv, kc, vc, att, s));
      TF_TRY(seq_gemm(m, cx, KC_SEQ_GEMM, 1, lw.w_o, s, &pending));
      TF_TRY(seq_resid_ln(m, cx, lw.b_o, pending, lw.ln2_g, lw.ln2_b, s));
      TF_TRY(seq_gemm(m, cx, KC_SEQ_GEMM, 0, lw.w_1, s, &ns, lw.b_1, reinterpret_cast<bf16*>(m->mlp)));
      if (ns > 0)  // the GEMM left partial tiles: sum them, add the bias, apply GELU
        TF_TRY(launch_seq(m, KC_SEQ_LN, seq::seq_bias_gelu_kernel, dim3((B * (m->hid / 4) + 255) / 256), 256, 0, cx.part, ns,
                          lw.b_1, mlp, B, m->hid, cx.step_ctr, s, L - 1, m->seq_check_steps));
      TF_TRY(seq_gemm(m, cx, KC_SEQ_GEMM, 2, lw.w_2, s, &pending));
      pending_bias = lw.b_2;
    }
    if (tail) {
      TF_TRY(seq_tail(m, cx, g, labels, v, u, pending_bias, pending, 0, s));
      continue;
    }
    if (fused) {  // the head normalises h itself (statistics from the last MLP-down projection)
      const seq::SeqLnA lnf{hrow, cx.stats, bw.lnf_g, bw.lnf_b};
      TF_TRY(seq_gemm(m, cx, KC_SEQ_GEMM, 0, bw.w_out, s, &ns, nullptr, nullptr, nullptr, &lnf));
    } else {
      TF_TRY(seq_resid_ln(m, cx, pending_bias, pending, bw.lnf_g, bw.lnf_b, s));
      TF_TRY(seq_gemm(m, cx, KC_SEQ_GEMM, 0, bw.w_out, s, &ns));
    }
    TF_TRY(seq_update_embed(m, cx, g, labels, v, u, ns, 0, s));
  }
  return check_launch("sequential step kernels");
}

static int seq_unroll(int n_steps) {  // steps per graph: a divisor of n_steps close to 16, so no step is a no-op
  int best = 1;
  for (int c = 1; c <= 32 && c <= n_steps; ++c)
    if (n_steps % c == 0) best = c;
  return best >= 4 ? best : (n_steps < 16 ? n_steps : 16);
}

// How many chains decode a batch of B samples side by side.  Measured (one block, ms): width 512, 4 layers, batch 64:
// 34.8 / 28.3 / 28.4 with 1 / 2 / 4 chains; width 1024, 8 layers, batch 64: 82.0 / 76.0 / 86.1; 1024 tokens, batch 16:
// 287 / 303 / 359.  A chain of 16 samples takes as long as one of 64: the block's time is the length of the dependent
// kernel chain, and a split only hides the small throughput-bound part (attention over the cache, partial sums), while
// every chain streams the weights again.  So: two chains from 32 samples up, otherwise one.
static int seq_chain_count(const tf_model* m, int B) {
  int n = m->seq_chains_force > 0 ? m->seq_chains_force : (B >= 32 ? 2 : 1);
  if (n > tf_model::MAX_CHAINS) n = tf_model::MAX_CHAINS;
  while (n > 1 && B / n < 4) n /= 2;  // at least four samples per chain
  return n < 1 ? 1 : n;
}

// all decoding steps of one chain, enqueued on m->stream (the chain's stream)
static int run_sequential_chain(tf_model* m, const SeqCtx& cx, int g, const int* labels, const float* v, float* u) {
  const int n_steps = m->L - 1;
  CU_OK(cudaMemsetAsync(cx.step_ctr, 0, sizeof(int), m->stream));
  CU_OK(cudaMemsetAsync(cx.tickets, 0, tf_model::SEQ_TICKETS * sizeof(int), m->stream));  // after an aborted launch
  m->cur_rows = cx.B;
  if (seq_tail_fused(m)) TF_TRY(seq_tail(m, cx, g, labels, v, u, nullptr, 0, 1, 0));
  else TF_TRY(seq_update_embed(m, cx, g, labels, v, u, 0, 1, 0));
  if ((m->prof_on && m->prof_mode == 1) || !m->use_graphs) {  // direct launches (per-kernel events need them)
    for (int t = 0; t < n_steps; ++t) {
      TF_TRY(seq_enqueue_steps(m, cx, g, labels, v, u, 1));
      TF_TRY(launch_seq(m, KC_CTRL, seq::seq_advance_kernel, dim3(1), 32, 0, cx.step_ctr, 1));
    }
    return check_launch("sequential block");
  }
  cudaStream_t run_stream = m->stream;
  auto key = std::make_tuple(g, cx.b0, cx.B, m->seq_variant);
  auto it = m->seq_graphs.find(key);
  if (it == m->seq_graphs.end()) {
    tf_model::SeqGraph sg;
    sg.unroll = seq_unroll(n_steps);
    const int64_t before = m->launches;
    cudaGraph_t graph = nullptr;
    m->stream = m->cap_stream;
    cudaError_t e = cudaStreamBeginCapture(m->cap_stream, cudaStreamCaptureModeThreadLocal);
    int r = TF_OK;
    if (e == cudaSuccess) {
      r = seq_enqueue_steps(m, cx, g, labels, v, u, sg.unroll);
      if (r == TF_OK) r = launch_seq(m, KC_CTRL, seq::seq_advance_kernel, dim3(1), 32, 0, cx.step_ctr, sg.unroll);
      e = cudaStreamEndCapture(m->cap_stream, &graph);
    }
    m->stream = run_stream;
    sg.nodes = (int)(m->launches - before);
    m->launches = before;
    if (e != cudaSuccess || r != TF_OK || !graph) {
      if (graph) cudaGraphDestroy(graph);
      cudaGetLastError();
      return r != TF_OK ? r : fail(TF_ECUDA, "capturing the sequential-step graph failed: %s", cudaGetErrorString(e));
    }
    e = cudaGraphInstantiate(&sg.exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e != cudaSuccess) return fail(TF_ECUDA, "cudaGraphInstantiate: %s", cudaGetErrorString(e));
    it = m->seq_graphs.emplace(key, sg).first;
  }
  const tf_model::SeqGraph& sg = it->second;
  const int replays = (n_steps + sg.unroll - 1) / sg.unroll;  // steps past n_steps return at once
  for (int i = 0; i < replays; ++i) CU_OK(cudaGraphLaunch(sg.exec, run_stream));
  m->launches += (int64_t)replays * sg.nodes;
  return TF_OK;
}

static int run_sequential_block_bf16(tf_model* m, int g, int B, const int* labels, const float* v, float* u) {
  const int n_steps = m->L - 1;
  cudaStream_t user = m->stream;
  const bool direct = (m->prof_on && m->prof_mode == 1) || !m->use_graphs;
  m->seq_check_steps = direct ? 0 : (n_steps % seq_unroll(n_steps) != 0);
  const int nch = direct ? 1 : seq_chain_count(m, B);
  if (nch == 1) {
    SeqCtx cx;
    cx.b0 = 0; cx.B = B; cx.step_ctr = m->step_ctr; cx.part = m->seq_part;
    cx.tickets = m->seq_tickets; cx.stats = m->seq_stats;
    return run_sequential_chain(m, cx, g, labels, v, u);
  }
  // fork: the chains start once everything enqueued on the caller's stream so far has completed; join: the caller's
  // stream continues once every chain has finished
  CU_OK(cudaEventRecord(m->seq_fork, user));
  int r = TF_OK;
  for (int c = 0; c < nch && r == TF_OK; ++c) {
    SeqCtx cx;
    cx.b0 = (int)((int64_t)B * c / nch);
    cx.B = (int)((int64_t)B * (c + 1) / nch) - cx.b0;
    cx.step_ctr = m->step_ctr + 16 * c;
    cx.part = m->seq_part + (size_t)cx.b0 * m->seq_part_row_floats;
    cx.tickets = m->seq_tickets + (size_t)c * tf_model::SEQ_TICKETS;
    cx.stats = m->seq_stats + (size_t)c * 16 * m->cfg.max_batch;
    m->stream = m->seq_streams[c];
    cudaError_t e = cudaStreamWaitEvent(m->stream, m->seq_fork, 0);
    if (e != cudaSuccess) r = fail(TF_ECUDA, "cudaStreamWaitEvent: %s", cudaGetErrorString(e));
    if (r == TF_OK) r = run_sequential_chain(m, cx, g, labels, v, u);
    if (r == TF_OK && (e = cudaEventRecord(m->seq_join[c], m->stream)) != cudaSuccess)
      r = fail(TF_ECUDA, "cudaEventRecord: %s", cudaGetErrorString(e));
    if (r == TF_OK && (e = cudaStreamWaitEvent(user, m->seq_join[c], 0)) != cudaSuccess)
      r = fail(TF_ECUDA, "cudaStreamWaitEvent: %s", cudaGetErrorString(e));
  }
  m->stream = user;
  return r;
}

// ------------------------------------------------------------------------------------------------
// Jacobi block (Algorithm 1) with per-sample stopping and active-set compaction
// ------------------------------------------------------------------------------------------------
// A recorded device-side timeout is reported once and the word is cleared, so the model stays usable: kernels
// launched after the word was set returned without work, the ones launched after this call run normally.
static int report_timeout(tf_model* m) {
  const int code = m->ctrl_host[2];
  cudaMemsetAsync(m->err, 0, sizeof(int), m->stream);
  cudaStreamSynchronize(m->stream);
  return fail(TF_ETIMEOUT, "device-side wait expired (code %d)", code);
}

static int read_ctrl(tf_model* m) {
  CU_OK(cudaMemcpyAsync(m->ctrl_host, m->ctrl, 2 * sizeof(int), cudaMemcpyDeviceToHost, m->stream));
  CU_OK(cudaMemcpyAsync(m->ctrl_host + 3, m->ctrl + 2, 2 * sizeof(int), cudaMemcpyDeviceToHost, m->stream));
  CU_OK(cudaMemcpyAsync(m->ctrl_host + 2, m->err, sizeof(int), cudaMemcpyDeviceToHost, m->stream));
  CU_OK(cudaStreamSynchronize(m->stream));
  if (m->ctrl_host[2] != 0) return report_timeout(m);
  if (m->ctrl_host[1] != 0) return fail(TF_ENONFINITE, "non-finite value in the convergence reduction");
  return TF_OK;
}

// synchronise the stream and turn a recorded device-side timeout into an error
static int sync_check(tf_model* m) {
  CU_OK(cudaMemcpyAsync(m->ctrl_host + 2, m->err, sizeof(int), cudaMemcpyDeviceToHost, m->stream));
  CU_OK(cudaStreamSynchronize(m->stream));
  if (m->ctrl_host[2] != 0) return report_timeout(m);
  return TF_OK;
}

// Class labels come from the caller's device memory and index the class-embedding table: copy them into the
// model-owned array (a fixed address for captured graphs) clamped to [0, n_classes), and fail with TF_EINVAL when one
// was out of range -- no kernel ever indexes the table with an unchecked id.
static int take_labels(tf_model* m, const int** labels, int B) {
  if (!*labels) return TF_OK;
  if (m->cfg.n_classes <= 0) {  // an unconditional model has no table: the labels are not read at all
    *labels = nullptr;
    return TF_OK;
  }
  LAUNCH(m, KC_CTRL, labels_check_kernel, (B + 127) / 128, 128, 0, *labels, m->labels_own, B, m->cfg.n_classes, m->ctrl + CTRL_LABEL_FLAG);
  TF_TRY(check_launch("labels_check_kernel"));
  CU_OK(cudaMemcpyAsync(m->ctrl_host + 5, m->ctrl + CTRL_LABEL_FLAG, sizeof(int), cudaMemcpyDeviceToHost, m->stream));
  CU_OK(cudaStreamSynchronize(m->stream));
  if (m->ctrl_host[5] != 0) {
    CU_OK(cudaMemsetAsync(m->ctrl + CTRL_LABEL_FLAG, 0, sizeof(int), m->stream));
    return fail(TF_EINVAL, "a class label lies outside [0, %d)", m->cfg.n_classes);
  }
  *labels = m->labels_own;
  return TF_OK;
}

// Options of one inverse call beyond the policy (all optional; see tf_jacobi_opts in tarflow.h).
struct InvOpts {
  int init_mode = 0;
  const float* u0_img = nullptr;        // [n_blocks][B][C][H][W]
  const float* tau_block = nullptr;     // host [n_blocks]
  int fallback_sweeps = 0;
  float* states_img = nullptr;          // out [n_blocks][B][C][H][W]
  const float* ref_img = nullptr;       // in  [n_blocks][B][C][H][W]
};

static int layout(tf_model* m, float* img, float* seq, int B, int to_seq);
template <class T>
static int run_sequential_any(tf_model* m, int g, int B, const int* labels, const float* v, float* u);
template <class T>
static int maf_pass(tf_model* m, int g, int n_slots, const float* u_src, const int* idx, int mode, const float* v, float* u_upd,
                    bool hp, int only_col);

// one causal pass of a Jacobi sweep over the listed slots, whichever flow the model is
template <class T>
static int sweep_pass(tf_model* m, int g, int n_slots, const float* u_src, const int* idx, const int* labels, const float* v,
                      float* u_upd, bool hp) {
  if (m->is_maf) return maf_pass<T>(m, g, n_slots, u_src, idx, 0, v, u_upd, hp, -1);
  return run_pass<T>(m, g, n_slots, u_src, idx, labels, PASS_JACOBI, v, u_upd, hp);
}

template <class T>
static int run_jacobi_block(tf_model* m, int g, int B, const int* labels, const float* v, float* u, float tau,
                            int max_iters, const InvOpts& op, int* sweeps_out, int* iters_row) {
  const size_t n = (size_t)B * m->L * m->D, img = (size_t)B * m->cfg.C * m->cfg.H * m->cfg.W;
  if (op.init_mode == 0) CU_OK(cudaMemsetAsync(u, 0, n * sizeof(float), m->stream));
  else if (op.init_mode == 1) CU_OK(cudaMemcpyAsync(u, v, n * sizeof(float), cudaMemcpyDeviceToDevice, m->stream));
  else TF_TRY(layout(m, const_cast<float*>(op.u0_img) + (size_t)g * img, u, B, 1));
  const bool l2 = m->trace_on && op.ref_img != nullptr && m->trace_l2 != nullptr;
  if (l2) TF_TRY(layout(m, const_cast<float*>(op.ref_img) + (size_t)g * img, m->ref_seq, B, 1));
  // precision policy (bf16 engine): which sweeps of a sample use two-term operands
  int start_phase = 0;
  float sw = -1.f;  // never escalate
  if (sizeof(T) == 2) {
    if (m->precision_mode == 2) start_phase = 1;
    else if (m->precision_mode == 0 && tau >= 0.f && tau < m->single_ok_tau) sw = m->switch_threshold;
  }
  LAUNCH(m, KC_CTRL, jacobi_begin_kernel, (B + 1023) / 1024 < 64 ? (B + 1023) / 1024 : 64, 256, 0, m->maxdiff, m->idx, m->phase,
         m->ctrl, B, start_phase, tau, sw);
  int n_active = B, n_hp = start_phase ? B : 0, t = 0;
  const int cap = (op.fallback_sweeps > 0 && op.fallback_sweeps < max_iters) ? op.fallback_sweeps : max_iters;
  // everything one sweep launches: the pass over the single-term samples, the pass over the two-term samples, the
  // sweep control (which takes the sweep number and the thresholds from device memory)
  auto enqueue_sweep = [&](int n_lp, int n_hpp) -> int {
    if (n_lp > 0) TF_TRY(sweep_pass<T>(m, g, n_lp, u, m->idx, labels, v, u, false));
    if (n_hpp > 0) TF_TRY(sweep_pass<T>(m, g, n_hpp, u, m->idx + n_lp, labels, v, u, true));
    const int na = n_lp + n_hpp;
    if (na <= FIN_CHUNK || m->fin_code == nullptr) {
      LAUNCH_PDL(m, KC_CTRL, jacobi_finalize_kernel, 1, 256, 0, m->maxdiff, m->idx, m->idx_tmp, m->phase, m->ctrl, iters_row);
    } else {  // large batches: count / scan / scatter over all SMs; the new slot list is written to the other buffer
      const int nblk = (na + FIN_CHUNK - 1) / FIN_CHUNK;
      LAUNCH(m, KC_CTRL, jacobi_finalize_count_kernel, nblk, FIN_CHUNK, 0, m->maxdiff, m->idx, m->phase, m->ctrl, iters_row,
             m->fin_code, m->fin_cnt, m->fin_top, m->fin_flag, nblk);
      LAUNCH(m, KC_CTRL, jacobi_finalize_scan_kernel, 1, 256, 0, m->fin_cnt, m->fin_top, m->fin_flag, m->ctrl, nblk);
      LAUNCH(m, KC_CTRL, jacobi_finalize_scatter_kernel, nblk, FIN_CHUNK, 0, m->idx, m->idx_tmp, m->fin_code, m->fin_cnt, m->ctrl,
             nblk);
      int* sw_idx = m->idx; m->idx = m->idx_tmp; m->idx_tmp = sw_idx;
    }
    return check_launch("sweep control kernels");
  };
  while (t < cap && n_active > 0) {
    ++t;
    const int n_lp = n_active - n_hp;
    // Few rows: a sweep is a chain of short kernels whose launch cost exceeds their run time, so the whole sweep is
    // captured once per (block, single-term slots, two-term slots) and replayed as a graph afterwards.
    const bool as_graph = m->use_graphs && m->cap_stream != nullptr && !m->prof_on && n_active <= FIN_CHUNK && (int64_t)n_active * m->L <= m->sweep_graph_rows;
    if (as_graph) {
      const auto key = std::make_tuple(g, n_lp, n_hp, (const void*)v, (const void*)u, (const void*)labels, (const void*)iters_row);
      auto it = m->sweep_graphs.find(key);
      if (it == m->sweep_graphs.end() && m->sweep_graphs.size() < 2048) {
        tf_model::SeqGraph sg;
        const int64_t before = m->launches;
        cudaStream_t user = m->stream;
        cudaGraph_t graph = nullptr;
        m->stream = m->cap_stream;
        cudaError_t e = cudaStreamBeginCapture(m->cap_stream, cudaStreamCaptureModeRelaxed);
        int r = TF_OK;
        if (e == cudaSuccess) {
          r = enqueue_sweep(n_lp, n_hp);
          e = cudaStreamEndCapture(m->cap_stream, &graph);
        }
        m->stream = user;
        sg.nodes = (int)(m->launches - before);
        m->launches = before;
        if (e != cudaSuccess || r != TF_OK || !graph) {
          if (graph) cudaGraphDestroy(graph);
          cudaGetLastError();
          return r != TF_OK ? r : fail(TF_ECUDA, "capturing a sweep graph failed: %s", cudaGetErrorString(e));
        }
        e = cudaGraphInstantiate(&sg.exec, graph, 0);
        cudaGraphDestroy(graph);
        if (e != cudaSuccess) return fail(TF_ECUDA, "cudaGraphInstantiate: %s", cudaGetErrorString(e));
        it = m->sweep_graphs.emplace(key, sg).first;
      }
      if (it != m->sweep_graphs.end()) {
        CU_OK(cudaGraphLaunch(it->second.exec, m->stream));
        m->launches += it->second.nodes;
      } else {
        TF_TRY(enqueue_sweep(n_lp, n_hp));
      }
    } else {
      TF_TRY(enqueue_sweep(n_lp, n_hp));
    }
    if (l2 && t <= m->trace_l2_sweeps) {
      LAUNCH(m, KC_CTRL, l2_distance_kernel, B, 256, 0, u, m->ref_seq,
             m->trace_l2 + ((size_t)g * m->trace_l2_sweeps + (t - 1)) * m->cfg.max_batch, m->L * m->D);
      m->trace_l2_count[g] = t;
    }
    if (tau >= 0.f || t == cap || m->trace_on) {
      const int before = n_active;
      TF_TRY(read_ctrl(m));
      n_active = m->ctrl_host[0];
      n_hp = m->ctrl_host[4];
      if (m->trace_on) {
        float top;
        memcpy(&top, &m->ctrl_host[3], sizeof(float));
        m->trace.push_back({g, t, before, top});
      }
    }
  }
  *sweeps_out = t;
  if (tau >= 0.f && n_active > 0 && cap < max_iters) {
    // Fall-back: the samples still in the active list are decoded sequentially from the block's input (Eq. 5), as a
    // dense batch of their own; their count becomes sweeps + L - 1.
    const int nf = m->L * m->D, nb = n_active;
    int gb = (int)(((size_t)nb * nf + 255) / 256);
    if (gb > 148 * 16) gb = 148 * 16;
    LAUNCH(m, KC_LAYOUT, gather_rows_kernel, gb, 256, 0, v, m->cmp_v, m->idx, nb, nf, 1);
    const int* lab_c = nullptr;
    if (labels) {
      LAUNCH(m, KC_LAYOUT, gather_int_kernel, (nb + 127) / 128, 128, 0, labels, m->cmp_labels, m->idx, nb);
      lab_c = m->cmp_labels;
    }
    TF_TRY(check_launch("gather kernels"));
    m->seq_variant = 1;
    int r = run_sequential_any<T>(m, g, nb, lab_c, m->cmp_v, m->cmp_u);
    m->seq_variant = 0;
    TF_TRY(r);
    LAUNCH(m, KC_LAYOUT, gather_rows_kernel, gb, 256, 0, m->cmp_u, u, m->idx, nb, nf, 0);
    LAUNCH(m, KC_CTRL, add_int_rows_kernel, (nb + 127) / 128, 128, 0, iters_row, m->idx, nb, m->L - 1);
    TF_TRY(check_launch("scatter kernels"));
    *sweeps_out = t + m->L - 1;
    return TF_OK;
  }
  return (tau >= 0.f && n_active > 0) ? TF_MAXITER : TF_OK;
}

// ------------------------------------------------------------------------------------------------
// whole-model drivers
// ------------------------------------------------------------------------------------------------
static int layout(tf_model* m, float* img, float* seq, int B, int to_seq) {
  size_t n = (size_t)B * m->cfg.C * m->cfg.H * m->cfg.W;
  int blocks = (int)((n + 255) / 256);
  if (blocks > 148 * 16) blocks = 148 * 16;
  LAUNCH(m, KC_LAYOUT, patchify_kernel, blocks, 256, 0, img, seq, B, m->cfg.C, m->cfg.H, m->cfg.W, m->cfg.patch, to_seq);
  return check_launch("patchify_kernel");
}

template <class T>
static int run_sequential_any(tf_model* m, int g, int B, const int* labels, const float* v, float* u) {
  const bool unit = m->prof_on && m->prof_mode == 2;  // time the whole block as one unit of class seq_block
  if (unit) {
    m->cur_rows = (int64_t)B * (m->L - 1);
    m->pre(KC_SEQ_BLOCK);
    m->prof_suspend = true;
  }
  int r;
  if constexpr (sizeof(T) == 2) r = run_sequential_block_bf16(m, g, B, labels, v, u);
  else r = run_sequential_block<T>(m, g, B, labels, v, u);
  if (unit) {
    m->prof_suspend = false;
    m->cur_rows = (int64_t)B * (m->L - 1);
    const int64_t keep = m->launches;
    m->post(KC_SEQ_BLOCK);
    m->launches = keep;
  }
  return r;
}

template <class T>
static int inverse_impl(tf_model* m, const float* z, const int* labels, int B, const uint8_t* policy, float tau,
                        int max_iters, const InvOpts& op, float* x, int* iters_block_host, int* iters_sample_dev) {
  const int K = m->cfg.n_blocks;
  const size_t img = (size_t)B * m->cfg.C * m->cfg.H * m->cfg.W;
  float *v = m->seq_a, *u = m->seq_b;
  m->trace.clear();
  m->trace_l2_count.assign(K, 0);
  TF_TRY(take_labels(m, &labels, B));
  TF_TRY(layout(m, const_cast<float*>(z), v, B, 1));
  int status = TF_OK;
  for (int g = 0; g < K; ++g) {
    int* iters_row = m->iters_sample + (size_t)g * m->cfg.max_batch;
    int sweeps = m->L - 1;
    if (m->block_ev[g]) cudaEventRecord(m->block_ev[g], m->stream);
    if (policy[g] == 0) {
      TF_TRY(run_sequential_any<T>(m, g, B, labels, v, u));
      LAUNCH(m, KC_CTRL, fill_int_kernel, (B + 127) / 128, 128, 0, iters_row, B, m->L - 1);
    } else {
      const float tau_g = op.tau_block ? op.tau_block[g] : tau;
      int r = run_jacobi_block<T>(m, g, B, labels, v, u, tau_g, max_iters, op, &sweeps, iters_row);
      if (r < 0) return r;
      if (r == TF_MAXITER) status = TF_MAXITER;
    }
    if (iters_block_host) iters_block_host[g] = sweeps;
    if (op.states_img) TF_TRY(layout(m, op.states_img + (size_t)g * img, u, B, 0));
    float* tmp = v; v = u; u = tmp;
  }
  if (m->block_ev[K]) cudaEventRecord(m->block_ev[K], m->stream);
  m->block_ev_valid = true;
  TF_TRY(layout(m, x, v, B, 0));
  if (iters_sample_dev) {
    for (int g = 0; g < K; ++g)
      CU_OK(cudaMemcpyAsync(iters_sample_dev + (size_t)g * B, m->iters_sample + (size_t)g * m->cfg.max_batch,
                            B * sizeof(int), cudaMemcpyDeviceToDevice, m->stream));
  }
  TF_TRY(sync_check(m));
  return status;
}

template <class T>
static int forward_impl(tf_model* m, const float* x, const int* labels, int B, float* z, float* logdet) {
  float *u = m->seq_a, *v = m->seq_b;
  TF_TRY(take_labels(m, &labels, B));
  TF_TRY(layout(m, const_cast<float*>(x), u, B, 1));
  if (logdet) CU_OK(cudaMemsetAsync(logdet, 0, B * sizeof(float), m->stream));
  for (int g = m->cfg.n_blocks - 1; g >= 0; --g) {
    TF_TRY(run_pass<T>(m, g, B, u, nullptr, labels, PASS_FORWARD, nullptr, nullptr, false));
    LAUNCH(m, KC_AFFINE, forward_affine_kernel, B, 256, 0, m->o, u, v, logdet, m->L, m->D, g & 1);
    TF_TRY(check_launch("forward_affine_kernel"));
    float* tmp = v; v = u; u = tmp;
  }
  TF_TRY(layout(m, z, u, B, 0));
  return sync_check(m);
}

// ------------------------------------------------------------------------------------------------
// second workload: MLP-based autoregressive flow (App. E.3).  One pass = cast -> three masked linear layers.
//   mode 0: Jacobi update in the last layer's epilogue (only_col >= 0: one step of sequential decoding)
//   mode 1: forward direction, the raw (mu, alpha) go to m->o
// The layer permutation (reversal on odd layers) and the MADE masks are folded into the weights when they are
// loaded, so every buffer here is in the sample's own dimension order.
// ------------------------------------------------------------------------------------------------
template <class T>
static int maf_pass(tf_model* m, int g, int n_slots, const float* u_src, const int* idx, int mode, const float* v, float* u_upd,
                    bool hp, int only_col) {
  const tf_model::MafBlock& bw = m->maf_blocks[g];
  const int D = m->L, H = m->maf_H, M = n_slots;
  T* a0 = reinterpret_cast<T*>(m->maf_a0);
  T* h1 = reinterpret_cast<T*>(m->maf_h1);
  T* h2 = reinterpret_cast<T*>(m->maf_h2);
  T* a0_lo = hp ? reinterpret_cast<T*>(m->maf_a0_lo) : nullptr;
  T* h1_lo = hp ? reinterpret_cast<T*>(m->maf_h1_lo) : nullptr;
  T* h2_lo = hp ? reinterpret_cast<T*>(m->maf_h2_lo) : nullptr;
  m->cur_rows = M;
  int cb = (int)(((size_t)M * ((D & 3) == 0 ? D / 4 : D) + 255) / 256);
  if (cb > 148 * 16) cb = 148 * 16;
  LAUNCH(m, KC_EMBED, (maf_cast_rows_kernel<T>), cb, 256, 0, u_src, idx, a0, a0_lo, M, D);
  TF_TRY(check_launch("maf_cast_rows_kernel"));
  if constexpr (sizeof(T) == 2) {
    const CUtensorMap* sm = m->maf_store_maps;
    TF_TRY(gemm<T>(m, KC_GEMM_MLP1, a0, &m->maf_map[0][0], hp ? &m->maf_map[0][1] : nullptr, bw.w1, M,
                   EpiStoreTma<ACT_RELU>{bw.b1, sm + 0, hp ? sm + 1 : nullptr}));
    TF_TRY(gemm<T>(m, KC_GEMM_MLP2, h1, &m->maf_map[1][0], hp ? &m->maf_map[1][1] : nullptr, bw.w2, M,
                   EpiStoreTma<ACT_RELU>{bw.b2, sm + 2, hp ? sm + 3 : nullptr}));
  } else {
    TF_TRY(gemm<T>(m, KC_GEMM_MLP1, a0, nullptr, nullptr, bw.w1, M, EpiStore<T, ACT_RELU>{h1, bw.b1, H, h1_lo}));
    TF_TRY(gemm<T>(m, KC_GEMM_MLP2, h1, nullptr, nullptr, bw.w2, M, EpiStore<T, ACT_RELU>{h2, bw.b2, H, h2_lo}));
  }
  const CUtensorMap* map2 = sizeof(T) == 2 ? &m->maf_map[2][0] : nullptr;
  const CUtensorMap* map2_lo = (sizeof(T) == 2 && hp) ? &m->maf_map[2][1] : nullptr;
  if (mode == 0) {
    if constexpr (sizeof(T) == 2) {
      // tensor-core engine: the raw (mu, alpha) leave through bulk stores, a row-per-warp kernel applies the update
      // (measured: 381 us for the fused lane-per-column epilogue against 85 + 60 us for the pair on 69 k rows)
      TF_TRY(gemm<T>(m, KC_GEMM_HEAD_UPDATE, h2, map2, map2_lo, bw.w3, M, EpiStoreF32Tma{bw.b3, m->maf_store_maps + 4}));
      LAUNCH(m, KC_AFFINE, maf_update_kernel, (M + 7) / 8, 256, 0, m->o, v, u_upd, m->maxdiff, idx, M, D, only_col);
      return check_launch("maf_update_kernel");
    } else {
      EpiMafUpdate epi{v, u_upd, m->maxdiff, idx, bw.b3, D, only_col};
      return gemm<T>(m, KC_GEMM_HEAD_UPDATE, h2, map2, map2_lo, bw.w3, M, epi);
    }
  }
  return gemm<T>(m, KC_GEMM_HEAD, h2, map2, map2_lo, bw.w3, M, EpiStore<float, ACT_NONE>{m->o, bw.b3, 2 * D});
}

template <class T>
static int maf_inverse_impl(tf_model* m, const float* z, int B, bool jacobi, float tau, int max_iters, int init_mode, float* x,
                            int* iters_block_host, int* iters_sample_dev) {
  const int K = m->cfg.n_blocks, D = m->L;
  const size_t n = (size_t)B * D;
  float *v = m->seq_a, *u = m->seq_b;
  m->trace.clear();
  m->trace_l2_count.assign(K, 0);
  CU_OK(cudaMemcpyAsync(v, z, n * sizeof(float), cudaMemcpyDeviceToDevice, m->stream));
  int status = TF_OK;
  InvOpts op;
  op.init_mode = init_mode;
  for (int g = 0; g < K; ++g) {
    int* iters_row = m->iters_sample + (size_t)g * m->cfg.max_batch;
    int sweeps = D;
    if (m->block_ev[g]) cudaEventRecord(m->block_ev[g], m->stream);
    if (!jacobi) {
      // Eq. 5: dimension i (in the layer's own order) is final after pass i; there is no cache, every pass is a whole one
      CU_OK(cudaMemsetAsync(u, 0, n * sizeof(float), m->stream));
      for (int i = 0; i < D; ++i)
        TF_TRY(maf_pass<T>(m, g, B, u, nullptr, 0, v, u, m->precision_mode == 2, (g & 1) ? D - 1 - i : i));
      LAUNCH(m, KC_CTRL, fill_int_kernel, (B + 127) / 128, 128, 0, iters_row, B, D);
      CU_OK(cudaMemsetAsync(m->maxdiff, 0, B * sizeof(float), m->stream));
    } else {
      int r = run_jacobi_block<T>(m, g, B, nullptr, v, u, tau, max_iters, op, &sweeps, iters_row);
      if (r < 0) return r;
      if (r == TF_MAXITER) status = TF_MAXITER;
    }
    if (iters_block_host) iters_block_host[g] = sweeps;
    float* tmp = v; v = u; u = tmp;
  }
  if (m->block_ev[K]) cudaEventRecord(m->block_ev[K], m->stream);
  m->block_ev_valid = true;
  CU_OK(cudaMemcpyAsync(x, v, n * sizeof(float), cudaMemcpyDeviceToDevice, m->stream));
  if (iters_sample_dev)
    for (int g = 0; g < K; ++g)
      CU_OK(cudaMemcpyAsync(iters_sample_dev + (size_t)g * B, m->iters_sample + (size_t)g * m->cfg.max_batch, B * sizeof(int),
                            cudaMemcpyDeviceToDevice, m->stream));
  TF_TRY(sync_check(m));
  return status;
}

template <class T>
static int maf_forward_impl(tf_model* m, const float* x, int B, float* z, float* logdet) {
  const int D = m->L;
  const size_t n = (size_t)B * D;
  float *u = m->seq_a, *v = m->seq_b;
  CU_OK(cudaMemcpyAsync(u, x, n * sizeof(float), cudaMemcpyDeviceToDevice, m->stream));
  if (logdet) CU_OK(cudaMemsetAsync(logdet, 0, B * sizeof(float), m->stream));
  for (int g = m->cfg.n_blocks - 1; g >= 0; --g) {
    TF_TRY(maf_pass<T>(m, g, B, u, nullptr, 1, nullptr, nullptr, false, -1));
    LAUNCH(m, KC_AFFINE, maf_forward_affine_kernel, B, 256, 0, m->o, u, v, logdet, D);
    TF_TRY(check_launch("maf_forward_affine_kernel"));
    float* tmp = v; v = u; u = tmp;
  }
  CU_OK(cudaMemcpyAsync(z, u, n * sizeof(float), cudaMemcpyDeviceToDevice, m->stream));
  return sync_check(m);
}

// ------------------------------------------------------------------------------------------------
// loading
// ------------------------------------------------------------------------------------------------
struct BlobReader {
  const float* p;
  const float* end;
  const float* take(size_t n) {
    const float* r = p;
    p += n;
    return r;
  }
};

static int upload_f32(tf_model* m, float** dst, const float* src, size_t n) {
  TF_TRY(dev_alloc(m, dst, n));
  CU_OK(cudaMemcpy(*dst, src, n * sizeof(float), cudaMemcpyHostToDevice));
  return TF_OK;
}

// matrix [N, K]: fp32 engine keeps fp32; bf16 engine converts on the device (round to nearest even)
static int upload_matrix(tf_model* m, Matrix* W, const float* src, int N, int K, float* staging) {
  W->N = N;
  W->K = K;
  size_t n = (size_t)N * K;
  if (m->cfg.dtype == 0) {
    float* w;
    TF_TRY(upload_f32(m, &w, src, n));
    W->w = w;
    return TF_OK;
  }
  bf16* w;
  TF_TRY(dev_alloc(m, &w, n));
  CU_OK(cudaMemcpy(staging, src, n * sizeof(float), cudaMemcpyHostToDevice));
  f32_to_bf16_kernel<<<148 * 4, 256>>>(staging, w, n);
  CU_OK(cudaDeviceSynchronize());
  W->w = w;
  W->bn = (N % 256 == 0) ? 256 : 128;
  TF_TRY(make_map_bf16(&W->map_seq, w, (uint64_t)N, (uint64_t)K, 128u));
  return make_map_bf16(&W->map, w, (uint64_t)N, (uint64_t)K, (uint32_t)W->bn);
}

static size_t block_floats(const tf_config& c, int L, int D) {
  size_t d = c.width, hid = (size_t)c.mlp_ratio * d;
  size_t n = d * D + d + (size_t)L * d + (size_t)c.n_classes * d;
  n += (size_t)c.n_layers * (2 * d + 3 * d * d + 3 * d + d * d + d + 2 * d + hid * d + hid + d * hid + d);
  n += 2 * d + 2 * (size_t)D * d + 2 * D;
  return n;
}

static int load_impl(tf_model* m, const void* blob, size_t nbytes) {
  const tf_config& c = m->cfg;
  const int L = m->L, D = m->D, d = m->d, hid = m->hid;
  const size_t want = 64 + 4 * block_floats(c, L, D) * c.n_blocks;
  if (nbytes != want) return fail(TF_ESIZE, "weight blob is %zu bytes, configuration needs %zu", nbytes, want);
  const int32_t* hdr = reinterpret_cast<const int32_t*>(blob);
  const int32_t expect[13] = {0x31574654, 1, c.C, c.H, c.W, c.patch, c.n_blocks, c.n_layers, c.width, c.n_heads,
                              c.mlp_ratio, c.n_classes, c.dtype};
  for (int i = 0; i < 13; ++i)
    if (hdr[i] != expect[i]) return fail(TF_ESIZE, "weight blob header field %d is %d, expected %d", i, hdr[i], expect[i]);

  int dev = 0;
  CU_OK(cudaGetDevice(&dev));
  CU_OK(cudaDeviceGetAttribute(&m->num_sms, cudaDevAttrMultiProcessorCount, dev));

  float* staging = nullptr;
  size_t max_mat = (size_t)hid * d;
  if ((size_t)3 * d * d > max_mat) max_mat = (size_t)3 * d * d;
  if (c.dtype == 1) CU_OK(cudaMalloc(&staging, max_mat * sizeof(float)));
  struct Guard { float* p; ~Guard() { if (p) cudaFree(p); } } guard{staging};

  BlobReader rd{reinterpret_cast<const float*>(reinterpret_cast<const char*>(blob) + 64), nullptr};
  m->blocks.resize(c.n_blocks);
  std::vector<float> tmp;
  for (int g = 0; g < c.n_blocks; ++g) {
    BlockW& bw = m->blocks[g];
    const float* w_in = rd.take((size_t)d * D);
    tmp.resize((size_t)d * D);
    for (int j = 0; j < d; ++j)
      for (int cc = 0; cc < D; ++cc) tmp[(size_t)cc * d + j] = w_in[(size_t)j * D + cc];
    TF_TRY(upload_f32(m, &bw.w_in_t, tmp.data(), tmp.size()));
    TF_TRY(upload_f32(m, &bw.b_in, rd.take(d), d));
    TF_TRY(upload_f32(m, &bw.pos, rd.take((size_t)L * d), (size_t)L * d));
    bw.cls = nullptr;
    if (c.n_classes > 0) TF_TRY(upload_f32(m, &bw.cls, rd.take((size_t)c.n_classes * d), (size_t)c.n_classes * d));
    bw.layers.resize(c.n_layers);
    for (LayerW& lw : bw.layers) {
      TF_TRY(upload_f32(m, &lw.ln1_g, rd.take(d), d));
      TF_TRY(upload_f32(m, &lw.ln1_b, rd.take(d), d));
      TF_TRY(upload_matrix(m, &lw.w_qkv, rd.take((size_t)3 * d * d), 3 * d, d, staging));
      TF_TRY(upload_f32(m, &lw.b_qkv, rd.take(3 * d), 3 * d));
      TF_TRY(upload_matrix(m, &lw.w_o, rd.take((size_t)d * d), d, d, staging));
      TF_TRY(upload_f32(m, &lw.b_o, rd.take(d), d));
      TF_TRY(upload_f32(m, &lw.ln2_g, rd.take(d), d));
      TF_TRY(upload_f32(m, &lw.ln2_b, rd.take(d), d));
      TF_TRY(upload_matrix(m, &lw.w_1, rd.take((size_t)hid * d), hid, d, staging));
      TF_TRY(upload_f32(m, &lw.b_1, rd.take(hid), hid));
      TF_TRY(upload_matrix(m, &lw.w_2, rd.take((size_t)d * hid), d, hid, staging));
      TF_TRY(upload_f32(m, &lw.b_2, rd.take(d), d));
    }
    TF_TRY(upload_f32(m, &bw.lnf_g, rd.take(d), d));
    TF_TRY(upload_f32(m, &bw.lnf_b, rd.take(d), d));
    // head: interleave rows so that outputs (2c, 2c+1) = (mu~_c, alpha~_c)
    const float* w_out = rd.take((size_t)2 * D * d);
    const float* b_out = rd.take((size_t)2 * D);
    tmp.resize((size_t)2 * D * d);
    std::vector<float> btmp(2 * D);
    for (int cc = 0; cc < D; ++cc) {
      memcpy(&tmp[(size_t)(2 * cc) * d], &w_out[(size_t)cc * d], d * sizeof(float));
      memcpy(&tmp[(size_t)(2 * cc + 1) * d], &w_out[(size_t)(D + cc) * d], d * sizeof(float));
      btmp[2 * cc] = b_out[cc];
      btmp[2 * cc + 1] = b_out[D + cc];
    }
    TF_TRY(upload_matrix(m, &bw.w_out, tmp.data(), 2 * D, d, staging));
    TF_TRY(upload_f32(m, &bw.b_out, btmp.data(), btmp.size()));
  }

  // workspace
  const size_t B = c.max_batch, M = B * L, esz = c.dtype == 1 ? 2 : 4;
  TF_TRY(dev_alloc(m, &m->seq_a, M * D));
  TF_TRY(dev_alloc(m, &m->seq_b, M * D));
  TF_TRY(dev_alloc(m, &m->cmp_v, M * D));
  TF_TRY(dev_alloc(m, &m->cmp_u, M * D));
  TF_TRY(dev_alloc(m, &m->ref_seq, M * D));
  TF_TRY(dev_alloc(m, &m->cmp_labels, B));
  TF_TRY(dev_alloc(m, &m->h, M * d));
  TF_TRY(dev_alloc(m, &m->o, M * 2 * D));
  TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->xn), M * d * esz));
  TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->qkv), M * 3 * d * esz));
  TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->att), M * d * esz));
  TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->mlp), M * hid * esz));
  TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->kcache), (size_t)c.n_layers * M * d * esz));
  TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->vcache), (size_t)c.n_layers * M * d * esz));
  if (c.dtype == 1) {
    TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->xn_lo), M * d * esz));
    TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->qkv_lo), M * 3 * d * esz));
    TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->att_lo), M * d * esz));
    TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->mlp_lo), M * hid * esz));
  }
  TF_TRY(dev_alloc(m, &m->maxdiff, B));
  TF_TRY(dev_alloc(m, &m->idx, B));
  TF_TRY(dev_alloc(m, &m->idx_tmp, B));
  TF_TRY(dev_alloc(m, &m->phase, B));
  if (B > (size_t)FIN_CHUNK) {
    const size_t nblk = (B + FIN_CHUNK - 1) / FIN_CHUNK;
    TF_TRY(dev_alloc(m, &m->fin_code, B));
    TF_TRY(dev_alloc(m, &m->fin_cnt, 2 * nblk));
    TF_TRY(dev_alloc(m, &m->fin_top, nblk));
    TF_TRY(dev_alloc(m, &m->fin_flag, nblk));
  }
  TF_TRY(dev_alloc(m, &m->ctrl, CTRL_WORDS));
  TF_TRY(dev_alloc(m, &m->err, 1));
  TF_TRY(dev_alloc(m, &m->iters_sample, (size_t)c.n_blocks * B));
  TF_TRY(dev_alloc(m, &m->io_z, B * c.C * c.H * c.W));
  TF_TRY(dev_alloc(m, &m->io_x, B * c.C * c.H * c.W));
  TF_TRY(dev_alloc(m, &m->io_labels, B));
  TF_TRY(dev_alloc(m, &m->labels_own, B));
  TF_TRY(dev_alloc(m, &m->step_ctr, 16 * tf_model::MAX_CHAINS));  // one counter per chain, 64 bytes apart
  if (c.dtype == 1) {  // partial tiles: up to 16 K slices of a [B, d] output, or d/256 slices of the widest one
    const size_t wide = (size_t)(hid > 3 * d ? hid : 3 * d);
    m->seq_part_row_floats = (size_t)16 * d;
    const size_t per_wide = (size_t)(d / 64 < 16 ? d / 64 : 16) * wide;
    if (per_wide > m->seq_part_row_floats) m->seq_part_row_floats = per_wide;
    m->seq_part_floats = m->seq_part_row_floats * B;
    TF_TRY(dev_alloc(m, &m->seq_part, m->seq_part_floats));
  }
  CU_OK(cudaMemset(m->step_ctr, 0, 16 * tf_model::MAX_CHAINS * sizeof(int)));
  CU_OK(cudaMemset(m->ctrl, 0, CTRL_WORDS * sizeof(int)));
  CU_OK(cudaMemset(m->err, 0, sizeof(int)));
  CU_OK(cudaMemset(m->iters_sample, 0, (size_t)c.n_blocks * B * sizeof(int)));
  CU_OK(cudaMallocHost(&m->ctrl_host, 8 * sizeof(int)));
  m->block_ev.assign(c.n_blocks + 1, nullptr);
  for (auto& e : m->block_ev) CU_OK(cudaEventCreate(&e));
  if (c.dtype == 1) {
    TF_TRY(make_map_bf16(&m->map_xn, m->xn, M, d, tc::BM));
    TF_TRY(make_map_bf16(&m->map_att, m->att, M, d, tc::BM));
    TF_TRY(make_map_bf16(&m->map_mlp, m->mlp, M, hid, tc::BM));
    TF_TRY(make_map_bf16(&m->map_xn_lo, m->xn_lo, M, d, tc::BM));
    TF_TRY(make_map_bf16(&m->map_att_lo, m->att_lo, M, d, tc::BM));
    TF_TRY(make_map_bf16(&m->map_mlp_lo, m->mlp_lo, M, hid, tc::BM));
    {
      CUtensorMap sm[tf_model::SM_COUNT];
      TF_TRY(make_map_store(&sm[tf_model::SM_QKV], m->qkv, M, 3 * d, 2));
      TF_TRY(make_map_store(&sm[tf_model::SM_QKV_LO], m->qkv_lo, M, 3 * d, 2));
      TF_TRY(make_map_store(&sm[tf_model::SM_MLP], m->mlp, M, hid, 2));
      TF_TRY(make_map_store(&sm[tf_model::SM_MLP_LO], m->mlp_lo, M, hid, 2));
      TF_TRY(make_map_store(&sm[tf_model::SM_H], m->h, M, d, 4));
      if (const char* e = getenv("TARFLOW_SMALL_M_ROWS")) m->small_m_rows = atoi(e);
      if (const char* e = getenv("TARFLOW_SPLIT_M_ROWS")) m->split_m_rows = atoi(e);
      if (const char* e = getenv("TARFLOW_SMALL_M_SPLIT")) m->small_m_split = atoi(e) != 0;
      if ((m->small_m_rows > 0 || m->split_m_rows > 0) && d % 128 == 0) {
        m->part_cap_rows = 8192;
        TF_TRY(dev_alloc(m, &m->sweep_part, (size_t)m->part_cap_rows * d));
        TF_TRY(make_map_store(&sm[tf_model::SM_PART], m->sweep_part, (uint64_t)m->part_cap_rows, d, 4));
        m->part_head_npad = (2 * m->D + 31) / 32 * 32;
        m->part_head_rows = (int)((size_t)m->part_cap_rows * d / m->part_head_npad);
        TF_TRY(make_map_store(&sm[tf_model::SM_PART_HEAD], m->sweep_part, (uint64_t)m->part_head_rows, m->part_head_npad, 4));
      } else {
        sm[tf_model::SM_PART] = sm[tf_model::SM_H];
        sm[tf_model::SM_PART_HEAD] = sm[tf_model::SM_H];
      }
      TF_TRY(make_map_3d(&sm[tf_model::SM_ATT3], m->att, B, L, d, 32));
      TF_TRY(make_map_3d(&m->map_qkv3, m->qkv, B, L, 3 * (uint64_t)d, attn_tc::BQ));
      TF_TRY(make_map_3d(&m->map_kv3, m->qkv, B, L, 3 * (uint64_t)d, attn_tc::BKV));
      TF_TRY(make_map_3d(&sm[tf_model::SM_ATT3_LO], m->att_lo, B, L, d, 32));
      TF_TRY(make_map_3d(&m->map_qkv3_lo, m->qkv_lo, B, L, 3 * (uint64_t)d, attn_tc::BQ));
      TF_TRY(make_map_3d(&m->map_kv3_lo, m->qkv_lo, B, L, 3 * (uint64_t)d, attn_tc::BKV));
      CU_OK(cudaFuncSetAttribute(attn_tc::attention_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 attn_tc::Cfg<false>::SMEM_BYTES));
      CU_OK(cudaFuncSetAttribute(attn_tc::attention_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 attn_tc::Cfg<true>::SMEM_BYTES));
      if (const char* e = getenv("TARFLOW_ATTN_TC_SPLIT")) m->use_tc_attention_split = atoi(e) != 0;
      if (const char* e = getenv("TARFLOW_ATTN_TC")) m->use_tc_attention = atoi(e) != 0;
      TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->store_maps), sizeof(sm)));
      CU_OK(cudaMemcpy(m->store_maps, sm, sizeof(sm), cudaMemcpyHostToDevice));
    }
    for (int r = 0; r < 3; ++r) {
      const uint32_t rt = 16u << r;
      TF_TRY(make_map_bf16(&m->map_seq_a[0][r], m->xn, M, d, rt));
      TF_TRY(make_map_bf16(&m->map_seq_a[1][r], m->att, M, d, rt));
      TF_TRY(make_map_bf16(&m->map_seq_a[2][r], m->mlp, M, hid, rt));
    }
    CU_OK(cudaFuncSetAttribute(seq::seq_gemm_tc_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, seq::gemm_tc_smem_bytes<16>()));
    CU_OK(cudaFuncSetAttribute(seq::seq_gemm_tc_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, seq::gemm_tc_smem_bytes<32>()));
    CU_OK(cudaFuncSetAttribute(seq::seq_gemm_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, seq::gemm_tc_smem_bytes<64>()));
    if (const char* e = getenv("TARFLOW_SEQ_MMA")) m->seq_use_tc = atoi(e) == 0;
    if (const char* e = getenv("TARFLOW_SEQ_FUSE_GELU")) m->seq_fuse_gelu = atoi(e) != 0;
    if (const char* e = getenv("TARFLOW_SEQ_FUSE_TAIL")) m->seq_fuse_tail = atoi(e) != 0;
    CU_OK(cudaFuncSetAttribute(seq::seq_gemm_tc_kernel<64, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, seq::gemm_tc_smem_bytes<64, 8>()));
    CU_OK(cudaFuncSetAttribute(seq::seq_gemm_tc_kernel<32, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, seq::gemm_tc_smem_bytes<32, 8>()));
    CU_OK(cudaFuncSetAttribute(seq::seq_gemm_tc_kernel<16, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, seq::gemm_tc_smem_bytes<16, 8>()));
    if (const char* e = getenv("TARFLOW_SEQ_KBN8")) m->seq_kbn8 = atoi(e) != 0;
    if (const char* e = getenv("TARFLOW_PAIR_GEMM")) m->use_pair_gemm = atoi(e) != 0;
    CU_OK(cudaFuncSetAttribute(attn::attention_mma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               attn::smem_bytes<true>()));
    CU_OK(cudaFuncSetAttribute(attn::attention_mma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               attn::smem_bytes<false>()));
    const int gsm = seq::gemm_smem_bytes(seq::KC);
    CU_OK(cudaFuncSetAttribute(seq::seq_gemm_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, gsm));
    CU_OK(cudaFuncSetAttribute(seq::seq_gemm_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, gsm));
    CU_OK(cudaFuncSetAttribute(seq::seq_gemm_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, gsm));
    CU_OK(cudaFuncSetAttribute(seq::seq_gemm_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, gsm));
    CU_OK(cudaStreamCreateWithFlags(&m->cap_stream, cudaStreamNonBlocking));
    for (int c = 0; c < tf_model::MAX_CHAINS; ++c) {
      CU_OK(cudaStreamCreateWithFlags(&m->seq_streams[c], cudaStreamNonBlocking));
      CU_OK(cudaEventCreateWithFlags(&m->seq_join[c], cudaEventDisableTiming));
    }
    CU_OK(cudaEventCreateWithFlags(&m->seq_fork, cudaEventDisableTiming));
    if (const char* e = getenv("TARFLOW_SEQ_CHAINS")) m->seq_chains_force = atoi(e);
    if (const char* e = getenv("TARFLOW_SEQ_KBN")) m->seq_kbn_force = atoi(e);
    if (const char* e = getenv("TARFLOW_SEQ_FIN")) m->seq_fin = atoi(e) != 0;
    if (const char* e = getenv("TARFLOW_SEQ_ATTN_THREADS")) m->seq_attn_threads = atoi(e);
    TF_TRY(dev_alloc(m, &m->seq_tickets, (size_t)tf_model::MAX_CHAINS * tf_model::SEQ_TICKETS));
    CU_OK(cudaMemset(m->seq_tickets, 0, (size_t)tf_model::MAX_CHAINS * tf_model::SEQ_TICKETS * sizeof(int)));
    TF_TRY(dev_alloc(m, &m->seq_stats, (size_t)tf_model::MAX_CHAINS * 16 * B));
    if (const char* e = getenv("TARFLOW_SWEEP_GRAPH_ROWS")) m->sweep_graph_rows = atoll(e);
    if (const char* e = getenv("TARFLOW_GRAPHS")) m->use_graphs = atoi(e) != 0;
  }
  CU_OK(cudaDeviceSynchronize());
  return TF_OK;
}

// ---- loading an MLP-based flow: masks and the layer permutation are applied to the weights here ----------------
// Degrees (MADE): input i has degree i + 1, hidden unit j of either hidden layer 1 + (j mod (D - 1)), output i degree
// i + 1.  A hidden unit keeps the weights from inputs / hidden units of degree <= its own, an output those from
// hidden units of degree < its own.  Odd layers act on the reversed dimension order: their first matrix gets its
// columns reversed and their output matrix / bias their rows, so the kernels work in the sample's own order.
static int maf_load_impl(tf_model* m, const void* blob, size_t nbytes, int D, int H) {
  const tf_config& c = m->cfg;
  const size_t per_block = (size_t)H * D + H + (size_t)H * H + H + (size_t)2 * D * H + 2 * D;
  const size_t want = 64 + 4 * per_block * c.n_blocks;
  if (nbytes != want) return fail(TF_ESIZE, "weight blob is %zu bytes, configuration needs %zu", nbytes, want);
  const int32_t* hdr = reinterpret_cast<const int32_t*>(blob);
  const int32_t expect[6] = {0x3146414D, 1, D, H, c.n_blocks, c.dtype};
  for (int i = 0; i < 6; ++i)
    if (hdr[i] != expect[i]) return fail(TF_ESIZE, "weight blob header field %d is %d, expected %d", i, hdr[i], expect[i]);
  int dev = 0;
  CU_OK(cudaGetDevice(&dev));
  CU_OK(cudaDeviceGetAttribute(&m->num_sms, cudaDevAttrMultiProcessorCount, dev));
  float* staging = nullptr;
  size_t max_mat = (size_t)H * H;
  if ((size_t)2 * D * H > max_mat) max_mat = (size_t)2 * D * H;
  if (c.dtype == 1) CU_OK(cudaMalloc(&staging, max_mat * sizeof(float)));
  struct Guard { float* p; ~Guard() { if (p) cudaFree(p); } } guard{staging};

  auto deg_hidden = [&](int j) { return 1 + j % (D > 1 ? D - 1 : 1); };
  BlobReader rd{reinterpret_cast<const float*>(reinterpret_cast<const char*>(blob) + 64), nullptr};
  m->maf_blocks.resize(c.n_blocks);
  std::vector<float> tmp, btmp(2 * D);
  for (int g = 0; g < c.n_blocks; ++g) {
    tf_model::MafBlock& bw = m->maf_blocks[g];
    const bool rev = (g & 1) != 0;
    const float* w1 = rd.take((size_t)H * D);
    tmp.assign((size_t)H * D, 0.f);
    for (int j = 0; j < H; ++j)
      for (int i = 0; i < D; ++i)
        if (deg_hidden(j) >= i + 1) tmp[(size_t)j * D + (rev ? D - 1 - i : i)] = w1[(size_t)j * D + i];
    TF_TRY(upload_matrix(m, &bw.w1, tmp.data(), H, D, staging));
    TF_TRY(upload_f32(m, &bw.b1, rd.take(H), H));
    const float* w2 = rd.take((size_t)H * H);
    tmp.assign((size_t)H * H, 0.f);
    for (int j = 0; j < H; ++j)
      for (int i = 0; i < H; ++i)
        if (deg_hidden(j) >= deg_hidden(i)) tmp[(size_t)j * H + i] = w2[(size_t)j * H + i];
    TF_TRY(upload_matrix(m, &bw.w2, tmp.data(), H, H, staging));
    TF_TRY(upload_f32(m, &bw.b2, rd.take(H), H));
    // output layer [mu | alpha] -> interleaved rows (2 i, 2 i + 1) = (mu_i, alpha_i) in the sample's own order
    const float* w3 = rd.take((size_t)2 * D * H);
    const float* b3 = rd.take((size_t)2 * D);
    tmp.assign((size_t)2 * D * H, 0.f);
    for (int i = 0; i < D; ++i) {
      const int r = rev ? D - 1 - i : i;  // position of the layer's dimension i in the sample's order
      for (int j = 0; j < H; ++j)
        if (i + 1 > deg_hidden(j)) {
          tmp[(size_t)(2 * r) * H + j] = w3[(size_t)i * H + j];
          tmp[(size_t)(2 * r + 1) * H + j] = w3[(size_t)(D + i) * H + j];
        }
      btmp[2 * r] = b3[i];
      btmp[2 * r + 1] = b3[D + i];
    }
    TF_TRY(upload_matrix(m, &bw.w3, tmp.data(), 2 * D, H, staging));
    TF_TRY(upload_f32(m, &bw.b3, btmp.data(), btmp.size()));
  }

  const size_t B = c.max_batch, esz = c.dtype == 1 ? 2 : 4;
  TF_TRY(dev_alloc(m, &m->seq_a, B * D));
  TF_TRY(dev_alloc(m, &m->seq_b, B * D));
  TF_TRY(dev_alloc(m, &m->o, B * 2 * D));
  TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->maf_a0), B * D * esz));
  TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->maf_a0_lo), B * D * esz));
  TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->maf_h1), B * H * esz));
  TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->maf_h1_lo), B * H * esz));
  TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->maf_h2), B * H * esz));
  TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->maf_h2_lo), B * H * esz));
  TF_TRY(dev_alloc(m, &m->maxdiff, B));
  TF_TRY(dev_alloc(m, &m->idx, B));
  TF_TRY(dev_alloc(m, &m->idx_tmp, B));
  TF_TRY(dev_alloc(m, &m->phase, B));
  if (B > (size_t)FIN_CHUNK) {
    const size_t nblk = (B + FIN_CHUNK - 1) / FIN_CHUNK;
    TF_TRY(dev_alloc(m, &m->fin_code, B));
    TF_TRY(dev_alloc(m, &m->fin_cnt, 2 * nblk));
    TF_TRY(dev_alloc(m, &m->fin_top, nblk));
    TF_TRY(dev_alloc(m, &m->fin_flag, nblk));
  }
  TF_TRY(dev_alloc(m, &m->ctrl, CTRL_WORDS));
  TF_TRY(dev_alloc(m, &m->err, 1));
  TF_TRY(dev_alloc(m, &m->iters_sample, (size_t)c.n_blocks * B));
  CU_OK(cudaMemset(m->ctrl, 0, CTRL_WORDS * sizeof(int)));
  CU_OK(cudaMemset(m->err, 0, sizeof(int)));
  CU_OK(cudaMemset(m->maxdiff, 0, B * sizeof(float)));
  CU_OK(cudaMemset(m->iters_sample, 0, (size_t)c.n_blocks * B * sizeof(int)));
  CU_OK(cudaMallocHost(&m->ctrl_host, 8 * sizeof(int)));
  m->block_ev.assign(c.n_blocks + 1, nullptr);
  for (auto& e : m->block_ev) CU_OK(cudaEventCreate(&e));
  if (c.dtype == 1) {
    void* bufs[3][2] = {{m->maf_a0, m->maf_a0_lo}, {m->maf_h1, m->maf_h1_lo}, {m->maf_h2, m->maf_h2_lo}};
    const int cols[3] = {D, H, H};
    for (int i = 0; i < 3; ++i)
      for (int t = 0; t < 2; ++t) TF_TRY(make_map_bf16(&m->maf_map[i][t], bufs[i][t], B, cols[i], tc::BM));
    CUtensorMap sm[5];
    TF_TRY(make_map_store(&sm[4], m->o, B, 2 * (uint64_t)D, 4));
    TF_TRY(make_map_store(&sm[0], m->maf_h1, B, H, 2));
    TF_TRY(make_map_store(&sm[1], m->maf_h1_lo, B, H, 2));
    TF_TRY(make_map_store(&sm[2], m->maf_h2, B, H, 2));
    TF_TRY(make_map_store(&sm[3], m->maf_h2_lo, B, H, 2));
    TF_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->maf_store_maps), sizeof(sm)));
    CU_OK(cudaMemcpy(m->maf_store_maps, sm, sizeof(sm), cudaMemcpyHostToDevice));
    if (const char* e = getenv("TARFLOW_PAIR_GEMM")) m->use_pair_gemm = atoi(e) != 0;
    if (const char* e = getenv("TARFLOW_SWEEP_GRAPH_ROWS")) m->sweep_graph_rows = atoll(e);
    CU_OK(cudaStreamCreateWithFlags(&m->cap_stream, cudaStreamNonBlocking));
  }
  CU_OK(cudaDeviceSynchronize());
  return TF_OK;
}

static int check_call(tf_model* m, int B, bool want_maf = false) {
  if (!m) return fail(TF_EINVAL, "model is NULL");
  if (m->is_maf != want_maf)
    return fail(TF_EINVAL, want_maf ? "this call needs a model loaded with tf_maf_load" : "this call needs a model loaded with tf_load");
  if (B < 1 || B > m->cfg.max_batch) return fail(TF_EINVAL, "B=%d outside [1, max_batch=%d]", B, m->cfg.max_batch);
  return TF_OK;
}

// ------------------------------------------------------------------------------------------------
// C ABI
// ------------------------------------------------------------------------------------------------
extern "C" {

const char* tf_last_error(void) { return g_err; }

int tf_load(const tf_config* cfg, const void* weights_host, size_t nbytes, tf_model** out) {
  g_err[0] = 0;
  if (!cfg || !weights_host || !out) return fail(TF_EINVAL, "NULL argument");
  *out = nullptr;
  const tf_config& c = *cfg;
  if (c.C < 1 || c.H < 1 || c.W < 1 || c.patch < 1 || c.H % c.patch || c.W % c.patch)
    return fail(TF_EINVAL, "image %dx%dx%d not divisible by patch %d", c.C, c.H, c.W, c.patch);
  if (c.n_blocks < 1 || c.n_layers < 1 || c.width < 4 || c.n_heads < 1 || c.width % c.n_heads || c.width % 4 ||
      c.mlp_ratio < 1 || c.n_classes < 0 || c.max_batch < 1)
    return fail(TF_EINVAL, "bad model dimensions");
  if (c.dtype != 0 && c.dtype != 1) return fail(TF_EINVAL, "dtype must be 0 (fp32) or 1 (bf16)");
  if (c.dtype == 1 && (c.width % 64 || c.width / c.n_heads != 64))
    return fail(TF_EINVAL, "bf16 engine needs width %% 64 == 0 and head_dim == 64");
  if (c.width > 2048) return fail(TF_EINVAL, "width > 2048 not supported");
  if (c.dtype == 1 && c.width > 1024) return fail(TF_EINVAL, "bf16 engine: width > 1024 not supported");
  tf_model* m = new (std::nothrow) tf_model();
  if (!m) return fail(TF_ENOMEM, "host allocation failed");
  m->cfg = c;
  m->L = (c.H / c.patch) * (c.W / c.patch);
  m->D = c.C * c.patch * c.patch;
  m->d = c.width;
  m->hid = c.mlp_ratio * c.width;
  m->hd = c.width / c.n_heads;
  if (m->L < 2) { delete m; return fail(TF_EINVAL, "need at least 2 tokens"); }
  int r = load_impl(m, weights_host, nbytes);
  if (r != TF_OK) {
    tf_free(m);
    return r;
  }
  *out = m;
  return TF_OK;
}

void tf_free(tf_model* m) {
  if (!m) return;
  cudaDeviceSynchronize();
  m->prof_collect();
  for (cudaEvent_t e : m->ev_pool) cudaEventDestroy(e);
  for (cudaEvent_t e : m->block_ev) if (e) cudaEventDestroy(e);
  for (auto& kv : m->seq_graphs) if (kv.second.exec) cudaGraphExecDestroy(kv.second.exec);
  for (auto& kv : m->sweep_graphs) if (kv.second.exec) cudaGraphExecDestroy(kv.second.exec);
  if (m->cap_stream) cudaStreamDestroy(m->cap_stream);
  for (int c = 0; c < tf_model::MAX_CHAINS; ++c) {
    if (m->seq_streams[c]) cudaStreamDestroy(m->seq_streams[c]);
    if (m->seq_join[c]) cudaEventDestroy(m->seq_join[c]);
  }
  if (m->seq_fork) cudaEventDestroy(m->seq_fork);
  for (void* p : m->allocs) cudaFree(p);
  if (m->guards_dev) cudaFree(m->guards_dev);
  if (m->guard_count) cudaFree(m->guard_count);
  if (m->ctrl_host) cudaFreeHost(m->ctrl_host);
  delete m;
}

int tf_forward(tf_model* m, const float* x_dev, const int32_t* labels_dev, int32_t B, float* z_dev, float* logdet_dev,
               void* cuda_stream) {
  g_err[0] = 0;
  TF_TRY(check_call(m, B));
  if (!x_dev || !z_dev) return fail(TF_EINVAL, "NULL buffer");
  if (m->cfg.n_classes > 0 && !labels_dev) return fail(TF_EINVAL, "class-conditional model needs labels");
  m->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  return m->cfg.dtype == 1 ? forward_impl<bf16>(m, x_dev, labels_dev, B, z_dev, logdet_dev)
                           : forward_impl<float>(m, x_dev, labels_dev, B, z_dev, logdet_dev);
}

static int inverse_checked(tf_model* m, const float* z_dev, const int32_t* labels_dev, int32_t B, const uint8_t* policy_host,
                           float tau, int32_t max_iters, const InvOpts& op, float* x_dev, int32_t* iters_block_host,
                           int32_t* iters_sample_dev, void* cuda_stream) {
  TF_TRY(check_call(m, B));
  if (!z_dev || !x_dev || !policy_host) return fail(TF_EINVAL, "NULL buffer");
  if (m->cfg.n_classes > 0 && !labels_dev) return fail(TF_EINVAL, "class-conditional model needs labels");
  if (max_iters < 1) return fail(TF_EINVAL, "max_iters must be >= 1");
  if (op.init_mode < 0 || op.init_mode > 2) return fail(TF_EINVAL, "init_mode must be 0, 1 or 2");
  if (op.init_mode == 2 && !op.u0_img) return fail(TF_EINVAL, "init_mode 2 needs u0_dev");
  if (op.fallback_sweeps < 0) return fail(TF_EINVAL, "fallback_sweeps must be >= 0");
  if (tau != tau) return fail(TF_EINVAL, "tau is NaN");
  for (int g = 0; g < m->cfg.n_blocks; ++g) {
    if (policy_host[g] > 1) return fail(TF_EINVAL, "policy[%d]=%d is neither 0 nor 1", g, (int)policy_host[g]);
    if (op.tau_block && op.tau_block[g] != op.tau_block[g]) return fail(TF_EINVAL, "tau_block[%d] is NaN", g);
  }
  m->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  return m->cfg.dtype == 1 ? inverse_impl<bf16>(m, z_dev, labels_dev, B, policy_host, tau, max_iters, op, x_dev,
                                                iters_block_host, iters_sample_dev)
                           : inverse_impl<float>(m, z_dev, labels_dev, B, policy_host, tau, max_iters, op, x_dev,
                                                 iters_block_host, iters_sample_dev);
}

int tf_inverse_jacobi(tf_model* m, const float* z_dev, const int32_t* labels_dev, int32_t B, const uint8_t* policy_host,
                      float tau, int32_t max_iters, int32_t init_mode, float* x_dev, int32_t* iters_block_host,
                      int32_t* iters_sample_dev, void* cuda_stream) {
  g_err[0] = 0;
  if (init_mode != 0 && init_mode != 1) return fail(TF_EINVAL, "init_mode must be 0 or 1");
  InvOpts op;
  op.init_mode = init_mode;
  return inverse_checked(m, z_dev, labels_dev, B, policy_host, tau, max_iters, op, x_dev, iters_block_host, iters_sample_dev,
                         cuda_stream);
}

int tf_inverse_jacobi_ex(tf_model* m, const float* z_dev, const int32_t* labels_dev, int32_t B, const uint8_t* policy_host,
                         float tau, int32_t max_iters, const tf_jacobi_opts* opts, float* x_dev, int32_t* iters_block_host,
                         int32_t* iters_sample_dev, void* cuda_stream) {
  g_err[0] = 0;
  InvOpts op;
  if (opts) {
    if (opts->struct_bytes != (int32_t)sizeof(tf_jacobi_opts)) return fail(TF_EINVAL, "tf_jacobi_opts.struct_bytes is %d, expected %d", opts->struct_bytes, (int)sizeof(tf_jacobi_opts));
    op.init_mode = opts->init_mode;
    op.u0_img = opts->u0_dev;
    op.tau_block = opts->tau_block_host;
    op.fallback_sweeps = opts->fallback_sweeps;
    op.states_img = opts->states_dev;
    op.ref_img = opts->ref_states_dev;
  }
  return inverse_checked(m, z_dev, labels_dev, B, policy_host, tau, max_iters, op, x_dev, iters_block_host, iters_sample_dev,
                         cuda_stream);
}

int tf_block_times(tf_model* m, float* ms_host, int32_t cap) {
  if (!m) return fail(TF_EINVAL, "model is NULL");
  const int K = m->cfg.n_blocks;
  if (!m->block_ev_valid) return 0;
  for (int g = 0; g < K && g < cap; ++g) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, m->block_ev[g], m->block_ev[g + 1]) != cudaSuccess) { cudaGetLastError(); return 0; }
    if (ms_host) ms_host[g] = ms;
  }
  return K;
}

int tf_inverse_sequential(tf_model* m, const float* z_dev, const int32_t* labels_dev, int32_t B, float* x_dev,
                          void* cuda_stream) {
  if (!m) return fail(TF_EINVAL, "model is NULL");
  std::vector<uint8_t> policy(m->cfg.n_blocks, 0);
  return tf_inverse_jacobi(m, z_dev, labels_dev, B, policy.data(), 0.f, 1, 0, x_dev, nullptr, nullptr, cuda_stream);
}

int tf_inverse_jacobi_host(tf_model* m, const float* z_host, const int32_t* labels_host, int32_t B,
                           const uint8_t* policy_host, float tau, int32_t max_iters, int32_t init_mode, float* x_host,
                           int32_t* iters_block_host, int32_t* iters_sample_host, void* cuda_stream) {
  g_err[0] = 0;
  TF_TRY(check_call(m, B));
  if (!z_host || !x_host) return fail(TF_EINVAL, "NULL buffer");
  if (m->cfg.n_classes > 0 && !labels_host) return fail(TF_EINVAL, "class-conditional model needs labels");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  size_t n = (size_t)B * m->cfg.C * m->cfg.H * m->cfg.W;
  CU_OK(cudaMemcpyAsync(m->io_z, z_host, n * sizeof(float), cudaMemcpyHostToDevice, st));
  if (labels_host) CU_OK(cudaMemcpyAsync(m->io_labels, labels_host, B * sizeof(int), cudaMemcpyHostToDevice, st));
  int r = tf_inverse_jacobi(m, m->io_z, labels_host ? m->io_labels : nullptr, B, policy_host, tau, max_iters, init_mode,
                            m->io_x, iters_block_host, nullptr, cuda_stream);
  if (r < 0) return r;
  CU_OK(cudaMemcpyAsync(x_host, m->io_x, n * sizeof(float), cudaMemcpyDeviceToHost, st));
  if (iters_sample_host)
    for (int g = 0; g < m->cfg.n_blocks; ++g)
      CU_OK(cudaMemcpyAsync(iters_sample_host + (size_t)g * B, m->iters_sample + (size_t)g * m->cfg.max_batch,
                            B * sizeof(int), cudaMemcpyDeviceToHost, st));
  CU_OK(cudaStreamSynchronize(st));
  return r;
}

int tf_maf_load(const tf_maf_config* cfg, const void* weights_host, size_t nbytes, tf_model** out) {
  g_err[0] = 0;
  if (!cfg || !weights_host || !out) return fail(TF_EINVAL, "NULL argument");
  *out = nullptr;
  if (cfg->D < 2 || cfg->hidden < 1 || cfg->n_blocks < 1 || cfg->max_batch < 1) return fail(TF_EINVAL, "bad model dimensions");
  if (cfg->dtype != 0 && cfg->dtype != 1) return fail(TF_EINVAL, "dtype must be 0 (fp32) or 1 (bf16)");
  if (cfg->dtype == 1 && (cfg->D % 8 || cfg->hidden % 64))
    return fail(TF_EINVAL, "bf16 engine needs D %% 8 == 0 and hidden %% 64 == 0");
  tf_model* m = new (std::nothrow) tf_model();
  if (!m) return fail(TF_ENOMEM, "host allocation failed");
  m->is_maf = true;
  m->small_m_rows = m->split_m_rows = 0;  // the MLP flow keeps one tile shape from 256 rows up: results do not depend on the batch
  m->cfg = tf_config{1, cfg->D, 1, 1, cfg->n_blocks, 2, cfg->hidden, 1, 1, 0, cfg->dtype, cfg->max_batch};
  m->L = cfg->D;  // D values per sample, token dimension 1
  m->D = 1;
  m->d = m->hid = m->maf_H = cfg->hidden;
  m->hd = cfg->hidden;
  int r = maf_load_impl(m, weights_host, nbytes, cfg->D, cfg->hidden);
  if (r != TF_OK) {
    tf_free(m);
    return r;
  }
  *out = m;
  return TF_OK;
}

int tf_maf_forward(tf_model* m, const float* x_dev, int32_t B, float* z_dev, float* logdet_dev, void* cuda_stream) {
  g_err[0] = 0;
  TF_TRY(check_call(m, B, true));
  if (!x_dev || !z_dev) return fail(TF_EINVAL, "NULL buffer");
  m->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  return m->cfg.dtype == 1 ? maf_forward_impl<bf16>(m, x_dev, B, z_dev, logdet_dev) : maf_forward_impl<float>(m, x_dev, B, z_dev, logdet_dev);
}

int tf_maf_inverse_sequential(tf_model* m, const float* z_dev, int32_t B, float* x_dev, void* cuda_stream) {
  g_err[0] = 0;
  TF_TRY(check_call(m, B, true));
  if (!z_dev || !x_dev) return fail(TF_EINVAL, "NULL buffer");
  m->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  return m->cfg.dtype == 1 ? maf_inverse_impl<bf16>(m, z_dev, B, false, 0.f, 1, 0, x_dev, nullptr, nullptr)
                           : maf_inverse_impl<float>(m, z_dev, B, false, 0.f, 1, 0, x_dev, nullptr, nullptr);
}

int tf_maf_inverse_jacobi(tf_model* m, const float* z_dev, int32_t B, float tau, int32_t max_iters, int32_t init_mode,
                          float* x_dev, int32_t* iters_block_host, int32_t* iters_sample_dev, void* cuda_stream) {
  g_err[0] = 0;
  TF_TRY(check_call(m, B, true));
  if (!z_dev || !x_dev) return fail(TF_EINVAL, "NULL buffer");
  if (max_iters < 1) return fail(TF_EINVAL, "max_iters must be >= 1");
  if (init_mode != 0 && init_mode != 1) return fail(TF_EINVAL, "init_mode must be 0 or 1");
  if (tau != tau) return fail(TF_EINVAL, "tau is NaN");
  m->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  return m->cfg.dtype == 1
             ? maf_inverse_impl<bf16>(m, z_dev, B, true, tau, max_iters, init_mode, x_dev, iters_block_host, iters_sample_dev)
             : maf_inverse_impl<float>(m, z_dev, B, true, tau, max_iters, init_mode, x_dev, iters_block_host, iters_sample_dev);
}

int tf_jacobi_update(const float* o_dev, const float* v_dev, float* u_dev, float* maxdiff_dev, int32_t B, int32_t L,
                     int32_t D, int32_t reversed, void* cuda_stream) {
  g_err[0] = 0;
  if (!o_dev || !v_dev || !u_dev || !maxdiff_dev) return fail(TF_EINVAL, "NULL buffer");
  if (B < 1 || L < 2 || D < 1) return fail(TF_EINVAL, "bad sizes");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  CU_OK(cudaMemsetAsync(maxdiff_dev, 0, B * sizeof(float), st));
  size_t n = (size_t)B * L * D;
  int blocks = (int)((n + 255) / 256);
  if (blocks > 148 * 8) blocks = 148 * 8;
  jacobi_update_kernel<<<blocks, 256, 0, st>>>(o_dev, v_dev, u_dev, maxdiff_dev, nullptr, B * L, L, D, reversed, 0);
  return check_launch("jacobi_update_kernel");
}

static int* g_gemm_err[kMaxDevices] = {nullptr};  // error word of the model-less GEMM entry point (one per device)

int tf_gemm_bf16(const void* a_dev, const void* w_dev, const float* bias_dev, float* c_dev, int32_t M, int32_t N,
                 int32_t K, void* cuda_stream) {
  g_err[0] = 0;
  if (!a_dev || !w_dev || !c_dev) return fail(TF_EINVAL, "NULL buffer");
  if (M < 1 || N < 8 || K < 64 || K % 64 || N % 8) return fail(TF_EINVAL, "need M>=1, N%%8==0, K%%64==0");
  const int dev = current_device();
  if (dev < 0) return fail(TF_EINVAL, "no current device with an ordinal below %d", kMaxDevices);
  if (!g_gemm_err[dev]) {
    CU_OK(cudaMalloc(&g_gemm_err[dev], sizeof(int)));
    CU_OK(cudaMemset(g_gemm_err[dev], 0, sizeof(int)));
  }
  int sms = 148;
  CU_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int bn = (N % 256 == 0) ? 256 : 128;
  CUtensorMap ma, mw;
  TF_TRY(make_map_bf16(&ma, a_dev, M, K, tc::BM));
  TF_TRY(make_map_bf16(&mw, w_dev, N, K, bn));
  EpiStore<float, false> epi{c_dev, bias_dev, N};
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (bn == 256) return launch_gemm_tc<256, 4>(nullptr, 0, st, ma, nullptr, mw, M, N, K, epi, g_gemm_err[dev], sms, nullptr);
  return launch_gemm_tc<128, 6>(nullptr, 0, st, ma, nullptr, mw, M, N, K, epi, g_gemm_err[dev], sms, nullptr);
}

int tf_gemm_status(void* cuda_stream) {
  g_err[0] = 0;
  CU_OK(cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(cuda_stream)));
  const int dev = current_device();
  if (dev < 0 || !g_gemm_err[dev]) return TF_OK;
  int e = 0;
  CU_OK(cudaMemcpy(&e, g_gemm_err[dev], sizeof(int), cudaMemcpyDeviceToHost));
  if (e != 0) {  // reported once, then cleared: later launches run normally
    CU_OK(cudaMemset(g_gemm_err[dev], 0, sizeof(int)));
    return fail(TF_ETIMEOUT, "device-side wait expired in tf_gemm_bf16 (code %d)", e);
  }
  return TF_OK;
}

// ------------------------------------------------------------------------------------------------
// Allocation-free skinny GEMM (see tf_skinny_gemm_noalloc in tarflow.h).  The split-K partial tiles and
// the step-counter word the kernel reads live in a static device array instead of cudaMalloc'd memory.
// ------------------------------------------------------------------------------------------------
#define TF_NOALLOC_HEADER_BYTES 256u
static __device__ __align__(256) unsigned char g_noalloc_scratch[TF_NOALLOC_SCRATCH_BYTES];
static unsigned char* g_noalloc_ptr[kMaxDevices] = {nullptr};  // device address of the array, per device ordinal

// c[m, n] = bias[n] + sum over K slices of part[s][m][n], slices added in index order
__global__ void noalloc_reduce_kernel(const float* __restrict__ part, const float* __restrict__ bias,
                                      float* __restrict__ c, int nsplit, int M, int N) {
  const size_t total = (size_t)M * N;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    float acc = bias ? bias[i % N] : 0.f;
    for (int sl = 0; sl < nsplit; ++sl) acc += part[(size_t)sl * total + i];
    c[i] = acc;
  }
}

int tf_skinny_gemm_noalloc(const void* a_dev, const void* w_dev, const float* bias_dev, float* c_dev, int32_t M, int32_t N,
                           int32_t K, void* cuda_stream) {
  g_err[0] = 0;
  if (!a_dev || !w_dev || !c_dev) return fail(TF_EINVAL, "NULL buffer");
  if (M < 1 || N < 8 || N % 8 || K < 256 || K % 256) return fail(TF_EINVAL, "need M >= 1, N %% 8 == 0, K %% 256 == 0");
  // the kernel reads A and W with 16-byte accesses and the reduction reads/writes 4-byte floats: a misaligned pointer
  // would fault on the device, so it is refused here
  if ((reinterpret_cast<uintptr_t>(a_dev) | reinterpret_cast<uintptr_t>(w_dev)) & 15)
    return fail(TF_EINVAL, "tf_skinny_gemm_noalloc: a_dev and w_dev must be 16-byte aligned");
  if ((reinterpret_cast<uintptr_t>(c_dev) | reinterpret_cast<uintptr_t>(bias_dev)) & 3)
    return fail(TF_EINVAL, "tf_skinny_gemm_noalloc: c_dev and bias_dev must be 4-byte aligned");
  const int klen = 256, ksplit = K / klen;
  const size_t need = (size_t)ksplit * M * N * sizeof(float);
  if (need > (size_t)TF_NOALLOC_SCRATCH_BYTES - TF_NOALLOC_HEADER_BYTES)
    return fail(TF_EINVAL, "tf_skinny_gemm_noalloc: (K/256)*M*N*4 = %zu bytes of partial tiles exceed the %zu-byte static scratch",
                need, (size_t)TF_NOALLOC_SCRATCH_BYTES - TF_NOALLOC_HEADER_BYTES);
  const int dev = current_device();
  if (dev < 0) return fail(TF_EINVAL, "no current device with an ordinal below %d", kMaxDevices);
  using Kern = void (*)(const bf16*, const bf16*, int, int, int, int, float*, const int*, int, int, int);
  Kern kern = seq::seq_gemm_kernel<8>;
  const int smem = seq::gemm_smem_bytes(klen);
  if (!g_noalloc_ptr[dev]) {  // once per device, with that device current: resolve the symbol to a device address
    unsigned char* p = nullptr;
    CU_OK(cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_noalloc_scratch));
    // the same limit tf_load sets for this kernel, so a model loaded earlier keeps its larger K slices
    CU_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, seq::gemm_smem_bytes(seq::KC)));
    g_noalloc_ptr[dev] = p;
  }
  unsigned char* base = g_noalloc_ptr[dev];
  int* step_word = reinterpret_cast<int*>(base);
  float* part = reinterpret_cast<float*>(base + TF_NOALLOC_HEADER_BYTES);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  // the array keeps whatever the last call left: the step word must read 0; the tiles are fully overwritten
  CU_OK(cudaMemsetAsync(step_word, 0, sizeof(int), st));
  dim3 grid((N + 7) / 8, ksplit, (M + seq::ROWS - 1) / seq::ROWS);
  kern<<<grid, seq::THREADS, smem, st>>>(reinterpret_cast<const bf16*>(a_dev), reinterpret_cast<const bf16*>(w_dev), M, N, K,
                                         klen, part, step_word, 0, 1, 0);
  TF_TRY(check_launch("seq_gemm_kernel (no-alloc)"));
  const size_t total = (size_t)M * N;
  int blocks = (int)((total + 255) / 256);
  if (blocks > 148 * 8) blocks = 148 * 8;
  noalloc_reduce_kernel<<<blocks, 256, 0, st>>>(part, bias_dev, c_dev, ksplit, M, N);
  return check_launch("noalloc_reduce_kernel");
}

int tf_selftest_wait_timeout(tf_model* m, int32_t limit_us, void* cuda_stream) {
  g_err[0] = 0;
  if (!m) return fail(TF_EINVAL, "model is NULL");
  if (limit_us < 1 || limit_us > 1000000) return fail(TF_EINVAL, "limit_us must lie in [1, 1000000]");
  m->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  LAUNCH(m, KC_CTRL, tc::wait_selftest_kernel, 1, 32, 0, m->err, (unsigned long long)limit_us * 1000ull);
  TF_TRY(check_launch("wait_selftest_kernel"));
  return sync_check(m);
}

int64_t tf_debug_check_guards(tf_model* m, void* cuda_stream) {
  g_err[0] = 0;
  if (!m) return fail(TF_EINVAL, "model is NULL");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  const int n = (int)m->guards.size();
  if (!m->guards_dev) {  // plain cudaMalloc: these two are not themselves guarded
    CU_OK(cudaMalloc(&m->guards_dev, (size_t)n * sizeof(unsigned char*)));
    CU_OK(cudaMalloc(&m->guard_count, sizeof(int)));
    CU_OK(cudaMemcpy(m->guards_dev, m->guards.data(), (size_t)n * sizeof(unsigned char*), cudaMemcpyHostToDevice));
  }
  CU_OK(cudaMemsetAsync(m->guard_count, 0, sizeof(int), st));
  guard_check_kernel<<<n, (int)(GUARD_BYTES / 4), 0, st>>>(m->guards_dev, m->guard_count, 0x01010101u * GUARD_BYTE);
  TF_TRY(check_launch("guard_check_kernel"));
  int bad = 0;
  CU_OK(cudaMemcpyAsync(&bad, m->guard_count, sizeof(int), cudaMemcpyDeviceToHost, st));
  CU_OK(cudaStreamSynchronize(st));
  if (bad != 0) fail(TF_OK, "%d guard words next to the model's device buffers were overwritten", bad);
  return bad;
}

int tf_profile_enable(tf_model* m, int32_t on) {
  if (!m) return fail(TF_EINVAL, "model is NULL");
  cudaDeviceSynchronize();
  m->prof_collect();
  for (int c = 0; c < KC_COUNT; ++c) { m->prof_ms[c] = 0; m->prof_n[c] = 0; m->prof_rows[c] = 0; }
  m->prof_on = on != 0;
  m->prof_mode = on == 2 ? 2 : (on != 0 ? 1 : 0);
  return TF_OK;
}

int tf_profile_read(tf_model* m, const char** names, double* ms, int64_t* launches, double* rows, int32_t cap) {
  if (!m) return fail(TF_EINVAL, "model is NULL");
  m->prof_collect();
  for (int c = 0; c < KC_COUNT && c < cap; ++c) {
    if (names) names[c] = kKernelClassNames[c];
    if (ms) ms[c] = m->prof_ms[c];
    if (launches) launches[c] = m->prof_n[c];
    if (rows) rows[c] = m->prof_rows[c];
  }
  return KC_COUNT;
}

int tf_set_precision(tf_model* m, int32_t mode, float switch_threshold, float single_ok_tau) {
  if (!m) return fail(TF_EINVAL, "model is NULL");
  if (mode < 0 || mode > 2) return fail(TF_EINVAL, "precision mode must be 0, 1 or 2");
  m->precision_mode = mode;
  m->switch_threshold = switch_threshold > 0.f ? switch_threshold : 0.03125f;
  m->single_ok_tau = single_ok_tau > 0.f ? single_ok_tau : 0.015625f;
  return TF_OK;
}

int tf_trace_enable(tf_model* m, int32_t on) {
  if (!m) return fail(TF_EINVAL, "model is NULL");
  m->trace_on = on != 0;
  m->trace.clear();
  m->trace_l2_count.assign(m->cfg.n_blocks, 0);
  if (m->trace_on && !m->trace_l2) {  // distance records: up to L + 2 sweeps per block
    m->trace_l2_sweeps = m->L + 2;
    TF_TRY(dev_alloc(m, &m->trace_l2, (size_t)m->cfg.n_blocks * m->trace_l2_sweeps * m->cfg.max_batch));
  }
  return TF_OK;
}

int tf_trace_read_l2(tf_model* m, int32_t block, int32_t B, float* l2_host, int32_t cap_sweeps) {
  if (!m) return fail(TF_EINVAL, "model is NULL");
  if (block < 0 || block >= m->cfg.n_blocks || B < 1 || B > m->cfg.max_batch) return fail(TF_EINVAL, "bad block or batch");
  if (!m->trace_l2 || m->trace_l2_count.empty()) return 0;
  const int n = m->trace_l2_count[block];
  for (int t = 0; t < n && t < cap_sweeps && l2_host; ++t)
    CU_OK(cudaMemcpy(l2_host + (size_t)t * B, m->trace_l2 + ((size_t)block * m->trace_l2_sweeps + t) * m->cfg.max_batch,
                     B * sizeof(float), cudaMemcpyDeviceToHost));
  return n;
}

int tf_trace_read(tf_model* m, int32_t* block, int32_t* sweep, int32_t* active, float* maxdiff, int32_t cap) {
  if (!m) return fail(TF_EINVAL, "model is NULL");
  int n = (int)m->trace.size();
  for (int i = 0; i < n && i < cap; ++i) {
    if (block) block[i] = m->trace[i].block;
    if (sweep) sweep[i] = m->trace[i].sweep;
    if (active) active[i] = m->trace[i].active;
    if (maxdiff) maxdiff[i] = m->trace[i].maxdiff;
  }
  return n;
}

int64_t tf_launch_count(tf_model* m) { return m ? m->launches : 0; }
int64_t tf_device_bytes(tf_model* m) { return m ? m->device_bytes : 0; }

}  // extern "C"

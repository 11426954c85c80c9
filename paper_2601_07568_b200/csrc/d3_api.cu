// C ABI of the d3 library (see include/d3.h): context, weight repacking, the forward pass as a
// sequence of kernel launches on one stream, the decision kernels and the generate loop.
#include "../../include/d3.h"
#include "../../include/d3_debug.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <string>
#include <tuple>
#include <utility>
#include <vector>

#include "attention.cuh"
#include "attention_tmem.cuh"
#include "chain.cuh"
#include "common.cuh"
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "gemm_pair.cuh"
#include "gemm_xt.cuh"
#include "small_kernels.cuh"

using namespace d3;
typedef __nv_bfloat16 bf16;

// ----------------------------------------------------------------------------- context
struct d3_ctx {
  d3_config cfg{};
  cudaStream_t stream = nullptr;
  bool is_bf16 = false;
  bool use_tc = false;
  bool fuse_qkv = false;
  bool fold_norm = false;  // tensor-core path: RMSNorm lives inside the matmuls (gains in the weight columns, row factors in the epilogues)
  void* xb = nullptr;      // bf16 copy of the residual stream (fold_norm)
  float* ssq = nullptr;    // [rows][ceil(d_model / 32)] chunk sums of squares of x (fold_norm)
  bool w_tiled = false;  // model matrices stored as contiguous 128 x 64 blocks (tensor-core path)
  size_t esz = 4;
  int n_sms = 148;
  // weights (context dtype), repacked
  void* tok_emb = nullptr;
  void* lm_head = nullptr;
  float* final_norm = nullptr;
  std::vector<void*> wqkv, wo, wgu, wd;
  std::vector<float*> attn_norm, ffn_norm;
  bool weights_loaded = false, prefilled = false;
  // cache and tables
  void* kv = nullptr;
  size_t kv_layer_elems = 0;  // elements of one K (or V) plane of one layer
  float *rope_cos = nullptr, *rope_sin = nullptr;
  // workspaces
  int max_rows = 0;
  float* x = nullptr;
  void* xn = nullptr;
  float* qkv_f32 = nullptr;
  void* q = nullptr;
  void* o = nullptr;
  void* h = nullptr;
  float4* stat_part = nullptr;
  float *conf = nullptr, *ent = nullptr;
  int* argmax = nullptr;
  int *prefix_len = nullptr, *pos_base = nullptr, *n_valid = nullptr, *kv_len = nullptr;
  uint32_t* error_word = nullptr;
  // tensor-core attention (bf16, d_head 128)
  bool attn_tc = false;
  CUtensorMap kv_tmap{};
  float* partial = nullptr;
  size_t partial_slots = 0;  // capacity in (tile, split) slots of 128*128 floats
  int* tile_count = nullptr;
  int n_tile_count = 0;
  // generate state
  GenState gen{};
  MbState mb{};           // multi-block decoding state (d3_generate_multiblock)
  int stat_rows = 0;      // rows the statistics buffers hold
  long long* host_counters = nullptr;  // pinned
  // taps
  int tap_layer = -1;
  float *tap_in = nullptr, *tap_out = nullptr;
  int tap_rows = 0;
  int last_rows = 0;
  int64_t launches = 0;
  std::map<std::string, int64_t> launches_by_kernel;  // the same, per kernel name
  int64_t dev_bytes = 0;
  // per-class kernel timing (off by default)
  bool prof_on = false;
  bool pdl = true;           // programmatic dependent launch between the kernels of a forward
  int* skip_flag = nullptr;  // device flag: non-zero turns the forward's kernels into no-ops
  int tune_producers = 0;
  int tune_attn_div = 0;  // experiment: key tiles per attention split
  int tune_pair = -1;     // -1: by row count; 0 / 1: one / two row tiles per matmul unit
  int tune_no_rr = 0;     // 1: wide matmuls on contiguous unit ranges
  int eos_id = -1;        // d3_generate stops a sequence once this id has been committed (< 0: never)
  long long last_early_stops = 0;
  float4* sample_part = nullptr;  // per (row, tile) sampling partials (temperature > 0)
  float temperature = 0.f;        // 0: greedy
  unsigned long long seed = 0;
  const int* draw_step = nullptr; // device step counters of the sequences for the next forward's noise (null: draw_step_add alone)
  int draw_step_add = 1;
  int explicit_step = 0;          // d3_denoise_step calls since the last prefill / commit
  int* hist_ids = nullptr;     // [max_batch, max_seq] ids of the stored prefix of every sequence
  int* refresh_ids = nullptr;  // [max_rows] input ids of a KV-refresh forward
  int cache_delay = 1;         // multi-block decoding: stabilizing rounds before a complete block is stored
  int refresh_every = 0;       // periodic KV-refresh in the generate loops (0: never)
  long long last_refreshes = 0;
  bool gen_fuse = true;   // d3_generate fuses finalize forwards with the next block's first step while the forward stays skinny
  int tune_strip = 0;     // skinny matmuls as column strips: 0 when it pays, 1 never, 2 with one CTA per SM, 3 whenever possible
  int tune_no_cluster = 0;  // 1: skinny matmuls on the unit-range kernel (L2 reduction) instead of clusters
  int tune_wide_tiles = -1;  // -1: by row count; 0 / 1: force 128- / 256-column tiles
  int tune_ring_kb = 0, tune_ctas_per_sm = 0;  // matmul tuning overrides (0 = default)
  int tune_strip_stages = 0;  // explicit pipeline depth of the column-strip kernel (0: from the ring size)
  int tune_chain = -1;        // skinny decode matmuls as chains (chain.cuh): -1 when the shapes allow, 0 never
  int chain_clusters = -1;    // clusters of the chain kernel that are resident at once (-1: not asked yet)
  int chain_qkv_ks = 2;       // K parts of the QKV matmul inside a chain
  int tune_chain_clusters = 0;  // 0: as many clusters as fit
  int tune_chain_l2 = -1;       // weight slabs the chain's L2 prefetch runs ahead (-1: default, 0: off)
  int tune_attn_shape = 0;      // experiment: keys per tile of the tcgen05 attention (0 = by rule, 64, 128)
  int tune_attn_tmem = -1;      // tcgen05 attention: -1 where measured faster, 0 never, 1 wherever the shape allows
  const int* live_n_valid = nullptr;  // set for the span of a forward whose sequences have rows_per_seq % 256 == 0 rows
  int live_rps = 0, live_rows = 0;    // (padded prompts): the pair kernel passes over row tiles without a live row
  int tune_cta_pairs = -1;      // wide matmuls on CTA pairs (cta_group::2): -1 when the shape allows, 0 never
  int pair_clusters = 0;        // CTA pairs of gemm_pair_kernel resident at once (asked once)
  int tune_xt = -1;             // 129..256-row matmuls with weights as the 128-row operand: -1 when the shape allows, 0 never
  unsigned int* chain_sync = nullptr;  // [operators of the program] border counters of a forward's chain launches
  void* chain_prog = nullptr;          // the forward's operators (tc::ChainOp) on the device
  int chain_prog_ops = 0;
  bool chain_prog_ready = false;
  CUtensorMap kv_tmap128{};            // the cache with boxes of 128 rows (attn_tmem_kernel)
  CUtensorMap kv_tmap32{};             // the cache with boxes of 32 rows (attention inside the chain)
  unsigned long long* commit_hist = nullptr;  // [COMMIT_HIST_BINS] commits per decision of the latest generate call
  struct ProfPair { cudaEvent_t a, b; int cls; };
  std::vector<ProfPair> prof_pool;
  size_t prof_used = 0;
  double prof_ms[D3_PROF_CLASSES] = {};
  int64_t prof_n[D3_PROF_CLASSES] = {};
  std::string last_error;
  std::vector<void*> allocs;
  std::map<std::tuple<const void*, int, int, int>, CUtensorMap> tmaps;
};

namespace {

const char* kVersion = "d3-b200 0.1";

int fail(d3_ctx* c, int code, const std::string& msg) {
  if (c) c->last_error = msg;
  return code;
}
#define CUDA_TRY(c, expr)                                                                         \
  do {                                                                                            \
    cudaError_t e_ = (expr);                                                                      \
    if (e_ != cudaSuccess)                                                                        \
      return fail((c), e_ == cudaErrorMemoryAllocation ? D3_ERR_OOM : D3_ERR_CUDA,                \
                  std::string(#expr) + ": " + cudaGetErrorString(e_));                            \
  } while (0)

int dev_alloc(d3_ctx* c, void** p, size_t bytes, bool zero = true) {
  if (bytes == 0) bytes = 16;
  cudaError_t e = cudaMalloc(p, bytes);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return fail(c, D3_ERR_OOM, "cudaMalloc of " + std::to_string(bytes) + " bytes: " + cudaGetErrorString(e));
  }
  c->allocs.push_back(*p);
  c->dev_bytes += static_cast<int64_t>(bytes);
  if (zero) {
    e = cudaMemsetAsync(*p, 0, bytes, c->stream);
    if (e != cudaSuccess) return fail(c, D3_ERR_CUDA, std::string("cudaMemsetAsync: ") + cudaGetErrorString(e));
  }
  return D3_OK;
}
#define ALLOC(c, ptr, bytes)                                                     \
  do {                                                                           \
    int rc_ = dev_alloc((c), reinterpret_cast<void**>(&(ptr)), (bytes));         \
    if (rc_ != D3_OK) return rc_;                                                \
  } while (0)

int check_launch(d3_ctx* c, const char* what) {
  c->launches++;
  c->launches_by_kernel[what]++;
  cudaError_t e = cudaPeekAtLastError();
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return fail(c, D3_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
  }
  return D3_OK;
}
#define LAUNCHED(c, what)                    \
  do {                                       \
    int rc_ = check_launch((c), (what));     \
    if (rc_ != D3_OK) return rc_;            \
  } while (0)
#define TRY(expr)                  \
  do {                             \
    int rc_ = (expr);              \
    if (rc_ != D3_OK) return rc_;  \
  } while (0)

// ---- optional per-class timing: an event pair around every launch of the class
void prof_flush(d3_ctx* c) {
  if (c->prof_used == 0) return;
  cudaStreamSynchronize(c->stream);
  for (size_t i = 0; i < c->prof_used; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->prof_pool[i].a, c->prof_pool[i].b) == cudaSuccess) {
      c->prof_ms[c->prof_pool[i].cls] += ms;
      c->prof_n[c->prof_pool[i].cls] += 1;
    }
  }
  c->prof_used = 0;
}
struct ProfScope {
  d3_ctx* c;
  long idx = -1;
  ProfScope(d3_ctx* ctx, int cls) : c(ctx) {
    if (!c->prof_on) return;
    if (c->prof_used == c->prof_pool.size()) {
      if (c->prof_pool.size() < 8192) {
        d3_ctx::ProfPair pp{};
        if (cudaEventCreate(&pp.a) != cudaSuccess || cudaEventCreate(&pp.b) != cudaSuccess) return;
        c->prof_pool.push_back(pp);
      } else {
        prof_flush(c);
      }
    }
    idx = static_cast<long>(c->prof_used++);
    c->prof_pool[idx].cls = cls;
    cudaEventRecord(c->prof_pool[idx].a, c->stream);
  }
  ~ProfScope() {
    if (idx >= 0) cudaEventRecord(c->prof_pool[idx].b, c->stream);
  }
};

// ---- tensor maps (driver entry point fetched through the runtime: no link against libcuda)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 row-major [rows, cols] matrix, box = [box_rows, 64 columns], 128-byte swizzle, zero fill.
// `swizzle` false: rows of the box land one after the other as they are (a block that is stored pre-swizzled).
int get_tmap(d3_ctx* c, const void* ptr, int rows, int cols, int box_rows, const CUtensorMap** out, bool swizzle = true) {
  auto key = std::make_tuple(ptr, rows, cols, swizzle ? box_rows : -box_rows);
  auto it = c->tmaps.find(key);
  if (it != c->tmaps.end()) {
    *out = &it->second;
    return D3_OK;
  }
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return fail(c, D3_ERR_CUDA, "cuTensorMapEncodeTiled entry point not found");
  if ((reinterpret_cast<uintptr_t>(ptr) & 15) != 0 || (cols % 8) != 0)
    return fail(c, D3_ERR_UNSUPPORTED, "tensor-core matmul needs 16-byte aligned operands and K % 8 == 0");
  CUtensorMap m;
  cuuint64_t gdim[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  cuuint64_t gstr[1] = {static_cast<cuuint64_t>(cols) * 2};
  cuuint32_t box[2] = {64, static_cast<cuuint32_t>(box_rows)};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstr, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(c, D3_ERR_CUDA, "cuTensorMapEncodeTiled failed with " + std::to_string(r));
  if (c->tmaps.size() > 4096) c->tmaps.clear();
  auto ins = c->tmaps.emplace(key, m);
  *out = &ins.first->second;
  return D3_OK;
}

// Up to this many rows a decode forward is bound by weight streaming, so twice the rows cost the same:
// d3_generate then fuses a block's finalize forward with the next block's first denoise step.
constexpr long long FUSE_MAX_ROWS = 64;

// ---- matmul dispatch
struct QkvExtra {
  RowMap rm;
  void* k_cache;
  void* v_cache;
};

// Launch with programmatic stream serialization: the kernel may become resident while the previous
// kernel of the stream is still running; everything it does before griddepcontrol.wait must be
// independent of that kernel.  Off while per-class timing is on, so that event pairs bracket one kernel.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(d3_ctx* c, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c->stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = (c->pdl && !c->prof_on) ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

template <int EPI, int BLOCK_N, int MT>
int launch_tc(d3_ctx* c, const CUtensorMap* tx, const CUtensorMap* tw, const tc::GemmParams& p, int n_ctas,
              size_t smem) {
  auto kern = tc::gemm_tc_kernel<EPI, BLOCK_N, MT>;
  static bool attr_set = false;
  if (!attr_set) {
    CUDA_TRY(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
    attr_set = true;
  }
  CUDA_TRY(c, launch_pdl(c, kern, dim3(n_ctas), dim3(tc::NUM_THREADS), smem, *tx, *tw, p));
  LAUNCHED(c, "gemm_tc_kernel");
  return D3_OK;
}

template <int BLOCK_N, int MT>
int dispatch_tc(d3_ctx* c, int epi, const CUtensorMap* tx, const CUtensorMap* tw, const tc::GemmParams& p, int n_ctas,
                size_t smem) {
  switch (epi) {
    case EPI_F32: return launch_tc<EPI_F32, BLOCK_N, MT>(c, tx, tw, p, n_ctas, smem);
    case EPI_T: return launch_tc<EPI_T, BLOCK_N, MT>(c, tx, tw, p, n_ctas, smem);
    case EPI_RESID: return launch_tc<EPI_RESID, BLOCK_N, MT>(c, tx, tw, p, n_ctas, smem);
    case EPI_SWIGLU: return launch_tc<EPI_SWIGLU, BLOCK_N, MT>(c, tx, tw, p, n_ctas, smem);
    case EPI_QKV: return launch_tc<EPI_QKV, BLOCK_N, MT>(c, tx, tw, p, n_ctas, smem);
    case EPI_STATS: return launch_tc<EPI_STATS, BLOCK_N, MT>(c, tx, tw, p, n_ctas, smem);
  }
  return fail(c, D3_ERR_INVALID_ARG, "unknown epilogue");
}

// Persistent CTAs; the (tile, K slab) units are dealt out evenly (see gemm_tc.cuh).
// `ctas_hint` > 0 forces the grid size (tests use it to move the segment borders around).
template <int BLOCK_N, int MT>
int run_linear_tc_bn(d3_ctx* c, const void* X, const void* W, int M, int N, int K, int epi, const EpiParams& ep,
                     int ctas_hint, const QkvExtra* qx, int w_tiled) {
  // m_tiles counts the row groups a unit covers: 128 rows, or 256 when two row tiles share a weight slab
  const int m_tiles = (M + 128 * MT - 1) / (128 * MT), n_tiles = (N + BLOCK_N - 1) / BLOCK_N;
  const int k_chunks = (K + 63) / 64;
  const long long tiles = static_cast<long long>(m_tiles) * n_tiles;
  if (tiles > c->n_tile_count) return fail(c, D3_ERR_SHAPE, "matmul has more output tiles than arrival counters");
  const int a_rows = MT == 2 ? 256 : (M >= 128 ? 128 : ((M + 31) / 32) * 32);
  tc::GemmParams p{};
  p.M = M; p.N = N; p.K = K;
  p.a_rows = a_rows;
  p.m_tiles = m_tiles; p.n_tiles = n_tiles; p.k_chunks = k_chunks;
  p.total_units = tiles * k_chunks;
  // skinny matmuls: two CTAs per SM (two sets of TMA-issuing threads keep more loads in flight)
  const int per_sm = c->tune_ctas_per_sm > 0 ? c->tune_ctas_per_sm : (M <= 128 ? 2 : 1);
  // at least eight K slabs per CTA: shorter ranges only add partial tiles
  long long n_ctas = std::min<long long>(static_cast<long long>(c->n_sms) * per_sm, std::max<long long>(1, p.total_units / 8));
  if (ctas_hint > 0) n_ctas = std::min<long long>(ctas_hint, p.total_units);
  // From 512 rows on the matmul is bound by the tensor pipe and by L2 reuse, not by balance: whole
  // tiles dealt round-robin in a banded order keep the CTAs of a moment on neighbouring tiles, so
  // weights are read from HBM once instead of once per row tile.
  if (BLOCK_N == 256 && MT == 1 && ctas_hint == 0 && !c->tune_no_rr) {
    p.rr = 1;
    p.gm = std::min(m_tiles, 16);
    n_ctas = std::min<long long>(c->n_sms, tiles);
  }
  n_ctas = std::min<long long>(n_ctas, std::min<long long>(tc::MAX_CTAS, static_cast<long long>(c->partial_slots / (2 * MT * (BLOCK_N / 128)))));
  const size_t stage_bytes = static_cast<size_t>(a_rows) * 128 + BLOCK_N * 128;
  // skinny matmuls are bound by HBM: keep the ring near 100 KB so that two CTAs (of this kernel, or
  // of this one and the next) share an SM; wide ones get all of shared memory
  const size_t ring = (c->tune_ring_kb > 0 ? c->tune_ring_kb : (M <= 128 ? 100 : 200)) * 1024;
  int stages = static_cast<int>(ring / stage_bytes);
  stages = std::max(2, std::min(stages, 16));
  p.stages = stages;
  p.partial = c->partial;
  p.tile_count = c->tile_count;
  p.error_word = c->error_word;
  p.skip_flag = c->skip_flag;
  p.w_tiled = w_tiled;
  p.n_producers = c->tune_producers > 0 ? c->tune_producers : 2;
  p.ep = ep;
  if (qx) {
    p.rope_cos = c->rope_cos; p.rope_sin = c->rope_sin;
    p.pos_base = qx->rm.pos_base; p.n_valid = qx->rm.n_valid; p.rows_per_seq = qx->rm.rows_per_seq;
    p.n_q_heads = c->cfg.n_q_heads; p.n_kv_heads = c->cfg.n_kv_heads; p.max_seq = c->cfg.max_seq;
    p.k_cache = static_cast<bf16*>(qx->k_cache); p.v_cache = static_cast<bf16*>(qx->v_cache);
  }
  const CUtensorMap *tx, *tw;
  TRY(get_tmap(c, X, M, K, a_rows, &tx));
  if (w_tiled) {
    if ((reinterpret_cast<uintptr_t>(W) & 15) != 0) return fail(c, D3_ERR_UNSUPPORTED, "tiled weights must be 16-byte aligned");
    p.w_packed = static_cast<const bf16*>(W);
    p.w_blocks = static_cast<long long>((N + 127) / 128) * k_chunks;
    tw = tx;  // unused by the kernel in this mode
  } else {
    TRY(get_tmap(c, W, N, K, BLOCK_N, &tw));
  }
  const size_t smem = tc::gemm_tc_smem_bytes(a_rows, BLOCK_N, stages);
  return dispatch_tc<BLOCK_N, MT>(c, epi, tx, tw, p, static_cast<int>(n_ctas), smem);
}

// Skinny matmuls (up to 128 rows by default, 256 on request): clusters of C CTAs own whole 128-column tiles and split K among
// their CTAs; the partial sums meet in distributed shared memory (gemm_ck_kernel).  C and the number
// of clusters are chosen so that the longest CTA has the fewest (tile, K slab) units.
template <int EPI>
int launch_ck(d3_ctx* c, const CUtensorMap* tx, const CUtensorMap* tw, const tc::GemmParams& p, const tc::ClusterSplit& cs,
              size_t smem) {
  auto kern = tc::gemm_ck_kernel<EPI>;
  static bool attr_set = false;
  if (!attr_set) {
    CUDA_TRY(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
    attr_set = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(cs.n_clusters * cs.C));
  cfg.blockDim = dim3(tc::NUM_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c->stream;
  cudaLaunchAttribute at[2];
  int na = 0;
  at[na].id = cudaLaunchAttributeClusterDimension;
  at[na].val.clusterDim.x = static_cast<unsigned>(cs.C);
  at[na].val.clusterDim.y = 1;
  at[na].val.clusterDim.z = 1;
  ++na;
  if (c->pdl && !c->prof_on) {
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = at;
  cfg.numAttrs = na;
  CUDA_TRY(c, cudaLaunchKernelEx(&cfg, kern, *tx, *tw, p, cs));
  LAUNCHED(c, "gemm_ck_kernel");
  return D3_OK;
}

int run_linear_ck(d3_ctx* c, const void* X, const void* W, int M, int N, int K, int epi, const EpiParams& ep,
                  int c_hint, const QkvExtra* qx, int w_tiled) {
  // up to 64 rows: one row tile with an X box of 32 or 64 rows; up to 256 rows: row tiles of 128
  const int a_rows = M <= 64 ? ((M + 31) / 32) * 32 : 128;
  const int m_tiles = (M + 127) / 128;
  const int T = m_tiles * ((N + 127) / 128), KC = (K + 63) / 64;
  if (epi != EPI_F32 && epi != EPI_T && epi != EPI_RESID) return fail(c, D3_ERR_UNSUPPORTED, "the cluster K-split kernel has elementwise epilogues only");
  // Cluster launches of this kernel get one CTA per SM, whatever its shared memory.  The kernel is
  // paced by its single-thread pipeline loops (a fixed time per K slab), so what counts is the number
  // of slabs a CTA walks through.  Either the clusters are all resident and loop over their tiles, or
  // every tile gets its own cluster and the grid runs in waves; a later wave overlaps the tail of the
  // one before it (measured: about three quarters of its length is added).
  const int slots = c->n_sms;
  tc::ClusterSplit cs{1, 1};
  long long best = -1;
  for (int C = 1; C <= 8; ++C) {
    if (C > KC) break;
    if (c_hint > 0 && C != c_hint) continue;
    const long long slabs = (KC + C - 1) / C;
    const int n_res = std::max(1, std::min(slots / C, T));
    const long long cost_res = static_cast<long long>((T + n_res - 1) / n_res) * slabs * 16;
    const long long waves = (static_cast<long long>(T) * C + slots - 1) / slots;
    // (with 128-row tiles the 200 KB of shared memory really leave one CTA per SM: whole waves)
    const long long cost_waves = a_rows <= 64 ? slabs * (4 + 3 * (waves - 1)) * 4  // slabs * (1 + 0.75 (waves - 1)) * 16
                                              : slabs * waves * 16;
    const bool by_waves = cost_waves < cost_res;
    const long long cost = (by_waves ? cost_waves : cost_res) + C;  // ties: smaller clusters
    if (best < 0 || cost < best) {
      best = cost;
      cs.C = C;
      cs.n_clusters = by_waves ? T : n_res;
    }
  }
  // skinny: ring + receive buffer stay near 100 KB, so that a CTA of the next kernel fits beside this
  // one; with 128-row tiles (32 KB stages, up to 64 KB of partials to receive) one CTA per SM
  const size_t stage_bytes = static_cast<size_t>(a_rows) * 128 + 128 * 128;
  const size_t recv_bytes = tc::gemm_ck_recv_bytes(a_rows, cs.C);
  // (64-row tiles: 108 KB buy a third 24 KB stage beside the 32 KB of partials, and two CTAs still share an SM)
  const size_t budget = (c->tune_ring_kb > 0 ? c->tune_ring_kb : (a_rows <= 32 ? 100 : a_rows <= 64 ? 108 : 200)) * 1024;
  int stages = static_cast<int>((budget > recv_bytes ? budget - recv_bytes : 0) / stage_bytes);
  stages = std::max(2, std::min(stages, 16));
  const size_t smem = tc::gemm_ck_smem_bytes(a_rows, stages, cs.C);
  tc::GemmParams p{};
  p.M = M; p.N = N; p.K = K;
  p.a_rows = a_rows;
  p.m_tiles = m_tiles; p.n_tiles = (N + 127) / 128; p.k_chunks = KC;
  p.total_units = static_cast<long long>(T) * KC;
  p.stages = stages;
  p.error_word = c->error_word;
  p.skip_flag = c->skip_flag;
  p.w_tiled = w_tiled;
  p.n_producers = 2;
  p.ep = ep;
  if (qx) {
    p.rope_cos = c->rope_cos; p.rope_sin = c->rope_sin;
    p.pos_base = qx->rm.pos_base; p.n_valid = qx->rm.n_valid; p.rows_per_seq = qx->rm.rows_per_seq;
    p.n_q_heads = c->cfg.n_q_heads; p.n_kv_heads = c->cfg.n_kv_heads; p.max_seq = c->cfg.max_seq;
    p.k_cache = static_cast<bf16*>(qx->k_cache); p.v_cache = static_cast<bf16*>(qx->v_cache);
  }
  const CUtensorMap *tx, *tw;
  TRY(get_tmap(c, X, M, K, a_rows, &tx));
  if (w_tiled) {
    if ((reinterpret_cast<uintptr_t>(W) & 15) != 0) return fail(c, D3_ERR_UNSUPPORTED, "tiled weights must be 16-byte aligned");
    p.w_packed = static_cast<const bf16*>(W);
    p.w_blocks = static_cast<long long>((N + 127) / 128) * KC;
    tw = tx;
  } else {
    TRY(get_tmap(c, W, N, K, 128, &tw));
  }
  switch (epi) {
    case EPI_F32: return launch_ck<EPI_F32>(c, tx, tw, p, cs, smem);
    case EPI_T: return launch_ck<EPI_T>(c, tx, tw, p, cs, smem);
    case EPI_RESID: return launch_ck<EPI_RESID>(c, tx, tw, p, cs, smem);
  }
  return fail(c, D3_ERR_INVALID_ARG, "unknown epilogue");
}

// Matmuls of 129..256 rows with few column tiles: weights as the 128-row MMA operand, a cluster per
// 128-column tile of the output splitting K (gemm_xt_kernel).  Returns D3_ERR_UNSUPPORTED (without a
// message) when the shape does not qualify; the caller then takes the unit-range kernel.
template <int EPI>
int launch_xt(d3_ctx* c, const CUtensorMap* tx, const tc::GemmParams& p, const tc::XtSplit& xs, int n_ctas, size_t smem) {
  auto kern = tc::gemm_xt_kernel<EPI>;
  static bool attr_set = false;
  if (!attr_set) {
    CUDA_TRY(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
    attr_set = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(n_ctas));
  cfg.blockDim = dim3(tc::XT_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c->stream;
  cudaLaunchAttribute at[2];
  int na = 0;
  if (xs.C > 1) {
    at[na].id = cudaLaunchAttributeClusterDimension;
    at[na].val.clusterDim.x = static_cast<unsigned>(xs.C);
    at[na].val.clusterDim.y = 1;
    at[na].val.clusterDim.z = 1;
    ++na;
  }
  if (c->pdl && !c->prof_on) {
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = at;
  cfg.numAttrs = na;
  CUDA_TRY(c, cudaLaunchKernelEx(&cfg, kern, *tx, p, xs));
  LAUNCHED(c, "gemm_xt_kernel");
  return D3_OK;
}

bool xt_usable(const d3_ctx* c, int M, int N, int K, int epi, int w_tiled, tc::XtSplit* xs, int* stages) {
  if (c->tune_xt == 0 || !w_tiled || M <= 128 || M > 256 || N % 128 != 0) return false;
  if (epi != EPI_F32 && epi != EPI_T && epi != EPI_RESID) return false;
  const int T = N / 128, KC = (K + 63) / 64;
  if (T > c->n_sms) return false;  // many column tiles: the unit-range kernel with row-tile pairs shares weight slabs already
  for (int C = 8; C >= 1; C >>= 1) {
    if (T * C > c->n_sms || KC < 4 * C) continue;
    const int n_cols = ((M + 32 * C - 1) / (32 * C)) * (32 * C);
    if (n_cols > 256) continue;
    const size_t stage_bytes = 128 * 128 + static_cast<size_t>(n_cols) * 128;
    int st = static_cast<int>((200 * 1024) / stage_bytes);
    st = std::max(2, std::min(st, 8));
    if (C > 1 && static_cast<size_t>(st) * stage_bytes < static_cast<size_t>(n_cols) * 512) continue;  // the staged partials live in the ring
    xs->C = C;
    xs->n_cols = n_cols;
    *stages = st;
    return true;
  }
  return false;
}

int run_linear_xt(d3_ctx* c, const void* X, const void* W, int M, int N, int K, int epi, const EpiParams& ep, const QkvExtra* qx,
                  const tc::XtSplit& xs, int stages) {
  if ((reinterpret_cast<uintptr_t>(W) & 15) != 0) return fail(c, D3_ERR_UNSUPPORTED, "tiled weights must be 16-byte aligned");
  tc::GemmParams p{};
  p.M = M; p.N = N; p.K = K;
  p.a_rows = xs.n_cols;
  p.k_chunks = (K + 63) / 64;
  p.stages = stages;
  p.error_word = c->error_word;
  p.skip_flag = c->skip_flag;
  p.w_tiled = 1;
  p.w_packed = static_cast<const bf16*>(W);
  p.w_blocks = static_cast<long long>(N / 128) * p.k_chunks;
  p.ep = ep;
  if (qx) {
    p.rope_cos = c->rope_cos; p.rope_sin = c->rope_sin;
    p.pos_base = qx->rm.pos_base; p.n_valid = qx->rm.n_valid; p.rows_per_seq = qx->rm.rows_per_seq;
    p.n_q_heads = c->cfg.n_q_heads; p.n_kv_heads = c->cfg.n_kv_heads; p.max_seq = c->cfg.max_seq;
    p.k_cache = static_cast<bf16*>(qx->k_cache); p.v_cache = static_cast<bf16*>(qx->v_cache);
  }
  const CUtensorMap* tx;
  TRY(get_tmap(c, X, M, K, xs.n_cols, &tx));
  const size_t smem = tc::gemm_xt_smem_bytes(xs.n_cols, stages);
  const int n_ctas = (N / 128) * xs.C;
  switch (epi) {
    case EPI_F32: return launch_xt<EPI_F32>(c, tx, p, xs, n_ctas, smem);
    case EPI_T: return launch_xt<EPI_T>(c, tx, p, xs, n_ctas, smem);
    case EPI_RESID: return launch_xt<EPI_RESID>(c, tx, p, xs, n_ctas, smem);
  }
  return fail(c, D3_ERR_INVALID_ARG, "unknown epilogue");
}

// Skinny matmuls with many columns as column strips over the whole K range (gemm_strip_kernel): the
// narrowest strip (a multiple of 16 columns that divides N) whose CTAs are all resident at once.
// Returns 0 when no strip width qualifies.
int strip_width(const d3_ctx* c, int M, int N, int w_tiled) {
  if (!w_tiled || M > 128 || c->tune_strip == 1) return 0;
  const int a_rows = ((M + 31) / 32) * 32;
  // above 64 rows a stage is 24-48 KB: one CTA per SM with all of shared memory as its ring
  const int per_sm = c->tune_ctas_per_sm > 0 ? c->tune_ctas_per_sm : ((c->tune_strip == 2 || a_rows > 64) ? 1 : 2);
  const int slots = c->n_sms * per_sm;
  if (c->tune_strip == 3) {  // tests: the narrowest strip the shape allows, whatever it costs
    for (int S = 16; S <= 256; S += 16)
      if (N % S == 0) return S;
    return 0;
  }
  for (int S = 16; S <= 256; S += 16) {
    // every CTA reads all of X: worth it while that is no more than its share of the weights
    if (N % S != 0 || N / S > slots || S < a_rows) continue;
    return N / S >= c->n_sms / 2 ? S : 0;  // most SMs must get a strip
  }
  return 0;
}

template <int EPI>
int launch_strip(d3_ctx* c, const CUtensorMap* tx, const tc::GemmParams& p, int S, int n_ctas, size_t smem) {
  static bool attr_set[2] = {false, false};
  // tensor memory: one accumulator of S columns per pipeline, the second one half way up
  const int wide = S * p.n_producers > 128 ? 1 : 0;
  auto kern = wide ? tc::gemm_strip_kernel<EPI, 256> : tc::gemm_strip_kernel<EPI, 128>;
  if (!attr_set[wide]) {
    CUDA_TRY(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
    attr_set[wide] = true;
  }
  CUDA_TRY(c, launch_pdl(c, kern, dim3(n_ctas), dim3(tc::STRIP_THREADS), smem, *tx, p, S));
  LAUNCHED(c, "gemm_strip_kernel");
  return D3_OK;
}

int run_linear_strip(d3_ctx* c, const void* X, const void* W, int M, int N, int K, int epi, const EpiParams& ep, int S,
                     const QkvExtra* qx) {
  if ((reinterpret_cast<uintptr_t>(W) & 15) != 0) return fail(c, D3_ERR_UNSUPPORTED, "tiled weights must be 16-byte aligned");
  const int a_rows = ((M + 31) / 32) * 32;
  const int KC = (K + 63) / 64;
  tc::GemmParams p{};
  p.M = M; p.N = N; p.K = K;
  p.a_rows = a_rows;
  p.m_tiles = 1; p.n_tiles = N / S; p.k_chunks = KC;
  p.total_units = static_cast<long long>(p.n_tiles) * KC;
  const int per_sm = c->tune_ctas_per_sm > 0 ? c->tune_ctas_per_sm : ((c->tune_strip == 2 || a_rows > 64) ? 1 : 2);
  const size_t ring = (c->tune_ring_kb > 0 ? c->tune_ring_kb : 200 / per_sm) * 1024;
  const size_t stage_bytes = static_cast<size_t>(a_rows + S) * 128;
  p.stages = std::max(2, std::min<int>(std::min<int>(static_cast<int>(ring / stage_bytes), KC), 32));
  const bool explicit_stages = c->tune_strip_stages > 0;
  if (explicit_stages) {
    p.stages = c->tune_strip_stages;
    if (p.stages < 2 || p.stages > 32 || p.stages > KC || static_cast<size_t>(p.stages) * stage_bytes > 200 * 1024)
      return fail(c, D3_ERR_UNSUPPORTED, "strip_stages outside 2..min(32, K slabs) or beyond 200 KB of shared memory");
  }
  p.error_word = c->error_word;
  p.skip_flag = c->skip_flag;
  p.w_tiled = 1;
  p.w_packed = static_cast<const bf16*>(W);
  p.w_blocks = static_cast<long long>((N + 127) / 128) * KC;
  p.gm = 1;  // K walk of CTA b starts at slab b mod KC
  // two issue pipelines per CTA while both accumulators fit 256 tensor-memory columns; each then owns
  // the stages of its parity, so the ring has an even number of them
  p.n_producers = (S <= 128 && KC >= 4 && c->tune_producers != 1) ? 2 : 1;
  if (p.n_producers == 2) {
    // every stage stays with one pipeline (stage s serves slabs s, s + stages, ...: the same parity
    // of slab index only when the count is even).  An odd count asked for by name is refused.
    if (explicit_stages && (p.stages & 1))
      return fail(c, D3_ERR_UNSUPPORTED, "two issue pipelines need an even number of stages");
    p.stages &= ~1;
  }
  p.ep = ep;
  if (qx) {
    p.rope_cos = c->rope_cos; p.rope_sin = c->rope_sin;
    p.pos_base = qx->rm.pos_base; p.n_valid = qx->rm.n_valid; p.rows_per_seq = qx->rm.rows_per_seq;
    p.n_q_heads = c->cfg.n_q_heads; p.n_kv_heads = c->cfg.n_kv_heads; p.max_seq = c->cfg.max_seq;
    p.k_cache = static_cast<bf16*>(qx->k_cache); p.v_cache = static_cast<bf16*>(qx->v_cache);
  }
  const CUtensorMap* tx;
  TRY(get_tmap(c, X, M, K, a_rows, &tx));
  const size_t smem = tc::gemm_strip_smem_bytes(a_rows, S, p.stages);
  switch (epi) {
    case EPI_F32: return launch_strip<EPI_F32>(c, tx, p, S, p.n_tiles, smem);
    case EPI_T: return launch_strip<EPI_T>(c, tx, p, S, p.n_tiles, smem);
    case EPI_RESID: return launch_strip<EPI_RESID>(c, tx, p, S, p.n_tiles, smem);
    case EPI_SWIGLU: return launch_strip<EPI_SWIGLU>(c, tx, p, S, p.n_tiles, smem);
    case EPI_QKV: return launch_strip<EPI_QKV>(c, tx, p, S, p.n_tiles, smem);
  }
  return fail(c, D3_ERR_INVALID_ARG, "unknown epilogue");
}

// ---- the decode forward as a chain (chain.cuh)
// Clusters of the chain kernel that can be resident at once with `smem` bytes per CTA (asked once per size).
int chain_max_clusters(d3_ctx* c, size_t smem) {
  static std::map<size_t, int> cache;
  auto it = cache.find(smem);
  if (it != cache.end()) return it->second;
  if (cudaFuncSetAttribute(tc::chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024) != cudaSuccess) {
    (void)cudaGetLastError();
    return 0;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(c->n_sms / tc::CHAIN_C * tc::CHAIN_C));
  cfg.blockDim = dim3(tc::CHAIN_THREADS);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = tc::CHAIN_C;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, tc::chain_kernel, &cfg) != cudaSuccess) {
    (void)cudaGetLastError();
    n = 0;
  }
  cache[smem] = n;
  return n;
}

constexpr int CHAIN_OPS_PER_LAYER = 5;  // QKV, attention, O-proj, gate/up, down

// Can a forward of bs x rows_per_seq rows run as a chain?  (bf16 tensor-core context with the fused QKV
// epilogue and folded norms; every (sequence, kv head) pair gets a cluster; all CTAs resident at once.)
bool chain_usable(d3_ctx* c, int bs, int rows_per_seq, int seg) {
  const d3_config& g = c->cfg;
  if (c->tune_chain == 0 || !c->use_tc || !c->fuse_qkv || !c->fold_norm || !c->w_tiled || !c->attn_tc) return false;
  const int M = bs * rows_per_seq;
  if (M > 64) return false;
  const int d = g.d_model, nq = g.n_q_heads * g.d_head, nkv = g.n_kv_heads * g.d_head, f = g.d_ffn;
  if (d % 32 != 0 || (nq + 2 * nkv) % 32 != 0 || (2 * f) % 16 != 0) return false;
  if ((nq + 63) / 64 < tc::CHAIN_C || (f + 63) / 64 < tc::CHAIN_C || (d + 63) / 64 < tc::CHAIN_C) return false;  // every rank of a K-split gets slabs
  if ((g.n_q_heads / g.n_kv_heads) * rows_per_seq > 64) return false;  // packed rows of a kv head: one attention tile
  if (seg > 0 && seg % 16 != 0) return false;                         // a 16-row group lies in one segment
  if (rows_per_seq % 16 != 0 && (g.n_q_heads / g.n_kv_heads) > 1) return false;
  return true;
}

// The program of a forward: QKV, attention, O-proj, gate/up, down per layer.  Built once (all
// buffers belong to the context) and kept on the device.
int chain_build_program(d3_ctx* c) {
  const d3_config& g = c->cfg;
  const int d = g.d_model, nq = g.n_q_heads * g.d_head, nkv = g.n_kv_heads * g.d_head, f = g.d_ffn;
  std::vector<tc::ChainOp> prog(static_cast<size_t>(g.n_layers) * CHAIN_OPS_PER_LAYER);
  auto after_norm = [&](EpiParams& ep) {
    ep.ssq_in = c->ssq; ep.ssq_chunks = (d + 31) / 32; ep.inv_k = 1.0f / static_cast<float>(d); ep.rms_eps = g.rms_eps;
  };
  auto updates_resid = [&](EpiParams& ep) {
    ep.yb = static_cast<bf16*>(c->xb); ep.ssq_out = c->ssq;
  };
  // activation tensor maps of a launch: 0 = attention output (O-proj), 1 = residual copy (QKV, gate/up), 2 = FFN hidden (down)
  for (int l = 0; l < g.n_layers; ++l) {
    tc::ChainOp* o = &prog[static_cast<size_t>(l) * CHAIN_OPS_PER_LAYER];
    for (int q = 0; q < CHAIN_OPS_PER_LAYER; ++q) {
      o[q] = tc::ChainOp{};
      o[q].layer = l;
      o[q].ks = tc::CHAIN_C;
    }
    o[0].kind = tc::CHAIN_KSPLIT; o[0].epi = EPI_QKV; o[0].ks = c->chain_qkv_ks; o[0].N = nq + 2 * nkv; o[0].K = d; o[0].x_map = 1;
    o[0].w = static_cast<const bf16*>(c->wqkv[l]);
    o[0].ep.y = c->q; o[0].ep.ldy = nq;
    after_norm(o[0].ep);
    o[1].kind = tc::CHAIN_ATTN; o[1].w = static_cast<const bf16*>(c->q); o[1].ep.y = c->o;
    o[2].kind = tc::CHAIN_KSPLIT; o[2].epi = EPI_RESID; o[2].N = d; o[2].K = nq; o[2].x_map = 0;
    o[2].w = static_cast<const bf16*>(c->wo[l]);
    o[2].ep.y = c->x; o[2].ep.ldy = d;
    updates_resid(o[2].ep);
    o[3].kind = tc::CHAIN_STRIP; o[3].epi = EPI_SWIGLU; o[3].N = 2 * f; o[3].K = d; o[3].x_map = 1;
    o[3].w = static_cast<const bf16*>(c->wgu[l]);
    o[3].ep.y = c->h; o[3].ep.ldy = f;
    after_norm(o[3].ep);
    o[4].kind = tc::CHAIN_KSPLIT; o[4].epi = EPI_RESID; o[4].N = d; o[4].K = f; o[4].x_map = 2;
    o[4].w = static_cast<const bf16*>(c->wd[l]);
    o[4].ep.y = c->x; o[4].ep.ldy = d;
    updates_resid(o[4].ep);
  }
  const size_t bytes = prog.size() * sizeof(tc::ChainOp);
  if (!c->chain_prog) {
    ALLOC(c, c->chain_prog, bytes);
    ALLOC(c, c->chain_sync, sizeof(unsigned int) * prog.size());
  }
  CUDA_TRY(c, cudaMemcpyAsync(c->chain_prog, prog.data(), bytes, cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));  // `prog` is a local
  c->chain_prog_ops = static_cast<int>(prog.size());
  // widest strips of the program, for the stage size and the receive buffer (they depend on the cluster count only)
  c->chain_prog_ready = true;
  return D3_OK;
}

// Launch operators [op_begin, op_end) of the forward's program.
int run_chain(d3_ctx* c, int op_begin, int op_end, const RowMap& rm) {
  ProfScope ps(c, D3_PROF_CHAIN);
  const d3_config& g = c->cfg;
  const int M = rm.bs * rm.rows_per_seq;
  const int a_rows = M <= 32 ? 32 : 64;
  const int d = g.d_model, nq = g.n_q_heads * g.d_head, nkv = g.n_kv_heads * g.d_head, f = g.d_ffn;
  // the grid: as many clusters as are resident at once (every CTA waits for every other at the borders)
  int n_clusters = c->chain_clusters;
  if (n_clusters < 0) {
    n_clusters = std::min(chain_max_clusters(c, 224 * 1024), c->n_sms / tc::CHAIN_C);
    c->chain_clusters = n_clusters;
  }
  if (c->tune_chain_clusters > 0) n_clusters = std::min(n_clusters, c->tune_chain_clusters);
  if (n_clusters < 8 || n_clusters < rm.bs * g.n_kv_heads)
    return fail(c, D3_ERR_UNSUPPORTED, "the chain kernel needs a resident cluster per (sequence, kv head) pair");
  const int n_cta = n_clusters * tc::CHAIN_C;
  auto strip_cols = [&](int N, int unit, int groups) { return ((N / unit + groups - 1) / groups) * unit; };
  const int qkv_cols = strip_cols(nq + 2 * nkv, 32, n_clusters * (tc::CHAIN_C / c->chain_qkv_ks));
  const int o_cols = strip_cols(d, 32, n_clusters);
  const int gu_cols = strip_cols(2 * f, 16, n_cta);
  const int max_strip = std::max(std::max(qkv_cols, o_cols), gu_cols);
  if (max_strip > 256) return fail(c, D3_ERR_UNSUPPORTED, "a chain strip would be wider than 256 columns");
  tc::ChainParams p{};
  p.prog = static_cast<const tc::ChainOp*>(c->chain_prog);
  p.op_begin = op_begin; p.op_end = op_end;
  p.M = M;
  p.a_rows = a_rows;
  p.w_stage_bytes = static_cast<uint32_t>(max_strip) * 128u;
  const size_t recv = std::max(std::max<size_t>(tc::chain_recv_bytes(a_rows, std::max(qkv_cols, o_cols)), sizeof(float) * tc::CHAIN_ARECV_FLOATS),
                               static_cast<size_t>(tc::CHAIN_ASTAGES) * tc::CHAIN_ASTAGE_BYTES);
  p.recv_bytes = static_cast<int>(recv);
  p.l2_ahead = c->tune_chain_l2 >= 0 ? c->tune_chain_l2 : 0;  // off by default: measured neutral at 12 slabs, slower beyond
  const size_t budget = (c->tune_ring_kb > 0 ? c->tune_ring_kb : 222) * 1024;  // whole CTA
  const size_t stage_bytes = static_cast<size_t>(a_rows) * 128 + p.w_stage_bytes;
  const size_t fixed = tc::chain_fixed_smem_bytes(recv, 16);
  int stages = static_cast<int>((budget > fixed ? budget - fixed : 0) / stage_bytes);
  stages = std::max(2, std::min(stages, 16));
  p.stages = stages;
  p.sync = c->chain_sync;
  p.error_word = c->error_word;
  p.skip_flag = c->skip_flag;
  p.rope_cos = c->rope_cos; p.rope_sin = c->rope_sin;
  p.rm = rm;
  p.n_q_heads = g.n_q_heads; p.n_kv_heads = g.n_kv_heads; p.max_seq = g.max_seq;
  p.kv_base = static_cast<bf16*>(c->kv);
  p.kv_plane_rows = static_cast<long long>(g.max_batch) * g.n_kv_heads * g.max_seq;
  p.scale_log2 = 1.4426950408889634f / std::sqrt(static_cast<float>(g.d_head));
  const CUtensorMap *t_o, *t_xb, *t_h;
  TRY(get_tmap(c, c->o, M, nq, a_rows, &t_o));
  TRY(get_tmap(c, c->xb, M, d, a_rows, &t_xb));
  TRY(get_tmap(c, c->h, M, f, a_rows, &t_h));
  const size_t smem = tc::chain_smem_bytes(a_rows, p.w_stage_bytes, stages, recv);
  if (smem > 224 * 1024) return fail(c, D3_ERR_UNSUPPORTED, "the chain kernel's shared memory does not fit");
  static bool attr_set = false;
  if (!attr_set) {
    CUDA_TRY(c, cudaFuncSetAttribute(tc::chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024));
    attr_set = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(n_cta));
  cfg.blockDim = dim3(tc::CHAIN_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c->stream;
  cudaLaunchAttribute at[2];
  int na = 0;
  at[na].id = cudaLaunchAttributeClusterDimension;
  at[na].val.clusterDim.x = tc::CHAIN_C;
  at[na].val.clusterDim.y = 1;
  at[na].val.clusterDim.z = 1;
  ++na;
  if (c->pdl && !c->prof_on) {
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = at;
  cfg.numAttrs = na;
  CUDA_TRY(c, cudaLaunchKernelEx(&cfg, tc::chain_kernel, *t_o, *t_xb, *t_h, c->kv_tmap32, p));
  LAUNCHED(c, "chain_kernel");
  return D3_OK;
}

// Tile width: 128 columns while weight streaming dominates, 256 when
// it is bound by the tensor pipe (from 512 rows on: a third less operand traffic per flop).
// Matmuls of more than 128 rows on CTA pairs (gemm_pair.cuh): 256 x 256 tiles, one cluster of two CTAs per tile at a time.
template <int EPI>
int launch_pair(d3_ctx* c, const CUtensorMap* tx, const CUtensorMap* tw, const tc::GemmParams& p, int tiles) {
  auto kern = tc::gemm_pair_kernel<EPI>;
  const size_t smem = tc::gemm_pair_smem_bytes();
  static bool attr_set = false;
  if (!attr_set) {
    CUDA_TRY(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    attr_set = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.blockDim = dim3(tc::PAIR_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c->stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 2;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  if (c->pair_clusters == 0) {  // pairs that are resident at once (a pair sits on the two SMs of one TPC)
    cfg.gridDim = dim3(static_cast<unsigned>(c->n_sms & ~1));
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n < 1) {
      (void)cudaGetLastError();
      n = 1;
    }
    c->pair_clusters = std::min(n, c->n_sms / 2);
  }
  cfg.gridDim = dim3(static_cast<unsigned>(2 * std::min(c->pair_clusters, tiles)));
  if (c->pdl && !c->prof_on) {
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 2;
  }
  CUDA_TRY(c, cudaLaunchKernelEx(&cfg, kern, *tx, *tw, p));
  LAUNCHED(c, "gemm_pair_kernel");
  return D3_OK;
}

bool pair_usable(const d3_ctx* c, int M, int N, int K, int epi, int w_tiled) {
  // from 129 rows on: at 129..256 rows a pair's tile holds all rows, so every weight block is staged once (measured
  // at 256 rows: QKV 58 -> 41 us and gate/up 77 -> 60 us per launch on the 8B shape, gate/up 69 -> 58 on the 7B one)
  return c->tune_cta_pairs != 0 && w_tiled && M > 128 && N % 256 == 0 && K % 64 == 0 &&
         static_cast<long long>(N / 128) * (K / 64) * 128 < (1ll << 31);
}

int run_linear_pair(d3_ctx* c, const void* X, const void* W, int M, int N, int K, int epi, const EpiParams& ep, const QkvExtra* qx) {
  tc::GemmParams p{};
  p.M = M; p.N = N; p.K = K;
  p.a_rows = 128;
  p.k_chunks = K / 64;
  p.m_tiles = (M + 255) / 256; p.n_tiles = N / 256;
  p.error_word = c->error_word;
  p.skip_flag = c->skip_flag;
  p.w_tiled = 1;
  if ((reinterpret_cast<uintptr_t>(W) & 15) != 0) return fail(c, D3_ERR_UNSUPPORTED, "tiled weights must be 16-byte aligned");
  p.w_packed = static_cast<const bf16*>(W);
  p.w_blocks = static_cast<long long>(N / 128) * p.k_chunks;
  p.ep = ep;
  if (c->live_n_valid != nullptr && M == c->live_rows) {
    p.live_n_valid = c->live_n_valid;
    p.live_rps = c->live_rps;
  }
  if (qx) {
    p.rope_cos = c->rope_cos; p.rope_sin = c->rope_sin;
    p.pos_base = qx->rm.pos_base; p.n_valid = qx->rm.n_valid; p.rows_per_seq = qx->rm.rows_per_seq;
    p.n_q_heads = c->cfg.n_q_heads; p.n_kv_heads = c->cfg.n_kv_heads; p.max_seq = c->cfg.max_seq;
    p.k_cache = static_cast<bf16*>(qx->k_cache); p.v_cache = static_cast<bf16*>(qx->v_cache);
  }
  const CUtensorMap *tx, *tw;
  TRY(get_tmap(c, X, M, K, 128, &tx));
  TRY(get_tmap(c, W, static_cast<int>(p.w_blocks) * 128, 64, 128, &tw, false));
  const int tiles = p.m_tiles * p.n_tiles;
  switch (epi) {
    case EPI_F32: return launch_pair<EPI_F32>(c, tx, tw, p, tiles);
    case EPI_T: return launch_pair<EPI_T>(c, tx, tw, p, tiles);
    case EPI_RESID: return launch_pair<EPI_RESID>(c, tx, tw, p, tiles);
    case EPI_SWIGLU: return launch_pair<EPI_SWIGLU>(c, tx, tw, p, tiles);
    case EPI_QKV: return launch_pair<EPI_QKV>(c, tx, tw, p, tiles);
    case EPI_STATS: return launch_pair<EPI_STATS>(c, tx, tw, p, tiles);
  }
  return fail(c, D3_ERR_INVALID_ARG, "unknown epilogue");
}

int run_linear_tc(d3_ctx* c, const void* X, const void* W, int M, int N, int K, int epi, const EpiParams& ep,
                  int ctas_hint, const QkvExtra* qx, int w_tiled) {
  // `ctas_hint` 1..8 on a skinny matmul forces the cluster size; larger hints ask for the unit-range kernel
  // Few column tiles and a long K (O-proj, down): clusters that split K and reduce through
  // distributed shared memory beat the L2 reduction of the unit-range kernel (measured at 32 rows on
  // the 8B shapes: 13 vs 16 us and 23 vs 25 us); cluster launches of this kernel get one CTA per SM
  // only, so the cluster size is chosen for a single wave (run_linear_ck).
  if (M <= 256 && !c->tune_no_cluster) {
    const int T = ((M + 127) / 128) * ((N + 127) / 128), KC = (K + 63) / 64;
    const bool elementwise = epi == EPI_F32 || epi == EPI_T || epi == EPI_RESID;
    if (elementwise && ctas_hint >= 1 && ctas_hint <= 8) return run_linear_ck(c, X, W, M, N, K, epi, ep, ctas_hint, qx, w_tiled);
    // few enough tiles that every tile gets a cluster of at least two resident CTAs.  By itself only
    // up to 128 rows (one row tile): at 256 rows the best cluster size is only level with the
    // unit-range kernel (measured on the 7B/8B shapes).
    if (elementwise && ctas_hint == 0 && M <= 128 && T * 2 <= c->n_sms && KC >= 16) return run_linear_ck(c, X, W, M, N, K, epi, ep, 0, qx, w_tiled);
  }
  if (ctas_hint < 0) {  // a strip width asked for by name
    const int S = -ctas_hint;
    if (!w_tiled || M > 128 || epi == EPI_STATS || S % 16 != 0 || S > 256 || N % S != 0)
      return fail(c, D3_ERR_UNSUPPORTED, "column strips need tiled weights, at most 128 rows and a width that is a multiple of 16, at most 256, and divides n");
    return run_linear_strip(c, X, W, M, N, K, epi, ep, S, qx);
  }
  if (ctas_hint == 0 && epi != EPI_STATS) {
    const int S = strip_width(c, M, N, w_tiled);
    // a residual epilogue that also writes chunk sums of squares needs whole 32-column chunks
    if (S > 0 && !(ep.ssq_out != nullptr && S % 32 != 0)) return run_linear_strip(c, X, W, M, N, K, epi, ep, S, qx);
  }
  if (ctas_hint == 0) {
    tc::XtSplit xs{};
    int xt_stages = 0;
    if (xt_usable(c, M, N, K, epi, w_tiled, &xs, &xt_stages)) return run_linear_xt(c, X, W, M, N, K, epi, ep, qx, xs, xt_stages);
  }
  if (ctas_hint == 0 && c->tune_wide_tiles < 0 && pair_usable(c, M, N, K, epi, w_tiled)) return run_linear_pair(c, X, W, M, N, K, epi, ep, qx);
  const bool wide = c->tune_wide_tiles >= 0 ? c->tune_wide_tiles != 0 : M >= 512;
  if (wide && N >= 256) return run_linear_tc_bn<256, 1>(c, X, W, M, N, K, epi, ep, ctas_hint, qx, w_tiled);
  // 129..511 rows: two row tiles per unit share each weight slab
  // (worth it when there are enough column tiles to give every SM whole tiles: with few tiles the
  // doubled partial tiles of split outputs cost more than the saved weight traffic)
  const bool pair = c->tune_pair >= 0 ? c->tune_pair != 0 : (M > 128 && (N + 127) / 128 >= c->n_sms);
  if (pair && M > 128) return run_linear_tc_bn<128, 2>(c, X, W, M, N, K, epi, ep, ctas_hint, qx, w_tiled);
  return run_linear_tc_bn<128, 1>(c, X, W, M, N, K, epi, ep, ctas_hint, qx, w_tiled);
}

template <typename T>
int run_linear_simt(d3_ctx* c, const void* X, const void* W, int M, int N, int K, int epi, const EpiParams& ep) {
  dim3 grid((N + simt::BN - 1) / simt::BN, (M + simt::BM - 1) / simt::BM);
  const T* x = static_cast<const T*>(X);
  const T* w = static_cast<const T*>(W);
  switch (epi) {
    case EPI_F32: simt::gemm_simt_kernel<T, EPI_F32><<<grid, simt::THREADS, 0, c->stream>>>(x, w, M, N, K, ep); break;
    case EPI_T: simt::gemm_simt_kernel<T, EPI_T><<<grid, simt::THREADS, 0, c->stream>>>(x, w, M, N, K, ep); break;
    case EPI_RESID: simt::gemm_simt_kernel<T, EPI_RESID><<<grid, simt::THREADS, 0, c->stream>>>(x, w, M, N, K, ep); break;
    case EPI_SWIGLU: simt::gemm_simt_kernel<T, EPI_SWIGLU><<<grid, simt::THREADS, 0, c->stream>>>(x, w, M, N, K, ep); break;
    case EPI_STATS: simt::gemm_simt_kernel<T, EPI_STATS><<<grid, simt::THREADS, 0, c->stream>>>(x, w, M, N, K, ep); break;
    default: return fail(c, D3_ERR_INVALID_ARG, "unknown epilogue");
  }
  LAUNCHED(c, "gemm_simt_kernel");
  return D3_OK;
}

int run_linear(d3_ctx* c, const void* X, const void* W, int M, int N, int K, int epi, const EpiParams& ep,
               int splits_hint = 0, const QkvExtra* qx = nullptr, int cls = D3_PROF_GEMM_OTHER, int w_tiled = 0) {
  if (M <= 0 || N <= 0 || K <= 0) return D3_OK;
  ProfScope ps(c, cls);
  if (c->use_tc) return run_linear_tc(c, X, W, M, N, K, epi, ep, splits_hint, qx, w_tiled);
  if (c->is_bf16) return run_linear_simt<bf16>(c, X, W, M, N, K, epi, ep);
  return run_linear_simt<float>(c, X, W, M, N, K, epi, ep);
}

// ---- typed launch helpers
template <typename T>
int launch_attention(d3_ctx* c, const void* q, const void* kc, const void* vc, void* out, const RowMap& rm) {
  const d3_config& g = c->cfg;
  dim3 grid((rm.rows_per_seq + attn::QT - 1) / attn::QT, g.n_q_heads, rm.bs);
  const float scale = 1.0f / std::sqrt(static_cast<float>(g.d_head));
  const T* qq = static_cast<const T*>(q);
  const T* kk = static_cast<const T*>(kc);
  const T* vv = static_cast<const T*>(vc);
  T* oo = static_cast<T*>(out);
  switch (g.d_head) {
    case 32: attn::attn_simt_kernel<T, 32><<<grid, attn::THREADS, 0, c->stream>>>(qq, kk, vv, oo, rm, g.n_q_heads, g.n_kv_heads, g.max_seq, scale); break;
    case 64: attn::attn_simt_kernel<T, 64><<<grid, attn::THREADS, 0, c->stream>>>(qq, kk, vv, oo, rm, g.n_q_heads, g.n_kv_heads, g.max_seq, scale); break;
    case 128: attn::attn_simt_kernel<T, 128><<<grid, attn::THREADS, 0, c->stream>>>(qq, kk, vv, oo, rm, g.n_q_heads, g.n_kv_heads, g.max_seq, scale); break;
    default: return fail(c, D3_ERR_UNSUPPORTED, "d_head must be 32, 64 or 128");
  }
  LAUNCHED(c, "attn_simt_kernel");
  return D3_OK;
}

// Tensor-core attention launch: warps per CTA from the packed rows per kv head, key splits so that
// about two CTAs per SM exist even at batch 1 (decode only; prefill has enough query tiles).
template <int NW, int KQ>
int launch_attn_tc(d3_ctx* c, const attn::AttnTcParams& p, dim3 grid) {
  auto kern = attn::attn_tc_kernel<NW, KQ>;
  static bool attr_set = false;
  if (!attr_set) {
    CUDA_TRY(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(attn::attn_tc_smem_bytes())));
    attr_set = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(NW * KQ * 32);
  cfg.dynamicSmemBytes = attn::attn_tc_smem_bytes();
  cfg.stream = c->stream;
  cudaLaunchAttribute at[2];
  int na = 0;
  if (grid.z > 1) {  // the key splits of one query tile form a cluster
    at[na].id = cudaLaunchAttributeClusterDimension;
    at[na].val.clusterDim.x = 1;
    at[na].val.clusterDim.y = 1;
    at[na].val.clusterDim.z = grid.z;
    ++na;
  }
  if (c->pdl && !c->prof_on) {
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = at;
  cfg.numAttrs = na;
  CUDA_TRY(c, cudaLaunchKernelEx(&cfg, kern, c->kv_tmap, p));
  LAUNCHED(c, "attn_tc_kernel");
  return D3_OK;
}

// CTAs of one attention instantiation that fit an SM (registers and shared memory), asked once.
template <int NW, int KQ>
int attn_ctas_per_sm() {
  static int cached = 0;
  if (cached == 0) {
    auto kern = attn::attn_tc_kernel<NW, KQ>;
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(attn::attn_tc_smem_bytes()));
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, NW * KQ * 32, attn::attn_tc_smem_bytes()) != cudaSuccess || n < 1) n = 1;
    cached = n;
  }
  return cached;
}

// tcgen05 attention launch.  Two shapes: 128-key tiles, one CTA per SM (long key ranges), and 64-key tiles, two CTAs
// per SM (a CTA that lives for a few tiles only: start-up and output of one overlap the tile loop of the other).
template <int KT, int SBUF>
int launch_attn_tmem(d3_ctx* c, const attn::AttnTcParams& p, dim3 grid) {
  auto kern = attn::attn_tmem_kernel<KT, SBUF>;
  const size_t smem = attn::TmLayout<KT, SBUF>::smem_bytes();
  static bool attr_set = false;
  if (!attr_set) {
    CUDA_TRY(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    attr_set = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(attn::TM_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c->stream;
  cudaLaunchAttribute at[2];
  int na = 0;
  if (grid.z > 1) {
    at[na].id = cudaLaunchAttributeClusterDimension;
    at[na].val.clusterDim.x = 1;
    at[na].val.clusterDim.y = 1;
    at[na].val.clusterDim.z = grid.z;
    ++na;
  }
  if (c->pdl && !c->prof_on) {
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = at;
  cfg.numAttrs = na;
  CUDA_TRY(c, cudaLaunchKernelEx(&cfg, kern, KT == 64 ? c->kv_tmap : c->kv_tmap128, p));
  LAUNCHED(c, "attn_tmem_kernel");
  return D3_OK;
}

// Decode-sized batches with several (sequence, kv head) pairs per SM: one persistent CTA per SM streams through its pairs.
bool attn_stream_usable(const d3_ctx* c, const RowMap& rm) {
  const d3_config& g = c->cfg;
  const int R = (g.n_q_heads / g.n_kv_heads) * rm.rows_per_seq;
  return R <= 128 && rm.rows_per_seq % 8 == 0 && rm.rows_per_seq <= 256 &&
         static_cast<long long>(rm.bs) * rm.rows_per_seq < (1ll << 31);
}
int run_attention_tmem_stream(d3_ctx* c, const void* q, int layer, void* out, const RowMap& rm) {
  const d3_config& g = c->cfg;
  auto kern = attn::attn_tmem_stream_kernel;
  const size_t smem = attn::TmStream::smem_bytes((g.n_q_heads / g.n_kv_heads) * rm.rows_per_seq);
  static bool attr_set = false;
  if (!attr_set) {
    CUDA_TRY(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(attn::TmStream::smem_bytes(64))));
    attr_set = true;
  }
  attn::AttnTcParams p{};
  p.q = static_cast<const bf16*>(q);
  p.out = static_cast<bf16*>(out);
  p.rm = rm;
  p.hq = g.n_q_heads; p.hkv = g.n_kv_heads; p.max_seq = g.max_seq;
  const long long plane_rows = static_cast<long long>(g.max_batch) * g.n_kv_heads * g.max_seq;
  p.k_row0 = (static_cast<long long>(layer) * 2 + 0) * plane_rows;
  p.v_row0 = (static_cast<long long>(layer) * 2 + 1) * plane_rows;
  p.n_splits = 1;
  p.scale_log2 = 1.4426950408889634f / std::sqrt(static_cast<float>(g.d_head));
  p.error_word = c->error_word;
  const CUtensorMap* tq;
  TRY(get_tmap(c, q, rm.bs * rm.rows_per_seq, g.n_q_heads * 128, rm.rows_per_seq, &tq));
  const int pairs = rm.bs * g.n_kv_heads;
  CUDA_TRY(c, launch_pdl(c, kern, dim3(static_cast<unsigned>(std::min(c->n_sms, pairs))), dim3(attn::TM_THREADS), smem, c->kv_tmap128, *tq, p));
  LAUNCHED(c, "attn_tmem_stream_kernel");
  return D3_OK;
}

int run_attention_tmem(d3_ctx* c, const void* q, int layer, void* out, const RowMap& rm) {
  const d3_config& g = c->cfg;
  const int group = g.n_q_heads / g.n_kv_heads;
  const int R = group * rm.rows_per_seq;
  const int q_tiles = (R + 127) / 128;
  const int pairs = rm.bs * g.n_kv_heads;
  // short key ranges (at most 8 tiles of 128 keys per CTA) and enough CTAs to fill two per SM: the small shape
  bool small = g.max_seq <= 1024 && pairs * q_tiles >= 2 * c->n_sms;
  if (c->tune_attn_shape > 0) small = c->tune_attn_shape == 64;
  const int kt = small ? 64 : 128;
  const int slots = c->n_sms * (small ? 2 : 1);
  int splits = 1;
  if (q_tiles <= 2 && pairs * q_tiles < slots) {
    // decode-sized: (sequence, kv head) pairs alone leave SMs idle, so the keys of a query tile are split over a
    // cluster (at most 8 CTAs, at least two key tiles each).  Cost of a split count: waves x key tiles per CTA.
    const int max_tiles = (g.max_seq + kt - 1) / kt;
    const int cap = std::max(1, std::min(8, max_tiles / 2));
    auto cost_of = [&](int s) {
      const long long waves = (static_cast<long long>(pairs) * q_tiles * s + slots - 1) / slots;
      return waves * ((max_tiles + s - 1) / s);
    };
    long long best = cost_of(1);
    for (int s = 2; s <= cap; ++s) best = std::min(best, cost_of(s));
    for (int s = 1; s <= cap; ++s)
      if (cost_of(s) * 100 <= best * 115) { splits = s; break; }
  }
  attn::AttnTcParams p{};
  p.q = static_cast<const bf16*>(q);
  p.out = static_cast<bf16*>(out);
  p.rm = rm;
  p.hq = g.n_q_heads; p.hkv = g.n_kv_heads; p.max_seq = g.max_seq;
  const long long plane_rows = static_cast<long long>(g.max_batch) * g.n_kv_heads * g.max_seq;
  p.k_row0 = (static_cast<long long>(layer) * 2 + 0) * plane_rows;
  p.v_row0 = (static_cast<long long>(layer) * 2 + 1) * plane_rows;
  p.n_splits = splits;
  p.scale_log2 = 1.4426950408889634f / std::sqrt(static_cast<float>(g.d_head));
  p.error_word = c->error_word;
  dim3 grid(q_tiles, pairs, splits);
  return small ? launch_attn_tmem<64, 2>(c, p, grid) : launch_attn_tmem<128, 2>(c, p, grid);
}

int run_attention_tc(d3_ctx* c, const void* q, int layer, void* out, const RowMap& rm) {
  const d3_config& g = c->cfg;
  const int group = g.n_q_heads / g.n_kv_heads;
  const int R = group * rm.rows_per_seq;
  // From 64 packed rows per kv head on (long blocks, fused finalize, grouped query heads, prefill) the tcgen05 kernel
  // is the faster one (measured: 60-70 against 84-110 us per layer at 64 rows x 4200-5100 keys, 27 against 33-37 at
  // 224 rows x 550-1000 keys, a third of the time on 4096-row prompts); at 32 rows the two are level on batches and
  // the mma.sync kernel, with its cheaper start, is ahead on a single sequence (15 against 19 us).
  if (c->tune_attn_shape == 2 ? attn_stream_usable(c, rm)
                              : (c->tune_attn_tmem < 0 && attn_stream_usable(c, rm) && rm.bs * g.n_kv_heads >= 2 * c->n_sms))
    return run_attention_tmem_stream(c, q, layer, out, rm);
  if (c->tune_attn_tmem == 1 || (c->tune_attn_tmem < 0 && R >= 64)) return run_attention_tmem(c, q, layer, out, rm);
  const int nw = R <= 32 ? 2 : (R <= 64 ? 4 : 8);
  const int q_tiles = (R + nw * 16 - 1) / (nw * 16);
  const int pairs = rm.bs * g.n_kv_heads;
  int splits = 1;
  const int slots = c->n_sms * (nw == 2 ? attn_ctas_per_sm<2, 4>() : nw == 4 ? attn_ctas_per_sm<4, 2>() : attn_ctas_per_sm<8, 1>());
  if (q_tiles <= 2 && pairs * q_tiles < slots) {
    // decode-sized: (sequence, kv head) pairs alone leave SMs idle, so the keys of a query tile are split
    // over a cluster (at most 8 CTAs, at least two key tiles each).  Cost of a split count:
    // (waves of resident CTAs) x (key tiles per CTA).
    const int max_tiles = (g.max_seq + attn::KT - 1) / attn::KT;
    const int cap = std::max(1, std::min(8, c->tune_attn_div > 0 ? max_tiles / c->tune_attn_div : max_tiles / 2));
    auto cost_of = [&](int s) {
      const long long waves = (static_cast<long long>(pairs) * q_tiles * s + slots - 1) / slots;
      return waves * ((max_tiles + s - 1) / s);
    };
    long long best = cost_of(1);
    for (int s = 2; s <= cap; ++s) best = std::min(best, cost_of(s));
    // larger clusters cost more than this count sees (co-scheduling, the merge: eight splits at a
    // 5120-key prefix took 160 us where two took 102): the smallest count within 15 % of the best
    for (int s = 1; s <= cap; ++s)
      if (cost_of(s) * 100 <= best * 115) { splits = s; break; }
  }
  attn::AttnTcParams p{};
  p.q = static_cast<const bf16*>(q);
  p.out = static_cast<bf16*>(out);
  p.rm = rm;
  p.hq = g.n_q_heads; p.hkv = g.n_kv_heads; p.max_seq = g.max_seq;
  const long long plane_rows = static_cast<long long>(g.max_batch) * g.n_kv_heads * g.max_seq;
  p.k_row0 = (static_cast<long long>(layer) * 2 + 0) * plane_rows;
  p.v_row0 = (static_cast<long long>(layer) * 2 + 1) * plane_rows;
  p.n_splits = splits;
  p.scale_log2 = 1.4426950408889634f / std::sqrt(static_cast<float>(g.d_head));
  p.error_word = c->error_word;
  dim3 grid(q_tiles, pairs, splits);
  switch (nw) {
    // eight warps per CTA whatever the rows: few row groups leave warps to split the keys of a tile
    case 2: return launch_attn_tc<2, 4>(c, p, grid);
    case 4: return launch_attn_tc<4, 2>(c, p, grid);
    default: return launch_attn_tc<8, 1>(c, p, grid);
  }
}

int run_attention(d3_ctx* c, const void* q, int layer, void* out, const RowMap& rm) {
  ProfScope ps(c, D3_PROF_ATTENTION);
  if (c->attn_tc) return run_attention_tc(c, q, layer, out, rm);
  const char* base = static_cast<const char*>(c->kv);
  const void* kc = base + (static_cast<size_t>(layer) * 2 + 0) * c->kv_layer_elems * c->esz;
  const void* vc = base + (static_cast<size_t>(layer) * 2 + 1) * c->kv_layer_elems * c->esz;
  if (c->is_bf16) return launch_attention<bf16>(c, q, kc, vc, out, rm);
  return launch_attention<float>(c, q, kc, vc, out, rm);
}

void* k_plane(d3_ctx* c, int layer) {
  return static_cast<char*>(c->kv) + (static_cast<size_t>(layer) * 2 + 0) * c->kv_layer_elems * c->esz;
}
void* v_plane(d3_ctx* c, int layer) {
  return static_cast<char*>(c->kv) + (static_cast<size_t>(layer) * 2 + 1) * c->kv_layer_elems * c->esz;
}

int run_rmsnorm(d3_ctx* c, const float* x, const float* gain, void* xn, int M) {
  ProfScope ps(c, D3_PROF_RMSNORM);
  const int d = c->cfg.d_model;
  if (c->is_bf16) CUDA_TRY(c, launch_pdl(c, rmsnorm_kernel<bf16>, dim3(M), dim3(256), 0, x, gain, static_cast<bf16*>(xn), d, c->cfg.rms_eps));
  else CUDA_TRY(c, launch_pdl(c, rmsnorm_kernel<float>, dim3(M), dim3(256), 0, x, gain, static_cast<float*>(xn), d, c->cfg.rms_eps));
  LAUNCHED(c, "rmsnorm_kernel");
  return D3_OK;
}

int run_stats_merge(d3_ctx* c, int M, int n_tiles, float* conf, float* ent, int* argmax, bool sampled = false) {
  ProfScope ps(c, D3_PROF_OTHER);
  if (sampled) {
    CUDA_TRY(c, launch_pdl(c, stats_merge_sample_kernel, dim3((M + 3) / 4), dim3(128), 0, static_cast<const float4*>(c->stat_part),
                           static_cast<const float4*>(c->sample_part), n_tiles, M, conf, ent, argmax));
    LAUNCHED(c, "stats_merge_sample_kernel");
    return D3_OK;
  }
  CUDA_TRY(c, launch_pdl(c, stats_merge_kernel, dim3((M + 3) / 4), dim3(128), 0, static_cast<const float4*>(c->stat_part), n_tiles, M, conf, ent, argmax));
  LAUNCHED(c, "stats_merge_kernel");
  return D3_OK;
}

// The transformer stack over M rows laid out as bs x rows_per_seq (row map already on the device).
//   head: 0 = none, 1 = fused statistics into ctx conf/ent/argmax, 2 = fp32 logits into `logits`.
//   seg: rows per segment when a sequence's rows are consecutive blocks that must not see later ones (0: one segment).
int forward(d3_ctx* c, const int* ids, int bs, int rows_per_seq, int head, float* logits, int seg = 0) {
  const d3_config& g = c->cfg;
  const int M = bs * rows_per_seq;
  if (M == 0) return D3_OK;
  if (M > c->max_rows) return fail(c, D3_ERR_SHAPE, "forward over more rows than the workspaces hold");
  const int d = g.d_model, nq = g.n_q_heads * g.d_head, nkv = g.n_kv_heads * g.d_head, f = g.d_ffn;
  RowMap rm{c->pos_base, c->n_valid, c->kv_len, rows_per_seq, bs, seg};
  c->last_rows = M;
  // Padded prompts: the matmuls on CTA pairs pass over 256-row tiles that hold no live row of their sequence (rows
  // beyond n_valid are computed by nobody's reader: attention, the cache write and the decisions skip them already).
  struct LiveRows {
    d3_ctx* c;
    LiveRows(d3_ctx* c_, const int* n_valid, int rps, int rows) : c(c_) {
      if (rps % 256 == 0) { c->live_n_valid = n_valid; c->live_rps = rps; c->live_rows = rows; }
    }
    ~LiveRows() { c->live_n_valid = nullptr; c->live_rps = 0; c->live_rows = 0; }
  } live_rows(c, c->n_valid, rows_per_seq, M);

  {
    ProfScope ps(c, D3_PROF_OTHER);
    if (c->is_bf16) CUDA_TRY(c, launch_pdl(c, embed_kernel<bf16>, dim3(M), dim3(128), 0, ids, static_cast<const bf16*>(c->tok_emb), c->x, d, g.vocab, c->error_word));
    else CUDA_TRY(c, launch_pdl(c, embed_kernel<float>, dim3(M), dim3(128), 0, ids, static_cast<const float*>(c->tok_emb), c->x, d, g.vocab, c->error_word));
    LAUNCHED(c, "embed_kernel");
    if (c->fold_norm) {
      CUDA_TRY(c, launch_pdl(c, row_prep_kernel, dim3(M), dim3(128), 0, static_cast<const float*>(c->x), static_cast<bf16*>(c->xb), c->ssq, d));
      LAUNCHED(c, "row_prep_kernel");
    }
  }
  // Folded RMSNorm: the matmuls after a norm read the bf16 copy of the residual stream and scale
  // their accumulator rows; the matmuls that update the residual stream refresh the copy and the
  // chunk sums of squares.
  const void* normed = c->fold_norm ? c->xb : c->xn;
  auto after_norm = [&](EpiParams& ep) {
    if (!c->fold_norm) return;
    ep.ssq_in = c->ssq; ep.ssq_chunks = (d + 31) / 32; ep.inv_k = 1.0f / static_cast<float>(d); ep.rms_eps = g.rms_eps;
  };
  auto updates_resid = [&](EpiParams& ep) {
    if (!c->fold_norm) return;
    ep.yb = static_cast<bf16*>(c->xb); ep.ssq_out = c->ssq;
  };

  if (chain_usable(c, bs, rows_per_seq, seg)) {
    // Skinny decode forward: all layers in one persistent launch (chain.cuh); a tapped layer cuts it.
    if (!c->chain_prog_ready) TRY(chain_build_program(c));
    CUDA_TRY(c, cudaMemsetAsync(c->chain_sync, 0, sizeof(unsigned int) * static_cast<size_t>(c->chain_prog_ops), c->stream));
    const int n_ops = c->chain_prog_ops;
    const bool tap = c->tap_layer >= 0 && c->tap_layer < g.n_layers && M <= c->tap_rows;
    if (!tap) {
      TRY(run_chain(c, 0, n_ops, rm));
    } else {
      // the residual stream enters layer L before its O-proj (QKV and attention only read it) and leaves it after down
      const int o_in = c->tap_layer * CHAIN_OPS_PER_LAYER + 2, o_out = (c->tap_layer + 1) * CHAIN_OPS_PER_LAYER;
      TRY(run_chain(c, 0, o_in, rm));
      CUDA_TRY(c, cudaMemcpyAsync(c->tap_in, c->x, sizeof(float) * M * d, cudaMemcpyDeviceToDevice, c->stream));
      TRY(run_chain(c, o_in, o_out, rm));
      CUDA_TRY(c, cudaMemcpyAsync(c->tap_out, c->x, sizeof(float) * M * d, cudaMemcpyDeviceToDevice, c->stream));
      if (o_out < n_ops) TRY(run_chain(c, o_out, n_ops, rm));
    }
  } else
  for (int l = 0; l < g.n_layers; ++l) {
    if (l == c->tap_layer && M <= c->tap_rows)
      CUDA_TRY(c, cudaMemcpyAsync(c->tap_in, c->x, sizeof(float) * M * d, cudaMemcpyDeviceToDevice, c->stream));
    if (!c->fold_norm) TRY(run_rmsnorm(c, c->x, c->attn_norm[l], c->xn, M));
    if (c->fuse_qkv) {
      EpiParams ep;
      ep.y = c->q; ep.ldy = nq;
      after_norm(ep);
      QkvExtra qx{rm, k_plane(c, l), v_plane(c, l)};
      TRY(run_linear(c, normed, c->wqkv[l], M, nq + 2 * nkv, d, EPI_QKV, ep, 0, &qx, D3_PROF_GEMM_QKV, c->w_tiled));
    } else {
      EpiParams ep;
      ep.y = c->qkv_f32; ep.ldy = nq + 2 * nkv;
      after_norm(ep);
      TRY(run_linear(c, normed, c->wqkv[l], M, nq + 2 * nkv, d, EPI_F32, ep, 0, nullptr, D3_PROF_GEMM_QKV, c->w_tiled));
      ProfScope ps(c, D3_PROF_OTHER);
      if (c->is_bf16)
        rope_kv_kernel<bf16><<<M, 256, 0, c->stream>>>(c->qkv_f32, static_cast<bf16*>(c->q), static_cast<bf16*>(k_plane(c, l)), static_cast<bf16*>(v_plane(c, l)), c->rope_cos, c->rope_sin, rm, g.n_q_heads, g.n_kv_heads, g.d_head, g.max_seq, c->error_word);
      else
        rope_kv_kernel<float><<<M, 256, 0, c->stream>>>(c->qkv_f32, static_cast<float*>(c->q), static_cast<float*>(k_plane(c, l)), static_cast<float*>(v_plane(c, l)), c->rope_cos, c->rope_sin, rm, g.n_q_heads, g.n_kv_heads, g.d_head, g.max_seq, c->error_word);
      LAUNCHED(c, "rope_kv_kernel");
    }
    TRY(run_attention(c, c->q, l, c->o, rm));
    {
      EpiParams ep;
      ep.y = c->x; ep.ldy = d;
      updates_resid(ep);
      TRY(run_linear(c, c->o, c->wo[l], M, d, nq, EPI_RESID, ep, 0, nullptr, D3_PROF_GEMM_O, c->w_tiled));
    }
    if (!c->fold_norm) TRY(run_rmsnorm(c, c->x, c->ffn_norm[l], c->xn, M));
    {
      EpiParams ep;
      ep.y = c->h; ep.ldy = f;
      after_norm(ep);
      TRY(run_linear(c, normed, c->wgu[l], M, 2 * f, d, EPI_SWIGLU, ep, 0, nullptr, D3_PROF_GEMM_GATE_UP, c->w_tiled));
    }
    {
      EpiParams ep;
      ep.y = c->x; ep.ldy = d;
      updates_resid(ep);
      TRY(run_linear(c, c->h, c->wd[l], M, d, f, EPI_RESID, ep, 0, nullptr, D3_PROF_GEMM_DOWN, c->w_tiled));
    }
    if (l == c->tap_layer && M <= c->tap_rows)
      CUDA_TRY(c, cudaMemcpyAsync(c->tap_out, c->x, sizeof(float) * M * d, cudaMemcpyDeviceToDevice, c->stream));
  }
  if (head == 0) return D3_OK;
  if (!c->fold_norm) TRY(run_rmsnorm(c, c->x, c->final_norm, c->xn, M));
  if (head == 1) {
    const int n_tiles = (g.vocab + 127) / 128;
    EpiParams ep;
    ep.scale = g.logit_scale; ep.mask_id = g.mask_id; ep.stat_part = c->stat_part; ep.n_tiles = n_tiles;
    const bool sampled = c->temperature > 0.f;
    if (sampled) {  // temperature sampling: Gumbel noise keyed by (seed; sequence, position, step)
      ep.sample_part = c->sample_part;
      ep.temperature = c->temperature;
      ep.seed_lo = static_cast<uint32_t>(c->seed & 0xffffffffull);
      ep.seed_hi = static_cast<uint32_t>(c->seed >> 32);
      ep.pos_base = c->pos_base;
      ep.rows_per_seq = rows_per_seq;
      ep.draw_step = c->draw_step;
      ep.draw_step_add = c->draw_step_add;
    }
    after_norm(ep);
    TRY(run_linear(c, normed, c->lm_head, M, g.vocab, d, EPI_STATS, ep, 0, nullptr, D3_PROF_GEMM_HEAD, c->w_tiled));
    TRY(run_stats_merge(c, M, n_tiles, c->conf, c->ent, c->argmax, sampled));
  } else {
    EpiParams ep;
    ep.y = logits; ep.ldy = g.vocab; ep.scale = g.logit_scale;
    after_norm(ep);
    TRY(run_linear(c, normed, c->lm_head, M, g.vocab, d, EPI_F32, ep, 0, nullptr, D3_PROF_GEMM_HEAD, c->w_tiled));
  }
  return D3_OK;
}

int check_device_error(d3_ctx* c) {
  uint32_t w = 0;
  CUDA_TRY(c, cudaMemcpyAsync(&w, c->error_word, sizeof(w), cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  const int rc = d3_status_of_error_word(w);
  if (rc == D3_ERR_DEVICE_TIMEOUT) return fail(c, rc, "a bounded device-side wait gave up");
  if (rc != D3_OK) return fail(c, rc, "device error word " + std::to_string(w) + " (bad token id, position or statistic)");
  return D3_OK;
}

template <typename T>
void cast_to_f32(d3_ctx* c, const void* src, float* dst, size_t n) {
  cast_to_f32_kernel<T><<<static_cast<unsigned>((n + 255) / 256), 256, 0, c->stream>>>(static_cast<const T*>(src), dst, n);
  c->launches++;
}

}  // namespace

// ----------------------------------------------------------------------------- create / destroy
extern "C" int d3_create(const d3_config* cfg, void* cuda_stream, d3_ctx** out) {
  if (!cfg || !out) return D3_ERR_INVALID_ARG;
  *out = nullptr;
  const d3_config& g = *cfg;
  if (g.n_layers <= 0 || g.d_model <= 0 || g.n_q_heads <= 0 || g.n_kv_heads <= 0 || g.d_ffn <= 0 || g.vocab <= 1 ||
      g.block <= 0 || g.max_batch <= 0 || g.max_seq <= 0 || g.mask_id < 0 || g.mask_id >= g.vocab)
    return D3_ERR_INVALID_ARG;
  if (g.dtype != D3_DTYPE_F32 && g.dtype != D3_DTYPE_BF16) return D3_ERR_INVALID_ARG;
  if (g.decide_mode != D3_DECIDE_CONFIDENCE && g.decide_mode != D3_DECIDE_ENTROPY) return D3_ERR_INVALID_ARG;
  if (!(g.rms_eps >= 0.f) || !(g.rope_theta > 0.f) || !std::isfinite(g.logit_scale)) return D3_ERR_INVALID_ARG;
  if (g.d_head != 32 && g.d_head != 64 && g.d_head != 128) return D3_ERR_UNSUPPORTED;
  if (g.n_q_heads % g.n_kv_heads != 0 || g.d_ffn % 64 != 0 || g.d_model % 8 != 0 || g.block > 128 ||
      g.block > g.max_seq)
    return D3_ERR_UNSUPPORTED;
  d3_ctx* c = new (std::nothrow) d3_ctx();
  if (!c) return D3_ERR_OOM;
  c->cfg = g;
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  c->is_bf16 = g.dtype == D3_DTYPE_BF16;
  c->esz = c->is_bf16 ? 2 : 4;
  c->use_tc = c->is_bf16 && g.gemm_impl == D3_GEMM_AUTO;
  c->fuse_qkv = c->use_tc && g.d_head == 128;
  c->w_tiled = c->use_tc;
  c->fold_norm = c->use_tc;
  auto bail = [&](int rc) {
    d3_destroy(c);
    return rc;
  };
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return bail(D3_ERR_CUDA);
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return bail(D3_ERR_CUDA);
  c->n_sms = prop.multiProcessorCount;
  if (c->use_tc && prop.major != 10) return bail(D3_ERR_UNSUPPORTED);

  const size_t d = g.d_model, nq = static_cast<size_t>(g.n_q_heads) * g.d_head,
               nkv = static_cast<size_t>(g.n_kv_heads) * g.d_head, f = g.d_ffn;
  long long pre_rows = g.max_prefill_rows > 0 ? g.max_prefill_rows : static_cast<long long>(g.max_batch) * g.max_seq;
  long long dec_rows = static_cast<long long>(g.max_batch) * g.block;
  // d3_generate may run the finalize forward of a block together with the first step of the next one
  // (2 * block rows per sequence) while that still is a skinny forward: room for it
  if (2 * dec_rows <= FUSE_MAX_ROWS) dec_rows *= 2;
  // and for a few blocks in flight per sequence (d3_generate_multiblock) while the forward stays
  // on the skinny kernels (128 rows)
  dec_rows = std::max<long long>(dec_rows, 128);
  c->max_rows = static_cast<int>(std::max(pre_rows, dec_rows));
  const size_t R = c->max_rows;
#define A_(ptr, bytes)                                                         \
  do {                                                                         \
    int rc_ = dev_alloc(c, reinterpret_cast<void**>(&(ptr)), (bytes));         \
    if (rc_ != D3_OK) return bail(rc_);                                        \
  } while (0)
  c->kv_layer_elems = static_cast<size_t>(g.max_batch) * g.n_kv_heads * g.max_seq * g.d_head;
  A_(c->kv, c->kv_layer_elems * 2 * g.n_layers * c->esz);
  A_(c->rope_cos, sizeof(float) * g.max_seq * (g.d_head / 2));
  A_(c->rope_sin, sizeof(float) * g.max_seq * (g.d_head / 2));
  A_(c->x, sizeof(float) * R * d);
  A_(c->xn, c->esz * R * std::max(d, nq));
  if (c->fold_norm) {
    A_(c->xb, sizeof(bf16) * R * d);
    A_(c->ssq, sizeof(float) * R * ((d + 31) / 32));
  }
  if (!c->fuse_qkv) A_(c->qkv_f32, sizeof(float) * R * (nq + 2 * nkv));
  A_(c->q, c->esz * R * nq);
  A_(c->o, c->esz * R * nq);
  A_(c->h, c->esz * R * f);
  const size_t n_tiles = (g.vocab + 127) / 128;
  A_(c->stat_part, sizeof(float4) * static_cast<size_t>(dec_rows) * n_tiles);
  A_(c->sample_part, sizeof(float4) * static_cast<size_t>(dec_rows) * n_tiles);
  A_(c->conf, sizeof(float) * dec_rows);
  A_(c->ent, sizeof(float) * dec_rows);
  A_(c->argmax, sizeof(int) * dec_rows);
  A_(c->prefix_len, sizeof(int) * g.max_batch);
  A_(c->pos_base, sizeof(int) * g.max_batch);
  A_(c->n_valid, sizeof(int) * g.max_batch);
  A_(c->kv_len, sizeof(int) * g.max_batch);
  A_(c->error_word, sizeof(uint32_t));
  if (c->use_tc) {
    c->partial_slots = 2048;
    A_(c->partial, c->partial_slots * 128 * 128 * sizeof(float));
    c->n_tile_count = 1 << 16;
    A_(c->tile_count, sizeof(int) * c->n_tile_count);
  }
  if (c->use_tc && g.d_head == 128) {
    const long long kv_rows = static_cast<long long>(g.n_layers) * 2 * g.max_batch * g.n_kv_heads * g.max_seq;
    if (kv_rows < (1ll << 31)) {
      const CUtensorMap* tm = nullptr;
      int rc_ = get_tmap(c, c->kv, static_cast<int>(kv_rows), 128, attn::KT, &tm);
      if (rc_ != D3_OK) return bail(rc_);
      c->kv_tmap = *tm;
      rc_ = get_tmap(c, c->kv, static_cast<int>(kv_rows), 128, tc::CHAIN_AKT, &tm);
      if (rc_ != D3_OK) return bail(rc_);
      c->kv_tmap32 = *tm;
      rc_ = get_tmap(c, c->kv, static_cast<int>(kv_rows), 128, 128, &tm);
      if (rc_ != D3_OK) return bail(rc_);
      c->kv_tmap128 = *tm;
      c->attn_tc = true;
    }
  }
  A_(c->gen.mode, sizeof(int) * g.max_batch);
  A_(c->gen.block_idx, sizeof(int) * g.max_batch);
  A_(c->gen.step, sizeof(int) * g.max_batch);
  c->gen.prefix_len = c->prefix_len;
  A_(c->gen.ids, sizeof(int) * dec_rows);
  A_(c->gen.mask, sizeof(uint8_t) * dec_rows);
  A_(c->gen.prev, sizeof(int) * dec_rows);
  c->stat_rows = static_cast<int>(dec_rows);
  c->mb.prefix_len = c->prefix_len;
  c->mb.counters = nullptr;  // shares gen.counters (set below)
  A_(c->mb.lo, sizeof(int) * g.max_batch);
  A_(c->mb.n_win, sizeof(int) * g.max_batch);
  A_(c->mb.ids, sizeof(int) * static_cast<size_t>(g.max_batch) * MB_MAX_WINDOW * g.block);
  A_(c->mb.mask, sizeof(uint8_t) * static_cast<size_t>(g.max_batch) * MB_MAX_WINDOW * g.block);
  A_(c->mb.fwd_ids, sizeof(int) * static_cast<size_t>(g.max_batch) * MB_MAX_WINDOW * g.block);
  A_(c->gen.fwd_ids, sizeof(int) * 2 * static_cast<size_t>(g.max_batch) * g.block);
  A_(c->gen.counters, sizeof(long long) * 8);
  A_(c->commit_hist, sizeof(unsigned long long) * COMMIT_HIST_BINS);
  c->gen.commit_hist = c->commit_hist;
  c->mb.commit_hist = c->commit_hist;
  c->gen.error_word = c->error_word;
  c->mb.error_word = c->error_word;
  A_(c->hist_ids, sizeof(int) * static_cast<size_t>(g.max_batch) * g.max_seq);
  A_(c->refresh_ids, sizeof(int) * R);
  A_(c->gen.refresh_flag, sizeof(int) * g.max_batch);
  A_(c->mb.stab, sizeof(int) * static_cast<size_t>(g.max_batch) * MB_MAX_WINDOW);
  c->gen.hist = c->hist_ids;
  c->mb.hist = c->hist_ids;
  if (cudaMallocHost(reinterpret_cast<void**>(&c->host_counters), sizeof(long long) * 8) != cudaSuccess)
    return bail(D3_ERR_OOM);
  c->tap_rows = static_cast<int>(dec_rows);
  A_(c->tap_in, sizeof(float) * dec_rows * d);
  A_(c->tap_out, sizeof(float) * dec_rows * d);
#undef A_
  // RoPE table in double precision on the host
  {
    const int half = g.d_head / 2;
    std::vector<float> cs(static_cast<size_t>(g.max_seq) * half), sn(cs.size());
    for (int k = 0; k < half; ++k) {
      const double inv = std::pow(static_cast<double>(g.rope_theta), -2.0 * k / g.d_head);
      for (int p = 0; p < g.max_seq; ++p) {
        const double a = p * inv;
        cs[static_cast<size_t>(p) * half + k] = static_cast<float>(std::cos(a));
        sn[static_cast<size_t>(p) * half + k] = static_cast<float>(std::sin(a));
      }
    }
    if (cudaMemcpyAsync(c->rope_cos, cs.data(), cs.size() * 4, cudaMemcpyHostToDevice, c->stream) != cudaSuccess ||
        cudaMemcpyAsync(c->rope_sin, sn.data(), sn.size() * 4, cudaMemcpyHostToDevice, c->stream) != cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess)
      return bail(D3_ERR_CUDA);
  }
  *out = c;
  return D3_OK;
}

extern "C" void d3_destroy(d3_ctx* c) {
  if (!c) return;
  cudaStreamSynchronize(c->stream);
  for (auto& pp : c->prof_pool) {
    cudaEventDestroy(pp.a);
    cudaEventDestroy(pp.b);
  }
  for (void* p : c->allocs) cudaFree(p);
  if (c->host_counters) cudaFreeHost(c->host_counters);
  delete c;
}

// ----------------------------------------------------------------------------- weights
namespace {
int upload(d3_ctx* c, void* dst, const void* src, size_t bytes, int src_is_device) {
  CUDA_TRY(c, cudaMemcpyAsync(dst, src, bytes, src_is_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, c->stream));
  return D3_OK;
}
int load_gain(d3_ctx* c, float** dst, const void* src, int src_is_device, void* tmp) {
  const size_t d = c->cfg.d_model;
  if (!*dst) ALLOC(c, *dst, sizeof(float) * d);
  if (!src) {
    std::vector<float> ones(d, 1.0f);
    CUDA_TRY(c, cudaMemcpyAsync(*dst, ones.data(), sizeof(float) * d, cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    return D3_OK;
  }
  TRY(upload(c, tmp, src, c->esz * d, src_is_device));
  if (c->is_bf16) cast_to_f32<bf16>(c, tmp, *dst, d);
  else cast_to_f32<float>(c, tmp, *dst, d);
  return D3_OK;
}
}  // namespace

// Elements of the stored form of an [n, k] matrix: row-major as given, or padded to whole
// 128 x 64 blocks for the tiled layout.
static size_t stored_elems(const d3_ctx* c, size_t n, size_t k) {
  if (!c->w_tiled) return n * k;
  return ((n + 127) / 128) * ((k + 63) / 64) * 128 * 64;
}

namespace {
// Final store of one assembled row-major matrix `rm` [n, k]: tiled blocks on the tensor-core path,
// a plain copy otherwise (then `rm` already is the final buffer and nothing is done).
int finish_matrix(d3_ctx* c, void* rm, void* dst, size_t n, size_t k, const float* fold_gain = nullptr) {
  if (!c->w_tiled) return D3_OK;
  if (fold_gain != nullptr && c->fold_norm) {  // the norm in front of this matmul becomes a row factor: its gains go into the columns
    // rows go in grid.y, chunked to the 65535 limit
    for (size_t r0 = 0; r0 < n; r0 += 65535) {
      const unsigned rows = static_cast<unsigned>(std::min<size_t>(65535, n - r0));
      scale_columns_kernel<<<dim3(static_cast<unsigned>((k + 255) / 256), rows), 256, 0, c->stream>>>(
          static_cast<bf16*>(rm) + r0 * k, fold_gain, static_cast<int>(k));
    }
    TRY(check_launch(c, "scale_columns_kernel"));
  }
  dim3 grid(static_cast<unsigned>((k + 63) / 64), static_cast<unsigned>((n + 127) / 128));
  pack_tiled_kernel<<<grid, 256, 0, c->stream>>>(static_cast<const bf16*>(rm), static_cast<bf16*>(dst), static_cast<int>(n),
                                                 static_cast<int>(k));
  return check_launch(c, "pack_tiled_kernel");
}
}  // namespace

extern "C" int d3_load_weights(d3_ctx* c, const d3_weights* w, int src_is_device) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!w || !w->tok_emb || !w->lm_head || !w->wq || !w->wk || !w->wv || !w->wo || !w->w_gate || !w->w_up || !w->w_down)
    return fail(c, D3_ERR_INVALID_ARG, "null weight pointer");
  const d3_config& g = c->cfg;
  const size_t d = g.d_model, nq = static_cast<size_t>(g.n_q_heads) * g.d_head,
               nkv = static_cast<size_t>(g.n_kv_heads) * g.d_head, f = g.d_ffn, V = g.vocab, e = c->esz;
  for (int l = 0; l < g.n_layers; ++l)
    if (!w->wq[l] || !w->wk[l] || !w->wv[l] || !w->wo[l] || !w->w_gate[l] || !w->w_up[l] || !w->w_down[l])
      return fail(c, D3_ERR_INVALID_ARG, "null per-layer weight pointer");
  if (!c->tok_emb) {
    ALLOC(c, c->tok_emb, V * d * e);
    ALLOC(c, c->lm_head, stored_elems(c, V, d) * e);
    c->wqkv.assign(g.n_layers, nullptr); c->wo.assign(g.n_layers, nullptr);
    c->wgu.assign(g.n_layers, nullptr); c->wd.assign(g.n_layers, nullptr);
    c->attn_norm.assign(g.n_layers, nullptr); c->ffn_norm.assign(g.n_layers, nullptr);
    for (int l = 0; l < g.n_layers; ++l) {
      ALLOC(c, c->wqkv[l], stored_elems(c, nq + 2 * nkv, d) * e);
      ALLOC(c, c->wo[l], stored_elems(c, d, nq) * e);
      ALLOC(c, c->wgu[l], stored_elems(c, 2 * f, d) * e);
      ALLOC(c, c->wd[l], stored_elems(c, d, f) * e);
    }
  }
  // Staging: tg / tu take one uploaded source matrix each; on the tiled path `rm` holds the
  // assembled row-major matrix (RoPE-pair permuted q/k rows + v, interleaved gate/up, or a matrix as
  // given) before it is cut into blocks; otherwise matrices are assembled in place.
  void *tg = nullptr, *tu = nullptr, *tgain = nullptr, *rm = nullptr;
  const size_t rm_elems = std::max(std::max(V * d, 2 * f * d), std::max((nq + 2 * nkv) * d, d * nq));
  cudaError_t ea = cudaMalloc(&tg, std::max(f, nq) * d * e);
  if (ea == cudaSuccess) ea = cudaMalloc(&tu, f * d * e);
  if (ea == cudaSuccess) ea = cudaMalloc(&tgain, d * e);
  if (ea == cudaSuccess && c->w_tiled) ea = cudaMalloc(&rm, rm_elems * e);
  if (ea != cudaSuccess) {
    (void)cudaGetLastError();
    cudaFree(tg); cudaFree(tu); cudaFree(tgain); cudaFree(rm);
    return fail(c, D3_ERR_OOM, std::string("staging buffers for the weight load: ") + cudaGetErrorString(ea));
  }
  int rc = D3_OK;
  auto step = [&](int r) { if (rc == D3_OK) rc = r; };
  auto target = [&](void* final_buf) { return c->w_tiled ? rm : final_buf; };
  step(upload(c, c->tok_emb, w->tok_emb, V * d * e, src_is_device));
  step(load_gain(c, &c->final_norm, w->final_norm, src_is_device, tgain));
  step(upload(c, target(c->lm_head), w->lm_head, V * d * e, src_is_device));
  step(finish_matrix(c, rm, c->lm_head, V, d, c->final_norm));
  for (int l = 0; l < g.n_layers && rc == D3_OK; ++l) {
    step(load_gain(c, &c->attn_norm[l], w->attn_norm ? w->attn_norm[l] : nullptr, src_is_device, tgain));
    step(load_gain(c, &c->ffn_norm[l], w->ffn_norm ? w->ffn_norm[l] : nullptr, src_is_device, tgain));
    // ---- q, k (rows permuted so that each RoPE pair of a head is adjacent) and v
    char* qkv = static_cast<char*>(target(c->wqkv[l]));
    for (int which = 0; which < 2 && rc == D3_OK; ++which) {
      const size_t rows = which == 0 ? nq : nkv;
      char* dst = qkv + (which == 0 ? 0 : nq * d * e);
      step(upload(c, tg, which == 0 ? w->wq[l] : w->wk[l], rows * d * e, src_is_device));
      if (rc != D3_OK) break;
      if (c->is_bf16)
        pack_rope_rows_kernel<bf16><<<static_cast<unsigned>(rows), 128, 0, c->stream>>>(static_cast<const bf16*>(tg), reinterpret_cast<bf16*>(dst), g.d_head, g.d_model);
      else
        pack_rope_rows_kernel<float><<<static_cast<unsigned>(rows), 128, 0, c->stream>>>(static_cast<const float*>(tg), reinterpret_cast<float*>(dst), g.d_head, g.d_model);
      step(check_launch(c, "pack_rope_rows_kernel"));
    }
    step(upload(c, qkv + (nq + nkv) * d * e, w->wv[l], nkv * d * e, src_is_device));
    step(finish_matrix(c, rm, c->wqkv[l], nq + 2 * nkv, d, c->attn_norm[l]));
    // ---- o, down: as given
    step(upload(c, target(c->wo[l]), w->wo[l], d * nq * e, src_is_device));
    step(finish_matrix(c, rm, c->wo[l], d, nq));
    step(upload(c, target(c->wd[l]), w->w_down[l], d * f * e, src_is_device));
    step(finish_matrix(c, rm, c->wd[l], d, f));
    // ---- gate / up: rows interleaved
    step(upload(c, tg, w->w_gate[l], f * d * e, src_is_device));
    step(upload(c, tu, w->w_up[l], f * d * e, src_is_device));
    if (rc == D3_OK) {
      void* gu = target(c->wgu[l]);
      if (c->is_bf16)
        interleave_gate_up_kernel<bf16><<<static_cast<unsigned>(2 * f), 128, 0, c->stream>>>(static_cast<const bf16*>(tg), static_cast<const bf16*>(tu), static_cast<bf16*>(gu), g.d_ffn, g.d_model);
      else
        interleave_gate_up_kernel<float><<<static_cast<unsigned>(2 * f), 128, 0, c->stream>>>(static_cast<const float*>(tg), static_cast<const float*>(tu), static_cast<float*>(gu), g.d_ffn, g.d_model);
      step(check_launch(c, "interleave_gate_up_kernel"));
    }
    step(finish_matrix(c, rm, c->wgu[l], 2 * f, d, c->ffn_norm[l]));
    // the staging buffers are reused by the next matrix: everything above is stream-ordered
  }
  cudaError_t es = cudaStreamSynchronize(c->stream);
  cudaFree(tg); cudaFree(tu); cudaFree(tgain); cudaFree(rm);
  if (rc != D3_OK) return rc;
  if (es != cudaSuccess) return fail(c, D3_ERR_CUDA, std::string("sync after weight load: ") + cudaGetErrorString(es));
  c->weights_loaded = true;
  return D3_OK;
}

// ----------------------------------------------------------------------------- decoding path
extern "C" int d3_prefill(d3_ctx* c, const int32_t* prompt_ids, const int32_t* prompt_lens, int32_t bs, int32_t p_max) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!prompt_lens || (!prompt_ids && p_max > 0) || bs <= 0 || p_max < 0) return fail(c, D3_ERR_INVALID_ARG, "bad prefill arguments");
  if (!c->weights_loaded) return fail(c, D3_ERR_STATE, "d3_prefill before d3_load_weights");
  if (bs > c->cfg.max_batch || p_max > c->cfg.max_seq || static_cast<long long>(bs) * p_max > c->max_rows)
    return fail(c, D3_ERR_SHAPE, "prefill larger than max_batch / max_seq / max_prefill_rows");
  prefill_rowmap_kernel<<<(bs + 63) / 64, 64, 0, c->stream>>>(prompt_lens, bs, p_max, c->prefix_len, c->pos_base, c->n_valid, c->kv_len);
  LAUNCHED(c, "prefill_rowmap_kernel");
  TRY(forward(c, prompt_ids, bs, p_max, 0, nullptr));
  if (p_max > 0) {
    hist_store_kernel<<<bs, 128, 0, c->stream>>>(prompt_ids, p_max, c->prefix_len, 0, nullptr, c->hist_ids, c->cfg.max_seq);
    LAUNCHED(c, "hist_store_kernel");
  }
  c->prefilled = true;
  c->explicit_step = 0;
  return D3_OK;
}

// One forward over the stored prefixes (flags null: every sequence; else the flagged ones, and only
// sequences with active[b] > 0 when that is given); their K/V are overwritten in place.
static int refresh_forward(d3_ctx* c, int bs, int* flags, const int* active, long long* pending) {
  std::vector<int> pl(bs);
  CUDA_TRY(c, cudaMemcpyAsync(pl.data(), c->prefix_len, sizeof(int) * bs, cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  int p_max = 0;
  for (int b = 0; b < bs; ++b) p_max = std::max(p_max, pl[b]);
  if (p_max > c->cfg.max_seq || static_cast<long long>(bs) * p_max > c->max_rows)
    return fail(c, D3_ERR_SHAPE, "KV-refresh: bs * longest stored prefix exceeds the workspaces (raise max_prefill_rows at d3_create)");
  if (p_max == 0) return D3_OK;
  refresh_rowmap_kernel<<<bs, 128, 0, c->stream>>>(c->hist_ids, c->cfg.max_seq, c->prefix_len, flags, active, p_max, 0, c->refresh_ids,
                                                   c->pos_base, c->n_valid, c->kv_len, pending);
  LAUNCHED(c, "refresh_rowmap_kernel");
  TRY(forward(c, c->refresh_ids, bs, p_max, 0, nullptr));
  return D3_OK;
}

extern "C" int d3_refresh_cache(d3_ctx* c, int32_t bs) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (bs <= 0) return fail(c, D3_ERR_INVALID_ARG, "bad refresh_cache arguments");
  if (!c->prefilled) return fail(c, D3_ERR_STATE, "d3_refresh_cache before d3_prefill");
  if (bs > c->cfg.max_batch) return fail(c, D3_ERR_SHAPE, "bs > max_batch");
  return refresh_forward(c, bs, nullptr, nullptr, nullptr);
}

extern "C" int d3_set_cache_policy(d3_ctx* c, int32_t cache_delay, int32_t refresh_every) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (cache_delay < 1 || cache_delay > 16 || refresh_every < 0) return fail(c, D3_ERR_INVALID_ARG, "cache_delay must be 1..16 and refresh_every >= 0");
  c->cache_delay = cache_delay;
  c->refresh_every = refresh_every;
  return D3_OK;
}
extern "C" int64_t d3_refresh_count(d3_ctx* c) { return c ? c->last_refreshes : 0; }

extern "C" int d3_denoise_step(d3_ctx* c, int32_t* block_ids, uint8_t* mask, float threshold, int32_t bs,
                               int32_t* out_pos, int32_t* out_ids, int32_t* out_count) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!block_ids || !mask || !out_pos || !out_ids || !out_count || bs <= 0 || std::isnan(threshold))
    return fail(c, D3_ERR_INVALID_ARG, "bad denoise_step arguments");
  if (!c->prefilled) return fail(c, D3_ERR_STATE, "d3_denoise_step before d3_prefill");
  if (bs > c->cfg.max_batch) return fail(c, D3_ERR_SHAPE, "bs > max_batch");
  const int B = c->cfg.block;
  decode_rowmap_kernel<<<(bs + 63) / 64, 64, 0, c->stream>>>(c->prefix_len, bs, B, c->pos_base, c->n_valid, c->kv_len);
  LAUNCHED(c, "decode_rowmap_kernel");
  c->draw_step = nullptr;  // sampling noise of the explicit calls: steps counted since the last prefill / commit
  c->draw_step_add = ++c->explicit_step;
  TRY(forward(c, block_ids, bs, B, 1, nullptr));
  unmask_kernel<<<bs, 32, 0, c->stream>>>(c->conf, c->ent, c->argmax, block_ids, mask, B, threshold, c->cfg.decide_mode, out_pos, out_ids, out_count, c->error_word);
  LAUNCHED(c, "unmask_kernel");
  return D3_OK;
}

extern "C" int d3_commit_block(d3_ctx* c, const int32_t* block_ids, int32_t bs) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!block_ids || bs <= 0) return fail(c, D3_ERR_INVALID_ARG, "bad commit_block arguments");
  if (!c->prefilled) return fail(c, D3_ERR_STATE, "d3_commit_block before d3_prefill");
  if (bs > c->cfg.max_batch) return fail(c, D3_ERR_SHAPE, "bs > max_batch");
  const int B = c->cfg.block;
  decode_rowmap_kernel<<<(bs + 63) / 64, 64, 0, c->stream>>>(c->prefix_len, bs, B, c->pos_base, c->n_valid, c->kv_len);
  LAUNCHED(c, "decode_rowmap_kernel");
  TRY(forward(c, block_ids, bs, B, 0, nullptr));
  hist_store_kernel<<<bs, 128, 0, c->stream>>>(block_ids, B, nullptr, B, c->prefix_len, c->hist_ids, c->cfg.max_seq);
  LAUNCHED(c, "hist_store_kernel");
  add_prefix_kernel<<<(bs + 63) / 64, 64, 0, c->stream>>>(c->prefix_len, bs, B);
  LAUNCHED(c, "add_prefix_kernel");
  c->explicit_step = 0;
  return D3_OK;
}

extern "C" int d3_generate(d3_ctx* c, int32_t gen_len, float threshold, int32_t bs, int32_t* out_ids,
                           int32_t* commit_step, d3_stats* host_stats) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!out_ids || bs <= 0 || gen_len <= 0 || std::isnan(threshold)) return fail(c, D3_ERR_INVALID_ARG, "bad generate arguments");
  if (!c->prefilled) return fail(c, D3_ERR_STATE, "d3_generate before d3_prefill");
  const int B = c->cfg.block;
  if (bs > c->cfg.max_batch || gen_len % B != 0) return fail(c, D3_ERR_SHAPE, "bs > max_batch or gen_len not a multiple of the block size");
  {  // prefix + gen_len must fit the cache
    std::vector<int> pl(bs);
    CUDA_TRY(c, cudaMemcpyAsync(pl.data(), c->prefix_len, sizeof(int) * bs, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    for (int b = 0; b < bs; ++b)
      if (pl[b] + gen_len > c->cfg.max_seq) return fail(c, D3_ERR_SHAPE, "prefix + gen_len exceeds max_seq");
  }
  const int n_blocks = gen_len / B;
  const int64_t launches0 = c->launches;
  GenState g = c->gen;
  g.out_ids = out_ids;
  g.commit_step = commit_step;
  gen_init_kernel<<<bs, 32, 0, c->stream>>>(g, bs, B, c->cfg.mask_id, gen_len);
  LAUNCHED(c, "gen_init_kernel");
  const long long max_iter = static_cast<long long>(n_blocks) * (B + 1) + 1;
  // (a refresh falls between a block's finalize forward and the next block's first step: no fusing then)
  const int fuse = (c->gen_fuse && c->refresh_every == 0 && 2ll * bs * B <= FUSE_MAX_ROWS && 2ll * c->cfg.max_batch * B <= FUSE_MAX_ROWS) ? 1 : 0;
  long long steps = 0;
  c->last_refreshes = 0;
  c->draw_step = g.step;  // sampling noise: each sequence's step within its block (the counter is bumped after the forward)
  c->draw_step_add = 1;
  int R = B;  // rows per sequence of the next forward: 2B while some sequence runs a fused finalize + first step
  for (long long it = 0; it < max_iter; ++it) {
    gen_rowmap_kernel<<<bs, 64, 0, c->stream>>>(g, bs, B, R, c->cfg.mask_id, c->pos_base, c->n_valid, c->kv_len);
    LAUNCHED(c, "gen_rowmap_kernel");
    TRY(forward(c, g.fwd_ids, bs, R, 1, nullptr, R > B ? B : 0));
    gen_advance_kernel<<<bs, 32, 0, c->stream>>>(g, c->conf, c->ent, c->argmax, bs, B, R, n_blocks, gen_len, threshold, c->cfg.decide_mode, c->cfg.mask_id, fuse, c->eos_id,
                                                 c->cfg.max_seq, c->refresh_every);
    LAUNCHED(c, "gen_advance_kernel");
    ++steps;
    CUDA_TRY(c, cudaMemcpyAsync(c->host_counters, g.counters, sizeof(long long) * 8, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    if (c->host_counters[4] <= 0) break;
    if (c->host_counters[7] > 0) {  // some sequences stored a block that completes a refresh period
      c->last_refreshes += c->host_counters[7];
      TRY(refresh_forward(c, bs, g.refresh_flag, nullptr, g.counters + 7));
    }
    R = c->host_counters[5] > 0 ? 2 * B : B;
  }
  c->last_early_stops = c->host_counters[6];
  if (host_stats) {
    std::memset(host_stats, 0, sizeof(*host_stats));
    host_stats->denoise_forwards = c->host_counters[0];
    host_stats->finalize_forwards = c->host_counters[1];
    host_stats->tokens_committed = c->host_counters[2];
    host_stats->forced_commits = c->host_counters[3];
    host_stats->steps = steps;
    host_stats->kernel_launches = c->launches - launches0;
  }
  if (c->host_counters[4] > 0) return fail(c, D3_ERR_STATE, "generate loop did not finish within its step bound");
  return check_device_error(c);
}

extern "C" int d3_generate_multiblock(d3_ctx* c, int32_t gen_len, float threshold, int32_t bs, int32_t max_active,
                                      int32_t* out_ids, int32_t* commit_round, d3_stats* host_stats) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!out_ids || bs <= 0 || gen_len <= 0 || std::isnan(threshold) || max_active < 1 || max_active > MB_MAX_WINDOW)
    return fail(c, D3_ERR_INVALID_ARG, "bad generate_multiblock arguments");
  if (!c->prefilled) return fail(c, D3_ERR_STATE, "d3_generate_multiblock before d3_prefill");
  const int B = c->cfg.block;
  if (bs > c->cfg.max_batch || gen_len % B != 0) return fail(c, D3_ERR_SHAPE, "bs > max_batch or gen_len not a multiple of the block size");
  if (static_cast<long long>(bs) * max_active * B > std::min<long long>(c->stat_rows, c->max_rows))
    return fail(c, D3_ERR_SHAPE, "bs * max_active * block rows exceed the workspaces (raise max_batch at d3_create)");
  {
    std::vector<int> pl(bs);
    CUDA_TRY(c, cudaMemcpyAsync(pl.data(), c->prefix_len, sizeof(int) * bs, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    for (int b = 0; b < bs; ++b)
      if (pl[b] + gen_len > c->cfg.max_seq) return fail(c, D3_ERR_SHAPE, "prefix + gen_len exceeds max_seq");
  }
  const int n_blocks = gen_len / B;
  const int W = MB_MAX_WINDOW;
  const int64_t launches0 = c->launches;
  MbState g = c->mb;
  g.counters = c->gen.counters;
  g.out_ids = out_ids;
  g.commit_round = commit_round;
  mb_init_kernel<<<bs, 64, 0, c->stream>>>(g, bs, B, W, c->cfg.mask_id, gen_len);
  LAUNCHED(c, "mb_init_kernel");
  const long long max_iter = static_cast<long long>(n_blocks) * (B + c->cache_delay) + 1;
  long long rounds = 0;
  c->last_refreshes = 0;
  int R = B;
  for (long long it = 0; it < max_iter; ++it) {
    mb_rowmap_kernel<<<bs, 64, 0, c->stream>>>(g, bs, B, W, R, c->cfg.mask_id, c->pos_base, c->n_valid, c->kv_len);
    LAUNCHED(c, "mb_rowmap_kernel");
    c->draw_step = nullptr;  // sampling noise of a round: keyed by the round
    c->draw_step_add = static_cast<int>(rounds + 1);
    TRY(forward(c, g.fwd_ids, bs, R, 1, nullptr, B));
    ++rounds;
    mb_advance_kernel<<<bs, 32, 0, c->stream>>>(g, c->conf, c->ent, c->argmax, bs, B, W, R, n_blocks, gen_len, threshold,
                                                c->cfg.decide_mode, c->cfg.mask_id, max_active, static_cast<int>(rounds), c->cache_delay,
                                                c->cfg.max_seq, c->eos_id);
    LAUNCHED(c, "mb_advance_kernel");
    CUDA_TRY(c, cudaMemcpyAsync(c->host_counters, g.counters, sizeof(long long) * 8, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    if (c->host_counters[4] <= 0) break;
    if (c->refresh_every > 0 && rounds % c->refresh_every == 0) {  // periodic KV-refresh of the sequences still decoding
      c->last_refreshes += c->host_counters[4];
      TRY(refresh_forward(c, bs, nullptr, g.n_win, nullptr));
    }
    R = static_cast<int>(std::max<long long>(1, c->host_counters[5])) * B;
  }
  if (host_stats) {
    std::memset(host_stats, 0, sizeof(*host_stats));
    host_stats->denoise_forwards = c->host_counters[0];
    host_stats->finalize_forwards = c->host_counters[1];
    host_stats->tokens_committed = c->host_counters[2];
    host_stats->forced_commits = c->host_counters[3];
    host_stats->steps = rounds;
    host_stats->kernel_launches = c->launches - launches0;
  }
  c->last_early_stops = c->host_counters[7];
  if (c->host_counters[4] > 0) return fail(c, D3_ERR_STATE, "multi-block loop did not finish within its round bound");
  return check_device_error(c);
}

extern "C" int d3_trajectory_rank(d3_ctx* c, const int32_t* commit_step, int32_t bs, int32_t gen_len, int32_t* rank) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!commit_step || !rank || bs <= 0 || gen_len <= 0) return fail(c, D3_ERR_INVALID_ARG, "bad trajectory_rank arguments");
  if (gen_len % c->cfg.block != 0) return fail(c, D3_ERR_SHAPE, "gen_len not a multiple of the block size");
  trajectory_rank_kernel<<<bs, 32, 0, c->stream>>>(commit_step, gen_len, c->cfg.block, rank);
  LAUNCHED(c, "trajectory_rank_kernel");
  return D3_OK;
}
extern "C" int d3_noisy_sequence(d3_ctx* c, const int32_t* y, const int32_t* rank, const int32_t* s, const int32_t* k,
                                 const int32_t* m, int32_t bs, int32_t n, int32_t* out) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!y || !rank || !s || !k || !m || !out || bs <= 0 || n <= 0) return fail(c, D3_ERR_INVALID_ARG, "bad noisy_sequence arguments");
  if (bs > 65535) return fail(c, D3_ERR_SHAPE, "more than 65535 sequences in one call");
  noisy_sequence_kernel<<<dim3((n + 255) / 256, bs), 256, 0, c->stream>>>(y, rank, s, k, m, n, c->cfg.mask_id, out);
  LAUNCHED(c, "noisy_sequence_kernel");
  return D3_OK;
}

extern "C" int d3_set_sampling(d3_ctx* c, float temperature, uint64_t seed) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!(temperature >= 0.f) || !std::isfinite(temperature)) return fail(c, D3_ERR_INVALID_ARG, "temperature must be finite and >= 0");
  c->temperature = temperature;
  c->seed = seed;
  return D3_OK;
}

extern "C" int d3_set_eos(d3_ctx* c, int32_t eos_id) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (eos_id >= c->cfg.vocab || eos_id == c->cfg.mask_id) return fail(c, D3_ERR_INVALID_ARG, "eos id outside the vocabulary or equal to the mask id");
  c->eos_id = eos_id < 0 ? -1 : eos_id;
  return D3_OK;
}
extern "C" int64_t d3_early_stops(d3_ctx* c) { return c ? c->last_early_stops : 0; }

extern "C" int d3_get_step_stats(d3_ctx* c, float* conf, float* entropy, int32_t* argmax, int32_t bs) {
  if (!c || bs <= 0 || bs > c->cfg.max_batch) return D3_ERR_INVALID_ARG;
  const size_t n = static_cast<size_t>(bs) * c->cfg.block;
  if (conf) CUDA_TRY(c, cudaMemcpyAsync(conf, c->conf, n * 4, cudaMemcpyDeviceToDevice, c->stream));
  if (entropy) CUDA_TRY(c, cudaMemcpyAsync(entropy, c->ent, n * 4, cudaMemcpyDeviceToDevice, c->stream));
  if (argmax) CUDA_TRY(c, cudaMemcpyAsync(argmax, c->argmax, n * 4, cudaMemcpyDeviceToDevice, c->stream));
  return D3_OK;
}

extern "C" int d3_forward_logits(d3_ctx* c, const int32_t* block_ids, int32_t bs, float* logits) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!block_ids || !logits || bs <= 0) return fail(c, D3_ERR_INVALID_ARG, "bad forward_logits arguments");
  if (!c->prefilled) return fail(c, D3_ERR_STATE, "d3_forward_logits before d3_prefill");
  if (bs > c->cfg.max_batch) return fail(c, D3_ERR_SHAPE, "bs > max_batch");
  const int B = c->cfg.block;
  decode_rowmap_kernel<<<(bs + 63) / 64, 64, 0, c->stream>>>(c->prefix_len, bs, B, c->pos_base, c->n_valid, c->kv_len);
  LAUNCHED(c, "decode_rowmap_kernel");
  return forward(c, block_ids, bs, B, 2, logits);
}

extern "C" int d3_denoise_window(d3_ctx* c, const int32_t* window_ids, int32_t bs, int32_t n_win, float* conf,
                                 float* entropy, int32_t* argmax) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!window_ids || bs <= 0 || n_win < 1 || n_win > MB_MAX_WINDOW) return fail(c, D3_ERR_INVALID_ARG, "bad denoise_window arguments");
  if (!c->prefilled) return fail(c, D3_ERR_STATE, "d3_denoise_window before d3_prefill");
  const int B = c->cfg.block;
  const long long rows = static_cast<long long>(bs) * n_win * B;
  if (bs > c->cfg.max_batch || rows > std::min<long long>(c->stat_rows, c->max_rows))
    return fail(c, D3_ERR_SHAPE, "bs * n_win * block rows exceed the workspaces (raise max_batch at d3_create)");
  decode_rowmap_kernel<<<(bs + 63) / 64, 64, 0, c->stream>>>(c->prefix_len, bs, n_win * B, c->pos_base, c->n_valid, c->kv_len);
  LAUNCHED(c, "decode_rowmap_kernel");
  c->draw_step = nullptr;
  c->draw_step_add = ++c->explicit_step;
  TRY(forward(c, window_ids, bs, n_win * B, 1, nullptr, B));
  const size_t n = static_cast<size_t>(rows);
  if (conf) CUDA_TRY(c, cudaMemcpyAsync(conf, c->conf, n * 4, cudaMemcpyDeviceToDevice, c->stream));
  if (entropy) CUDA_TRY(c, cudaMemcpyAsync(entropy, c->ent, n * 4, cudaMemcpyDeviceToDevice, c->stream));
  if (argmax) CUDA_TRY(c, cudaMemcpyAsync(argmax, c->argmax, n * 4, cudaMemcpyDeviceToDevice, c->stream));
  return D3_OK;
}

extern "C" int d3_set_tap(d3_ctx* c, int32_t layer) {
  if (!c || layer >= c->cfg.n_layers) return D3_ERR_INVALID_ARG;
  c->tap_layer = layer < 0 ? -1 : layer;
  return D3_OK;
}

extern "C" int d3_read_tap(d3_ctx* c, float* resid_in, float* resid_out, int32_t rows) {
  if (!c || rows <= 0 || rows > c->tap_rows) return D3_ERR_INVALID_ARG;
  const size_t n = static_cast<size_t>(rows) * c->cfg.d_model * sizeof(float);
  if (resid_in) CUDA_TRY(c, cudaMemcpyAsync(resid_in, c->tap_in, n, cudaMemcpyDeviceToDevice, c->stream));
  if (resid_out) CUDA_TRY(c, cudaMemcpyAsync(resid_out, c->tap_out, n, cudaMemcpyDeviceToDevice, c->stream));
  return D3_OK;
}

extern "C" int d3_read_kv(d3_ctx* c, int32_t layer, int32_t seq, int32_t pos0, int32_t n, float* k_out, float* v_out) {
  if (!c) return D3_ERR_INVALID_ARG;
  const d3_config& g = c->cfg;
  if (layer < 0 || layer >= g.n_layers || seq < 0 || seq >= g.max_batch || pos0 < 0 || n <= 0 || pos0 + n > g.max_seq)
    return fail(c, D3_ERR_INVALID_ARG, "bad read_kv range");
  for (int hh = 0; hh < g.n_kv_heads; ++hh) {
    const size_t off = ((static_cast<size_t>(seq) * g.n_kv_heads + hh) * g.max_seq + pos0) * g.d_head;
    const size_t cnt = static_cast<size_t>(n) * g.d_head;
    for (int which = 0; which < 2; ++which) {
      float* dst = which == 0 ? k_out : v_out;
      if (!dst) continue;
      const char* src = static_cast<const char*>(which == 0 ? k_plane(c, layer) : v_plane(c, layer)) + off * c->esz;
      if (c->is_bf16) cast_to_f32<bf16>(c, src, dst + static_cast<size_t>(hh) * cnt, cnt);
      else cast_to_f32<float>(c, src, dst + static_cast<size_t>(hh) * cnt, cnt);
    }
  }
  cudaError_t e = cudaPeekAtLastError();
  if (e != cudaSuccess) return fail(c, D3_ERR_CUDA, std::string("cast_to_f32_kernel: ") + cudaGetErrorString(e));
  return D3_OK;
}

extern "C" int d3_get_state(d3_ctx* c, int32_t* prefix_len, int32_t bs) {
  if (!c || !prefix_len || bs <= 0 || bs > c->cfg.max_batch) return D3_ERR_INVALID_ARG;
  CUDA_TRY(c, cudaMemcpyAsync(prefix_len, c->prefix_len, sizeof(int) * bs, cudaMemcpyDeviceToDevice, c->stream));
  return D3_OK;
}
extern "C" int d3_set_state(d3_ctx* c, const int32_t* prefix_len, int32_t bs) {
  if (!c || !prefix_len || bs <= 0 || bs > c->cfg.max_batch) return D3_ERR_INVALID_ARG;
  CUDA_TRY(c, cudaMemcpyAsync(c->prefix_len, prefix_len, sizeof(int) * bs, cudaMemcpyDeviceToDevice, c->stream));
  c->prefilled = true;
  return D3_OK;
}

// ----------------------------------------------------------------------------- single operators
extern "C" int d3_op_linear(d3_ctx* c, const void* x, const void* w, void* y, int32_t m, int32_t n, int32_t k,
                            int32_t epilogue, int32_t splits) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!x || !w || !y || m <= 0 || n <= 0 || k <= 0 || epilogue < 0 || epilogue > 3)
    return fail(c, D3_ERR_INVALID_ARG, "bad op_linear arguments");
  if (epilogue == EPI_SWIGLU && n % 2 != 0) return fail(c, D3_ERR_SHAPE, "SwiGLU epilogue needs an even n");
  EpiParams ep;
  ep.y = y;
  ep.ldy = epilogue == EPI_SWIGLU ? n / 2 : n;
  return run_linear(c, x, w, m, n, k, epilogue, ep, splits);
}

extern "C" int64_t d3_packed_weight_elems(int32_t n, int32_t k) {
  if (n <= 0 || k <= 0) return 0;
  return static_cast<int64_t>((n + 127) / 128) * ((k + 63) / 64) * 128 * 64;
}

extern "C" int d3_pack_weight(d3_ctx* c, const void* w, int32_t n, int32_t k, void* packed) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!w || !packed || n <= 0 || k <= 0) return fail(c, D3_ERR_INVALID_ARG, "bad pack_weight arguments");
  if (!c->is_bf16) return fail(c, D3_ERR_UNSUPPORTED, "the tiled layout exists for bfloat16 only");
  dim3 grid(static_cast<unsigned>((k + 63) / 64), static_cast<unsigned>((n + 127) / 128));
  pack_tiled_kernel<<<grid, 256, 0, c->stream>>>(static_cast<const bf16*>(w), static_cast<bf16*>(packed), n, k);
  LAUNCHED(c, "pack_tiled_kernel");
  return D3_OK;
}

extern "C" int d3_op_linear_packed(d3_ctx* c, const void* x, const void* w_packed, void* y, int32_t m, int32_t n,
                                   int32_t k, int32_t epilogue, int32_t splits) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!x || !w_packed || !y || m <= 0 || n <= 0 || k <= 0 || epilogue < 0 || epilogue > 3)
    return fail(c, D3_ERR_INVALID_ARG, "bad op_linear_packed arguments");
  if (!c->use_tc) return fail(c, D3_ERR_UNSUPPORTED, "the tiled layout is read by the tensor-core matmul only");
  if (epilogue == EPI_SWIGLU && n % 2 != 0) return fail(c, D3_ERR_SHAPE, "SwiGLU epilogue needs an even n");
  EpiParams ep;
  ep.y = y;
  ep.ldy = epilogue == EPI_SWIGLU ? n / 2 : n;
  return run_linear(c, x, w_packed, m, n, k, epilogue, ep, splits, nullptr, D3_PROF_GEMM_OTHER, 1);
}

extern "C" int d3_op_lm_head_stats(d3_ctx* c, const void* x, const void* w, int32_t m, int32_t vocab, int32_t k,
                                   float scale, int32_t mask_id, float* conf, float* entropy, int32_t* argmax) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!x || !w || !conf || !entropy || !argmax || m <= 0 || vocab <= 0 || k <= 0)
    return fail(c, D3_ERR_INVALID_ARG, "bad op_lm_head_stats arguments");
  const int n_tiles = (vocab + 127) / 128;
  const size_t cap = static_cast<size_t>(c->cfg.max_batch) * c->cfg.block * ((c->cfg.vocab + 127) / 128);
  if (static_cast<size_t>(m) * n_tiles > cap) return fail(c, D3_ERR_SHAPE, "m * vocab tiles exceed the statistics workspace");
  EpiParams ep;
  ep.scale = scale; ep.mask_id = mask_id; ep.stat_part = c->stat_part; ep.n_tiles = n_tiles;
  TRY(run_linear(c, x, w, m, vocab, k, EPI_STATS, ep));
  return run_stats_merge(c, m, n_tiles, conf, entropy, argmax);
}

extern "C" int d3_op_attention(d3_ctx* c, const void* q, int32_t layer, int32_t bs, int32_t rows,
                               const int32_t* kv_len, void* out) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!q || !out || !kv_len || layer < 0 || layer >= c->cfg.n_layers || bs <= 0 || bs > c->cfg.max_batch || rows <= 0)
    return fail(c, D3_ERR_INVALID_ARG, "bad op_attention arguments");
  // all rows live, positions irrelevant here
  decode_rowmap_kernel<<<(bs + 63) / 64, 64, 0, c->stream>>>(kv_len, bs, rows, c->pos_base, c->n_valid, c->kv_len);
  LAUNCHED(c, "decode_rowmap_kernel");
  RowMap rm{c->pos_base, c->n_valid, kv_len, rows, bs, 0};
  return run_attention(c, q, layer, out, rm);
}

extern "C" int d3_op_write_kv(d3_ctx* c, int32_t layer, int32_t seq, int32_t pos0, int32_t n, const float* k, const float* v) {
  if (!c) return D3_ERR_INVALID_ARG;
  const d3_config& g = c->cfg;
  if (!k || !v || layer < 0 || layer >= g.n_layers || seq < 0 || seq >= g.max_batch || pos0 < 0 || n <= 0 || pos0 + n > g.max_seq)
    return fail(c, D3_ERR_INVALID_ARG, "bad op_write_kv range");
  for (int hh = 0; hh < g.n_kv_heads; ++hh) {
    const size_t off = ((static_cast<size_t>(seq) * g.n_kv_heads + hh) * g.max_seq + pos0) * g.d_head;
    const size_t cnt = static_cast<size_t>(n) * g.d_head;
    for (int which = 0; which < 2; ++which) {
      const float* src = (which == 0 ? k : v) + static_cast<size_t>(hh) * cnt;
      char* dst = static_cast<char*>(which == 0 ? k_plane(c, layer) : v_plane(c, layer)) + off * c->esz;
      const unsigned blocks = static_cast<unsigned>((cnt + 255) / 256);
      if (c->is_bf16) cast_from_f32_kernel<bf16><<<blocks, 256, 0, c->stream>>>(src, reinterpret_cast<bf16*>(dst), cnt);
      else cast_from_f32_kernel<float><<<blocks, 256, 0, c->stream>>>(src, reinterpret_cast<float*>(dst), cnt);
      LAUNCHED(c, "cast_from_f32_kernel");
    }
  }
  return D3_OK;
}

extern "C" int d3_op_unmask(d3_ctx* c, const float* conf, const float* entropy, const int32_t* argmax,
                            int32_t* block_ids, uint8_t* mask, float threshold, int32_t bs, int32_t* out_pos,
                            int32_t* out_ids, int32_t* out_count) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (!conf || !entropy || !argmax || !block_ids || !mask || !out_pos || !out_ids || !out_count || bs <= 0 ||
      std::isnan(threshold))
    return fail(c, D3_ERR_INVALID_ARG, "bad op_unmask arguments");
  unmask_kernel<<<bs, 32, 0, c->stream>>>(conf, entropy, argmax, block_ids, mask, c->cfg.block, threshold, c->cfg.decide_mode, out_pos, out_ids, out_count, c->error_word);
  LAUNCHED(c, "unmask_kernel");
  return D3_OK;
}

// ----------------------------------------------------------------------------- misc
extern "C" int d3_get_error_word(d3_ctx* c, uint32_t* word) {
  if (!c || !word) return D3_ERR_INVALID_ARG;
  CUDA_TRY(c, cudaMemcpyAsync(word, c->error_word, sizeof(uint32_t), cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  return D3_OK;
}
extern "C" void d3_tuning_defaults(d3_tuning* t) {
  if (!t) return;
  std::memset(t, 0, sizeof(*t));
  t->cluster_k_split = -1;
  t->row_tile_pairs = -1;
  t->round_robin = 1;
  t->chain = -1;
  t->chain_l2_ahead = -1;
  t->weights_as_rows = -1;
  t->attention_tmem = -1;
  t->cta_pairs = -1;
}
extern "C" int d3_set_tuning(d3_ctx* c, const d3_tuning* t) {
  if (!c || !t) return D3_ERR_INVALID_ARG;
  if (t->ring_kb < 0 || t->ring_kb > 224 || t->ctas_per_sm < 0 || t->ctas_per_sm > 3 || t->producers < 0 || t->producers > 2 ||
      (t->tile_columns != 0 && t->tile_columns != 128 && t->tile_columns != 256) || t->attn_key_tiles < 0 || t->attn_key_tiles > 7 ||
      t->cluster_k_split < -1 || t->cluster_k_split > 0 || t->row_tile_pairs < -1 || t->row_tile_pairs > 1 ||
      (t->round_robin != 0 && t->round_robin != 1) || t->column_strips < 0 || t->column_strips > 3 || t->strip_stages < 0 ||
      t->strip_stages > 32 || t->chain < -1 || t->chain > 0 || t->chain_clusters < 0 || t->chain_l2_ahead < -1 || t->chain_l2_ahead > 256 || t->weights_as_rows < -1 || t->weights_as_rows > 0 ||
      ((t->attention_tmem < -1 || t->attention_tmem > 2) && t->attention_tmem != 64 && t->attention_tmem != 128) ||
      t->cta_pairs < -1 || t->cta_pairs > 0)
    return fail(c, D3_ERR_INVALID_ARG, "d3_set_tuning: a field is outside its range");
  c->tune_ring_kb = t->ring_kb;
  c->tune_ctas_per_sm = t->ctas_per_sm;
  c->tune_producers = t->producers;
  c->tune_wide_tiles = t->tile_columns == 0 ? -1 : (t->tile_columns == 256 ? 1 : 0);
  c->tune_attn_div = t->attn_key_tiles;
  c->tune_no_cluster = t->cluster_k_split == 0 ? 1 : 0;
  c->tune_pair = t->row_tile_pairs;
  c->tune_no_rr = t->round_robin ? 0 : 1;
  c->tune_strip = t->column_strips;
  c->tune_strip_stages = t->strip_stages;
  c->tune_chain = t->chain;
  c->tune_chain_clusters = t->chain_clusters;
  c->tune_chain_l2 = t->chain_l2_ahead;
  c->tune_xt = t->weights_as_rows;
  c->tune_attn_tmem = t->attention_tmem > 1 ? 1 : t->attention_tmem;
  c->tune_attn_shape = t->attention_tmem > 1 ? t->attention_tmem : 0;
  c->tune_cta_pairs = t->cta_pairs;
  return D3_OK;
}
extern "C" int d3_set_fused_finalize(d3_ctx* c, int on) {
  if (!c) return D3_ERR_INVALID_ARG;
  c->gen_fuse = on != 0;
  return D3_OK;
}
extern "C" int d3_clear_error_word(d3_ctx* c) {
  if (!c) return D3_ERR_INVALID_ARG;
  CUDA_TRY(c, cudaMemsetAsync(c->error_word, 0, sizeof(uint32_t), c->stream));
  return D3_OK;
}
extern "C" int d3_debug_stall_probe(d3_ctx* c, int32_t limit_us) {
  if (!c) return D3_ERR_INVALID_ARG;
  if (limit_us < 1 || limit_us > 2000000) return fail(c, D3_ERR_INVALID_ARG, "limit_us must be 1..2000000");
  if (!c->use_tc) return fail(c, D3_ERR_UNSUPPORTED, "the probe runs the tensor-core matmul kernel (bfloat16 contexts only)");
  // One CTA, one 32 x 128 x 64 unit, no loads issued: the MMA-issuing thread's wait for the first
  // stage runs out, it raises the abort flag and the error word, the epilogue warps see the flag at
  // their next check, every role falls through to the final barrier and tensor memory is released.
  // No copy and no MMA is in flight at any time.
  tc::GemmParams p{};
  p.M = 32; p.N = 128; p.K = 64;
  p.a_rows = 32;
  p.m_tiles = 1; p.n_tiles = 1; p.k_chunks = 1;
  p.total_units = 1;
  p.stages = 2;
  p.partial = c->partial;
  p.tile_count = c->tile_count;
  p.error_word = c->error_word;
  p.skip_flag = nullptr;
  p.wait_limit_us = static_cast<uint32_t>(limit_us);
  p.stall = 1;
  p.n_producers = 1;
  p.w_tiled = 1;
  p.w_packed = static_cast<const bf16*>(c->xb);  // never read
  p.w_blocks = 1;
  p.ep.y = c->x;
  p.ep.ldy = c->cfg.d_model;
  const CUtensorMap* tx;
  TRY(get_tmap(c, c->xb, 32, 64, 32, &tx));
  const size_t smem = tc::gemm_tc_smem_bytes(32, 128, p.stages);
  TRY((launch_tc<EPI_F32, 128, 1>(c, tx, tx, p, 1, smem)));
  return check_device_error(c);
}
extern "C" int d3_status_of_error_word(uint32_t w) {
  if (w & ERRW_MBAR_TIMEOUT) return D3_ERR_DEVICE_TIMEOUT;
  if (w) return D3_ERR_INVALID_ARG;
  return D3_OK;
}
extern "C" int d3_commit_histogram(d3_ctx* c, int64_t* hist, int32_t n) {
  if (!c || !hist || n <= 0) return D3_ERR_INVALID_ARG;
  unsigned long long h[COMMIT_HIST_BINS];
  CUDA_TRY(c, cudaMemcpyAsync(h, c->commit_hist, sizeof(h), cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  for (int i = 0; i < n; ++i) hist[i] = i < COMMIT_HIST_BINS ? static_cast<int64_t>(h[i]) : 0;
  return D3_OK;
}
extern "C" int d3_set_overlap(d3_ctx* c, int on) {
  if (!c) return D3_ERR_INVALID_ARG;
  c->pdl = on != 0;
  return D3_OK;
}
extern "C" int d3_profile_enable(d3_ctx* c, int on) {
  if (!c) return D3_ERR_INVALID_ARG;
  prof_flush(c);
  if (on) {
    for (int i = 0; i < D3_PROF_CLASSES; ++i) {
      c->prof_ms[i] = 0.0;
      c->prof_n[i] = 0;
    }
  }
  c->prof_on = on != 0;
  return D3_OK;
}
extern "C" int d3_profile_read(d3_ctx* c, double* ms, int64_t* launches) {
  if (!c || !ms || !launches) return D3_ERR_INVALID_ARG;
  prof_flush(c);
  for (int i = 0; i < D3_PROF_CLASSES; ++i) {
    ms[i] = c->prof_ms[i];
    launches[i] = c->prof_n[i];
  }
  return D3_OK;
}
extern "C" int64_t d3_launch_count(d3_ctx* c) { return c ? c->launches : 0; }
extern "C" int64_t d3_launch_count_of(d3_ctx* c, const char* kernel) {
  if (!c || !kernel) return 0;
  auto it = c->launches_by_kernel.find(kernel);
  return it == c->launches_by_kernel.end() ? 0 : it->second;
}
extern "C" int64_t d3_device_bytes(d3_ctx* c) { return c ? c->dev_bytes : 0; }

extern "C" const char* d3_strerror(int code) {
  switch (code) {
    case D3_OK: return "ok";
    case D3_ERR_INVALID_ARG: return "invalid argument";
    case D3_ERR_SHAPE: return "shape outside the configured limits";
    case D3_ERR_OOM: return "out of device memory";
    case D3_ERR_CUDA: return "CUDA call failed";
    case D3_ERR_DEVICE_TIMEOUT: return "bounded device-side wait gave up";
    case D3_ERR_STATE: return "call out of order";
    case D3_ERR_UNSUPPORTED: return "unsupported configuration";
  }
  return "unknown error";
}
extern "C" const char* d3_last_error(d3_ctx* c) { return c ? c->last_error.c_str() : ""; }
extern "C" const char* d3_version(void) { return kVersion; }

// ----------------------------------------------------------------------------- allocation-free variant
// LM-head statistics for callers that must not allocate device memory (see include/d3.h).  The
// per-tile partial statistics, which the context-based entry point keeps in a buffer from cudaMalloc,
// live here in a fixed array inside the loaded module.
static __device__ __align__(256) float4 g_static_stat_part[D3_STATIC_MAX_PARTIALS];

namespace {
constexpr int kMaxDevices = 64;
float4* g_static_stat_ptr[kMaxDevices] = {};  // device address of the array, per device ordinal

// `g_static_stat_part` names a host-side handle in host code, not a device address: resolve it once
// per device, with that device current, and cache the result.
int static_scratch(float4** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return D3_ERR_CUDA;
  if (!g_static_stat_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_stat_part) != cudaSuccess || !p) {
      (void)cudaGetLastError();
      return D3_ERR_CUDA;
    }
    g_static_stat_ptr[dev] = static_cast<float4*>(p);
  }
  *out = g_static_stat_ptr[dev];
  return D3_OK;
}

template <typename T>
int lm_head_stats_static(const void* x, const void* w, int m, int vocab, int k, float scale, int mask_id, float* conf,
                         float* entropy, int* argmax, float4* part, cudaStream_t stream) {
  const int n_tiles = (vocab + simt::BN - 1) / simt::BN;
  EpiParams ep;
  ep.scale = scale; ep.mask_id = mask_id; ep.stat_part = part; ep.n_tiles = n_tiles;
  dim3 grid(n_tiles, (m + simt::BM - 1) / simt::BM);
  simt::gemm_simt_kernel<T, EPI_STATS><<<grid, simt::THREADS, 0, stream>>>(static_cast<const T*>(x), static_cast<const T*>(w), m, vocab, k, ep);
  if (cudaPeekAtLastError() != cudaSuccess) {
    (void)cudaGetLastError();
    return D3_ERR_CUDA;
  }
  stats_merge_kernel<<<(m + 3) / 4, 128, 0, stream>>>(part, n_tiles, m, conf, entropy, argmax);
  if (cudaPeekAtLastError() != cudaSuccess) {
    (void)cudaGetLastError();
    return D3_ERR_CUDA;
  }
  return D3_OK;
}
}  // namespace

extern "C" int d3_lm_head_stats_static(const void* x, const void* w, int32_t dtype, int32_t m, int32_t vocab, int32_t k,
                                       float scale, int32_t mask_id, float* conf, float* entropy, int32_t* argmax,
                                       void* cuda_stream) {
  if (!x || !w || !conf || !entropy || !argmax || m <= 0 || vocab <= 0 || k <= 0) return D3_ERR_INVALID_ARG;
  if (dtype != D3_DTYPE_F32 && dtype != D3_DTYPE_BF16) return D3_ERR_INVALID_ARG;
  const long long n_tiles = (static_cast<long long>(vocab) + simt::BN - 1) / simt::BN;
  if (static_cast<long long>(m) * n_tiles > D3_STATIC_MAX_PARTIALS) return D3_ERR_SHAPE;
  float4* part = nullptr;
  int rc = static_scratch(&part);
  if (rc != D3_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  // Every partial that the merge reads is written by the matmul launch before it, so nothing in
  // the shared array has to start at zero and stale contents of earlier calls are never read.
  if (dtype == D3_DTYPE_BF16)
    return lm_head_stats_static<bf16>(x, w, m, vocab, k, scale, mask_id, conf, entropy, argmax, part, stream);
  return lm_head_stats_static<float>(x, w, m, vocab, k, scale, mask_id, conf, entropy, argmax, part, stream);
}

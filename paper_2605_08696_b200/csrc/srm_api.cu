// Host runtime and C ABI of the SRM decode library (see include/srm.h for the contract).
// Everything here is argument checking, buffer carving and kernel launches; all arithmetic
// of the path runs in the kernels included below.
#include "../../include/srm.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "common.cuh"
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "gemm_tc_splitk.cuh"
#include "mixer.cuh"
#include "mixer_stream.cuh"
#include "mixer_proj.cuh"
#include "mixer_variants.cuh"
#include "mixer_model_variants.cuh"
#include "prefill.cuh"
#include "prefill_scan.cuh"
#include "select.cuh"
#include "select_topp.cuh"
#include "step_small.cuh"

using namespace srm;

namespace {

int g_last_cuda_error = 0;

#define SRM_CUDA(expr)                                  \
  do {                                                  \
    cudaError_t e__ = (expr);                           \
    if (e__ != cudaSuccess) {                           \
      g_last_cuda_error = (int)e__;                     \
      return SRM_ERR_CUDA;                              \
    }                                                   \
  } while (0)

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

struct Slot { size_t off = 0, bytes = 0; int elem = 4; };

struct Layout {
  Slot global[SRM_T_COUNT];
  std::vector<Slot> layer;     // [L][SRM_T_COUNT]
  size_t total = 0;
};

bool is_global_tensor(int t) { return t == SRM_T_E || t == SRM_T_LNF_G || t == SRM_T_LNF_B || t == SRM_T_W_LM; }

bool config_ok(const srm_config* c) {
  if (c == nullptr) return false;
  if (c->n_layers < 1 || c->d_model < 64 || c->d_model > 2048 || c->d_model % 64) return false;
  if (c->n_heads < 2 || c->n_heads > kPrefillMaxHeads || c->n_heads % 2 || c->d_model % (4 * c->n_heads)) return false;
  if (c->ffn_mult < 1 || c->vocab < 8 || c->vocab % 8 || c->n_ctx < 1) return false;
  if (c->dtype != SRM_DTYPE_FP32 && c->dtype != SRM_DTYPE_BF16) return false;
  if (c->state_dtype != SRM_DTYPE_FP32 && c->state_dtype != SRM_DTYPE_BF16 && c->state_dtype != SRM_DTYPE_FP16) return false;
  if (!(c->ln_eps > 0.f)) return false;
  if (c->mixer != SRM_MIXER_MIXED && c->mixer != SRM_MIXER_COMBINED && c->mixer != SRM_MIXER_KERNEL) return false;
  if (c->mixer != SRM_MIXER_MIXED) {
    // the further mixers: no head projections, cache in fp32 or fp16, rows of at most 1024 channels
    if ((c->flags & SRM_FLAG_HEAD_PROJ) || c->state_dtype == SRM_DTYPE_BF16 || c->d_model > 1024) return false;
    if (c->mixer == SRM_MIXER_KERNEL && (c->kernel_size < 1 || c->kernel_size > 16 || c->kernel_size > c->d_model)) return false;
  }
  return true;
}

// d-vectors of cache per sample and layer: 1 (mixed heads), 2 (combined heads: both sum terms), k (kernel of size k)
int cache_planes(const srm_config& c) {
  return c.mixer == SRM_MIXER_COMBINED ? 2 : c.mixer == SRM_MIXER_KERNEL ? c.kernel_size : 1;
}

size_t tensor_elems(const srm_config& c, int t) {
  const size_t d = c.d_model, F = (size_t)c.ffn_mult * d, V = c.vocab, n = c.n_ctx;
  const size_t h = c.mixer == SRM_MIXER_KERNEL ? (size_t)c.kernel_size : (size_t)c.n_heads;   // filters take the heads' place
  switch (t) {
    case SRM_T_E: case SRM_T_W_LM: return V * d;
    case SRM_T_ALPHA: case SRM_T_ALPHA_COL: return h * n;
    case SRM_T_BETA: return n * d;
    case SRM_T_LAMBDA: case SRM_T_LAMBDA_COL: return h;
    case SRM_T_W_COMB: return 2 * h;
    case SRM_T_W1: case SRM_T_W2: return F * d;
    case SRM_T_W_IN: case SRM_T_W_OUT: return d * d;
    case SRM_T_B1: return F;
    default: return d;
  }
}

Layout make_layout(const srm_config& c) {
  Layout L;
  const int wbytes = c.dtype == SRM_DTYPE_BF16 ? 2 : 4;
  auto is_matrix = [](int t) {
    return t == SRM_T_E || t == SRM_T_W1 || t == SRM_T_W2 || t == SRM_T_W_LM || t == SRM_T_W_IN || t == SRM_T_W_OUT;
  };
  size_t off = 0;
  auto place = [&](int t) {
    Slot s;
    s.elem = is_matrix(t) ? wbytes : 4;
    s.bytes = tensor_elems(c, t) * s.elem;
    s.off = off;
    off = align_up(off + s.bytes, 256);
    return s;
  };
  L.global[SRM_T_E] = place(SRM_T_E);
  L.layer.resize((size_t)c.n_layers * SRM_T_COUNT);
  for (int l = 0; l < c.n_layers; ++l)
  {
    for (int t = SRM_T_LN1_G; t <= SRM_T_B2; ++t) L.layer[(size_t)l * SRM_T_COUNT + t] = place(t);
    if (c.flags & SRM_FLAG_HEAD_PROJ) {
      L.layer[(size_t)l * SRM_T_COUNT + SRM_T_W_IN] = place(SRM_T_W_IN);
      L.layer[(size_t)l * SRM_T_COUNT + SRM_T_W_OUT] = place(SRM_T_W_OUT);
    }
    if (c.mixer == SRM_MIXER_COMBINED)
      for (int t = SRM_T_ALPHA_COL; t <= SRM_T_W_COMB; ++t) L.layer[(size_t)l * SRM_T_COUNT + t] = place(t);
  }
  L.global[SRM_T_LNF_G] = place(SRM_T_LNF_G);
  L.global[SRM_T_LNF_B] = place(SRM_T_LNF_B);
  L.global[SRM_T_W_LM] = place(SRM_T_W_LM);
  L.total = off;
  return L;
}

// ---- TMA descriptors ------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// Row-major [rows, cols] matrix of 2-byte (bf16) or 4-byte (fp32) elements; the box is 128 bytes of
// one row (the swizzle span) x box_rows rows.
int make_tmap(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int box_rows, int elem_bytes) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) { g_last_cuda_error = (int)cudaErrorNotSupported; return SRM_ERR_CUDA; }
  cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t gstride[1] = {(cuuint64_t)cols * (cuuint64_t)elem_bytes};
  cuuint32_t box[2] = {(cuuint32_t)(128 / elem_bytes), (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                  const_cast<void*>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { g_last_cuda_error = 10000 + (int)r; return SRM_ERR_CUDA; }
  return SRM_OK;
}

// cudaFuncAttributeMaxDynamicSharedMemorySize is a per-device setting: remember which (kernel, device) pairs have
// it, so that a model on a second device of the process gets it too. Safe from several host threads.
int ensure_dynamic_smem(const void* func, int bytes) {
  static std::mutex mu;
  static std::vector<std::pair<const void*, int>> done;      // (kernel, device ordinal)
  int dev = -1;
  SRM_CUDA(cudaGetDevice(&dev));
  std::lock_guard<std::mutex> lock(mu);
  for (const auto& e : done)
    if (e.first == func && e.second == dev) return SRM_OK;
  SRM_CUDA(cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  done.emplace_back(func, dev);
  return SRM_OK;
}

struct TmapCacheEntry { const void* base; int64_t rows, cols; int box_rows, elem_bytes; CUtensorMap map; };

std::atomic<unsigned long long> g_kernel_launches{0};     // kernels launched by this library since load (all threads)

struct ProfRecord { cudaEvent_t start, stop; int cls; };

}  // namespace

struct srm_model {
  srm_config cfg;
  const uint8_t* w;
  Layout layout;
  int device = 0;
  int num_sms = 0;
  bool head_proj() const { return (cfg.flags & SRM_FLAG_HEAD_PROJ) != 0; }
  bool tc_ready = false;                 // smem attribute set for the tensor-core kernels
  int tc_clusters = 0;                   // CTA pairs of the tensor-core kernel that are resident at once
  std::vector<TmapCacheEntry> tmaps;     // weight and activation descriptors, built on first use
  // One decode step captured as a CUDA graph for srm_generate (launch-bound batches): the stream it is
  // captured on, the instantiated graph, and what it was captured for.
  cudaStream_t cap_stream = nullptr;
  cudaGraphExec_t step_exec = nullptr;
  uint64_t step_launches = 0;            // kernels in the captured step
  struct StepKey {
    const srm_state* s = nullptr; const void* ws = nullptr; size_t ws_bytes = 0; const int32_t* out = nullptr;
    int64_t out_stride = 0; srm_sampling samp = {};
    bool ragged = false;                 // per-sample positions: the captured kernels then take the position vector
    bool operator==(const StepKey& o) const {
      return ragged == o.ragged && s == o.s && ws == o.ws && ws_bytes == o.ws_bytes && out == o.out && out_stride == o.out_stride &&
             samp.mode == o.samp.mode && samp.top_k == o.samp.top_k && samp.temperature == o.samp.temperature &&
             samp.top_p == o.samp.top_p &&
             samp.seed == o.samp.seed && samp.sample_idx_base == o.samp.sample_idx_base;
    }
  } step_key;
  bool profiling = false;                // bracket every launch with CUDA events on its stream
  std::vector<ProfRecord> prof;          // open records, folded into the totals by srm_profile_read
  std::vector<cudaEvent_t> event_pool;
  unsigned long long prof_launches[SRM_KERNEL_CLASS_COUNT] = {};
  double prof_ms[SRM_KERNEL_CLASS_COUNT] = {};

  const void* ptr(int layer, int t) const {
    const Slot& s = is_global_tensor(t) ? layout.global[t] : layout.layer[(size_t)layer * SRM_T_COUNT + t];
    return w + s.off;
  }
  const float* fptr(int layer, int t) const { return reinterpret_cast<const float*>(ptr(layer, t)); }
  int act_bytes() const { return cfg.dtype == SRM_DTYPE_BF16 ? 2 : 4; }
  int state_bytes() const { return cfg.state_dtype == SRM_DTYPE_FP32 ? 4 : 2; }
  int64_t F() const { return (int64_t)cfg.ffn_mult * cfg.d_model; }

  // Copies the descriptor out: the cache may reallocate or be cleared by a later insertion.
  int tmap(const void* base, int64_t rows, int64_t cols, int box_rows, int elem_bytes, CUtensorMap* out) {
    for (auto& e : tmaps)
      if (e.base == base && e.rows == rows && e.cols == cols && e.box_rows == box_rows && e.elem_bytes == elem_bytes) {
        *out = e.map;
        return SRM_OK;
      }
    if (tmaps.size() >= 4096) tmaps.clear();
    TmapCacheEntry e{base, rows, cols, box_rows, elem_bytes, {}};
    int rc = make_tmap(&e.map, base, rows, cols, box_rows, elem_bytes);
    if (rc != SRM_OK) return rc;
    tmaps.push_back(e);
    *out = e.map;
    return SRM_OK;
  }
};

struct srm_state {
  srm_model* m;
  int64_t B;
  uint8_t* base;
  size_t nbytes;
  uint32_t* status;       // device status word (header)
  int32_t* last_tok;      // [B]
  int32_t* pos_dev;       // [B] per-sample positions, used after srm_prefill_ragged
  float* thr;             // [B] candidate threshold of each sample's next top-k selection (0: none yet)
  uint8_t* S;             // [L, B, d] in state dtype
  int64_t pos;            // position of the next token (ragged: of the longest sample)
  bool ragged = false;    // samples have their own positions (pos_dev)

  // Layer l: planes() consecutive slabs [B, d] (plane_elems() elements apart)
  int planes() const { return cache_planes(m->cfg); }
  int64_t plane_elems() const { return B * (int64_t)m->cfg.d_model; }
  void* layer_ptr(int l) const { return S + (size_t)l * planes() * B * m->cfg.d_model * m->state_bytes(); }
};

namespace {

// Counts the launch and, when profiling is on, records an event before and after it.
struct LaunchScope {
  srm_model* m; cudaStream_t st; cudaEvent_t stop = nullptr;
  LaunchScope(const srm_model& model, int cls, cudaStream_t stream) : m(const_cast<srm_model*>(&model)), st(stream) {
    ++g_kernel_launches;
    if (!m->profiling) return;
    cudaEvent_t ev[2];
    for (auto& e : ev) {
      if (!m->event_pool.empty()) { e = m->event_pool.back(); m->event_pool.pop_back(); }
      else if (cudaEventCreate(&e) != cudaSuccess) return;
    }
    cudaEventRecord(ev[0], st);
    stop = ev[1];
    m->prof.push_back(ProfRecord{ev[0], ev[1], cls});
  }
  ~LaunchScope() { if (stop != nullptr) cudaEventRecord(stop, st); }
};

constexpr size_t kStateHeader = 256;

size_t state_bytes_for(const srm_config& c, int64_t B) {
  const size_t sb = c.state_dtype == SRM_DTYPE_FP32 ? 4 : 2;
  return kStateHeader + 3 * align_up((size_t)B * 4, 256) + (size_t)c.n_layers * cache_planes(c) * B * c.d_model * sb;
}

// ---- workspace carving ----------------------------------------------------------------------
// Scratch of the small-batch step kernel (step_small.cuh): partial sums of the down projection
// [8][64, d] fp32, the per-CTA results of the LM-head slabs [256][64] and the grid-barrier word.
size_t small_scratch_bytes(const srm_config& c) {
  return align_up((size_t)8 * sb::kMaxRows * c.d_model * 4, 256) + align_up((size_t)256 * sb::kMaxRows * 8, 256) + 256;
}

struct DecodeWs {
  float* x; void* a; void* H; float* logits;
  uint8_t* small;         // small_scratch_bytes
  float* q;               // head projections only
  int32_t* order;         // split-K down projection: one word per (tile of x, CTA of the pair, epilogue warp)
  size_t order_bytes;
  int64_t rows;
};
struct PrefillWs { float* x; void* a; void* H; void* a_last; float* logits; float* q; int64_t samples; };

// The down projection of a decode step may be split along K between CTA pairs (gemm_tc_splitk.cuh).
bool splitk_enabled(const srm_config& c) {
  return c.dtype == SRM_DTYPE_BF16 && !(c.flags & (SRM_FLAG_SIMT_GEMM | SRM_FLAG_NO_SPLITK));
}
size_t splitk_order_bytes(int64_t M, int64_t N) {
  return align_up(tc::split_order_words(((M + tc::BM - 1) / tc::BM) * ((N + tc::BN - 1) / tc::BN)) * 4, 256);
}
size_t decode_ws_bytes(const srm_model& m, int64_t rows) {
  const size_t d = m.cfg.d_model, F = m.F(), V = m.cfg.vocab, ab = m.act_bytes();
  return align_up(rows * d * 4, 256) + align_up(rows * d * ab, 256) + align_up(rows * F * ab, 256) +
         align_up(rows * V * 4, 256) + (m.head_proj() ? align_up(rows * d * 4, 256) : 0) +
         (splitk_enabled(m.cfg) ? splitk_order_bytes(rows, m.cfg.d_model) : 0) + small_scratch_bytes(m.cfg);
}
size_t prefill_ws_bytes(const srm_model& m, int64_t samples, int n) {
  const size_t d = m.cfg.d_model, F = m.F(), V = m.cfg.vocab, ab = m.act_bytes(), rows = (size_t)samples * n;
  return align_up(rows * d * 4, 256) + align_up(rows * d * ab, 256) + align_up(rows * F * ab, 256) +
         align_up(samples * d * ab, 256) + align_up(samples * V * 4, 256) +
         (m.head_proj() ? align_up(rows * d * 4, 256) : 0);
}
int64_t fit_rows(size_t ws_bytes, int64_t want, size_t (*need)(const srm_model&, int64_t, int), const srm_model& m, int n) {
  if (need(m, 1, n) > ws_bytes) return 0;
  int64_t lo = 1, hi = want;            // largest r in [1, want] with need(r) <= ws_bytes
  while (lo < hi) {
    const int64_t mid = lo + (hi - lo + 1) / 2;
    if (need(m, mid, n) <= ws_bytes) lo = mid; else hi = mid - 1;
  }
  return lo;
}
size_t decode_need(const srm_model& m, int64_t r, int) { return decode_ws_bytes(m, r); }
size_t prefill_need(const srm_model& m, int64_t r, int n) { return prefill_ws_bytes(m, r, n); }

DecodeWs carve_decode(const srm_model& m, void* ws, int64_t rows) {
  const size_t d = m.cfg.d_model, F = m.F(), ab = m.act_bytes();
  uint8_t* p = static_cast<uint8_t*>(ws);
  DecodeWs w;
  w.rows = rows;
  w.x = reinterpret_cast<float*>(p); p += align_up(rows * d * 4, 256);
  w.a = p; p += align_up(rows * d * ab, 256);
  w.H = p; p += align_up(rows * F * ab, 256);
  w.logits = reinterpret_cast<float*>(p); p += align_up(rows * (size_t)m.cfg.vocab * 4, 256);
  w.q = m.head_proj() ? reinterpret_cast<float*>(p) : nullptr;
  if (m.head_proj()) p += align_up(rows * d * 4, 256);
  w.order_bytes = splitk_enabled(m.cfg) ? splitk_order_bytes(rows, m.cfg.d_model) : 0;
  w.order = w.order_bytes ? reinterpret_cast<int32_t*>(p) : nullptr;
  p += w.order_bytes;
  w.small = p;
  return w;
}
PrefillWs carve_prefill(const srm_model& m, void* ws, int64_t samples, int n) {
  const size_t d = m.cfg.d_model, F = m.F(), ab = m.act_bytes(), rows = (size_t)samples * n;
  uint8_t* p = static_cast<uint8_t*>(ws);
  PrefillWs w;
  w.samples = samples;
  w.x = reinterpret_cast<float*>(p); p += align_up(rows * d * 4, 256);
  w.a = p; p += align_up(rows * d * ab, 256);
  w.H = p; p += align_up(rows * F * ab, 256);
  w.a_last = p; p += align_up(samples * d * ab, 256);
  w.logits = reinterpret_cast<float*>(p); p += align_up(samples * (size_t)m.cfg.vocab * 4, 256);
  w.q = m.head_proj() ? reinterpret_cast<float*>(p) : nullptr;
  return w;
}

// ---- kernel launchers -------------------------------------------------------------------------
// Every kernel goes through here: programmatic stream serialization lets the next kernel's blocks be
// scheduled and run their set-up while this one drains; each kernel orders itself with pdl_wait().
template <typename... KArgs, typename... Args>
cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Calls f(WT{}, ST{}) with the weight / activation type and the cache storage type of the configuration.
template <typename F>
int dispatch_types(const srm_config& c, F&& f) {
  const bool wb = c.dtype == SRM_DTYPE_BF16;
  switch (c.state_dtype) {
    case SRM_DTYPE_BF16: return wb ? f(bf16{}, bf16{}) : f(float{}, bf16{});
    case SRM_DTYPE_FP16: return wb ? f(bf16{}, fp16{}) : f(float{}, fp16{});
    default: return wb ? f(bf16{}, float{}) : f(float{}, float{});
  }
}

template <int NV, typename WT, typename ST>
int launch_mixer_stream(const MixerParams& p, int num_sms, cudaStream_t st) {
  const int warps = mixer_stream_warps(p.d, (int)sizeof(ST));
  const size_t smem = mixer_stream_smem(p.d, (int)sizeof(ST), warps);
  int rc = ensure_dynamic_smem(reinterpret_cast<const void*>(mixer_stream_kernel<NV, WT, ST>), kStreamSmemBudget);
  if (rc != SRM_OK) return rc;
  const unsigned grid = (unsigned)(p.R < num_sms ? p.R : num_sms);
  SRM_CUDA(launch_kernel(mixer_stream_kernel<NV, WT, ST>, dim3(grid), dim3(warps * 32), smem, st, p));
  return SRM_OK;
}

template <typename WT, typename ST>
int launch_mixer_nv(const MixerParams& p, int num_sms, cudaStream_t st) {
  const int nv = (p.d + 127) / 128;
  // whole 128-channel vectors per lane, each inside one head: the streaming kernel
  const bool fast = p.d % 128 == 0 && (p.d / p.h) % 128 == 0 && p.h <= 8 && mixer_stream_warps(p.d, (int)sizeof(ST)) >= 1;
  if (fast && nv == 4) return launch_mixer_stream<4, WT, ST>(p, num_sms, st);
  if (fast && nv == 8) return launch_mixer_stream<8, WT, ST>(p, num_sms, st);
  if (fast && nv == 12) return launch_mixer_stream<12, WT, ST>(p, num_sms, st);
  if (fast && nv == 16) return launch_mixer_stream<16, WT, ST>(p, num_sms, st);
  const unsigned grid = (unsigned)((p.R + kMixerWarps - 1) / kMixerWarps);
  const dim3 blk(kMixerWarps * 32);
  if (nv <= 1) SRM_CUDA(launch_kernel(mixer_step_kernel<1, WT, ST>, dim3(grid), dim3(blk), 0, st, p));
  else if (nv <= 2) SRM_CUDA(launch_kernel(mixer_step_kernel<2, WT, ST>, dim3(grid), dim3(blk), 0, st, p));
  else if (nv <= 4) SRM_CUDA(launch_kernel(mixer_step_kernel<4, WT, ST>, dim3(grid), dim3(blk), 0, st, p));
  else if (nv <= 6) SRM_CUDA(launch_kernel(mixer_step_kernel<6, WT, ST>, dim3(grid), dim3(blk), 0, st, p));
  else if (nv <= 8) SRM_CUDA(launch_kernel(mixer_step_kernel<8, WT, ST>, dim3(grid), dim3(blk), 0, st, p));
  else if (nv <= 12) SRM_CUDA(launch_kernel(mixer_step_kernel<12, WT, ST>, dim3(grid), dim3(blk), 0, st, p));
  else SRM_CUDA(launch_kernel(mixer_step_kernel<16, WT, ST>, dim3(grid), dim3(blk), 0, st, p));
  return SRM_OK;
}

int launch_mixer(const srm_model& m, int layer, int t, int64_t R, const int32_t* tok, float* x, void* S, void* a,
                 uint32_t* status, cudaStream_t st, const int32_t* ctr = nullptr, const int32_t* pos = nullptr) {
  if (R <= 0) return SRM_OK;
  LaunchScope scope(m, SRM_KERNEL_MIXER, st);
  MixerParams p;
  p.x = x; p.tok = tok; p.E = m.ptr(-1, SRM_T_E); p.S = S; p.a = a;
  p.ln1_g = m.fptr(layer, SRM_T_LN1_G); p.ln1_b = m.fptr(layer, SRM_T_LN1_B);
  p.ln2_g = m.fptr(layer, SRM_T_LN2_G); p.ln2_b = m.fptr(layer, SRM_T_LN2_B);
  p.alpha = m.fptr(layer, SRM_T_ALPHA); p.beta = m.fptr(layer, SRM_T_BETA); p.lam = m.fptr(layer, SRM_T_LAMBDA);
  p.R = R; p.d = m.cfg.d_model; p.h = m.cfg.n_heads; p.n_ctx = m.cfg.n_ctx; p.t = t; p.vocab = m.cfg.vocab;
  p.eps = m.cfg.ln_eps; p.status = status; p.ctr = ctr; p.pos = pos;
  return dispatch_types(m.cfg, [&](auto w, auto c) { return launch_mixer_nv<decltype(w), decltype(c)>(p, m.num_sms, st); });
}

// Fused step of the combined-head / kernel-size-k mixers on R rows at position t (mixer_model_variants.cuh).
// S: plane 0 of the rows' cache, planes `plane` elements apart; x, a rows x_stride elements apart.
template <typename WT, typename ST>
int launch_mixer_variant_t(const VariantParams& p, bool kernel_mix, cudaStream_t st) {
  const unsigned grid = (unsigned)((p.R + kMixerWarps - 1) / kMixerWarps);
  const dim3 blk(kMixerWarps * 32);
  const int nv = (p.d + 127) / 128;
#define SRM_VARIANT_LAUNCH(NV)                                                                                          \
  do {                                                                                                                  \
    if (kernel_mix) SRM_CUDA(launch_kernel(mixer_variant_step_kernel<NV, WT, ST, true>, dim3(grid), dim3(blk), 0, st, p)); \
    else SRM_CUDA(launch_kernel(mixer_variant_step_kernel<NV, WT, ST, false>, dim3(grid), dim3(blk), 0, st, p));           \
  } while (0)
  if (nv <= 1) SRM_VARIANT_LAUNCH(1);
  else if (nv <= 4) SRM_VARIANT_LAUNCH(4);
  else SRM_VARIANT_LAUNCH(8);
#undef SRM_VARIANT_LAUNCH
  return SRM_OK;
}

int launch_mixer_variant(const srm_model& m, int layer, int t, int64_t R, const int32_t* tok, int64_t tok_stride, float* x,
                         void* a, int64_t x_stride, void* S, int64_t plane, uint32_t* status, cudaStream_t st,
                         const int32_t* ctr = nullptr, int cls = SRM_KERNEL_MIXER) {
  if (R <= 0) return SRM_OK;
  LaunchScope scope(m, cls, st);
  const srm_config& c = m.cfg;
  VariantParams p;
  p.x = x; p.tok = tok; p.E = m.ptr(-1, SRM_T_E); p.S = S; p.a = a;
  p.ln1_g = m.fptr(layer, SRM_T_LN1_G); p.ln1_b = m.fptr(layer, SRM_T_LN1_B);
  p.ln2_g = m.fptr(layer, SRM_T_LN2_G); p.ln2_b = m.fptr(layer, SRM_T_LN2_B);
  p.alpha = m.fptr(layer, SRM_T_ALPHA); p.beta = m.fptr(layer, SRM_T_BETA); p.lam = m.fptr(layer, SRM_T_LAMBDA);
  const bool comb = c.mixer == SRM_MIXER_COMBINED;
  p.alpha_col = comb ? m.fptr(layer, SRM_T_ALPHA_COL) : nullptr;
  p.lam_col = comb ? m.fptr(layer, SRM_T_LAMBDA_COL) : nullptr;
  p.w_comb = comb ? m.fptr(layer, SRM_T_W_COMB) : nullptr;
  p.R = R; p.x_stride = x_stride; p.tok_stride = tok_stride; p.plane = plane;
  p.d = c.d_model; p.h = c.n_heads; p.k = c.kernel_size; p.n_ctx = c.n_ctx; p.t = t; p.vocab = c.vocab;
  p.eps = c.ln_eps; p.status = status; p.ctr = ctr;
  const bool wb = c.dtype == SRM_DTYPE_BF16, half_cache = c.state_dtype == SRM_DTYPE_FP16;
  const bool km = c.mixer == SRM_MIXER_KERNEL;
  if (wb) return half_cache ? launch_mixer_variant_t<bf16, fp16>(p, km, st) : launch_mixer_variant_t<bf16, float>(p, km, st);
  return half_cache ? launch_mixer_variant_t<float, fp16>(p, km, st) : launch_mixer_variant_t<float, float>(p, km, st);
}

template <typename WT>
int launch_norm_t(const float* x, int64_t R, int64_t stride, int64_t offset, const float* g, const float* b, float eps,
                  int d, void* out, cudaStream_t st, const int32_t* row_len = nullptr) {
  const int nv = (d + 127) / 128;
  const unsigned grid = (unsigned)((R + kMixerWarps - 1) / kMixerWarps);
  const dim3 blk(kMixerWarps * 32);
  WT* o = reinterpret_cast<WT*>(out);
  if (nv <= 1) SRM_CUDA(launch_kernel(norm_rows_kernel<1, WT>, dim3(grid), dim3(blk), 0, st, x, R, stride, offset, g, b, eps, d, o, row_len));
  else if (nv <= 2) SRM_CUDA(launch_kernel(norm_rows_kernel<2, WT>, dim3(grid), dim3(blk), 0, st, x, R, stride, offset, g, b, eps, d, o, row_len));
  else if (nv <= 4) SRM_CUDA(launch_kernel(norm_rows_kernel<4, WT>, dim3(grid), dim3(blk), 0, st, x, R, stride, offset, g, b, eps, d, o, row_len));
  else if (nv <= 6) SRM_CUDA(launch_kernel(norm_rows_kernel<6, WT>, dim3(grid), dim3(blk), 0, st, x, R, stride, offset, g, b, eps, d, o, row_len));
  else if (nv <= 8) SRM_CUDA(launch_kernel(norm_rows_kernel<8, WT>, dim3(grid), dim3(blk), 0, st, x, R, stride, offset, g, b, eps, d, o, row_len));
  else if (nv <= 12) SRM_CUDA(launch_kernel(norm_rows_kernel<12, WT>, dim3(grid), dim3(blk), 0, st, x, R, stride, offset, g, b, eps, d, o, row_len));
  else SRM_CUDA(launch_kernel(norm_rows_kernel<16, WT>, dim3(grid), dim3(blk), 0, st, x, R, stride, offset, g, b, eps, d, o, row_len));
  SRM_CUDA(cudaGetLastError());
  return SRM_OK;
}

// out[r, :] = LN(x[r * stride + offset, :]; g, b) in the activation type
int launch_norm(const srm_model& m, const float* x, int64_t R, int64_t stride, int64_t offset, const float* g,
                const float* b, void* out, cudaStream_t st) {
  if (R <= 0) return SRM_OK;
  LaunchScope scope(m, SRM_KERNEL_NORM, st);
  if (m.cfg.dtype == SRM_DTYPE_BF16) return launch_norm_t<bf16>(x, R, stride, offset, g, b, m.cfg.ln_eps, m.cfg.d_model, out, st);
  return launch_norm_t<float>(x, R, stride, offset, g, b, m.cfg.ln_eps, m.cfg.d_model, out, st);
}

int launch_final_norm(const srm_model& m, const float* x, int64_t R, int64_t stride, int64_t offset, void* out,
                      cudaStream_t st, const int32_t* row_len = nullptr) {
  if (R <= 0) return SRM_OK;
  LaunchScope scope(m, SRM_KERNEL_NORM, st);
  const float* g = m.fptr(-1, SRM_T_LNF_G);
  const float* b = m.fptr(-1, SRM_T_LNF_B);
  if (m.cfg.dtype == SRM_DTYPE_BF16) return launch_norm_t<bf16>(x, R, stride, offset, g, b, m.cfg.ln_eps, m.cfg.d_model, out, st, row_len);
  return launch_norm_t<float>(x, R, stride, offset, g, b, m.cfg.ln_eps, m.cfg.d_model, out, st, row_len);
}

template <typename T>
int launch_gemm_simt(int epi, int64_t M, int64_t N, int64_t K, const void* A, const void* W, const float* bias,
                     void* out, cudaStream_t st) {
  const dim3 grid((unsigned)((N + kSimtBN - 1) / kSimtBN), (unsigned)((M + kSimtBM - 1) / kSimtBM));
  const T* a = reinterpret_cast<const T*>(A);
  const T* w = reinterpret_cast<const T*>(W);
  if (epi == kEpiBiasGelu) SRM_CUDA(launch_kernel(gemm_simt_kernel<T, kEpiBiasGelu>, dim3(grid), dim3(256), 0, st, a, w, bias, out, M, N, K));
  else if (epi == kEpiBiasResidual) SRM_CUDA(launch_kernel(gemm_simt_kernel<T, kEpiBiasResidual>, dim3(grid), dim3(256), 0, st, a, w, bias, out, M, N, K));
  else SRM_CUDA(launch_kernel(gemm_simt_kernel<T, kEpiPlain>, dim3(grid), dim3(256), 0, st, a, w, bias, out, M, N, K));
  SRM_CUDA(cudaGetLastError());
  return SRM_OK;
}

int ensure_tc_ready(srm_model& m) {
  if (m.tc_ready) return SRM_OK;
  SRM_CUDA(cudaFuncSetAttribute(tc::gemm_tc_kernel<kEpiBiasGelu>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes));
  SRM_CUDA(cudaFuncSetAttribute(tc::gemm_tc_kernel<kEpiBiasResidual>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes));
  SRM_CUDA(cudaFuncSetAttribute(tc::gemm_tc_kernel<kEpiPlain>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes));
  SRM_CUDA(cudaFuncSetAttribute(tc::gemm_tc_kernel<kEpiArgmax>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes));
  SRM_CUDA(cudaFuncSetAttribute(tc::gemm_tc_kernel<kEpiCollect>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes));
  SRM_CUDA(cudaFuncSetAttribute(tc::gemm_tc_splitk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * (m.num_sms / 2));
  cfg.blockDim = dim3(tc::kThreads);
  cfg.dynamicSmemBytes = tc::kSmemBytes;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  int clusters = 0;
  SRM_CUDA(cudaOccupancyMaxActiveClusters(&clusters, tc::gemm_tc_kernel<kEpiPlain>, &cfg));
  if (clusters < 1) { g_last_cuda_error = (int)cudaErrorLaunchOutOfResources; return SRM_ERR_CUDA; }
  m.tc_clusters = clusters < m.num_sms / 2 ? clusters : m.num_sms / 2;
  m.tc_ready = true;
  return SRM_OK;
}

// How many of the last tiles of a launch run as two half-width pieces (gemm_tc.cuh): the r tiles of a last, partly
// filled round when their 2 r halves still fit in one round (they then end after three quarters of a tile's time
// with nearly every pair busy); none with SRM_FLAG_NO_TAIL_SPLIT.
int gemm_tail_tiles(const srm_model& m, int64_t tiles) {
  if (m.cfg.flags & SRM_FLAG_NO_TAIL_SPLIT) return 0;
  const int64_t r = tiles % m.tc_clusters;
  return (r > 0 && 2 * r <= m.tc_clusters) ? (int)r : 0;
}

int launch_gemm_tc(srm_model& m, int epi, int64_t M, int64_t N, int64_t K, const void* A, const void* W,
                   const float* bias, void* out, uint32_t* status, cudaStream_t st) {
  int rc = ensure_tc_ready(m);
  if (rc != SRM_OK) return rc;
  CUtensorMap ta, tb, td, tb64;
  if ((rc = m.tmap(A, M, K, tc::kRowsPerCta, 2, &ta)) != SRM_OK) return rc;
  if ((rc = m.tmap(W, N, K, tc::kRowsPerCta, 2, &tb)) != SRM_OK) return rc;
  if ((rc = m.tmap(W, N, K, tc::kHalfN / 2, 2, &tb64)) != SRM_OK) return rc;      // W rows of a half-width piece
  if (epi == kEpiArgmax) td = ta;       // no output matrix: the descriptor is not used
  else if ((rc = m.tmap(out, M, N, tc::kOutBoxRows, epi == kEpiBiasGelu ? 2 : 4, &td)) != SRM_OK) return rc;
  const uint8_t* wb = static_cast<const uint8_t*>(W);
  const int w_static = wb >= m.w && wb < m.w + m.layout.total;      // inside the weight blob
  const int64_t tiles = ((M + tc::BM - 1) / tc::BM) * ((N + tc::BN - 1) / tc::BN);
  const int tail = gemm_tail_tiles(m, tiles);
  tc::GemmArgs g{M, N, K, bias, out, status, w_static};
  g.tail_tiles = tail;
  const int64_t pieces = tiles + tail;
  const unsigned grid = 2u * (unsigned)(pieces < m.tc_clusters ? pieces : m.tc_clusters);
  if (epi == kEpiBiasGelu) SRM_CUDA(launch_kernel(tc::gemm_tc_kernel<kEpiBiasGelu>, dim3(grid), dim3(tc::kThreads), tc::kSmemBytes, st, ta, tb, td, tb64, g));
  else if (epi == kEpiBiasResidual) SRM_CUDA(launch_kernel(tc::gemm_tc_kernel<kEpiBiasResidual>, dim3(grid), dim3(tc::kThreads), tc::kSmemBytes, st, ta, tb, td, tb64, g));
  else if (epi == kEpiArgmax) SRM_CUDA(launch_kernel(tc::gemm_tc_kernel<kEpiArgmax>, dim3(grid), dim3(tc::kThreads), tc::kSmemBytes, st, ta, tb, td, tb64, g));
  else SRM_CUDA(launch_kernel(tc::gemm_tc_kernel<kEpiPlain>, dim3(grid), dim3(tc::kThreads), tc::kSmemBytes, st, ta, tb, td, tb64, g));
  SRM_CUDA(cudaGetLastError());
  return SRM_OK;
}

int launch_gemm(srm_model& m, int epi, int64_t M, int64_t N, int64_t K, const void* A, const void* W,
                const float* bias, void* out, uint32_t* status, cudaStream_t st, int cls = -1) {
  if (M <= 0) return SRM_OK;
  if (cls < 0) cls = epi == kEpiBiasGelu ? SRM_KERNEL_GEMM_UP : epi == kEpiBiasResidual ? SRM_KERNEL_GEMM_DOWN : SRM_KERNEL_GEMM_LM;
  LaunchScope scope(m, cls, st);
  if (epi == kEpiArgmax) return launch_gemm_tc(m, epi, M, N, K, A, W, bias, out, status, st);
  if (m.cfg.dtype == SRM_DTYPE_FP32) return launch_gemm_simt<float>(epi, M, N, K, A, W, bias, out, st);
  if (m.cfg.flags & SRM_FLAG_SIMT_GEMM) return launch_gemm_simt<bf16>(epi, M, N, K, A, W, bias, out, st);
  return launch_gemm_tc(m, epi, M, N, K, A, W, bias, out, status, st);
}

// out[M, N] += A[M, K] W[N, K]^T + bias with K shared out between CTA pairs. `order`: zeroed words (split_order_words).
// Returns SRM_ERR_UNSUPPORTED when the shape does not call for it (whole tiles per pair lose nothing, or too
// few tiles): the caller then takes the unsplit kernel.
int launch_gemm_splitk(srm_model& m, int64_t M, int64_t N, int64_t K, const void* A, const void* W, const float* bias,
                       float* out, int32_t* order, uint32_t* status, cudaStream_t st, bool only_if_faster = false) {
  if (M <= 0) return SRM_OK;
  int rc = ensure_tc_ready(m);
  if (rc != SRM_OK) return rc;
  tc::SplitPlan P;
  const int64_t tiles = ((M + tc::BM - 1) / tc::BM) * ((N + tc::BN - 1) / tc::BN);
  if (K % tc::BK || !tc::split_plan(tiles, (int)(K / tc::BK), m.tc_clusters, &P)) return SRM_ERR_UNSUPPORTED;
  if (only_if_faster && tc::split_saved_kb(P) < tc::kSplitWorthKb) return SRM_ERR_UNSUPPORTED;
  LaunchScope scope(m, SRM_KERNEL_GEMM_DOWN, st);
  CUtensorMap ta, tb, td;
  if ((rc = m.tmap(A, M, K, tc::kRowsPerCta, 2, &ta)) != SRM_OK) return rc;
  if ((rc = m.tmap(W, N, K, tc::kRowsPerCta, 2, &tb)) != SRM_OK) return rc;
  if ((rc = m.tmap(out, M, N, tc::kOutBoxRows, 4, &td)) != SRM_OK) return rc;
  const uint8_t* wb = static_cast<const uint8_t*>(W);
  const int w_static = wb >= m.w && wb < m.w + m.layout.total;
  tc::SplitArgs g{M, N, K, bias, status, order, w_static};
  SRM_CUDA(launch_kernel(tc::gemm_tc_splitk_kernel, dim3(2u * (unsigned)P.pairs), dim3(tc::kThreads), tc::kSmemBytes, st,
                         ta, tb, td, g, P));
  SRM_CUDA(cudaGetLastError());
  return SRM_OK;
}

float topk_z0(int top_k, int V) {
  // threshold start of the streaming kernel: the normal quantile that leaves about 2.5 k (at least 96: the set also
  // yields the row's next candidate threshold, which wants a tail to measure) of the V logits above it
  // (rational approximation 26.2.23 of Abramowitz & Stegun; only a starting point, the kernel adapts)
  double pr = (2.5 * top_k > 96.0 ? 2.5 * top_k : 96.0) / (double)V;
  if (pr > 0.45) pr = 0.45;
  const double tt = std::sqrt(-2.0 * std::log(pr));
  return (float)(tt - (2.515517 + 0.802853 * tt + 0.010328 * tt * tt) /
                          (1.0 + 1.432788 * tt + 0.189269 * tt * tt + 0.001308 * tt * tt * tt));
}

int check_sampling(const srm_model& m, const srm_sampling* s) {
  if (s == nullptr) return SRM_ERR_INVALID_ARG;
  if (s->mode == SRM_SELECT_GREEDY) return SRM_OK;
  if (s->mode == SRM_SELECT_TOPP) {
    return (s->top_p > 0.f && s->top_p <= 1.f && s->temperature > 0.f) ? SRM_OK : SRM_ERR_INVALID_ARG;
  }
  if (s->mode != SRM_SELECT_TOPK) return SRM_ERR_INVALID_ARG;
  if (s->top_k < 1 || s->top_k > kTopKMax || s->top_k > m.cfg.vocab || !(s->temperature > 0.f)) return SRM_ERR_INVALID_ARG;
  return SRM_OK;
}

int launch_select(const srm_model& m, int64_t R, const float* logits, const srm_sampling& s, uint64_t sample_base,
                  int step, const SelectOut& out, uint32_t* status, cudaStream_t st) {
  if (R <= 0) return SRM_OK;
  LaunchScope scope(m, SRM_KERNEL_SELECT, st);
  const int V = m.cfg.vocab;
  if (s.mode == SRM_SELECT_GREEDY) {
    SRM_CUDA(launch_kernel(select_greedy_kernel, dim3((unsigned)R), dim3(kSelThreads), 0, st, logits, R, V, out, status));
  } else if (s.mode == SRM_SELECT_TOPP) {
    const float inv_t = 1.0f / s.temperature;
    const size_t scratch = ((sizeof(ToppScratch) + 15) & ~size_t(15)) + sizeof(ToppHist);
    if (V <= kToppSmemFloats) {
      const size_t smem = scratch + (size_t)V * 4;
      int rc = ensure_dynamic_smem(reinterpret_cast<const void*>(select_topp_kernel<true>),
                                   (int)(scratch + (size_t)kToppSmemFloats * 4));
      if (rc != SRM_OK) return rc;
      SRM_CUDA(launch_kernel(select_topp_kernel<true>, dim3((unsigned)R), dim3(kToppThreads), smem, st, logits, R, V,
                             s.top_p, inv_t, s.seed, sample_base, step, out, status));
    } else {
      // the scratch alone exceeds the default dynamic shared-memory limit
      int rc = ensure_dynamic_smem(reinterpret_cast<const void*>(select_topp_kernel<false>), (int)scratch);
      if (rc != SRM_OK) return rc;
      SRM_CUDA(launch_kernel(select_topp_kernel<false>, dim3((unsigned)R), dim3(kToppThreads), scratch, st, logits, R, V,
                             s.top_p, inv_t, s.seed, sample_base, step, out, status));
    }
  } else {
    const float inv_t = 1.0f / s.temperature;
    const float z0 = topk_z0(s.top_k, V);
    SRM_CUDA(launch_kernel(select_topk_stream_kernel, dim3((unsigned)R), dim3(kSelThreads), 0, st, logits, R, V, s.top_k,
                           inv_t, z0, s.seed, sample_base, step, out, status));
    // rows the streaming kernel could not settle (marked -1): the radix selection, reading the row from
    // global memory; every other block exits at once
    SRM_CUDA(launch_kernel(select_topk_kernel<false>, dim3((unsigned)R), dim3(kSelThreads), 0, st, logits, R, V, s.top_k,
                           inv_t, s.seed, sample_base, step, out, status, 1));
    ++g_kernel_launches;
  }
  SRM_CUDA(cudaGetLastError());
  return SRM_OK;
}

// True when token selection can be fused into the LM-head GEMM: greedy rule, tensor-core path, and the
// caller does not ask for the logits.
bool can_fuse_greedy(const srm_model& m, const srm_sampling& s, const float* logits_out) {
  return s.mode == SRM_SELECT_GREEDY && logits_out == nullptr && m.cfg.dtype == SRM_DTYPE_BF16 &&
         !(m.cfg.flags & SRM_FLAG_SIMT_GEMM);
}

// LM head with the argmax fused into its epilogue: `part` receives uint2 [argmax_slots(V)][R] partial
// results (it needs argmax_slots(V) * R * 8 bytes, never more than the R x V fp32 logits would), a small
// second kernel reduces them per row and writes the tokens.
int launch_lm_head_greedy(srm_model& m, int64_t R, const void* a, void* part, const SelectOut& out, uint32_t* status,
                          cudaStream_t st) {
  if (R <= 0) return SRM_OK;
  const int V = m.cfg.vocab;
  int rc = launch_gemm(m, kEpiArgmax, R, V, m.cfg.d_model, a, m.ptr(-1, SRM_T_W_LM), nullptr, part, status, st);
  if (rc != SRM_OK) return rc;
  LaunchScope scope(m, SRM_KERNEL_SELECT, st);
  const unsigned grid = (unsigned)((R + kArgmaxRows - 1) / kArgmaxRows);
  SRM_CUDA(launch_kernel(argmax_reduce_kernel, dim3(grid), dim3(kArgmaxRows * kArgmaxLanes), 0, st, reinterpret_cast<const uint2*>(part), R,
                                                                   tc::argmax_slots(V), V, out));
  SRM_CUDA(cudaGetLastError());
  return SRM_OK;
}

// True when top-k selection can be fused into the LM-head GEMM (candidates collected in the epilogue, no logits
// written): tensor-core path, no logits requested, k small enough for three times k candidates to sit well
// inside a list, and a workspace whose logits and hidden-layer areas are large enough for the lists and for the
// rows handed back (V >= 2048, F >= 2 d).
bool can_fuse_topk(const srm_model& m, const srm_sampling& s, const float* logits_out) {
  return s.mode == SRM_SELECT_TOPK && logits_out == nullptr && m.cfg.dtype == SRM_DTYPE_BF16 &&
         !(m.cfg.flags & (SRM_FLAG_SIMT_GEMM | SRM_FLAG_NO_FUSED_TOPK)) && s.top_k <= kFusedTopkMaxK &&
         (size_t)m.cfg.vocab * 4 >= (size_t)kFusedTopkCap * 8 && m.cfg.ffn_mult >= 2;
}

// LM head with top-k / temperature / Philox selection and no logits in HBM. `lists` (the logits area of the
// workspace) receives the per-row candidate lists; `scratch` (the hidden-layer area, free after the last down
// projection) holds the activation rows handed back, their indices and the counters. Rows the merge kernel
// cannot settle (no threshold yet, too few or too many candidates) get their logits from a second LM-head
// launch over just those rows, written over the (then dead) lists, and the streaming selection.
int launch_lm_head_topk(srm_model& m, int64_t R, const void* a, void* lists, void* scratch, const float* thr,
                        const srm_sampling& s, uint64_t sample_base, int step, const SelectOut& out, uint32_t* status,
                        uint32_t* handed_back, cudaStream_t st) {
  if (R <= 0) return SRM_OK;
  const int V = m.cfg.vocab, d = m.cfg.d_model;
  const size_t row_bytes = (size_t)d * 2;
  uint8_t* p = static_cast<uint8_t*>(scratch);
  void* a_fb = p; p += align_up((size_t)R * row_bytes, 256);
  int32_t* fb_rows = reinterpret_cast<int32_t*>(p); p += align_up((size_t)R * 4, 256);
  uint32_t* cnt = reinterpret_cast<uint32_t*>(p); p += align_up((size_t)R * 4, 256);
  uint32_t* n_fb = reinterpret_cast<uint32_t*>(p);
  SRM_CUDA(cudaMemsetAsync(cnt, 0, align_up((size_t)R * 4, 256) + 256, st));       // counters and n_fb
  int rc = ensure_tc_ready(m);
  if (rc != SRM_OK) return rc;
  const float inv_t = 1.0f / s.temperature;
  CUtensorMap ta, tb;
  {
    LaunchScope scope(m, SRM_KERNEL_GEMM_LM, st);
    if ((rc = m.tmap(a, R, d, tc::kRowsPerCta, 2, &ta)) != SRM_OK) return rc;
    if ((rc = m.tmap(m.ptr(-1, SRM_T_W_LM), V, d, tc::kRowsPerCta, 2, &tb)) != SRM_OK) return rc;
    CUtensorMap tb64;
    if ((rc = m.tmap(m.ptr(-1, SRM_T_W_LM), V, d, tc::kHalfN / 2, 2, &tb64)) != SRM_OK) return rc;
    const int64_t tiles = ((R + tc::BM - 1) / tc::BM) * ((V + tc::BN - 1) / tc::BN);
    tc::GemmArgs g{R, V, d, nullptr, lists, status, 1, thr, cnt, kFusedTopkCap, nullptr, gemm_tail_tiles(m, tiles)};
    const int64_t pieces = tiles + g.tail_tiles;
    const unsigned grid = 2u * (unsigned)(pieces < m.tc_clusters ? pieces : m.tc_clusters);
    SRM_CUDA(launch_kernel(tc::gemm_tc_kernel<kEpiCollect>, dim3(grid), dim3(tc::kThreads), tc::kSmemBytes, st, ta, tb, ta, tb64, g));
  }
  {
    LaunchScope scope(m, SRM_KERNEL_SELECT, st);
    SRM_CUDA(launch_kernel(topk_merge_kernel, dim3((unsigned)R), dim3(kSelThreads), 0, st,
                           reinterpret_cast<const unsigned long long*>(lists), cnt, thr, kFusedTopkCap, R, s.top_k, inv_t, s.seed,
                           sample_base, step, out, reinterpret_cast<const uint4*>(a), reinterpret_cast<uint4*>(a_fb),
                           (int)(row_bytes / 16), fb_rows, n_fb, handed_back));
  }
  {
    // the rows handed back: logits of the first *n_fb rows of a_fb only (no tile when there is none)
    LaunchScope scope(m, SRM_KERNEL_GEMM_LM, st);
    CUtensorMap tf, td;
    if ((rc = m.tmap(a_fb, R, d, tc::kRowsPerCta, 2, &tf)) != SRM_OK) return rc;
    if ((rc = m.tmap(lists, R, V, tc::kOutBoxRows, 4, &td)) != SRM_OK) return rc;
    tc::GemmArgs g{R, V, d, nullptr, lists, status, 0, nullptr, nullptr, 0, n_fb, 0};
    const int64_t tiles = ((R + tc::BM - 1) / tc::BM) * ((V + tc::BN - 1) / tc::BN);
    const unsigned grid = 2u * (unsigned)(tiles < m.tc_clusters ? tiles : m.tc_clusters);
    SRM_CUDA(launch_kernel(tc::gemm_tc_kernel<kEpiPlain>, dim3(grid), dim3(tc::kThreads), tc::kSmemBytes, st, tf, tb, td, tb, g));
  }
  {
    LaunchScope scope(m, SRM_KERNEL_SELECT, st);
    SelectOut o = out;
    o.row_map = fb_rows;
    o.n_rows = n_fb;
    const float* lg = reinterpret_cast<const float*>(lists);
    SRM_CUDA(launch_kernel(select_topk_stream_kernel, dim3((unsigned)R), dim3(kSelThreads), 0, st, lg, R, V, s.top_k, inv_t,
                           topk_z0(s.top_k, V), s.seed, sample_base, step, o, status));
    SRM_CUDA(launch_kernel(select_topk_kernel<false>, dim3((unsigned)R), dim3(kSelThreads), 0, st, lg, R, V, s.top_k, inv_t,
                           s.seed, sample_base, step, o, status, 1));
    ++g_kernel_launches;
  }
  SRM_CUDA(cudaGetLastError());
  return SRM_OK;
}

// From this many prompts per pass the scan kernel (one warp per prompt) is the faster prefill mixer.
constexpr int64_t kPrefillScanMinSamples = 384;

template <int NV, typename WT, typename ST>
int launch_prefill_scan(const PrefillParams& p, int num_sms, cudaStream_t st) {
  const int warps = prefill_scan_warps(p.d, p.Bp, num_sms);
  const size_t smem = prefill_scan_smem(p.d, warps);
  int rc = ensure_dynamic_smem(reinterpret_cast<const void*>(prefill_scan_kernel<NV, WT, ST>), kScanSmemBudget);
  if (rc != SRM_OK) return rc;
  const unsigned grid = (unsigned)(p.Bp < num_sms ? p.Bp : num_sms);
  SRM_CUDA(launch_kernel(prefill_scan_kernel<NV, WT, ST>, dim3(grid), dim3(warps * 32), smem, st, p));
  SRM_CUDA(cudaGetLastError());
  return SRM_OK;
}

template <typename WT, typename ST>
int launch_prefill_scan_nv(const PrefillParams& p, int num_sms, cudaStream_t st) {
  switch (p.d / 128) {
    case 4: return launch_prefill_scan<4, WT, ST>(p, num_sms, st);
    case 8: return launch_prefill_scan<8, WT, ST>(p, num_sms, st);
    case 12: return launch_prefill_scan<12, WT, ST>(p, num_sms, st);
    default: return launch_prefill_scan<16, WT, ST>(p, num_sms, st);
  }
}

int launch_prefill_mixer(const srm_model& m, int layer, int64_t Bp, int n, const int32_t* tok, float* x, void* S,
                         void* a, uint32_t* status, cudaStream_t st, const int32_t* len = nullptr) {
  if (Bp <= 0) return SRM_OK;
  LaunchScope scope(m, SRM_KERNEL_PREFILL_MIXER, st);
  PrefillParams p;
  p.x = x; p.tok = tok; p.E = m.ptr(-1, SRM_T_E); p.S = S; p.a = a;
  p.ln1_g = m.fptr(layer, SRM_T_LN1_G); p.ln1_b = m.fptr(layer, SRM_T_LN1_B);
  p.ln2_g = m.fptr(layer, SRM_T_LN2_G); p.ln2_b = m.fptr(layer, SRM_T_LN2_B);
  p.alpha = m.fptr(layer, SRM_T_ALPHA); p.beta = m.fptr(layer, SRM_T_BETA); p.lam = m.fptr(layer, SRM_T_LAMBDA);
  p.Bp = Bp; p.n = n; p.d = m.cfg.d_model; p.h = m.cfg.n_heads; p.n_ctx = m.cfg.n_ctx; p.vocab = m.cfg.vocab;
  p.eps = m.cfg.ln_eps; p.status = status; p.len = len;
  const size_t smem = (size_t)kPrefillTile * m.cfg.d_model * 4;
  const int nv = p.d / 128;
  const bool scan_shape = p.d % 128 == 0 && (p.d / p.h) % 128 == 0 && p.h <= 8 && (nv == 4 || nv == 8 || nv == 12 || nv == 16);
  if (scan_shape && Bp >= kPrefillScanMinSamples) {        // many prompts: one warp walks each prompt's positions
    return dispatch_types(m.cfg, [&](auto w, auto c) { return launch_prefill_scan_nv<decltype(w), decltype(c)>(p, m.num_sms, st); });
  }
  auto go = [&](auto kernel) -> int {
    SRM_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));   // smem depends on d: set per launch
    SRM_CUDA(launch_kernel(kernel, dim3((unsigned)Bp), dim3(kPrefillThreads), smem, st, p));
    SRM_CUDA(cudaGetLastError());
    return SRM_OK;
  };
  return dispatch_types(m.cfg, [&](auto w, auto c) { return go(prefill_mixer_kernel<decltype(w), decltype(c)>); });
}

// Token-mixing block with head projections (Eq. 10) on `rows` rows of the residual stream:
//   [x = E[tok]];  a = LN1(x);  q = a W_in^T;  y, S' = mixer(q, S);  x += y W_out^T;  a = LN2(x).
// Decode: t >= 0, one position, S [rows, d] in/out. Prefill: t < 0, `samples` prompts of n positions
// (rows = samples * n), sequence-parallel mixing, S [samples, d] out.
template <typename WT, typename ST>
int launch_mix_proj_t(bool prefill, const MixProjParams& p, int64_t vecs, cudaStream_t st) {
  const unsigned grid = (unsigned)((vecs + kMixProjThreads - 1) / kMixProjThreads);
  if (prefill) SRM_CUDA(launch_kernel(mixer_proj_prefill_kernel<WT, ST>, dim3(grid), dim3(kMixProjThreads), 0, st, p));
  else SRM_CUDA(launch_kernel(mixer_proj_step_kernel<WT, ST>, dim3(grid), dim3(kMixProjThreads), 0, st, p));
  return SRM_OK;
}

int launch_mixer_block_proj(srm_model& m, int layer, int t, int64_t rows, int64_t samples, int n, const int32_t* tok,
                            float* x, void* S, void* a, float* q, uint32_t* status, cudaStream_t st,
                            const int32_t* ctr = nullptr, const int32_t* pos = nullptr) {
  if (rows <= 0) return SRM_OK;
  const srm_config& c = m.cfg;
  const int d = c.d_model;
  const bool prefill = t < 0;
  const bool wb = c.dtype == SRM_DTYPE_BF16;
  int rc;
  if (tok != nullptr) {
    LaunchScope scope(m, prefill ? SRM_KERNEL_PREFILL_MIXER : SRM_KERNEL_MIXER, st);
    const unsigned grid = (unsigned)((rows * (d / 4) + kMixProjThreads - 1) / kMixProjThreads);
    if (wb) SRM_CUDA(launch_kernel(embed_rows_kernel<bf16>, dim3(grid), dim3(kMixProjThreads), 0, st, tok,
                                   reinterpret_cast<const bf16*>(m.ptr(-1, SRM_T_E)), x, rows, d, c.vocab, status));
    else SRM_CUDA(launch_kernel(embed_rows_kernel<float>, dim3(grid), dim3(kMixProjThreads), 0, st, tok,
                                reinterpret_cast<const float*>(m.ptr(-1, SRM_T_E)), x, rows, d, c.vocab, status));
  }
  if ((rc = launch_norm(m, x, rows, 1, 0, m.fptr(layer, SRM_T_LN1_G), m.fptr(layer, SRM_T_LN1_B), a, st))) return rc;
  if ((rc = launch_gemm(m, kEpiPlain, rows, d, d, a, m.ptr(layer, SRM_T_W_IN), nullptr, q, status, st, SRM_KERNEL_GEMM_PROJ))) return rc;
  {
    LaunchScope scope(m, prefill ? SRM_KERNEL_PREFILL_MIXER : SRM_KERNEL_MIXER, st);
    MixProjParams p;
    p.q = q; p.S = S; p.y = a;
    p.alpha = m.fptr(layer, SRM_T_ALPHA); p.beta = m.fptr(layer, SRM_T_BETA); p.lam = m.fptr(layer, SRM_T_LAMBDA);
    p.R = prefill ? samples : rows; p.d = d; p.h = c.n_heads; p.n_ctx = c.n_ctx; p.t = prefill ? 0 : t; p.n = n;
    p.ctr = prefill ? nullptr : ctr;
    p.pos = pos;                                   // decode: per-row positions; prefill: prompt lengths
    p.status = status;
    const int64_t vecs = p.R * (d / 4);
    rc = dispatch_types(c, [&](auto w, auto cs) { return launch_mix_proj_t<decltype(w), decltype(cs)>(prefill, p, vecs, st); });
    if (rc) return rc;
  }
  if ((rc = launch_gemm(m, kEpiBiasResidual, rows, d, d, a, m.ptr(layer, SRM_T_W_OUT), nullptr, x, status, st, SRM_KERNEL_GEMM_PROJ))) return rc;
  return launch_norm(m, x, rows, 1, 0, m.fptr(layer, SRM_T_LN2_G), m.fptr(layer, SRM_T_LN2_B), a, st);
}

// One decode step for rows [b0, b0 + R) of the state.
int decode_chunk(srm_model& m, srm_state& s, int64_t b0, int64_t R, const int32_t* tok_in, const srm_sampling& samp,
                 int step, const SelectOut& out_all, float* logits_out, const DecodeWs& w, cudaStream_t st,
                 const int32_t* ctr) {
  const srm_config& c = m.cfg;
  const int d = c.d_model;
  const int64_t F = m.F();
  const int t = (int)(s.pos < c.n_ctx ? s.pos : c.n_ctx - 1);
  const int32_t* pos = s.ragged ? s.pos_dev + b0 : nullptr;       // samples of different lengths: a position per row
  int rc;
  // the down projection shares K out between CTA pairs where that is the faster kernel for R rows
  bool split = false;
  if (w.order != nullptr && F % tc::BK == 0) {
    if ((rc = ensure_tc_ready(m))) return rc;
    tc::SplitPlan P;
    const int64_t tiles = ((R + tc::BM - 1) / tc::BM) * ((d + tc::BN - 1) / tc::BN);
    split = tc::split_plan(tiles, (int)(F / tc::BK), m.tc_clusters, &P) && tc::split_saved_kb(P) >= tc::kSplitWorthKb;
  }
  if (split) SRM_CUDA(cudaMemsetAsync(w.order, 0, w.order_bytes, st));
  for (int l = 0; l < c.n_layers; ++l) {
    uint8_t* Sl = static_cast<uint8_t*>(s.layer_ptr(l)) + (size_t)b0 * d * m.state_bytes();
    if (c.mixer != SRM_MIXER_MIXED) {
      if ((rc = launch_mixer_variant(m, l, t, R, l == 0 ? tok_in + b0 : nullptr, 1, w.x, w.a, d, Sl, s.plane_elems(), s.status,
                                     st, ctr))) return rc;
    } else if (m.head_proj()) {
      if ((rc = launch_mixer_block_proj(m, l, t, R, R, 1, l == 0 ? tok_in + b0 : nullptr, w.x, Sl, w.a, w.q, s.status, st, ctr, pos))) return rc;
    } else if ((rc = launch_mixer(m, l, t, R, l == 0 ? tok_in + b0 : nullptr, w.x, Sl, w.a, s.status, st, ctr, pos))) return rc;
    if ((rc = launch_gemm(m, kEpiBiasGelu, R, F, d, w.a, m.ptr(l, SRM_T_W1), m.fptr(l, SRM_T_B1), w.H, s.status, st))) return rc;
    rc = split ? launch_gemm_splitk(m, R, d, F, w.H, m.ptr(l, SRM_T_W2), m.fptr(l, SRM_T_B2), w.x, w.order, s.status, st, true)
               : SRM_ERR_UNSUPPORTED;
    if (rc == SRM_ERR_UNSUPPORTED)
      rc = launch_gemm(m, kEpiBiasResidual, R, d, F, w.H, m.ptr(l, SRM_T_W2), m.fptr(l, SRM_T_B2), w.x, s.status, st);
    if (rc) return rc;
  }
  if ((rc = launch_final_norm(m, w.x, R, 1, 0, w.a, st))) return rc;
  SelectOut o = out_all;
  o.last_tok += b0;
  if (o.tok_out) o.tok_out += b0;
  if (o.store) o.store += b0 * o.store_stride;
  if (o.pos) o.pos += b0;
  if (o.thr_out) o.thr_out += b0;
  if (can_fuse_greedy(m, samp, logits_out)) return launch_lm_head_greedy(m, R, w.a, w.logits, o, s.status, st);
  if (can_fuse_topk(m, samp, logits_out))
    return launch_lm_head_topk(m, R, w.a, w.logits, w.H, s.thr + b0, samp, samp.sample_idx_base + (uint64_t)b0, step, o,
                               s.status, s.status + kCtrHandedBack, st);
  float* lg = logits_out != nullptr ? logits_out + b0 * c.vocab : w.logits;
  if ((rc = launch_gemm(m, kEpiPlain, R, c.vocab, d, w.a, m.ptr(-1, SRM_T_W_LM), nullptr, lg, s.status, st))) return rc;
  return launch_select(m, R, lg, samp, samp.sample_idx_base + (uint64_t)b0, step, o, s.status, st);
}

// ---- small batches: the whole step in one cooperative kernel (step_small.cuh) ----------------------
struct SmallPlan { sb::Params p; int grid; size_t smem; };

// Whether a batch of B samples takes the single-kernel step, and its slab plan. Mixed heads, bf16 weights, at most
// 64 samples and 1024 channels; everything else takes the kernel-per-operation path.
bool small_step_plan(const srm_model& m, const srm_state& s, SmallPlan* P) {
  const srm_config& c = m.cfg;
  if (c.dtype != SRM_DTYPE_BF16 || (c.flags & (SRM_FLAG_SIMT_GEMM | SRM_FLAG_NO_SMALL_BATCH | SRM_FLAG_HEAD_PROJ))) return false;
  if (c.mixer != SRM_MIXER_MIXED || s.ragged || s.B > sb::kMaxRows || c.d_model > 1024 || m.num_sms < 16 || m.num_sms > 256) return false;
  const int d = c.d_model, F = (int)m.F(), V = c.vocab, G = m.num_sms;
  if (F % 32 || d % 64) return false;
  sb::Params& p = P->p;
  p.up_cols = ((F + G - 1) / G + 15) / 16 * 16;
  p.up_ctas = (F + p.up_cols - 1) / p.up_cols;
  p.dn_cols = 64;
  p.dn_nslabs = d / 64;
  int ks = G / p.dn_nslabs;
  ks = ks > 8 ? 8 : ks;
  if (ks < 1) return false;
  p.dn_klen = ((F + ks - 1) / ks + 31) / 32 * 32;
  p.dn_kslabs = (F + p.dn_klen - 1) / p.dn_klen;
  p.lm_cols = ((V + G - 1) / G + sb::kLmChunkCols - 1) / sb::kLmChunkCols * sb::kLmChunkCols;
  p.lm_ctas = (V + p.lm_cols - 1) / p.lm_cols;
  P->grid = G;
  P->smem = 128 + (size_t)sb::act_region_bytes(d, p.dn_klen) + (size_t)sb::weight_region_bytes(d, p.up_cols, p.dn_cols, p.dn_klen);
  return P->smem <= (size_t)sb::kSmemBytes;
}

template <typename ST>
int launch_step_small_t(const SmallPlan& P, cudaStream_t st) {
  int rc = ensure_dynamic_smem(reinterpret_cast<const void*>(sb::step_small_kernel<ST>), sb::kSmemBytes);
  if (rc != SRM_OK) return rc;
  int per_sm = 0;
  SRM_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sb::step_small_kernel<ST>, sb::kThreads, P.smem));
  if (per_sm < 1) return SRM_ERR_UNSUPPORTED;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)P.grid);
  cfg.blockDim = dim3(sb::kThreads);
  cfg.dynamicSmemBytes = P.smem;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeCooperative;           // all CTAs resident at once: the kernel has grid-wide barriers
  attr.val.cooperative = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  SRM_CUDA(cudaLaunchKernelEx(&cfg, sb::step_small_kernel<ST>, P.p));
  return SRM_OK;
}

// One decode step of all B <= 64 samples of the state. SRM_ERR_UNSUPPORTED: take the ordinary path.
int decode_step_small(srm_model& m, srm_state& s, SmallPlan& P, const int32_t* tok_in, const srm_sampling& samp, int step,
                      const SelectOut& out, float* logits_out, const DecodeWs& w, cudaStream_t st, const int32_t* ctr) {
  const srm_config& c = m.cfg;
  sb::Params& p = P.p;
  p.B = (int)s.B; p.d = c.d_model; p.F = (int)m.F(); p.V = c.vocab; p.h = c.n_heads; p.n_ctx = c.n_ctx; p.L = c.n_layers;
  p.t = (int)(s.pos < c.n_ctx ? s.pos : c.n_ctx - 1);
  p.eps = c.ln_eps;
  p.tok_in = tok_in;
  p.E = reinterpret_cast<const bf16*>(m.ptr(-1, SRM_T_E));
  p.W_lm = reinterpret_cast<const bf16*>(m.ptr(-1, SRM_T_W_LM));
  p.lnf_g = m.fptr(-1, SRM_T_LNF_G); p.lnf_b = m.fptr(-1, SRM_T_LNF_B);
  p.layer0 = sb::LayerW{m.fptr(0, SRM_T_LN1_G), m.fptr(0, SRM_T_LN1_B), m.fptr(0, SRM_T_LN2_G), m.fptr(0, SRM_T_LN2_B),
                        m.fptr(0, SRM_T_ALPHA), m.fptr(0, SRM_T_BETA), m.fptr(0, SRM_T_LAMBDA), m.fptr(0, SRM_T_B1),
                        m.fptr(0, SRM_T_B2), reinterpret_cast<const bf16*>(m.ptr(0, SRM_T_W1)),
                        reinterpret_cast<const bf16*>(m.ptr(0, SRM_T_W2))};
  p.layer_bytes = c.n_layers > 1 ? (int64_t)(m.layout.layer[SRM_T_COUNT + SRM_T_LN1_G].off - m.layout.layer[SRM_T_LN1_G].off) : 0;
  p.S = s.layer_ptr(0);
  p.layer_stride = (int64_t)s.B * c.d_model * m.state_bytes();
  p.x = w.x; p.a = reinterpret_cast<bf16*>(w.a); p.H = reinterpret_cast<bf16*>(w.H);
  uint8_t* q = w.small;
  p.part = reinterpret_cast<float*>(q); q += align_up((size_t)8 * sb::kMaxRows * c.d_model * 4, 256);
  p.best = reinterpret_cast<unsigned long long*>(q); q += align_up((size_t)256 * sb::kMaxRows * 8, 256);
  p.bar = reinterpret_cast<uint32_t*>(q);
  p.status = s.status;
  p.ctr = ctr;
  p.greedy = samp.mode == SRM_SELECT_GREEDY ? 1 : 0;
  p.logits = logits_out != nullptr ? logits_out : (p.greedy ? nullptr : w.logits);
  p.out = out;
  SRM_CUDA(cudaMemsetAsync(p.bar, 0, 256, st));
  int rc;
  {
    LaunchScope scope(m, SRM_KERNEL_STEP_SMALL, st);
    if (c.state_dtype == SRM_DTYPE_FP16) rc = launch_step_small_t<fp16>(P, st);
    else if (c.state_dtype == SRM_DTYPE_BF16) rc = launch_step_small_t<bf16>(P, st);
    else rc = launch_step_small_t<float>(P, st);
  }
  if (rc != SRM_OK || p.greedy) return rc;
  return launch_select(m, s.B, p.logits, samp, samp.sample_idx_base, step, out, s.status, st);
}

// Rows per decode pass for a batch of B rows when the workspace holds up to `fit` rows. Up to kOnePassRows the
// batch runs as one pass. Beyond that it is cut into the fewest equal passes of at most kMaxPassRows rows, each a
// whole number of 256-row tiles: a larger pass pushes the activations of a layer (H, x, a: 14 KB per row for
// d = 1024) out of L2 between the GEMMs, a smaller one leaves rounds of tiles partly empty. Measured at 32768
// rows, d = 1024: 4096 / 5888 / 8192 / 9472 / 16384 / 32768 rows per pass take 11.95 / 11.75 / 11.35 / 11.24 /
// 11.49 / 11.68 ms per step; at 16384 rows, d = 1536: 4608 / 9472 / 16384 rows take 17.67 / 16.84 / 17.33 ms.
constexpr int64_t kOnePassRows = 12288, kMaxPassRows = 10240;
int64_t choose_pass_rows(int64_t B, int64_t fit) {
  if (fit < B && fit < kMaxPassRows) return fit;              // the workspace decides
  if (B <= kOnePassRows && fit >= B) return B;
  const int64_t passes = (B + kMaxPassRows - 1) / kMaxPassRows;
  int64_t rows = (B + passes - 1) / passes;
  rows = (rows + tc::BM - 1) / tc::BM * tc::BM;
  return rows < fit ? rows : fit;
}

// `ctr` non-null: position, Philox step and store column come from the device-side counters (graph replay).
int decode_step_impl(srm_model* m, srm_state* s, const int32_t* d_tok_in, const srm_sampling* samp, int step,
                     int32_t* d_tok_out, int32_t* d_store, int64_t store_stride, int64_t store_col,
                     float* d_logits_out, void* d_ws, size_t ws_bytes, cudaStream_t st, const int32_t* ctr = nullptr) {
  if (m == nullptr || s == nullptr || s->m != m || d_ws == nullptr) return SRM_ERR_INVALID_ARG;
  int rc = check_sampling(*m, samp);
  if (rc) return rc;
  if (!aligned(d_ws, 256) || !aligned(d_tok_in, 4) || !aligned(d_tok_out, 4) || !aligned(d_logits_out, 16)) return SRM_ERR_ALIGNMENT;
  if (s->pos >= m->cfg.n_ctx) return SRM_ERR_CTX_OVERFLOW;
  const int64_t fit = fit_rows(ws_bytes, s->B, decode_need, *m, 0);
  if (fit < 1) return SRM_ERR_BUFFER_TOO_SMALL;
  const int64_t rows = choose_pass_rows(s->B, fit);
  const DecodeWs w = carve_decode(*m, d_ws, rows);
  const int32_t* tok_in = d_tok_in != nullptr ? d_tok_in : s->last_tok;
  SelectOut out{s->last_tok, d_tok_out, d_store, store_stride, store_col, 1, ctr, s->ragged ? s->pos_dev : nullptr,
                nullptr, nullptr, samp->mode == SRM_SELECT_TOPK ? s->thr : nullptr};
  SmallPlan small;
  if (rows >= s->B && small_step_plan(*m, *s, &small)) {
    rc = decode_step_small(*m, *s, small, tok_in, *samp, step, out, d_logits_out, w, st, ctr);
    if (rc != SRM_ERR_UNSUPPORTED) {
      if (rc == SRM_OK) s->pos += 1;
      return rc;
    }
  }
  for (int64_t b0 = 0; b0 < s->B; b0 += rows) {
    const int64_t R = (s->B - b0 < rows) ? s->B - b0 : rows;
    if ((rc = decode_chunk(*m, *s, b0, R, tok_in, *samp, step, out, d_logits_out, w, st, ctr))) return rc;
  }
  s->pos += 1;
  return SRM_OK;
}

}  // namespace

// ================================ C ABI =========================================================
extern "C" {

size_t srm_weights_bytes(const srm_config* cfg) {
  if (!config_ok(cfg)) return 0;
  return make_layout(*cfg).total;
}

int srm_weight_slot(const srm_config* cfg, int32_t layer, int32_t tensor, size_t* offset, size_t* nbytes,
                    int32_t* elem_bytes) {
  if (!config_ok(cfg) || tensor < 0 || tensor >= SRM_T_COUNT) return SRM_ERR_INVALID_ARG;
  const Layout L = make_layout(*cfg);
  Slot s;
  if (is_global_tensor(tensor)) {
    s = L.global[tensor];
  } else {
    if (layer < 0 || layer >= cfg->n_layers) return SRM_ERR_INVALID_ARG;
    if ((tensor == SRM_T_W_IN || tensor == SRM_T_W_OUT) && !(cfg->flags & SRM_FLAG_HEAD_PROJ)) return SRM_ERR_INVALID_ARG;
    s = L.layer[(size_t)layer * SRM_T_COUNT + tensor];
  }
  if (offset) *offset = s.off;
  if (nbytes) *nbytes = s.bytes;
  if (elem_bytes) *elem_bytes = s.elem;
  return SRM_OK;
}

size_t srm_state_bytes(const srm_config* cfg, int64_t B) {
  if (!config_ok(cfg) || B < 1) return 0;
  return state_bytes_for(*cfg, B);
}

size_t srm_workspace_bytes(const srm_config* cfg, int64_t B_chunk, int32_t n_prefill_max) {
  if (!config_ok(cfg) || B_chunk < 1 || n_prefill_max < 0) return 0;
  srm_model tmp;
  tmp.cfg = *cfg;
  size_t need = decode_ws_bytes(tmp, B_chunk);
  if (n_prefill_max > 0) {
    const size_t p = prefill_ws_bytes(tmp, 1, n_prefill_max);
    if (p > need) need = p;
  }
  return need;
}

int srm_create(const srm_config* cfg, const void* d_weights, size_t nbytes, srm_model** out) {
  if (out == nullptr || d_weights == nullptr) return SRM_ERR_INVALID_ARG;
  *out = nullptr;
  if (cfg == nullptr) return SRM_ERR_INVALID_ARG;
  if (!config_ok(cfg)) return SRM_ERR_UNSUPPORTED;
  if (!aligned(d_weights, 256)) return SRM_ERR_ALIGNMENT;
  srm_model* m = new (std::nothrow) srm_model();
  if (m == nullptr) return SRM_ERR_INVALID_ARG;
  m->cfg = *cfg;
  m->w = static_cast<const uint8_t*>(d_weights);
  m->layout = make_layout(*cfg);
  if (nbytes < m->layout.total) { delete m; return SRM_ERR_BUFFER_TOO_SMALL; }
  cudaError_t e = cudaGetDevice(&m->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&m->num_sms, cudaDevAttrMultiProcessorCount, m->device);
  if (e != cudaSuccess) { g_last_cuda_error = (int)e; delete m; return SRM_ERR_CUDA; }
  m->tmaps.reserve(256);
  *out = m;
  return SRM_OK;
}

int srm_destroy(srm_model* m) {
  if (m != nullptr) {
    if (m->step_exec != nullptr) cudaGraphExecDestroy(m->step_exec);
    if (m->cap_stream != nullptr) cudaStreamDestroy(m->cap_stream);
    for (auto& r : m->prof) { cudaEventDestroy(r.start); cudaEventDestroy(r.stop); }
    for (auto& e : m->event_pool) cudaEventDestroy(e);
  }
  delete m;
  return SRM_OK;
}

int srm_profile_enable(srm_model* m, int on) {
  if (m == nullptr) return SRM_ERR_INVALID_ARG;
  m->profiling = on != 0;
  return SRM_OK;
}

int srm_profile_read(srm_model* m, int32_t kernel_class, uint64_t* launches, double* total_ms) {
  if (m == nullptr || kernel_class < 0 || kernel_class >= SRM_KERNEL_CLASS_COUNT) return SRM_ERR_INVALID_ARG;
  for (auto& r : m->prof) {
    SRM_CUDA(cudaEventSynchronize(r.stop));
    float ms = 0.f;
    SRM_CUDA(cudaEventElapsedTime(&ms, r.start, r.stop));
    m->prof_launches[r.cls] += 1;
    m->prof_ms[r.cls] += ms;
    m->event_pool.push_back(r.start);
    m->event_pool.push_back(r.stop);
  }
  m->prof.clear();
  if (launches) *launches = m->prof_launches[kernel_class];
  if (total_ms) *total_ms = m->prof_ms[kernel_class];
  return SRM_OK;
}

int srm_profile_reset(srm_model* m) {
  if (m == nullptr) return SRM_ERR_INVALID_ARG;
  int rc = srm_profile_read(m, 0, nullptr, nullptr);
  if (rc) return rc;
  for (int i = 0; i < SRM_KERNEL_CLASS_COUNT; ++i) { m->prof_launches[i] = 0; m->prof_ms[i] = 0.0; }
  return SRM_OK;
}

uint64_t srm_kernel_launches(void) { return g_kernel_launches; }

int64_t srm_decode_pass_rows(int64_t B, int64_t ws_rows) { return B < 1 || ws_rows < 1 ? 0 : choose_pass_rows(B, ws_rows); }

int srm_state_create(srm_model* m, int64_t B, void* d_state, size_t nbytes, void* stream, srm_state** out) {
  if (out == nullptr) return SRM_ERR_INVALID_ARG;
  *out = nullptr;
  if (m == nullptr || d_state == nullptr || B < 1) return SRM_ERR_INVALID_ARG;
  if (!aligned(d_state, 256)) return SRM_ERR_ALIGNMENT;
  if (nbytes < state_bytes_for(m->cfg, B)) return SRM_ERR_BUFFER_TOO_SMALL;
  srm_state* s = new (std::nothrow) srm_state();
  if (s == nullptr) return SRM_ERR_INVALID_ARG;
  s->m = m; s->B = B; s->base = static_cast<uint8_t*>(d_state); s->nbytes = state_bytes_for(m->cfg, B);
  s->status = reinterpret_cast<uint32_t*>(s->base);
  s->last_tok = reinterpret_cast<int32_t*>(s->base + kStateHeader);
  s->pos_dev = reinterpret_cast<int32_t*>(s->base + kStateHeader + align_up((size_t)B * 4, 256));
  s->thr = reinterpret_cast<float*>(s->base + kStateHeader + 2 * align_up((size_t)B * 4, 256));
  s->S = s->base + kStateHeader + 3 * align_up((size_t)B * 4, 256);
  s->pos = 0;
  int rc = srm_state_reset(s, stream);
  if (rc != SRM_OK) { delete s; return rc; }
  *out = s;
  return SRM_OK;
}

int srm_state_destroy(srm_state* s) {
  if (s != nullptr && s->m != nullptr && s->m->step_key.s == s && s->m->step_exec != nullptr) {
    cudaGraphExecDestroy(s->m->step_exec);        // the captured step refers to this state's buffers
    s->m->step_exec = nullptr;
    s->m->step_key = srm_model::StepKey();
  }
  delete s;
  return SRM_OK;
}

int srm_state_reset(srm_state* s, void* stream) {
  if (s == nullptr) return SRM_ERR_INVALID_ARG;
  SRM_CUDA(cudaMemsetAsync(s->base, 0, s->nbytes, static_cast<cudaStream_t>(stream)));
  s->pos = 0;
  s->ragged = false;
  return SRM_OK;
}

int64_t srm_state_pos(const srm_state* s) { return s ? s->pos : -1; }

int srm_state_set_pos(srm_state* s, int64_t pos) {
  if (s == nullptr || pos < 0 || pos > s->m->cfg.n_ctx) return SRM_ERR_INVALID_ARG;
  if (s->ragged) return SRM_ERR_INVALID_ARG;            // the positions live on the device, one per sample
  s->pos = pos;
  return SRM_OK;
}

int srm_state_adopt_positions(srm_state* s, int64_t max_pos) {
  if (s == nullptr || max_pos < 1 || max_pos > s->m->cfg.n_ctx) return SRM_ERR_INVALID_ARG;
  s->pos = max_pos;
  s->ragged = true;
  return SRM_OK;
}

int srm_state_is_ragged(const srm_state* s) { return s != nullptr && s->ragged ? 1 : 0; }

void* srm_state_layer_ptr(const srm_state* s, int32_t layer) {
  if (s == nullptr || layer < 0 || layer >= s->m->cfg.n_layers) return nullptr;
  return s->layer_ptr(layer);
}

int32_t* srm_state_last_token_ptr(const srm_state* s) { return s ? s->last_tok : nullptr; }

int32_t srm_cache_planes(const srm_config* cfg) { return config_ok(cfg) ? cache_planes(*cfg) : 0; }

float* srm_state_topk_threshold_ptr(const srm_state* s) { return s ? s->thr : nullptr; }

int srm_state_topk_handed_back(srm_state* s, void* stream, uint64_t* rows) {
  if (s == nullptr || rows == nullptr) return SRM_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t v = 0;
  SRM_CUDA(cudaMemcpyAsync(&v, s->status + kCtrHandedBack, 4, cudaMemcpyDeviceToHost, st));
  SRM_CUDA(cudaStreamSynchronize(st));
  *rows = v;
  return SRM_OK;
}

int srm_status(srm_state* s, void* stream, uint32_t* flags) {
  if (s == nullptr) return SRM_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t f = 0;
  SRM_CUDA(cudaMemcpyAsync(&f, s->status, 4, cudaMemcpyDeviceToHost, st));
  SRM_CUDA(cudaMemsetAsync(s->status, 0, 4, st));
  SRM_CUDA(cudaStreamSynchronize(st));
  if (flags) *flags = f;
  return f ? SRM_ERR_DEVICE_STATUS : SRM_OK;
}

}  // extern "C"

namespace {

// Sequence-parallel prefill of `P` prompts, each standing for `replicas` consecutive samples of the state
// (replicas == 1: the plain prefill). A prompt is run once; with replicas > 1 its per-layer cache goes to a
// staging area at the end of the workspace and is then copied to the rows of its replicas, and every replica
// selects its own first token from the prompt's last-position logits.
int prefill_impl(srm_model* m, srm_state* s, const int32_t* d_tokens, int64_t P, int32_t n, int64_t replicas,
                 const srm_sampling* samp, int32_t* d_first_tok, float* d_logits_last, void* d_ws, size_t ws_bytes,
                 cudaStream_t st, const int32_t* d_len = nullptr) {
  const srm_config& c = m->cfg;
  const int d = c.d_model;
  const int64_t F = m->F();
  const size_t row_bytes = (size_t)d * m->state_bytes();
  const int planes = cache_planes(c);
  const size_t stage_per_prompt = replicas > 1 ? align_up((size_t)c.n_layers * planes * row_bytes, 256) : 0;
  // largest number of prompts per pass whose workspace and staging both fit
  int64_t Bp = fit_rows(ws_bytes, P, prefill_need, *m, n);
  while (Bp >= 1 && prefill_ws_bytes(*m, Bp, n) + (size_t)Bp * stage_per_prompt > ws_bytes) --Bp;
  if (Bp < 1) return SRM_ERR_BUFFER_TOO_SMALL;
  const PrefillWs w = carve_prefill(*m, d_ws, Bp, n);
  uint8_t* stage = static_cast<uint8_t*>(d_ws) + align_up(prefill_ws_bytes(*m, Bp, n), 256);
  int rc;
  for (int64_t p0 = 0; p0 < P; p0 += Bp) {
    const int64_t np = (P - p0 < Bp) ? P - p0 : Bp;
    const int64_t rows = np * n;
    const int64_t b0 = p0 * replicas, nb = np * replicas;          // state rows of this pass
    for (int l = 0; l < c.n_layers; ++l) {
      uint8_t* Sl = replicas > 1 ? stage + (size_t)l * planes * np * row_bytes
                                 : static_cast<uint8_t*>(s->layer_ptr(l)) + (size_t)b0 * row_bytes;
      if (c.mixer != SRM_MIXER_MIXED) {
        // the sequence form of these mixers through their recurrence: one launch per position over all prompts of the
        // pass, the (zeroed) cache updated in place; rows of one prompt are n apart in x and a
        const int64_t plane = replicas > 1 ? np * (int64_t)d : s->plane_elems();
        for (int pl = 0; pl < planes; ++pl)          // the recurrence starts from an empty cache
          SRM_CUDA(cudaMemsetAsync(Sl + (size_t)pl * plane * m->state_bytes(), 0, (size_t)np * row_bytes, st));
        for (int t = 0; t < n; ++t)
          if ((rc = launch_mixer_variant(*m, l, t, np, l == 0 ? d_tokens + p0 * n + t : nullptr, n, w.x + (size_t)t * d,
                                         static_cast<uint8_t*>(w.a) + (size_t)t * d * m->act_bytes(), (int64_t)n * d, Sl, plane,
                                         s->status, st, nullptr, SRM_KERNEL_PREFILL_MIXER))) return rc;
      } else if (m->head_proj()) {
        if ((rc = launch_mixer_block_proj(*m, l, -1, rows, np, n, l == 0 ? d_tokens + p0 * n : nullptr, w.x, Sl, w.a, w.q, s->status, st,
                                          nullptr, d_len ? d_len + p0 : nullptr))) return rc;
      } else if ((rc = launch_prefill_mixer(*m, l, np, n, l == 0 ? d_tokens + p0 * n : nullptr, w.x, Sl, w.a, s->status, st,
                                            d_len ? d_len + p0 : nullptr))) return rc;
      if ((rc = launch_gemm(*m, kEpiBiasGelu, rows, F, d, w.a, m->ptr(l, SRM_T_W1), m->fptr(l, SRM_T_B1), w.H, s->status, st))) return rc;
      if ((rc = launch_gemm(*m, kEpiBiasResidual, rows, d, F, w.H, m->ptr(l, SRM_T_W2), m->fptr(l, SRM_T_B2), w.x, s->status, st))) return rc;
      for (int pl = 0; replicas > 1 && pl < planes; ++pl) {
        LaunchScope scope(*m, SRM_KERNEL_PREFILL_MIXER, st);
        const int64_t vpr = (int64_t)row_bytes / 16, total = nb * vpr;
        const uint8_t* src = Sl + (size_t)pl * np * row_bytes;
        uint8_t* dst = static_cast<uint8_t*>(s->layer_ptr(l)) + ((size_t)pl * s->B + (size_t)b0) * row_bytes;
        SRM_CUDA(launch_kernel(broadcast_rows_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st,
                               reinterpret_cast<const uint4*>(src), reinterpret_cast<uint4*>(dst), np, replicas, vpr));
      }
    }
    // LM head on the last prompt position only; selection per state row
    if ((rc = launch_final_norm(*m, w.x, np, n, n - 1, w.a_last, st, d_len ? d_len + p0 : nullptr))) return rc;
    SelectOut o{s->last_tok + b0, d_first_tok ? d_first_tok + b0 : nullptr, nullptr, 0, 0, replicas, nullptr, nullptr,
                nullptr, nullptr, samp->mode == SRM_SELECT_TOPK ? s->thr + b0 : nullptr};
    if (replicas == 1 && can_fuse_greedy(*m, *samp, d_logits_last)) {
      if ((rc = launch_lm_head_greedy(*m, np, w.a_last, w.logits, o, s->status, st))) return rc;
      continue;
    }
    float* lg = d_logits_last != nullptr ? d_logits_last + p0 * c.vocab : w.logits;
    if ((rc = launch_gemm(*m, kEpiPlain, np, c.vocab, d, w.a_last, m->ptr(-1, SRM_T_W_LM), nullptr, lg, s->status, st))) return rc;
    if ((rc = launch_select(*m, nb, lg, *samp, samp->sample_idx_base + (uint64_t)b0, 0, o, s->status, st))) return rc;
  }
  s->pos = n;
  if (d_len != nullptr) {
    // from here on every sample has its own position: its prompt length (srm_prefill_ragged checked replicas == 1)
    ++g_kernel_launches;
    SRM_CUDA(launch_kernel(clamp_lengths_kernel, dim3((unsigned)((s->B + 255) / 256)), dim3(256), 0, st, d_len, s->pos_dev,
                           s->B, 1, (int)n));
    s->ragged = true;
  }
  return SRM_OK;
}

int prefill_check(srm_model* m, srm_state* s, const int32_t* d_tokens, int32_t n, const srm_sampling* samp,
                  const int32_t* d_first_tok, const float* d_logits_last, const void* d_ws) {
  if (m == nullptr || s == nullptr || s->m != m || d_tokens == nullptr || d_ws == nullptr || n < 1) return SRM_ERR_INVALID_ARG;
  int rc = check_sampling(*m, samp);
  if (rc) return rc;
  if (!aligned(d_ws, 256) || !aligned(d_tokens, 4) || !aligned(d_first_tok, 4) || !aligned(d_logits_last, 16)) return SRM_ERR_ALIGNMENT;
  if (s->pos != 0) return SRM_ERR_INVALID_ARG;           // the parallel form starts from an empty cache
  if (n > m->cfg.n_ctx) return SRM_ERR_CTX_OVERFLOW;
  return SRM_OK;
}

}  // namespace

extern "C" {

int srm_prefill(srm_model* m, srm_state* s, const int32_t* d_tokens, int32_t n, const srm_sampling* samp,
                int32_t* d_first_tok, float* d_logits_last, void* d_ws, size_t ws_bytes, void* stream) {
  int rc = prefill_check(m, s, d_tokens, n, samp, d_first_tok, d_logits_last, d_ws);
  if (rc) return rc;
  return prefill_impl(m, s, d_tokens, s->B, n, 1, samp, d_first_tok, d_logits_last, d_ws, ws_bytes,
                      static_cast<cudaStream_t>(stream));
}

int srm_prefill_ragged(srm_model* m, srm_state* s, const int32_t* d_tokens, int32_t n_max, const int32_t* d_lengths,
                       const srm_sampling* samp, int32_t* d_first_tok, float* d_logits_last, void* d_ws, size_t ws_bytes,
                       void* stream) {
  int rc = prefill_check(m, s, d_tokens, n_max, samp, d_first_tok, d_logits_last, d_ws);
  if (rc) return rc;
  if (d_lengths == nullptr) return SRM_ERR_INVALID_ARG;
  if (!aligned(d_lengths, 4)) return SRM_ERR_ALIGNMENT;
  if (m->cfg.mixer != SRM_MIXER_MIXED) return SRM_ERR_UNSUPPORTED;      // one position per sample: mixed heads only
  return prefill_impl(m, s, d_tokens, s->B, n_max, 1, samp, d_first_tok, d_logits_last, d_ws, ws_bytes,
                      static_cast<cudaStream_t>(stream), d_lengths);
}

int srm_prefill_replicated(srm_model* m, srm_state* s, const int32_t* d_tokens, int32_t n_prompts, int32_t n,
                           int32_t replicas, const srm_sampling* samp, int32_t* d_first_tok, float* d_logits_last,
                           void* d_ws, size_t ws_bytes, void* stream) {
  int rc = prefill_check(m, s, d_tokens, n, samp, d_first_tok, d_logits_last, d_ws);
  if (rc) return rc;
  if (n_prompts < 1 || replicas < 1 || (int64_t)n_prompts * replicas != s->B) return SRM_ERR_INVALID_ARG;
  return prefill_impl(m, s, d_tokens, n_prompts, n, replicas, samp, d_first_tok, d_logits_last, d_ws, ws_bytes,
                      static_cast<cudaStream_t>(stream));
}

int srm_decode_step(srm_model* m, srm_state* s, const int32_t* d_tok_in, const srm_sampling* samp, int32_t step,
                    int32_t* d_tok_out, float* d_logits_out, void* d_ws, size_t ws_bytes, void* stream) {
  return decode_step_impl(m, s, d_tok_in, samp, step, d_tok_out, nullptr, 0, 0, d_logits_out, d_ws, ws_bytes,
                          static_cast<cudaStream_t>(stream));
}

}  // extern "C"

namespace {

// Whether srm_generate replays a captured step: worth it when the step is bound by the host's launch rate
// (about 50 kernels of a few microseconds each), i.e. for small batches.
bool use_step_graph(const srm_model& m, const srm_state& s, int steps) {
  if (m.profiling || (m.cfg.flags & SRM_FLAG_NO_GRAPH) || steps < 4) return false;
  if (m.cfg.flags & SRM_FLAG_GRAPH) return true;
  return s.B * (int64_t)m.cfg.d_model <= (int64_t)1 << 21;
}

// Captures one decode step (all its kernels, driven by the device-side counters, plus the kernel that
// advances them) on the model's own stream and instantiates it; reuses the previous graph when nothing it
// was captured for has changed. Nothing is executed here.
int prepare_step_graph(srm_model* m, srm_state* s, const srm_sampling* samp, int32_t* d_out, int64_t out_stride,
                       void* d_ws, size_t ws_bytes) {
  srm_model::StepKey key;
  key.s = s; key.ws = d_ws; key.ws_bytes = ws_bytes; key.out = d_out; key.out_stride = out_stride; key.samp = *samp;
  key.ragged = s->ragged;
  if (m->step_exec != nullptr && m->step_key == key) return SRM_OK;
  if (m->step_exec != nullptr) { cudaGraphExecDestroy(m->step_exec); m->step_exec = nullptr; }
  if (m->cap_stream == nullptr) SRM_CUDA(cudaStreamCreateWithFlags(&m->cap_stream, cudaStreamNonBlocking));
  int32_t* hdr = reinterpret_cast<int32_t*>(s->status);
  const int64_t pos0 = s->pos;
  SRM_CUDA(cudaStreamBeginCapture(m->cap_stream, cudaStreamCaptureModeRelaxed));
  int rc = decode_step_impl(m, s, nullptr, samp, 0, nullptr, d_out, out_stride, 0, nullptr, d_ws, ws_bytes,
                            m->cap_stream, hdr);
  cudaError_t e = cudaSuccess;
  if (rc == SRM_OK) {
    ++g_kernel_launches;
    e = launch_kernel(advance_counters_kernel, dim3(1), dim3(1), 0, m->cap_stream, hdr);
  }
  cudaGraph_t graph = nullptr;
  const cudaError_t e2 = cudaStreamEndCapture(m->cap_stream, &graph);
  s->pos = pos0;                                       // the captured step has not run
  if (rc != SRM_OK) { if (graph) cudaGraphDestroy(graph); return rc; }
  if (e != cudaSuccess || e2 != cudaSuccess || graph == nullptr) {
    if (graph) cudaGraphDestroy(graph);
    g_last_cuda_error = (int)(e != cudaSuccess ? e : e2);
    return SRM_ERR_CUDA;
  }
  e = cudaGraphInstantiate(&m->step_exec, graph, 0);
  cudaGraphDestroy(graph);
  if (e != cudaSuccess) { m->step_exec = nullptr; g_last_cuda_error = (int)e; return SRM_ERR_CUDA; }
  m->step_key = key;
  return SRM_OK;
}

}  // namespace

extern "C" {

int srm_generate(srm_model* m, srm_state* s, int32_t steps, int32_t first_step, const srm_sampling* samp,
                 int32_t* d_out, int64_t out_stride, void* d_ws, size_t ws_bytes, void* stream) {
  if (m == nullptr || s == nullptr || s->m != m || steps < 0 || (d_out != nullptr && out_stride < steps)) return SRM_ERR_INVALID_ARG;
  if (s->pos + steps > m->cfg.n_ctx) return SRM_ERR_CTX_OVERFLOW;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (samp != nullptr && d_ws != nullptr && use_step_graph(*m, *s, steps)) {
    const uint64_t launches0 = g_kernel_launches;
    int rc = prepare_step_graph(m, s, samp, d_out, out_stride, d_ws, ws_bytes);
    if (rc) return rc;
    const uint64_t per_step = g_kernel_launches - launches0;      // 0 when the graph was reused
    if (per_step) m->step_launches = per_step;
    g_kernel_launches = launches0;
    SRM_CUDA(launch_kernel(set_counters_kernel, dim3(1), dim3(1), 0, st, reinterpret_cast<int32_t*>(s->status),
                           (int)s->pos, (int)first_step, 0));
    ++g_kernel_launches;
    for (int j = 0; j < steps; ++j) SRM_CUDA(cudaGraphLaunch(m->step_exec, st));
    g_kernel_launches += (uint64_t)steps * m->step_launches;
    s->pos += steps;
    return SRM_OK;
  }
  for (int j = 0; j < steps; ++j) {
    int rc = decode_step_impl(m, s, nullptr, samp, first_step + j, nullptr, d_out, out_stride, j, nullptr, d_ws,
                              ws_bytes, st);
    if (rc) return rc;
  }
  return SRM_OK;
}

int srm_decode_step_host(srm_model* m, srm_state* s, const int32_t* h_tok_in, const srm_sampling* samp, int32_t step,
                         int32_t* h_tok_out, void* d_ws, size_t ws_bytes, void* stream) {
  if (m == nullptr || s == nullptr || h_tok_in == nullptr || h_tok_out == nullptr) return SRM_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the state's own last-token vector doubles as the device staging buffer
  SRM_CUDA(cudaMemcpyAsync(s->last_tok, h_tok_in, (size_t)s->B * 4, cudaMemcpyHostToDevice, st));
  int rc = decode_step_impl(m, s, nullptr, samp, step, nullptr, nullptr, 0, 0, nullptr, d_ws, ws_bytes, st);
  if (rc) return rc;
  SRM_CUDA(cudaMemcpyAsync(h_tok_out, s->last_tok, (size_t)s->B * 4, cudaMemcpyDeviceToHost, st));
  return SRM_OK;
}

// ---- decode step on the built-in scratch array --------------------------------------------------
}  // extern "C"

// Workspace for callers that cannot allocate: part of the module image, so it exists on every
// device that loads the library. In host code this name is only a handle for
// cudaGetSymbolAddress; kernels must be given the address that call returns.
static __device__ __align__(256) unsigned char g_static_scratch[SRM_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {};    // device address per device ordinal, looked up once
std::mutex g_static_scratch_mutex;

// Address of g_static_scratch on the current device (which must be `device`).
int static_scratch_address(int device, void** out) {
  int cur = -1;
  SRM_CUDA(cudaGetDevice(&cur));
  if (cur != device || cur < 0 || cur >= kMaxDevices) return SRM_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (g_static_scratch_addr[cur] == nullptr) {
    void* p = nullptr;
    SRM_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
    if (p == nullptr || !aligned(p, 256)) return SRM_ERR_ALIGNMENT;
    g_static_scratch_addr[cur] = p;
  }
  *out = g_static_scratch_addr[cur];
  return SRM_OK;
}
}  // namespace

extern "C" {

int srm_decode_step_static(srm_model* m, srm_state* s, const int32_t* d_tok_in, const srm_sampling* samp,
                           int32_t step, int32_t* d_tok_out, float* d_logits_out, void* stream) {
  if (m == nullptr || s == nullptr || s->m != m) return SRM_ERR_INVALID_ARG;
  if (decode_ws_bytes(*m, s->B) > (size_t)SRM_STATIC_SCRATCH_BYTES) return SRM_ERR_STATIC_SCRATCH;
  void* ws = nullptr;
  int rc = static_scratch_address(m->device, &ws);
  if (rc != SRM_OK) return rc;
  // Nothing in the workspace has to start at zero: the first mixer launch writes x and a, the up
  // projection writes H, the LM head writes the logits, each before anything reads them.
  return decode_step_impl(m, s, d_tok_in, samp, step, d_tok_out, nullptr, 0, 0, d_logits_out, ws,
                          (size_t)SRM_STATIC_SCRATCH_BYTES, static_cast<cudaStream_t>(stream));
}

// ---- single kernels ---------------------------------------------------------------------------
int srm_k_mixer_step(srm_model* m, int32_t layer, int32_t t, int64_t R, const int32_t* d_tok, float* d_x, void* d_S,
                     void* d_a, uint32_t* d_status, void* stream) {
  if (m == nullptr || R < 0) return SRM_ERR_INVALID_ARG;
  if (R == 0) return SRM_OK;
  if (d_x == nullptr || d_S == nullptr || d_a == nullptr) return SRM_ERR_INVALID_ARG;
  if (layer < 0 || layer >= m->cfg.n_layers || t < 0) return SRM_ERR_INVALID_ARG;
  if (t >= m->cfg.n_ctx) return SRM_ERR_CTX_OVERFLOW;
  if (!aligned(d_x, 16) || !aligned(d_S, 16) || !aligned(d_a, 16)) return SRM_ERR_ALIGNMENT;
  if (m->cfg.mixer != SRM_MIXER_MIXED)      // d_S: the planes [C][R, d] of these R rows
    return launch_mixer_variant(*m, layer, t, R, d_tok, 1, d_x, d_a, m->cfg.d_model, d_S, R * (int64_t)m->cfg.d_model, d_status,
                                static_cast<cudaStream_t>(stream));
  return launch_mixer(*m, layer, t, R, d_tok, d_x, d_S, d_a, d_status, static_cast<cudaStream_t>(stream));
}

namespace {
int device_sm_count(int* sms) {
  int dev = 0;
  SRM_CUDA(cudaGetDevice(&dev));
  SRM_CUDA(cudaDeviceGetAttribute(sms, cudaDevAttrMultiProcessorCount, dev));
  return SRM_OK;
}
}  // namespace

int srm_k_mixer_combined_step(int64_t R, int32_t d, int32_t n_heads, int32_t t, int32_t n_ctx, const float* d_z,
                              float* d_S_row, float* d_S_col, const float* d_alpha_row, const float* d_alpha_col,
                              const float* d_beta, const float* d_lam_row, const float* d_lam_col, const float* d_w,
                              float* d_y, void* stream) {
  if (R < 0 || d < 4 || n_heads < 1 || n_ctx < 1 || t < 0) return SRM_ERR_INVALID_ARG;
  if (t >= n_ctx) return SRM_ERR_CTX_OVERFLOW;
  if (d % n_heads || (d / n_heads) % 4) return SRM_ERR_UNSUPPORTED;
  if (R == 0) return SRM_OK;
  if (!d_z || !d_S_row || !d_S_col || !d_alpha_row || !d_alpha_col || !d_beta || !d_lam_row || !d_lam_col || !d_w || !d_y)
    return SRM_ERR_INVALID_ARG;
  if (!aligned(d_z, 16) || !aligned(d_S_row, 16) || !aligned(d_S_col, 16) || !aligned(d_beta, 16) || !aligned(d_y, 16))
    return SRM_ERR_ALIGNMENT;
  int sms = 0, rc = device_sm_count(&sms);
  if (rc != SRM_OK) return rc;
  CombinedParams p{R, d, n_heads, t, n_ctx, d_z, d_S_row, d_S_col, d_alpha_row, d_alpha_col, d_beta, d_lam_row, d_lam_col, d_w, d_y};
  // 8 blocks per SM, of which 5 are resident: measured 256 us per 65536 x 1024 against 273 us with exactly one
  // resident wave (each thread then walks more elements with three loads in flight)
  const int64_t blocks = (R * (d / 4) + kVariantThreads - 1) / kVariantThreads, cap = (int64_t)sms * 8;
  ++g_kernel_launches;
  SRM_CUDA(launch_kernel(combined_step_kernel, dim3((unsigned)(blocks < cap ? blocks : cap)), dim3(kVariantThreads), 0,
                         static_cast<cudaStream_t>(stream), p));
  return SRM_OK;
}

int srm_k_mixer_kernel_step(int64_t R, int32_t d, int32_t k, int32_t t, int32_t n_ctx, const float* d_z, float* d_P,
                            const float* d_alpha, const float* d_beta, const float* d_lam, float* d_y, void* stream) {
  if (R < 0 || d < 4 || k < 1 || n_ctx < 1 || t < 0) return SRM_ERR_INVALID_ARG;
  if (t >= n_ctx) return SRM_ERR_CTX_OVERFLOW;
  if (d % 4 || k > kKernelMixMaxK || k > d || kernel_mix_smem(d, k) > 200 * 1024) return SRM_ERR_UNSUPPORTED;
  if (R == 0) return SRM_OK;
  if (!d_z || !d_P || !d_alpha || !d_beta || !d_lam || !d_y) return SRM_ERR_INVALID_ARG;
  if (!aligned(d_z, 16) || !aligned(d_P, 16) || !aligned(d_y, 16)) return SRM_ERR_ALIGNMENT;
  int sms = 0, rc = device_sm_count(&sms);
  if (rc != SRM_OK) return rc;
  if ((rc = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel_mix_step_kernel), 200 * 1024)) != SRM_OK) return rc;
  KernelMixParams p{R, d, k, t, n_ctx, d_z, d_P, d_alpha, d_beta, d_lam, d_y};
  const size_t smem = kernel_mix_smem(d, k);
  // one wave of resident blocks: a second, partly filled wave would run at a fraction of the bandwidth
  int per_sm = 0;
  SRM_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel_mix_step_kernel, kVariantThreads, smem));
  const int64_t cap = (int64_t)sms * (per_sm < 1 ? 1 : per_sm);
  ++g_kernel_launches;
  SRM_CUDA(launch_kernel(kernel_mix_step_kernel, dim3((unsigned)(R < cap ? R : cap)), dim3(kVariantThreads), smem,
                         static_cast<cudaStream_t>(stream), p));
  return SRM_OK;
}

int srm_k_mixer_combined_scan(int64_t Bp, int32_t n, int32_t t0, int32_t d, int32_t n_heads, int32_t n_ctx, const float* d_Z,
                              float* d_S_row, float* d_S_col, const float* d_alpha_row, const float* d_alpha_col,
                              const float* d_beta, const float* d_lam_row, const float* d_lam_col, const float* d_w,
                              float* d_Y, void* stream) {
  if (Bp < 0 || n < 1 || d < 4 || n_heads < 1 || n_ctx < 1 || t0 < 0) return SRM_ERR_INVALID_ARG;
  if ((int64_t)t0 + n > n_ctx) return SRM_ERR_CTX_OVERFLOW;
  if (d % n_heads || (d / n_heads) % 4) return SRM_ERR_UNSUPPORTED;
  if (Bp == 0) return SRM_OK;
  if (!d_Z || !d_S_row || !d_S_col || !d_alpha_row || !d_alpha_col || !d_beta || !d_lam_row || !d_lam_col || !d_w || !d_Y)
    return SRM_ERR_INVALID_ARG;
  if (!aligned(d_Z, 16) || !aligned(d_S_row, 16) || !aligned(d_S_col, 16) || !aligned(d_beta, 16) || !aligned(d_Y, 16))
    return SRM_ERR_ALIGNMENT;
  int sms = 0, rc = device_sm_count(&sms);
  if (rc != SRM_OK) return rc;
  CombinedScanParams p{Bp, n, t0, d, n_heads, n_ctx, d_Z, d_S_row, d_S_col, d_alpha_row, d_alpha_col, d_beta, d_lam_row, d_lam_col, d_w, d_Y};
  const int64_t blocks = (Bp * (d / 4) + kVariantThreads - 1) / kVariantThreads, cap = (int64_t)sms * 8;
  ++g_kernel_launches;
  SRM_CUDA(launch_kernel(combined_scan_kernel, dim3((unsigned)(blocks < cap ? blocks : cap)), dim3(kVariantThreads), 0,
                         static_cast<cudaStream_t>(stream), p));
  return SRM_OK;
}

int srm_k_mixer_kernel_scan(int64_t Bp, int32_t n, int32_t t0, int32_t d, int32_t k, int32_t n_ctx, const float* d_Z, float* d_P,
                            const float* d_alpha, const float* d_beta, const float* d_lam, float* d_Y, void* stream) {
  if (Bp < 0 || n < 1 || d < 4 || k < 1 || n_ctx < 1 || t0 < 0) return SRM_ERR_INVALID_ARG;
  if ((int64_t)t0 + n > n_ctx) return SRM_ERR_CTX_OVERFLOW;
  if (d % 4 || k > kKernelMixMaxK || k > d || kernel_scan_smem(d, k) > 200 * 1024) return SRM_ERR_UNSUPPORTED;
  if (Bp == 0) return SRM_OK;
  if (!d_Z || !d_P || !d_alpha || !d_beta || !d_lam || !d_Y) return SRM_ERR_INVALID_ARG;
  if (!aligned(d_Z, 16) || !aligned(d_P, 16) || !aligned(d_Y, 16) || !aligned(d_beta, 16)) return SRM_ERR_ALIGNMENT;
  int sms = 0, rc = device_sm_count(&sms);
  if (rc != SRM_OK) return rc;
  if ((rc = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel_scan_kernel), 200 * 1024)) != SRM_OK) return rc;
  KernelScanParams p{Bp, n, t0, d, k, n_ctx, d_Z, d_P, d_alpha, d_beta, d_lam, d_Y};
  const size_t smem = kernel_scan_smem(d, k);
  int per_sm = 0;
  SRM_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel_scan_kernel, kVariantThreads, smem));
  const int64_t cap = (int64_t)sms * (per_sm < 1 ? 1 : per_sm);
  ++g_kernel_launches;
  SRM_CUDA(launch_kernel(kernel_scan_kernel, dim3((unsigned)(Bp < cap ? Bp : cap)), dim3(kVariantThreads), smem,
                         static_cast<cudaStream_t>(stream), p));
  return SRM_OK;
}

int srm_k_final_norm(srm_model* m, int64_t R, const float* d_x, void* d_a, void* stream) {
  if (m == nullptr || R < 0) return SRM_ERR_INVALID_ARG;
  if (R == 0) return SRM_OK;
  if (d_x == nullptr || d_a == nullptr) return SRM_ERR_INVALID_ARG;
  if (!aligned(d_x, 16) || !aligned(d_a, 16)) return SRM_ERR_ALIGNMENT;
  return launch_final_norm(*m, d_x, R, 1, 0, d_a, static_cast<cudaStream_t>(stream));
}

int srm_k_gemm(srm_model* m, int32_t epilogue, int64_t M, int64_t N, int64_t K, const void* d_A, const void* d_W,
               const float* d_bias, void* d_out, uint32_t* d_status, void* stream) {
  if (m == nullptr || M < 0 || N < 1 || K < 1) return SRM_ERR_INVALID_ARG;
  if (M == 0) return SRM_OK;
  if (d_A == nullptr || d_W == nullptr || d_out == nullptr) return SRM_ERR_INVALID_ARG;
  if (epilogue < 0 || epilogue > 2 || (epilogue == kEpiBiasGelu && d_bias == nullptr)) return SRM_ERR_INVALID_ARG;
  if (K % 64 || N % 8) return SRM_ERR_UNSUPPORTED;
  if (!aligned(d_A, 16) || !aligned(d_W, 16) || !aligned(d_out, 16) || !aligned(d_bias, 16)) return SRM_ERR_ALIGNMENT;
  return launch_gemm(*m, epilogue, M, N, K, d_A, d_W, d_bias, d_out, d_status, static_cast<cudaStream_t>(stream));
}

size_t srm_k_gemm_splitk_order_bytes(int64_t M, int64_t N) {
  if (M < 1 || N < 1) return 0;
  return splitk_order_bytes(M, N);
}

int srm_k_gemm_splitk(srm_model* m, int64_t M, int64_t N, int64_t K, const void* d_A, const void* d_W,
                      const float* d_bias, float* d_out, void* d_order, size_t order_bytes, uint32_t* d_status,
                      void* stream) {
  if (m == nullptr || M < 0 || N < 1 || K < 1) return SRM_ERR_INVALID_ARG;
  if (M == 0) return SRM_OK;
  if (d_A == nullptr || d_W == nullptr || d_out == nullptr || d_order == nullptr) return SRM_ERR_INVALID_ARG;
  if (m->cfg.dtype != SRM_DTYPE_BF16 || (m->cfg.flags & SRM_FLAG_SIMT_GEMM) || K % 64 || N % 8) return SRM_ERR_UNSUPPORTED;
  if (!aligned(d_A, 16) || !aligned(d_W, 16) || !aligned(d_out, 16) || !aligned(d_bias, 16) || !aligned(d_order, 256)) return SRM_ERR_ALIGNMENT;
  const size_t need = splitk_order_bytes(M, N);
  if (order_bytes < need) return SRM_ERR_BUFFER_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = ensure_tc_ready(*m);
  if (rc != SRM_OK) return rc;
  tc::SplitPlan P;
  if (!tc::split_plan(((M + tc::BM - 1) / tc::BM) * ((N + tc::BN - 1) / tc::BN), (int)(K / 64), m->tc_clusters, &P)) return SRM_ERR_UNSUPPORTED;
  SRM_CUDA(cudaMemsetAsync(d_order, 0, need, st));
  return launch_gemm_splitk(*m, M, N, K, d_A, d_W, d_bias, d_out, static_cast<int32_t*>(d_order), d_status, st);
}

int64_t srm_k_gemm_splitk_plan(int64_t M, int64_t N, int64_t K, int32_t pairs, int32_t pair, int64_t* pieces, int64_t max_pieces) {
  if (M < 1 || N < 1 || K < 64 || K % 64 || pairs < 1 || pair < 0 || pair >= pairs || max_pieces < 0) return SRM_ERR_INVALID_ARG;
  if (max_pieces > 0 && pieces == nullptr) return SRM_ERR_INVALID_ARG;
  tc::SplitPlan P;
  const int64_t m_tiles = (M + tc::BM - 1) / tc::BM;
  if (!tc::split_plan(m_tiles * ((N + tc::BN - 1) / tc::BN), (int)(K / 64), pairs, &P)) return SRM_ERR_UNSUPPORTED;
  tc::SplitCursor cur;
  cur.init(P, pair);
  tc::SplitPiece pc;
  int64_t n = 0;
  while (cur.next(P, &pc)) {
    if (n < max_pieces) {
      int64_t* o = pieces + 4 * n;
      o[0] = pc.tile % m_tiles; o[1] = pc.tile / m_tiles; o[2] = pc.kb0; o[3] = pc.kb1;
    }
    ++n;
  }
  return n;
}

int srm_k_lm_head_greedy(srm_model* m, int64_t R, const void* d_a, void* d_part, size_t part_bytes, int32_t* d_tok,
                         uint32_t* d_status, void* stream) {
  if (m == nullptr || R < 0) return SRM_ERR_INVALID_ARG;
  if (R == 0) return SRM_OK;
  if (d_a == nullptr || d_part == nullptr || d_tok == nullptr) return SRM_ERR_INVALID_ARG;
  if (m->cfg.dtype != SRM_DTYPE_BF16) return SRM_ERR_UNSUPPORTED;
  if (!aligned(d_a, 16) || !aligned(d_part, 16)) return SRM_ERR_ALIGNMENT;
  if (part_bytes < (size_t)tc::argmax_slots(m->cfg.vocab) * (size_t)R * 8) return SRM_ERR_BUFFER_TOO_SMALL;
  SelectOut o{d_tok, nullptr, nullptr, 0, 0, 1};
  return launch_lm_head_greedy(*m, R, d_a, d_part, o, d_status, static_cast<cudaStream_t>(stream));
}

int srm_k_select(srm_model* m, int64_t R, const float* d_logits, const srm_sampling* samp, int32_t step,
                 int32_t* d_tok, uint32_t* d_status, void* stream) {
  if (m == nullptr || R < 0) return SRM_ERR_INVALID_ARG;
  if (R == 0) return SRM_OK;
  if (d_logits == nullptr || d_tok == nullptr) return SRM_ERR_INVALID_ARG;
  int rc = check_sampling(*m, samp);
  if (rc) return rc;
  if (!aligned(d_logits, 16)) return SRM_ERR_ALIGNMENT;
  SelectOut o{d_tok, nullptr, nullptr, 0, 0, 1};
  return launch_select(*m, R, d_logits, *samp, samp->sample_idx_base, step, o, d_status, static_cast<cudaStream_t>(stream));
}

int srm_k_prefill_mixer(srm_model* m, int32_t layer, int64_t Bp, int32_t n, const int32_t* d_tok, float* d_x, void* d_S,
                        void* d_a, uint32_t* d_status, void* stream) {
  if (m == nullptr || Bp < 0 || n < 1) return SRM_ERR_INVALID_ARG;
  if (Bp == 0) return SRM_OK;
  if (d_x == nullptr || d_S == nullptr || d_a == nullptr) return SRM_ERR_INVALID_ARG;
  if (layer < 0 || layer >= m->cfg.n_layers) return SRM_ERR_INVALID_ARG;
  if (n > m->cfg.n_ctx) return SRM_ERR_CTX_OVERFLOW;
  if (!aligned(d_x, 16) || !aligned(d_S, 16) || !aligned(d_a, 16)) return SRM_ERR_ALIGNMENT;
  if (m->cfg.mixer != SRM_MIXER_MIXED) return SRM_ERR_UNSUPPORTED;
  return launch_prefill_mixer(*m, layer, Bp, n, d_tok, d_x, d_S, d_a, d_status, static_cast<cudaStream_t>(stream));
}

const char* srm_strerror(int code) {
  switch (code) {
    case SRM_OK: return "ok";
    case SRM_ERR_INVALID_ARG: return "invalid argument";
    case SRM_ERR_UNSUPPORTED: return "unsupported shape or configuration";
    case SRM_ERR_ALIGNMENT: return "misaligned device pointer";
    case SRM_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case SRM_ERR_CTX_OVERFLOW: return "position would exceed n_ctx";
    case SRM_ERR_CUDA: return "CUDA call failed (see srm_last_cuda_error)";
    case SRM_ERR_DEVICE_STATUS: return "device status flags set";
    case SRM_ERR_STATIC_SCRATCH: return "batch needs more scratch than the library's built-in array holds";
    default: return "unknown error";
  }
}

int srm_last_cuda_error(void) { return g_last_cuda_error; }

const char* srm_version(void) { return "srm-b200 0.1 (sm_100a)"; }

}  // extern "C"

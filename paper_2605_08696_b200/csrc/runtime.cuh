// Host runtime of the SRM decode library, part 1: error handling, the weight-blob layout, TMA descriptors, the model
// and state handles, the launch counter / CUDA-event profiler, and the carving of the caller's workspace.
// Included by srm_api.cu only (one translation unit).
#pragma once
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
#include "ffn_fused.cuh"
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
  std::vector<std::pair<int, tc::FfnPlan>> ffn_plans;   // work lists of the fused feed-forward kernel, by row blocks
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

// Partial-product planes of a small pass's down projection (GemmArgs::k_slices): up to 8 planes of the pass's rows
// (padded to whole 256-row tiles) x d floats, never more than one 256 x 256 fp32 tile per CTA pair of the largest
// device (tiles x ranges stays within the pairs). Only for the models whose mixer adds them (mixer_stream_kernel).
constexpr int kMaxKSlices = 8;
bool kslice_model(const srm_config& c) {
  const int d = c.d_model, nv = d / 128, se = c.state_dtype == SRM_DTYPE_FP32 ? 4 : 2;
  return c.dtype == SRM_DTYPE_BF16 && !(c.flags & (SRM_FLAG_SIMT_GEMM | SRM_FLAG_NO_KSLICE | SRM_FLAG_HEAD_PROJ)) &&
         c.mixer == SRM_MIXER_MIXED && d % 128 == 0 && (d / c.n_heads) % 128 == 0 && c.n_heads <= 8 &&
         (nv == 4 || nv == 8 || nv == 12 || nv == 16) && mixer_stream_warps(d, se) >= 1 && ((size_t)c.ffn_mult * d) % 64 == 0;
}
size_t kslice_bytes(const srm_config& c, int64_t rows) {
  if (!kslice_model(c)) return 0;
  const size_t rows_pad = (size_t)(rows + tc::BM - 1) / tc::BM * tc::BM;
  const size_t want = (size_t)kMaxKSlices * rows_pad * c.d_model * 4, cap = (size_t)96 * tc::BM * tc::BN * 4;
  return align_up(want < cap ? want : cap, 256);
}

struct DecodeWs {
  float* x; void* a; void* H; float* logits;
  float* part;            // kslice_bytes
  size_t part_bytes;
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
         (splitk_enabled(m.cfg) ? splitk_order_bytes(rows, m.cfg.d_model) : 0) + small_scratch_bytes(m.cfg) +
         kslice_bytes(m.cfg, rows);
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
  w.small = p; p += small_scratch_bytes(m.cfg);
  w.part_bytes = kslice_bytes(m.cfg, rows);
  w.part = w.part_bytes ? reinterpret_cast<float*>(p) : nullptr;
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

}  // namespace

// Host runtime of the SRM decode library, part 2: one launcher per kernel, the decode step of a pass of rows, the
// choice of the pass size and the decode step of a whole batch. Everything here is argument set-up and launches;
// all arithmetic of the path runs in the kernels. Included by srm_api.cu only (one translation unit).
#pragma once

#include "runtime.cuh"

namespace {

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

// ps: partial products of the previous layer's down projection still to be added into x (mixer_stream_kernel only).
int launch_mixer(const srm_model& m, int layer, int t, int64_t R, const int32_t* tok, float* x, void* S, void* a,
                 uint32_t* status, cudaStream_t st, const int32_t* ctr = nullptr, const int32_t* pos = nullptr,
                 const PartialSum& ps = PartialSum()) {
  if (R <= 0) return SRM_OK;
  LaunchScope scope(m, SRM_KERNEL_MIXER, st);
  MixerParams p;
  p.part = ps.part; p.n_part = ps.n_part; p.part_plane = ps.plane; p.part_bias = ps.bias;
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
                  int d, void* out, cudaStream_t st, const int32_t* row_len = nullptr, const PartialSum& ps = PartialSum()) {
  const int nv = (d + 127) / 128;
  const unsigned grid = (unsigned)((R + kMixerWarps - 1) / kMixerWarps);
  const dim3 blk(kMixerWarps * 32);
  WT* o = reinterpret_cast<WT*>(out);
  if (nv <= 1) SRM_CUDA(launch_kernel(norm_rows_kernel<1, WT>, dim3(grid), dim3(blk), 0, st, x, R, stride, offset, g, b, eps, d, o, row_len, ps));
  else if (nv <= 2) SRM_CUDA(launch_kernel(norm_rows_kernel<2, WT>, dim3(grid), dim3(blk), 0, st, x, R, stride, offset, g, b, eps, d, o, row_len, ps));
  else if (nv <= 4) SRM_CUDA(launch_kernel(norm_rows_kernel<4, WT>, dim3(grid), dim3(blk), 0, st, x, R, stride, offset, g, b, eps, d, o, row_len, ps));
  else if (nv <= 6) SRM_CUDA(launch_kernel(norm_rows_kernel<6, WT>, dim3(grid), dim3(blk), 0, st, x, R, stride, offset, g, b, eps, d, o, row_len, ps));
  else if (nv <= 8) SRM_CUDA(launch_kernel(norm_rows_kernel<8, WT>, dim3(grid), dim3(blk), 0, st, x, R, stride, offset, g, b, eps, d, o, row_len, ps));
  else if (nv <= 12) SRM_CUDA(launch_kernel(norm_rows_kernel<12, WT>, dim3(grid), dim3(blk), 0, st, x, R, stride, offset, g, b, eps, d, o, row_len, ps));
  else SRM_CUDA(launch_kernel(norm_rows_kernel<16, WT>, dim3(grid), dim3(blk), 0, st, x, R, stride, offset, g, b, eps, d, o, row_len, ps));
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
                      cudaStream_t st, const int32_t* row_len = nullptr, const PartialSum& ps = PartialSum()) {
  if (R <= 0) return SRM_OK;
  LaunchScope scope(m, SRM_KERNEL_NORM, st);
  const float* g = m.fptr(-1, SRM_T_LNF_G);
  const float* b = m.fptr(-1, SRM_T_LNF_B);
  if (m.cfg.dtype == SRM_DTYPE_BF16) return launch_norm_t<bf16>(x, R, stride, offset, g, b, m.cfg.ln_eps, m.cfg.d_model, out, st, row_len, ps);
  return launch_norm_t<float>(x, R, stride, offset, g, b, m.cfg.ln_eps, m.cfg.d_model, out, st, row_len, ps);
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
  SRM_CUDA(cudaFuncSetAttribute(tc::ffn_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes));
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

// k_slices > 1 (epilogue kEpiPlain only; K / 64 a multiple of k_slices): out is k_slices planes of plane_rows x N
// partial products (GemmArgs::k_slices).
int launch_gemm_tc(srm_model& m, int epi, int64_t M, int64_t N, int64_t K, const void* A, const void* W,
                   const float* bias, void* out, uint32_t* status, cudaStream_t st, int k_slices = 1, int64_t plane_rows = 0) {
  int rc = ensure_tc_ready(m);
  if (rc != SRM_OK) return rc;
  CUtensorMap ta, tb, td, tb64;
  if ((rc = m.tmap(A, M, K, tc::kRowsPerCta, 2, &ta)) != SRM_OK) return rc;
  if ((rc = m.tmap(W, N, K, tc::kRowsPerCta, 2, &tb)) != SRM_OK) return rc;
  if ((rc = m.tmap(W, N, K, tc::kHalfN / 2, 2, &tb64)) != SRM_OK) return rc;      // W rows of a half-width piece
  if (epi == kEpiArgmax) td = ta;       // no output matrix: the descriptor is not used
  else if ((rc = m.tmap(out, k_slices > 1 ? k_slices * plane_rows : M, N, tc::kOutBoxRows, epi == kEpiBiasGelu ? 2 : 4, &td)) != SRM_OK) return rc;
  const uint8_t* wb = static_cast<const uint8_t*>(W);
  const int w_static = wb >= m.w && wb < m.w + m.layout.total;      // inside the weight blob
  const int64_t tiles = ((M + tc::BM - 1) / tc::BM) * ((N + tc::BN - 1) / tc::BN);
  const int tail = k_slices > 1 ? 0 : gemm_tail_tiles(m, tiles);
  tc::GemmArgs g{M, N, K, bias, out, status, w_static};
  g.tail_tiles = tail;
  g.k_slices = k_slices > 1 ? k_slices : 1;
  g.plane_rows = plane_rows;
  const int64_t pieces = (tiles + tail) * g.k_slices;
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

// ---- the feed-forward block as one kernel (ffn_fused.cuh) --------------------------------------
tc::FfnShape ffn_shape(int64_t M, int d, int64_t F) {
  return tc::FfnShape{(int)((M + tc::BM - 1) / tc::BM), (int)(F / tc::BN), d / tc::BK, d / tc::BN, (int)(F / tc::BK)};
}
size_t ffn_ready_bytes(int64_t M, int64_t F) { return align_up((size_t)((M + tc::BM - 1) / tc::BM) * (size_t)(F / tc::BN) * 4, 256); }

// Whether M rows of this model can take the fused kernel (shape limits of the plan and of whole 256-wide tiles).
bool ffn_fused_shape_ok(const srm_model& m, int64_t M) {
  const srm_config& c = m.cfg;
  if (c.dtype != SRM_DTYPE_BF16 || (c.flags & SRM_FLAG_SIMT_GEMM)) return false;
  const int64_t F = m.F();
  if (c.d_model % tc::BN || F % tc::BN || M < 1 || M > (int64_t)tc::kFfnMaxRb * tc::BM) return false;
  return tc::ffn_shape_ok(ffn_shape(M, c.d_model, F), 2);
}

// Whether the decode step takes it for a pass of M rows: from two tiles per CTA pair. With fewer the chain up tile ->
// epilogue -> counter -> down tile is longer than two launches that overlap through programmatic dependent launch,
// and the down projection of such a pass runs over ranges of K instead (down_k_slices). Measured on the mid model
// (74 pairs, 20 tiles per 256 rows), ms per step, one kernel / two launches / two launches with ranges of K: 512 rows
// 0.73 / 0.64 / 0.50, 1024: 0.76 / 0.71 / 0.59, 1536: 0.80 / 0.81 / 0.75, 2048: 0.89 / 0.93 / 0.92, 2304: 0.94 / 0.99 /
// 0.99, 3072: 1.14 / 1.24 / -, 4096: 1.47 / 1.51 / -.
bool ffn_fused_worthwhile(const srm_model& m, int64_t M) {
  const tc::FfnShape s = ffn_shape(M, m.cfg.d_model, m.F());
  return m.tc_clusters >= 2 && (int64_t)s.Rb * (s.Cu + s.Cd) >= 2 * (int64_t)m.tc_clusters;
}

// `ready`: ffn_ready_bytes(M, F) bytes of zeroed words. SRM_ERR_UNSUPPORTED: take the two launches.
int launch_ffn_fused(srm_model& m, int layer, int64_t M, const void* a, void* H, float* x, int32_t* ready, uint32_t* status,
                     cudaStream_t st) {
  if (M <= 0) return SRM_OK;
  if (!ffn_fused_shape_ok(m, M)) return SRM_ERR_UNSUPPORTED;
  int rc = ensure_tc_ready(m);
  if (rc != SRM_OK) return rc;
  const int d = m.cfg.d_model;
  const int64_t F = m.F();
  const tc::FfnShape shape = ffn_shape(M, d, F);
  if (m.tc_clusters < 2 || !tc::ffn_shape_ok(shape, m.tc_clusters)) return SRM_ERR_UNSUPPORTED;
  const tc::FfnPlan* plan = nullptr;
  for (const auto& e : m.ffn_plans)
    if (e.first == shape.Rb) plan = &e.second;
  if (plan == nullptr) {
    m.ffn_plans.emplace_back(shape.Rb, tc::FfnPlan{});
    if (!tc::ffn_make_plan(shape, m.tc_clusters, &m.ffn_plans.back().second)) { m.ffn_plans.pop_back(); return SRM_ERR_UNSUPPORTED; }
    plan = &m.ffn_plans.back().second;
  }
  LaunchScope scope(m, SRM_KERNEL_FFN, st);
  CUtensorMap ta, tw1, tw1h, ths, th, tw2, tx;
  const void* W1 = m.ptr(layer, SRM_T_W1);
  const void* W2 = m.ptr(layer, SRM_T_W2);
  if ((rc = m.tmap(a, M, d, tc::kRowsPerCta, 2, &ta)) != SRM_OK) return rc;
  if ((rc = m.tmap(W1, F, d, tc::kRowsPerCta, 2, &tw1)) != SRM_OK) return rc;
  if ((rc = m.tmap(W1, F, d, tc::kHalfN / 2, 2, &tw1h)) != SRM_OK) return rc;        // W1 rows of a half-width piece
  if ((rc = m.tmap(H, M, F, tc::kOutBoxRows, 2, &ths)) != SRM_OK) return rc;
  if ((rc = m.tmap(H, M, F, tc::kRowsPerCta, 2, &th)) != SRM_OK) return rc;
  if ((rc = m.tmap(W2, d, F, tc::kRowsPerCta, 2, &tw2)) != SRM_OK) return rc;
  if ((rc = m.tmap(x, M, d, tc::kOutBoxRows, 4, &tx)) != SRM_OK) return rc;
  tc::FfnArgs g{M, d, (int)F, m.fptr(layer, SRM_T_B1), m.fptr(layer, SRM_T_B2), status, ready, 1};
  SRM_CUDA(launch_kernel(tc::ffn_fused_kernel, dim3(2u * (unsigned)m.tc_clusters), dim3(tc::kThreads), tc::kSmemBytes, st,
                         ta, tw1, tw1h, ths, th, tw2, tx, g, *plan));
  SRM_CUDA(cudaGetLastError());
  return SRM_OK;
}

// Ranges the K dimension of a small down projection is cut into (GemmArgs::k_slices): the largest power of two up
// to kMaxKSlices that divides the k-blocks, leaves at least four k-blocks per range and keeps tiles x ranges within the CTA
// pairs; 1 (no cut) when the tiles alone fill half the pairs. Depends on the tile count, so rows of passes of very
// different sizes see sums in another order (last bits); equal-sized passes and all smaller ones agree bit for bit.
int down_k_slices(int64_t tiles, int k_blocks, int pairs) {
  if (tiles < 1 || 2 * tiles > pairs) return 1;
  int ks = 1;
  while (ks < kMaxKSlices && k_blocks % (2 * ks) == 0 && k_blocks / (2 * ks) >= 4 && tiles * 2 * ks <= pairs) ks *= 2;
  return ks;
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
  // the feed-forward block as one kernel: its per-layer counters sit in the logits area, which nothing uses before
  // the LM head
  const size_t ready_layer = ffn_ready_bytes(R, F);
  bool fused_ffn = !(c.flags & SRM_FLAG_NO_FUSED_FFN) && ffn_fused_shape_ok(m, R) &&
                   ready_layer * c.n_layers <= align_up((size_t)w.rows * c.vocab * 4, 256);
  if (fused_ffn) {
    if ((rc = ensure_tc_ready(m))) return rc;
    fused_ffn = ffn_fused_worthwhile(m, R);
  }
  if (fused_ffn) SRM_CUDA(cudaMemsetAsync(w.logits, 0, ready_layer * c.n_layers, st));
  else if (split) SRM_CUDA(cudaMemsetAsync(w.order, 0, w.order_bytes, st));
  // A small pass (the down projection has less than half as many tiles as there are CTA pairs): its K dimension is
  // cut into ranges so that all pairs work on it; the partial products go to planes of their own in the workspace
  // and the next consumer of x (the next layer's mixer, the final norm) adds them in a fixed order.
  PartialSum ps_none, ps;
  int k_slices = 1;
  const int64_t plane_rows = (R + tc::BM - 1) / tc::BM * tc::BM;
  if (!fused_ffn && !split && w.part != nullptr) {
    if ((rc = ensure_tc_ready(m))) return rc;
    k_slices = down_k_slices(plane_rows / tc::BM * ((d + tc::BN - 1) / tc::BN), (int)(F / tc::BK), m.tc_clusters);
    while (k_slices > 1 && (size_t)k_slices * plane_rows * d * 4 > w.part_bytes) k_slices /= 2;
  }
  if (k_slices > 1) ps = PartialSum{w.part, k_slices, plane_rows * (int64_t)d, nullptr};
  for (int l = 0; l < c.n_layers; ++l) {
    uint8_t* Sl = static_cast<uint8_t*>(s.layer_ptr(l)) + (size_t)b0 * d * m.state_bytes();
    if (c.mixer != SRM_MIXER_MIXED) {
      if ((rc = launch_mixer_variant(m, l, t, R, l == 0 ? tok_in + b0 : nullptr, 1, w.x, w.a, d, Sl, s.plane_elems(), s.status,
                                     st, ctr))) return rc;
    } else if (m.head_proj()) {
      if ((rc = launch_mixer_block_proj(m, l, t, R, R, 1, l == 0 ? tok_in + b0 : nullptr, w.x, Sl, w.a, w.q, s.status, st, ctr, pos))) return rc;
    } else {
      PartialSum pl = l > 0 ? ps : ps_none;                // what layer l - 1's down projection left in planes
      if (l > 0) pl.bias = m.fptr(l - 1, SRM_T_B2);
      if ((rc = launch_mixer(m, l, t, R, l == 0 ? tok_in + b0 : nullptr, w.x, Sl, w.a, s.status, st, ctr, pos, pl))) return rc;
    }
    if (fused_ffn) {
      int32_t* ready = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(w.logits) + (size_t)l * ready_layer);
      rc = launch_ffn_fused(m, l, R, w.a, w.H, w.x, ready, s.status, st);
      if (rc == SRM_OK) continue;
      if (rc != SRM_ERR_UNSUPPORTED) return rc;
      fused_ffn = false;                                   // (no plan for this shape: decided at the first layer)
      if (split) SRM_CUDA(cudaMemsetAsync(w.order, 0, w.order_bytes, st));
    }
    if ((rc = launch_gemm(m, kEpiBiasGelu, R, F, d, w.a, m.ptr(l, SRM_T_W1), m.fptr(l, SRM_T_B1), w.H, s.status, st))) return rc;
    rc = split ? launch_gemm_splitk(m, R, d, F, w.H, m.ptr(l, SRM_T_W2), m.fptr(l, SRM_T_B2), w.x, w.order, s.status, st, true)
               : SRM_ERR_UNSUPPORTED;
    if (rc == SRM_ERR_UNSUPPORTED) {
      if (k_slices > 1) {
        LaunchScope scope(m, SRM_KERNEL_GEMM_DOWN, st);
        rc = launch_gemm_tc(m, kEpiPlain, R, d, F, w.H, m.ptr(l, SRM_T_W2), nullptr, w.part, s.status, st, k_slices, plane_rows);
      } else {
        rc = launch_gemm(m, kEpiBiasResidual, R, d, F, w.H, m.ptr(l, SRM_T_W2), m.fptr(l, SRM_T_B2), w.x, s.status, st);
      }
    }
    if (rc) return rc;
  }
  if (k_slices > 1) ps.bias = m.fptr(c.n_layers - 1, SRM_T_B2);
  if ((rc = launch_final_norm(m, w.x, R, 1, 0, w.a, st, nullptr, k_slices > 1 ? ps : ps_none))) return rc;
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

// C ABI of the SRM decode library (see include/srm.h for the contract): argument checking and the calls into the
// host runtime (runtime.cuh: layout, handles, workspace; launchers.cuh: kernel launches and the decode step).
#include "launchers.cuh"

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

size_t srm_prefill_workspace_bytes(const srm_config* cfg, int64_t samples, int32_t n) {
  if (!config_ok(cfg) || samples < 1 || n < 1) return 0;
  srm_model tmp;
  tmp.cfg = *cfg;
  return prefill_ws_bytes(tmp, samples, n);
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
// Rows per feed-forward kernel of a prefill pass (mid, 4096 prompts x 256 tokens: 4096 / 8192 / 16384 rows per slab take
// 0.327 / 0.310 / 0.303 s; 16384 is the most one plan holds).
constexpr int64_t kPrefillFfnRows = 16384;

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
      // The feed-forward block over the rows of the pass: in slabs of kPrefillFfnRows rows, each as ONE kernel
      // (ffn_fused.cuh: a slab's hidden activations are consumed from L2 as they are
      // produced instead of crossing HBM twice), where the model's shape allows and the slab counters fit in the
      // logits area (free until the LM head); else, and for a short last slab, up projection then down projection.
      const size_t slab_ready = ffn_ready_bytes(kPrefillFfnRows, F);
      const int64_t n_slabs = (rows + kPrefillFfnRows - 1) / kPrefillFfnRows;
      bool slabs = !(c.flags & SRM_FLAG_NO_FUSED_FFN) && rows >= kPrefillFfnRows && ffn_fused_shape_ok(*m, kPrefillFfnRows) &&
                   (size_t)n_slabs * slab_ready <= align_up((size_t)np * c.vocab * 4, 256);
      if (slabs) {
        if ((rc = ensure_tc_ready(*m))) return rc;
        slabs = ffn_fused_worthwhile(*m, kPrefillFfnRows);
      }
      if (slabs) SRM_CUDA(cudaMemsetAsync(w.logits, 0, (size_t)n_slabs * slab_ready, st));
      for (int64_t r0 = 0; slabs && r0 < rows; r0 += kPrefillFfnRows) {
        const int64_t nr = rows - r0 < kPrefillFfnRows ? rows - r0 : kPrefillFfnRows;
        uint8_t* a_s = static_cast<uint8_t*>(w.a) + (size_t)r0 * d * m->act_bytes();
        uint8_t* H_s = static_cast<uint8_t*>(w.H) + (size_t)r0 * F * m->act_bytes();
        float* x_s = w.x + (size_t)r0 * d;
        int32_t* ready = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(w.logits) + (size_t)(r0 / kPrefillFfnRows) * slab_ready);
        rc = ffn_fused_worthwhile(*m, nr) ? launch_ffn_fused(*m, l, nr, a_s, H_s, x_s, ready, s->status, st) : SRM_ERR_UNSUPPORTED;
        if (rc == SRM_ERR_UNSUPPORTED) {
          if ((rc = launch_gemm(*m, kEpiBiasGelu, nr, F, d, a_s, m->ptr(l, SRM_T_W1), m->fptr(l, SRM_T_B1), H_s, s->status, st))) return rc;
          rc = launch_gemm(*m, kEpiBiasResidual, nr, d, F, H_s, m->ptr(l, SRM_T_W2), m->fptr(l, SRM_T_B2), x_s, s->status, st);
        }
        if (rc) return rc;
      }
      if (!slabs) {
        if ((rc = launch_gemm(*m, kEpiBiasGelu, rows, F, d, w.a, m->ptr(l, SRM_T_W1), m->fptr(l, SRM_T_B1), w.H, s->status, st))) return rc;
        if ((rc = launch_gemm(*m, kEpiBiasResidual, rows, d, F, w.H, m->ptr(l, SRM_T_W2), m->fptr(l, SRM_T_B2), w.x, s->status, st))) return rc;
      }
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
  // The caller has nothing to clear: the first mixer launch writes x and a, the up projection writes H, the LM head
  // writes the logits, each before anything reads them, and the few words that must start at zero (order words of a
  // split down projection, candidate counters of the fused top-k selection, the grid-barrier word of the small-batch
  // kernel) are cleared by the step itself with memsets on the stream.
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

size_t srm_k_ffn_ready_bytes(int64_t M, int64_t F) {
  if (M < 1 || F < tc::BN) return 0;
  return ffn_ready_bytes(M, F);
}

int srm_k_ffn(srm_model* m, int32_t layer, int64_t M, const void* d_a, void* d_H, float* d_x, void* d_ready,
              size_t ready_bytes, uint32_t* d_status, void* stream) {
  if (m == nullptr || M < 0 || layer < 0 || layer >= m->cfg.n_layers) return SRM_ERR_INVALID_ARG;
  if (M == 0) return SRM_OK;
  if (d_a == nullptr || d_H == nullptr || d_x == nullptr || d_ready == nullptr) return SRM_ERR_INVALID_ARG;
  if (!ffn_fused_shape_ok(*m, M)) return SRM_ERR_UNSUPPORTED;
  if (!aligned(d_a, 16) || !aligned(d_H, 16) || !aligned(d_x, 16) || !aligned(d_ready, 256)) return SRM_ERR_ALIGNMENT;
  const size_t need = ffn_ready_bytes(M, m->F());
  if (ready_bytes < need) return SRM_ERR_BUFFER_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  SRM_CUDA(cudaMemsetAsync(d_ready, 0, need, st));
  return launch_ffn_fused(*m, layer, M, d_a, d_H, d_x, static_cast<int32_t*>(d_ready), d_status, st);
}

int64_t srm_k_ffn_plan(int64_t M, int32_t d, int32_t F, int32_t pairs, int32_t* off, int32_t* items, int64_t max_items,
                       double* makespan, double* ideal) {
  if (M < 1 || d < tc::BN || F < tc::BN || pairs < 1 || max_items < 0 || off == nullptr) return SRM_ERR_INVALID_ARG;
  if (max_items > 0 && items == nullptr) return SRM_ERR_INVALID_ARG;
  if (d % tc::BN || F % tc::BN || M > (int64_t)tc::kFfnMaxRb * tc::BM) return SRM_ERR_UNSUPPORTED;
  const tc::FfnShape shape = ffn_shape(M, d, F);
  if (!tc::ffn_shape_ok(shape, pairs)) return SRM_ERR_UNSUPPORTED;
  tc::FfnPlan* plan = new (std::nothrow) tc::FfnPlan();
  if (plan == nullptr) return SRM_ERR_INVALID_ARG;
  if (!tc::ffn_make_plan(shape, pairs, plan)) { delete plan; return SRM_ERR_UNSUPPORTED; }
  for (int p = 0; p <= pairs; ++p) off[p] = plan->off[p];
  const int64_t n = plan->off[pairs];
  for (int64_t i = 0; i < n && i < max_items; ++i) {
    const uint16_t it = plan->item[i];
    items[3 * i] = tc::ffn_item_down(it) ? 1 : tc::ffn_item_half(it) ? (tc::ffn_item_noff(it) ? 3 : 2) : 0;
    items[3 * i + 1] = tc::ffn_item_rb(it);
    items[3 * i + 2] = tc::ffn_item_cb(it);
  }
  if (makespan != nullptr) *makespan = tc::ffn_simulate(shape, *plan);
  if (ideal != nullptr) *ideal = tc::ffn_ideal(shape, pairs);
  delete plan;
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

int srm_k_wait_probe(uint32_t* d_status, int64_t limit_cycles, int32_t* d_gave_up, void* stream) {
  if (d_status == nullptr || limit_cycles < 1 || limit_cycles > (1ll << 31)) return SRM_ERR_INVALID_ARG;
  ++g_kernel_launches;
  tc::wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(d_status, (long long)limit_cycles, d_gave_up);
  SRM_CUDA(cudaGetLastError());
  return SRM_OK;
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

// One token-adaptive quantised layer (Eq. 1, 3, 9; App. B.2) and the prefill of
// a stack of them, composed from the library's kernels.  Everything between
// the router and the residual write-back is sized by the device-side executed
// token count; the host never reads it.
#include <string.h>

#include "attention.cuh"
#include "router_select.cuh"
#include "rowops.cuh"
#include "wq_gemm.cuh"

namespace qtale {

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct LayerWs {
  unsigned char* router_ws;  // scratch of the selection kernel
  size_t router_ws_bytes;
  float* scores;
  int32_t* idx;
  int32_t* pos;
  int32_t* n_exec;
  int32_t* cu_exec;
  void* hn;     // bf16 [T, d]            normed activations (attention, then MLP)
  void* qkv;    // bf16 [T, (H + 2 Hkv) hd]
  float* cs;    // float2 [T, hd/2]       rotary cos / sin
  void* ao;     // bf16 [T, H hd]         attention output
  float* u;     // fp32 [T, d]            x + attention branch
  void* gu;     // bf16 [T, 2 F]          gate | up (only when SwiGLU is not fused)
  void* act;    // bf16 [T, F]
  void* splitk; // scratch of the split-K GEMMs of a decode step
  size_t splitk_bytes;
  size_t total;
};

static LayerWs carve(const qtale_layer_config* c, int T, int B, void* base) {
  LayerWs w;
  size_t off = 0;
  unsigned char* b = static_cast<unsigned char*>(base);
  auto take = [&](size_t bytes) {
    unsigned char* p = b ? b + off : nullptr;
    off += align_up(bytes, 256);
    return p;
  };
  const size_t t = (size_t)T;
  const int qd = c->n_heads * c->head_dim, kvd = c->n_kv_heads * c->head_dim;
  w.router_ws_bytes = qtale_router_select_workspace_bytes(T);
  w.router_ws = take(w.router_ws_bytes);
  w.scores = reinterpret_cast<float*>(take(t * 4));
  w.idx = reinterpret_cast<int32_t*>(take(t * 4));
  w.pos = reinterpret_cast<int32_t*>(take(t * 4));
  w.n_exec = reinterpret_cast<int32_t*>(take(256));
  w.cu_exec = reinterpret_cast<int32_t*>(take((size_t)(B + 1) * 4));
  w.hn = take(t * c->d * 2);
  w.qkv = take(t * (qd + 2 * kvd) * 2);
  w.cs = reinterpret_cast<float*>(take(t * (c->head_dim / 2) * 8));
  w.ao = take(t * qd * 2);
  w.u = reinterpret_cast<float*>(take(t * c->d * 4));
  w.gu = take(t * 2 * c->ffn * 2);
  w.act = take(t * c->ffn * 2);
  w.splitk_bytes = wq_splitk_workspace_bytes();
  w.splitk = take(w.splitk_bytes);
  w.total = off;
  return w;
}

static int check_config(const qtale_layer_config* c) {
  if (!c) return QTALE_ERR_NULL;
  if (c->bits != 0 && (c->bits < 2 || c->bits > 4)) return QTALE_ERR_BITS;
  if (c->group != 64 && c->group != 128) return QTALE_ERR_GROUP;
  if (c->d < 8 || c->d % 8 || c->n_heads < 1 || c->n_kv_heads < 1 ||
      c->n_heads % c->n_kv_heads || (c->head_dim != 64 && c->head_dim != 128) || c->ffn < 8 ||
      c->ffn % 8)
    return QTALE_ERR_SHAPE;
  if (c->select_mode < QTALE_SELECT_THRESHOLD || c->select_mode > QTALE_SELECT_FORCED)
    return QTALE_ERR_MODE;
  if (c->act_dtype != QTALE_ACT_BF16 && c->act_dtype != QTALE_ACT_F16) return QTALE_ERR_MODE;
  return QTALE_OK;
}

#define QTALE_TRY(expr)            \
  do {                             \
    int rc__ = (expr);             \
    if (rc__ != QTALE_OK) return rc__; \
  } while (0)

static int layer_forward_impl(const qtale_layer_config* c, const qtale_layer_weights* w, void* x,
                              int T, const int32_t* cu_seqlens, int B, const int32_t* pos0,
                              const uint8_t* valid, const float* scores_override,
                              const int32_t* forced_idx, int forced_n, const qtale_kv_cache* kv,
                              int phase, int32_t* n_exec_out, float* scores_out, const LayerWs& ws,
                              cudaStream_t s) {
  const int d = c->d, H = c->n_heads, Hkv = c->n_kv_heads, hd = c->head_dim, F = c->ffn;
  const int qd = H * hd, kvd = Hkv * hd, nqkv = qd + 2 * kvd;
  const int act = c->act_dtype;

  // 1. execute / bypass decision and index lists
  const int32_t* idx = ws.idx;
  if (c->select_mode == QTALE_SELECT_FORCED) {
    idx = forced_idx;
    QTALE_TRY(qtale_index_bookkeeping(forced_idx, forced_n, T, cu_seqlens, B, pos0, ws.n_exec,
                                      ws.cu_exec, ws.pos, s));
  } else {
    // top-k: without a padding mask every token is valid and k is known here; with one the
    // kernel counts the valid tokens first (the ratio refers to them, App. B.2)
    int k = 0;
    double ratio = -1.0;
    if (c->select_mode == QTALE_SELECT_TOPK) {
      if (valid) ratio = (double)c->ratio; else k = qtale_topk_count((double)c->ratio, T);
    }
    float* sc_buf = scores_out ? scores_out : ws.scores;
    if (!scores_override && w->router_h > 0) {
      // MLP router: its scores come from a kernel of their own and enter the selection as given
      QTALE_TRY(router_mlp_launch(x, T, d, w->router_w1, w->router_b1, w->router_w2, w->router_h,
                                  w->router_b2[0], w->router_b2[1], sc_buf, s));
      scores_override = sc_buf;
    }
    QTALE_TRY(router_select_launch(x, T, d, w->router_w, w->router_b, scores_override, valid,
                                   cu_seqlens, B, pos0, c->select_mode, c->theta, k, ratio,
                                   scores_out ? scores_out : ws.scores, ws.idx, ws.n_exec,
                                   ws.cu_exec, ws.pos, ws.router_ws, ws.router_ws_bytes, s,
                                   n_exec_out));
  }
  if (n_exec_out && c->select_mode == QTALE_SELECT_FORCED &&
      cudaMemcpyAsync(n_exec_out, ws.n_exec, sizeof(int32_t), cudaMemcpyDeviceToDevice, s) !=
          cudaSuccess)
    return QTALE_ERR_CUDA;

  // decode steps: the linears run with the K dimension split over the SMs (ticket words zeroed)
  void* sk = nullptr;
  if (phase == QTALE_PHASE_DECODE && T <= 64) {
    sk = ws.splitk;
    if (cudaMemsetAsync(sk, 0, wq_splitk_ticket_bytes(), s) != cudaSuccess) return QTALE_ERR_CUDA;
  }
  const size_t skb = ws.splitk_bytes;

  // 2. gather the executed tokens and apply the first RMSNorm; the same launch writes the
  //    rotary table of their (original) positions and, for the prefill attention's tiled loads,
  //    clears the value columns of the 128 rows after the executed count
  const bool fused_rope = w->qkv.row_mode != QTALE_WQ_ROWS_PLAIN;
  GatherExtras gx;
  gx.pos = ws.pos;
  gx.cs = reinterpret_cast<float2*>(ws.cs);
  gx.half = hd / 2;
  gx.rope_base = c->rope_theta;
  gx.tail = phase == QTALE_PHASE_DECODE ? nullptr : static_cast<uint4*>(ws.qkv);
  gx.tail_ld = nqkv;
  gx.tail_col0 = qd + kvd;
  gx.tail_cols = kvd;
  gx.tail_rows = 128;
  QTALE_TRY(launch_compact(x, idx, ws.n_exec, T, d, w->gamma1, c->rms_eps, act, nullptr, ws.hn, s, &gx));
  // 3. q, k, v projections, rotary embedding at the original positions in the epilogue
  if (fused_rope) {
    qtale_epilogue_args er;
    memset(&er, 0, sizeof(er));
    er.rope_cs = ws.cs;
    er.rope_features = qd + kvd;
    QTALE_TRY(wq_gemm_launch(ws.hn, d, ws.n_exec, T, &w->qkv, act, QTALE_EPI_ROPE, &er, ws.qkv, nqkv, s, sk, skb, 0));
  } else {
    QTALE_TRY(wq_gemm_launch(ws.hn, d, ws.n_exec, T, &w->qkv, act, QTALE_EPI_STORE_16, nullptr, ws.qkv,
                             nqkv, s, sk, skb, 0));
    QTALE_TRY(launch_rope(ws.qkv, ws.n_exec, T, nqkv, H + Hkv, hd, ws.cs, act, s));
  }
  // 5. attention among executed tokens (+ cache)
  if (kv) {
    QTALE_TRY(launch_kv_append(ws.qkv, ws.n_exec, T, nqkv, qd, kvd, hd, ws.cu_exec, B, kv->k, kv->v,
                               kv->kv_len, kv->cap, s));
  }
  if (phase == QTALE_PHASE_DECODE) {
    QTALE_TRY(launch_attn_decode(ws.qkv, nqkv, H, Hkv, hd, act, idx, ws.n_exec, T, kv->k, kv->v,
                                 kv->kv_len, kv->cap, ws.ao, qd, s));
  } else {
    QTALE_TRY(launch_attn_prefill(ws.qkv, nqkv, H, Hkv, hd, act, ws.cu_exec, B, T, ws.ao, qd, s));
  }
  // 6. output projection + residual: u = x[idx] + attention branch (fp32)
  qtale_epilogue_args e;
  memset(&e, 0, sizeof(e));
  e.idx = idx;
  e.resid = x;
  e.ld_resid = d;
  e.dst = nullptr;
  e.ld_dst = 0;
  QTALE_TRY(wq_gemm_launch(ws.ao, qd, ws.n_exec, T, &w->o, act, QTALE_EPI_RESID_F32, &e, ws.u, d, s, sk, skb, 1));
  // 7. second RMSNorm
  QTALE_TRY(launch_rmsnorm_f32(ws.u, ws.n_exec, T, d, w->gamma2, c->rms_eps, act, ws.hn, s));
  // 8. gate / up projections and SwiGLU
  if (w->gate_up.row_mode == QTALE_WQ_ROWS_SWIGLU) {
    QTALE_TRY(wq_gemm_launch(ws.hn, d, ws.n_exec, T, &w->gate_up, act, QTALE_EPI_SWIGLU, nullptr, ws.act,
                             F, s, sk, skb, 2));
  } else {
    QTALE_TRY(wq_gemm_launch(ws.hn, d, ws.n_exec, T, &w->gate_up, act, QTALE_EPI_STORE_16, nullptr,
                             ws.gu, 2 * F, s, sk, skb, 2));
    QTALE_TRY(launch_swiglu(ws.gu, ws.n_exec, T, F, ws.act, act, s));
  }
  // 9. down projection + residual scatter: x[idx] = bf16(u + MLP branch)   (Eq. 3)
  e.resid = ws.u;
  e.ld_resid = d;
  e.dst = x;
  e.ld_dst = d;
  QTALE_TRY(wq_gemm_launch(ws.act, F, ws.n_exec, T, &w->down, act, QTALE_EPI_RESID_SCATTER, &e, nullptr,
                           0, s, sk, skb, 3));
  return QTALE_OK;
}

static int check_weights(const qtale_layer_config* c, const qtale_layer_weights* w) {
  if (!w || !w->qkv.packed || !w->o.packed || !w->gate_up.packed || !w->down.packed ||
      !w->gamma1 || !w->gamma2)
    return QTALE_ERR_NULL;
  const int qd = c->n_heads * c->head_dim, kvd = c->n_kv_heads * c->head_dim;
  if (w->qkv.N != qd + 2 * kvd || w->qkv.K != c->d || w->o.N != c->d || w->o.K != qd ||
      w->gate_up.N != 2 * c->ffn || w->gate_up.K != c->d || w->down.N != c->d ||
      w->down.K != c->ffn)
    return QTALE_ERR_SHAPE;
  const qtale_wq_weight* all[4] = {&w->qkv, &w->o, &w->gate_up, &w->down};
  for (const qtale_wq_weight* q : all) {
    if (c->bits ? q->bits != c->bits : (q->bits < 2 || q->bits > 4)) return QTALE_ERR_BITS;
    if (q->group != c->group) return QTALE_ERR_GROUP;
    if (!aligned16(q->packed)) return QTALE_ERR_ALIGN;
  }
  const int rope_mode = c->head_dim == 64 ? QTALE_WQ_ROWS_ROPE64 : QTALE_WQ_ROWS_ROPE128;
  if ((w->qkv.row_mode != QTALE_WQ_ROWS_PLAIN && w->qkv.row_mode != rope_mode) ||
      w->o.row_mode != QTALE_WQ_ROWS_PLAIN || w->down.row_mode != QTALE_WQ_ROWS_PLAIN)
    return QTALE_ERR_MODE;
  return QTALE_OK;
}

}  // namespace qtale

using namespace qtale;

extern "C" {

size_t qtale_layer_workspace_bytes(const qtale_layer_config* cfg, int T_cap, int B_cap) {
  if (check_config(cfg) != QTALE_OK || T_cap < 1 || B_cap < 1) return 0;
  return carve(cfg, T_cap, B_cap, nullptr).total;
}

int qtale_layer_forward(const qtale_layer_config* cfg, const qtale_layer_weights* w, void* x_inout,
                        int T, const int32_t* cu_seqlens, int B, const int32_t* pos0,
                        const uint8_t* valid, const float* scores_override,
                        const int32_t* forced_idx, int forced_n, const qtale_kv_cache* kv,
                        int phase, int32_t* n_exec_out, float* scores_out, void* ws,
                        size_t ws_bytes, void* stream) {
  QTALE_TRY(check_config(cfg));
  QTALE_TRY(check_weights(cfg, w));
  if (!x_inout || !cu_seqlens || !ws) return QTALE_ERR_NULL;
  if (T < 1 || B < 1 || B > T) return QTALE_ERR_SHAPE;
  if (!aligned16(x_inout) || !aligned16(ws)) return QTALE_ERR_ALIGN;
  if (phase != QTALE_PHASE_PREFILL && phase != QTALE_PHASE_DECODE) return QTALE_ERR_MODE;
  if (phase == QTALE_PHASE_DECODE && (!kv || T != B)) return QTALE_ERR_SHAPE;
  if (kv && (!kv->k || !kv->v || !kv->kv_len || kv->cap < 1)) return QTALE_ERR_NULL;
  if (cfg->select_mode == QTALE_SELECT_FORCED) {
    if (forced_n < 0 || forced_n > T) return QTALE_ERR_CAPACITY;
    if (forced_n > 0 && !forced_idx) return QTALE_ERR_NULL;
  } else if (!scores_override) {
    if (w->router_h < 0 || w->router_h > 64) return QTALE_ERR_SHAPE;
    if (w->router_h == 0 && !w->router_w) return QTALE_ERR_NULL;
    if (w->router_h > 0 && (!w->router_w1 || !w->router_b1 || !w->router_w2)) return QTALE_ERR_NULL;
  }
  if (ws_bytes < qtale_layer_workspace_bytes(cfg, T, B)) return QTALE_ERR_WORKSPACE;
  const LayerWs lw = carve(cfg, T, B, ws);
  return layer_forward_impl(cfg, w, x_inout, T, cu_seqlens, B, pos0, valid, scores_override,
                            forced_idx, forced_n, kv, phase, n_exec_out, scores_out, lw,
                            static_cast<cudaStream_t>(stream));
}

size_t qtale_model_workspace_bytes(const qtale_model_config* cfg, int T_cap, int B_cap,
                                   int n_logit_rows) {
  if (!cfg) return 0;
  const size_t layer = qtale_layer_workspace_bytes(&cfg->layer, T_cap, B_cap);
  if (layer == 0) return 0;
  const size_t rows = n_logit_rows > 0 ? (size_t)n_logit_rows : 0;
  return layer + align_up(rows * cfg->layer.d * 2, 256) + 256;
}

int qtale_model_prefill(const qtale_model_config* cfg, const qtale_model_weights* w,
                        const int32_t* ids, int T, const int32_t* cu_seqlens, int B,
                        const uint8_t* valid, const qtale_kv_cache* caches,
                        const float* per_layer_ratio, void* hidden_out, float* logits_out,
                        const int32_t* logit_rows, int n_logit_rows, int32_t* per_layer_n_exec,
                        float* layer_scores_out, void* ws, size_t ws_bytes, void* stream) {
  if (!cfg || !w || !ids || !cu_seqlens || !hidden_out || !ws || !w->embed || !w->layers)
    return QTALE_ERR_NULL;
  QTALE_TRY(check_config(&cfg->layer));
  if (cfg->n_layers < 1 || cfg->vocab < 1 || T < 1 || B < 1 || B > T) return QTALE_ERR_SHAPE;
  if (logits_out && (!w->lm_head || !w->final_gamma || !logit_rows || n_logit_rows < 1))
    return QTALE_ERR_NULL;
  for (int l = 0; l < cfg->n_layers; ++l) QTALE_TRY(check_weights(&cfg->layer, &w->layers[l]));
  if (!aligned16(hidden_out) || !aligned16(ws) || !aligned16(w->embed)) return QTALE_ERR_ALIGN;
  const int n_rows = logits_out ? n_logit_rows : 0;
  if (ws_bytes < qtale_model_workspace_bytes(cfg, T, B, n_rows)) return QTALE_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int d = cfg->layer.d;

  const LayerWs lw = carve(&cfg->layer, T, B, ws);
  void* hrows = static_cast<unsigned char*>(ws) + lw.total;

  QTALE_TRY(launch_embed(w->embed, ids, T, d, cfg->vocab, hidden_out, s));
  for (int l = 0; l < cfg->n_layers; ++l) {
    qtale_layer_config lc = cfg->layer;
    if (per_layer_ratio) {
      lc.select_mode = QTALE_SELECT_TOPK;
      lc.ratio = per_layer_ratio[l];
    } else if (lc.select_mode == QTALE_SELECT_FORCED) {
      return QTALE_ERR_MODE;
    }
    if (caches && (!caches[l].k || !caches[l].v || !caches[l].kv_len || caches[l].cap < 1))
      return QTALE_ERR_NULL;
    QTALE_TRY(layer_forward_impl(&lc, &w->layers[l], hidden_out, T, cu_seqlens, B, nullptr,
                                 valid, nullptr, nullptr, 0, caches ? &caches[l] : nullptr,
                                 QTALE_PHASE_PREFILL,
                                 per_layer_n_exec ? per_layer_n_exec + l : nullptr,
                                 layer_scores_out ? layer_scores_out + (size_t)l * T : nullptr, lw,
                                 s));
  }
  if (logits_out) {
    QTALE_TRY(launch_compact(hidden_out, logit_rows, nullptr, n_logit_rows, d, w->final_gamma,
                             cfg->layer.rms_eps, QTALE_ACT_BF16, nullptr, hrows, s));
    QTALE_TRY(bf16_gemm_launch(hrows, d, nullptr, n_logit_rows, w->lm_head, cfg->vocab, d, d,
                               logits_out, cfg->vocab, s));
  }
  return QTALE_OK;
}

size_t qtale_model_decode_workspace_bytes(const qtale_model_config* cfg, int B_cap) {
  if (!cfg || B_cap < 1) return 0;
  const size_t layer = qtale_layer_workspace_bytes(&cfg->layer, B_cap, B_cap);
  if (layer == 0) return 0;
  return layer + align_up((size_t)B_cap * cfg->layer.d * 2, 256) + align_up((size_t)(B_cap + 1) * 4, 256);
}

int qtale_model_decode_step(const qtale_model_config* cfg, const qtale_model_weights* w,
                            const int32_t* ids, int B, int32_t* pos, const uint8_t* valid,
                            const qtale_kv_cache* caches, void* hidden_out, float* logits_out,
                            int32_t* next_ids_out, int32_t* per_layer_n_exec,
                            float* layer_scores_out, void* ws, size_t ws_bytes, void* stream) {
  if (!cfg || !w || !ids || !pos || !caches || !hidden_out || !ws || !w->embed || !w->layers)
    return QTALE_ERR_NULL;
  QTALE_TRY(check_config(&cfg->layer));
  if (cfg->n_layers < 1 || cfg->vocab < 1 || B < 1) return QTALE_ERR_SHAPE;
  if (cfg->layer.select_mode == QTALE_SELECT_FORCED) return QTALE_ERR_MODE;
  if ((logits_out || next_ids_out) && (!w->lm_head || !w->final_gamma)) return QTALE_ERR_NULL;
  if (next_ids_out && !logits_out) return QTALE_ERR_NULL;
  for (int l = 0; l < cfg->n_layers; ++l) {
    QTALE_TRY(check_weights(&cfg->layer, &w->layers[l]));
    if (!caches[l].k || !caches[l].v || !caches[l].kv_len || caches[l].cap < 1) return QTALE_ERR_NULL;
  }
  if (!aligned16(hidden_out) || !aligned16(ws) || !aligned16(w->embed)) return QTALE_ERR_ALIGN;
  if (ws_bytes < qtale_model_decode_workspace_bytes(cfg, B)) return QTALE_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int d = cfg->layer.d;
  const LayerWs lw = carve(&cfg->layer, B, B, ws);
  unsigned char* base = static_cast<unsigned char*>(ws) + lw.total;
  void* hrows = base;
  int32_t* cu = reinterpret_cast<int32_t*>(base + align_up((size_t)B * d * 2, 256));

  QTALE_TRY(launch_iota(cu, B + 1, s));  // one new token per sequence: cu_seqlens = 0, 1, ..., B
  QTALE_TRY(launch_embed(w->embed, ids, B, d, cfg->vocab, hidden_out, s));
  for (int l = 0; l < cfg->n_layers; ++l) {
    QTALE_TRY(layer_forward_impl(&cfg->layer, &w->layers[l], hidden_out, B, cu, B, pos, valid, nullptr,
                                 nullptr, 0, &caches[l], QTALE_PHASE_DECODE,
                                 per_layer_n_exec ? per_layer_n_exec + l : nullptr,
                                 layer_scores_out ? layer_scores_out + (size_t)l * B : nullptr, lw, s));
  }
  if (logits_out) {
    QTALE_TRY(launch_compact(hidden_out, cu, nullptr, B, d, w->final_gamma, cfg->layer.rms_eps,
                             QTALE_ACT_BF16, nullptr, hrows, s));
    QTALE_TRY(bf16_gemm_launch(hrows, d, nullptr, B, w->lm_head, cfg->vocab, d, d, logits_out,
                               cfg->vocab, s));
    if (next_ids_out) QTALE_TRY(launch_argmax_rows(logits_out, B, cfg->vocab, next_ids_out, s));
  }
  return launch_advance_pos(pos, valid, B, s);
}

}  // extern "C"

/*
 * qtale.h -- C ABI of libqtale: forward pass of a token-adaptive transformer
 * layer with low-bit group-quantised weights (QTALE, arXiv 2602.10431) on one
 * NVIDIA B200 (sm_100a).
 *
 * Per layer the path is: router score per token and execute / bypass decision
 * (Eq. 2, Eq. 9), gathering of the executed tokens into a dense tensor
 * (App. B.2), the layer function f_l on the executed tokens only with every
 * linear a b-bit group-quantised matmul (Eq. 1; Sec. 4.1 implementation
 * details), and the residual write-back x + f_l(x) for executed tokens while
 * bypassed tokens keep x (Eq. 3).
 *
 * Conventions
 *  - Every function returns an int status: QTALE_OK (0) or a negative
 *    QTALE_ERR_* code; qtale_strerror() names it.  Arguments are validated on
 *    the host; on error nothing is launched and no output is touched.
 *  - Unless a parameter says "host", every pointer is a DEVICE pointer owned
 *    by the caller, 16-byte aligned.  The library never allocates or frees
 *    device memory; scratch comes from a caller workspace whose size the
 *    matching *_workspace_bytes() query returns.
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *    Calls enqueue work and return without synchronising.  The number of
 *    executed tokens stays on the device (int32) and is never read back by
 *    the library.
 *  - The residual stream (layer input / output) is bf16, row-major, innermost
 *    dimension contiguous.  Tensors the layer keeps between its kernels
 *    (normed activations, q/k/v, attention output, SwiGLU activation, KV cache)
 *    are 16-bit in the format `act_dtype` selects: QTALE_ACT_BF16, or
 *    QTALE_ACT_F16 whose three extra significand bits keep the accumulated
 *    rounding error of a 4096-wide layer inside the max-abs 2e-2 bound (fp16's
 *    range, 65504, must then cover those tensors).  Accumulation is fp32.
 *    Tokens of all sequences are flattened: token t of the call belongs to
 *    sequence b with cu_seqlens[b] <= t < cu_seqlens[b+1].  cu_seqlens (device,
 *    int32 [B+1]) must satisfy 0 = cu_seqlens[0] <= ... <= cu_seqlens[B] = T
 *    (empty sequences are fine).  The host cannot see it, so the selection
 *    kernel checks it: a violation records QTALE_ERR_SHAPE in the device status
 *    word, tokens outside [cu_seqlens[0], cu_seqlens[B]) never execute, and no
 *    access leaves the B + 1 entries.
 *  - Workspaces need not be cleared by the caller, and may be reused between
 *    calls of different sizes: every kernel initialises what it reads.
 *  - A device-side wait that exceeds its iteration limit ends the kernel
 *    normally and records QTALE_ERR_TIMEOUT in a device status word that
 *    qtale_device_status() reads.
 */
#ifndef QTALE_H_
#define QTALE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define QTALE_OK 0
#define QTALE_ERR_NULL (-1)      /* a required pointer is NULL */
#define QTALE_ERR_ALIGN (-2)     /* pointer or pitch not 16-byte aligned */
#define QTALE_ERR_SHAPE (-3)     /* unsupported or inconsistent sizes */
#define QTALE_ERR_BITS (-4)      /* bits not in {2, 3, 4} */
#define QTALE_ERR_GROUP (-5)     /* group not in {64, 128} */
#define QTALE_ERR_WORKSPACE (-6) /* workspace too small */
#define QTALE_ERR_CAPACITY (-7)  /* a count exceeds the capacity of its buffer */
#define QTALE_ERR_TIMEOUT (-8)   /* a bounded device-side wait gave up */
#define QTALE_ERR_CUDA (-9)      /* a CUDA runtime / driver call failed */
#define QTALE_ERR_MODE (-10)     /* unknown mode / epilogue / phase / dtype */

#define QTALE_ACT_BF16 0
#define QTALE_ACT_F16 1

const char* qtale_strerror(int status);

/* Reads (synchronously, after cudaStreamSynchronize of `stream`) and clears
 * the device status word of the current device.  Returns QTALE_OK or the
 * first device-side error recorded since the last call. */
int qtale_device_status(void* stream);

/* ------------------------------------------------------------------------- */
/* Selection (Eq. 2, Eq. 9)                                                   */
/* ------------------------------------------------------------------------- */

#define QTALE_SELECT_THRESHOLD 0 /* execute iff p0 >= theta            (Eq. 9) */
#define QTALE_SELECT_TOPK 1      /* the k highest scores (extension, see below) */
#define QTALE_SELECT_FORCED 2    /* caller supplies the index list              */

/* k of top-k selection for a requested execution ratio: floor(ratio*n + 0.5),
 * clamped to [0, n].  Host function. */
int qtale_topk_count(double ratio, int n_valid);

/* Scratch of qtale_router_select for a call of T tokens: 16 KB of counters plus
 * 8 bytes per token (candidate list of the top-k selection). */
size_t qtale_router_select_workspace_bytes(int T);

/*
 * Router score, execute decision and ordered compaction in one launch.
 *
 * Score (Eq. 9 specialised to a linear two-class router): the router emits
 * two class logits (g0 execute, g1 bypass); with a linear router their
 * difference is z_t = w_router . x_t + bias and softmax([g0,g1])[0] =
 * 1 / (1 + exp(-z_t)).  The dot product is formed from fp32 partial sums of 8
 * products accumulated in fp64 (within about 1e-8 of an all-fp64 sum); the
 * logistic is evaluated in fp64 and the score is stored as fp32.  If scores_override != NULL the router is skipped and those
 * scores are used (and copied to scores_out).
 *
 * Decision: THRESHOLD: execute iff score >= theta (fp32 compare, ties
 * execute), one theta for all layers.  TOPK (not in the paper, which controls
 * the ratio through theta only): the k valid tokens of the call with the
 * highest scores, equal scores ordered by lower token index.  Tokens with
 * valid[t] == 0 (padding, App. B.2) never execute.
 *
 * Outputs: scores_out[T]; idx_out[T]: ascending token indices of executed
 * tokens in its first *n_exec_out entries (rest untouched); n_exec_out[1];
 * cu_exec_out[B+1]: offsets of each sequence's executed tokens inside idx_out;
 * pos_out[T]: for executed token i its position inside its sequence,
 * idx - cu_seqlens[b] + (pos0 ? pos0[b] : 0).
 *
 *   x          [T, d] bf16              w_router  [d] fp32
 *   valid      [T] uint8 or NULL        cu_seqlens [B+1] int32, pos0 [B] or NULL
 * Limits: d % 8 == 0, 1 <= T <= 2^24, 1 <= B <= T, 0 <= k <= T.
 */
int qtale_router_select(const void* x, int T, int d, const float* w_router, float bias,
                        const float* scores_override, const uint8_t* valid,
                        const int32_t* cu_seqlens, int B, const int32_t* pos0, int mode,
                        float theta, int k, float* scores_out, int32_t* idx_out,
                        int32_t* n_exec_out, int32_t* cu_exec_out, int32_t* pos_out, void* ws,
                        size_t ws_bytes, void* stream);

/*
 * Router as a small MLP (Eq. 2: "a lightweight MLP" produces the two class
 * logits; Eq. 9: the execute probability is their softmax):
 *   u = W1 x + b1,  a = max(u, 0),  (g0, g1) = W2 a + b2,  score = softmax(g)[0]
 *         = 1 / (1 + exp(-((W2[0] - W2[1]) . a + b2_execute - b2_bypass))).
 * The paper states neither the hidden width nor the activation; ReLU is this
 * library's reading.  The hidden layer runs on the tensor cores with fp64
 * accumulation across 64-feature chunks, so the scores agree with an fp64
 * evaluation to about 1e-7.  Feed scores_out to qtale_router_select as
 * scores_override (qtale_layer_forward does that when router_h > 0).
 *   x [T, d] bf16; w1 [h, d] bf16; b1 [h] fp32; w2 [2, h] fp32 (row 0 execute,
 *   row 1 bypass); scores_out [T] fp32.  Limits: d % 8 == 0, 1 <= h <= 64.
 */
int qtale_router_mlp_scores(const void* x, int T, int d, const void* w1, const float* b1,
                            const float* w2, int h, float b2_execute, float b2_bypass,
                            float* scores_out, void* stream);

/*
 * qtale_router_select for callers that must not allocate device memory.
 * (No counterpart in the paper: this is a packaging variant of the call above.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plugin inside
 * a host application that owns the whole memory pool and hands out no scratch,
 * a real-time or safety-checked loop that forbids allocator calls after start-up,
 * or a caller that simply has no buffer left to lend as `ws`.  Same arguments,
 * results and limits as qtale_router_select, minus the workspace: the kernel's
 * scratch (counters, histogram, per-CTA counts, top-k candidate list) sits in an
 * array that is part of the library's device image, sized for
 * QTALE_ROUTER_STATIC_MAX_TOKENS tokens (16 KB + 8 bytes per token = 528 KB), so
 * every GPU that loads the library holds that much until the process exits.  The
 * call itself performs no cudaMalloc / cudaFree and uses no allocating library
 * routine.
 *
 *  - Limit: T > QTALE_ROUTER_STATIC_MAX_TOKENS is refused with
 *    QTALE_ERR_CAPACITY (nothing is launched); use qtale_router_select with a
 *    workspace of your own for larger calls.
 *  - The first call on each device looks up the array's device address (one
 *    cudaGetSymbolAddress, result cached per device ordinal; the cache does not
 *    survive a cudaDeviceReset); make that first call outside any stream capture.
 *  - All calls on a device share the one array.  Its counters are cleared on the
 *    stream before every launch, so leftovers of the previous call are harmless,
 *    but two calls whose kernels overlap on the GPU (different streams) race on
 *    it: keep calls to this entry point on one stream, or order them yourself.
 */
#define QTALE_ROUTER_STATIC_MAX_TOKENS 65536
int qtale_router_select_static(const void* x, int T, int d, const float* w_router, float bias,
                               const float* scores_override, const uint8_t* valid,
                               const int32_t* cu_seqlens, int B, const int32_t* pos0, int mode,
                               float theta, int k, float* scores_out, int32_t* idx_out,
                               int32_t* n_exec_out, int32_t* cu_exec_out, int32_t* pos_out,
                               void* stream);

/*
 * Threshold for a requested execution ratio (Sec. 3.4, Eq. 9: one global theta
 * controls the ratio after training; App. A.1 searches it on a grid).  Given
 * the router scores of a calibration batch pooled over all layers, returns the
 * theta for which the share of valid scores with score >= theta is `ratio`:
 * theta = the k-th largest valid score, k = floor(ratio * n_valid + 0.5) (the
 * exact quantile, no histogram approximation); k = 0 gives theta = 2 (above
 * every probability).  *count_out = number of valid scores >= theta (k, or more
 * when scores tie at theta).  The accuracy-driven half of the paper's search
 * needs task data and is not part of this library.
 *   scores [n] fp32 device; valid [n] uint8 or NULL; theta_out [1] fp32 and
 *   count_out [1] int32 on the device; ws of qtale_theta_workspace_bytes().
 * Limits: 1 <= n <= 2^31, 0 <= ratio <= 1, scores must not be NaN.
 */
size_t qtale_theta_workspace_bytes(void);
int qtale_theta_for_ratio(const float* scores, const uint8_t* valid, size_t n, double ratio,
                          float* theta_out, int32_t* count_out, void* ws, size_t ws_bytes,
                          void* stream);

/* Bookkeeping for a caller-supplied ascending index list (QTALE_SELECT_FORCED):
 * fills n_exec_out, cu_exec_out and pos_out as qtale_router_select does.
 * idx [n] int32 device, 0 <= n <= T. */
int qtale_index_bookkeeping(const int32_t* idx, int n, int T, const int32_t* cu_seqlens, int B,
                            const int32_t* pos0, int32_t* n_exec_out, int32_t* cu_exec_out,
                            int32_t* pos_out, void* stream);

/* ------------------------------------------------------------------------- */
/* Gather / scatter (App. B.2; Eq. 3)                                          */
/* ------------------------------------------------------------------------- */

/*
 * Gather of the executed rows: xc[i,:] = x[idx[i],:] for i < *n_exec.
 * If rms_gamma != NULL also hn[i,:] = x[idx[i],:] / sqrt(mean(x^2) + eps) * gamma
 * (fp32 arithmetic, one rounding to act_dtype).  xc_out or hn_out may be NULL
 * (not both).  Rows i >= *n_exec of the outputs are left untouched.
 *   x [T, d] bf16; idx [T] int32; n_exec [1] int32; rms_gamma [d] fp32;
 *   xc_out [T, d] bf16 (byte copy), hn_out [T, d] act_dtype (capacity T rows).
 *   d % 8 == 0.
 */
int qtale_compact(const void* x, const int32_t* idx, const int32_t* n_exec, int T, int d,
                  const float* rms_gamma, float eps, int act_dtype, void* xc_out, void* hn_out,
                  void* stream);

/*
 * Residual scatter (Eq. 3, execute branch), in place:
 * x[idx[i],:] = bf16(float(xc[i,:]) + f[i,:]) for i < *n_exec; every other row
 * of x is left untouched (bypass branch).  xc bf16 [T, d]; f fp32 [T, d].
 */
int qtale_scatter_add(void* x_inout, const void* xc, const float* f, const int32_t* idx,
                      const int32_t* n_exec, int T, int d, void* stream);

/* ------------------------------------------------------------------------- */
/* Weight-only quantised GEMM (Sec. 4.1: 4-bit / 3-bit, per-group parameters) */
/* ------------------------------------------------------------------------- */

/* A quantised linear W[N, K] (y = x W^T) in the kernel-native layout written
 * by qtale_wq_repack.  Dequantisation: w = (code - zero) * scale with one
 * fp16 scale and one integer-valued fp16 zero-point per `group` consecutive
 * input features of a row. */
typedef struct {
  const void* packed; /* device copy of the repacked blob */
  int N, K;           /* logical shape */
  int bits;           /* 2, 3 or 4 */
  int group;          /* 64 or 128 */
  int row_mode;       /* QTALE_WQ_ROWS_* the blob was repacked with */
} qtale_wq_weight;

#define QTALE_WQ_ROWS_PLAIN 0  /* output feature n sits in tile n / 128, lane n % 128       */
#define QTALE_WQ_ROWS_SWIGLU 1 /* W = [gate; up] (N = 2F): each 128-row tile holds 64 gate
                                  rows and the matching 64 up rows, needed by EPI_SWIGLU   */
#define QTALE_WQ_ROWS_ROPE64 2  /* W = [Wq; Wk; Wv] with heads of 64 / 128 features: inside a  */
#define QTALE_WQ_ROWS_ROPE128 3 /* tile every feature sits next to its rotary partner half a
                                  head further (N % head_dim == 0), needed by EPI_ROPE      */

/*
 * Offline repack, HOST pointers.  Input is the interface layout: codes
 * row-major [N, row_bytes]; 4-bit: two codes per byte, even k in the low
 * nibble, row_bytes = ceil(K/2); 3-bit: little-endian bit stream along K,
 * row_bytes = ceil(3K/8); scales / zeros fp16 [N, ceil(K/group)].
 * Call with packed_out == NULL to get the blob size in *bytes; then with a
 * buffer of that size.  Rows are padded to a multiple of 128 and K to a
 * multiple of `group` with codes equal to the zero-point (weight 0).
 */
int qtale_wq_repack(const uint8_t* codes, const uint16_t* scales, const uint16_t* zeros, int N,
                    int K, int bits, int group, int row_mode, void* packed_out, size_t* bytes);

#define QTALE_EPI_STORE_16 0      /* y[m,n] = act_dtype(acc)                             */
#define QTALE_EPI_STORE_F32 1     /* y[m,n] = acc                                  (fp32) */
#define QTALE_EPI_RESID_F32 2     /* y[m,n] = float(resid[idx[m],n]) + acc         (fp32) */
#define QTALE_EPI_RESID_SCATTER 3 /* dst[idx[m],n] = bf16(resid_f32[m,n] + acc)    (Eq. 3) */
#define QTALE_EPI_SWIGLU 4        /* y[m,j] = act_dtype(silu(acc[m,j]) * acc[m,F+j]), N = 2F;
                                     needs QTALE_WQ_ROWS_SWIGLU weights                   */
#define QTALE_EPI_ROPE 5          /* y[m,:] = act_dtype(acc[m,:]) with the rotary embedding applied
                                     to the features below rope_features (query and key heads):
                                     (x_j, x_{j+hd/2}) -> (x_j c - x_{j+hd/2} s, x_{j+hd/2} c + x_j s)
                                     with (c, s) = rope_cs[m, j]; one rounding of the fp32 result;
                                     needs QTALE_WQ_ROWS_ROPE* weights                    */

typedef struct {
  const int32_t* idx;    /* [M_cap] row indices (RESID_F32, RESID_SCATTER) */
  const void* resid;     /* RESID_F32: bf16 [T, ld_resid] gathered by idx;
                            RESID_SCATTER: fp32 [M_cap, ld_resid] dense          */
  int ld_resid;          /* elements */
  void* dst;             /* RESID_SCATTER: bf16 [T, ld_dst], rows idx[m] written */
  int ld_dst;
  const void* rope_cs;   /* ROPE: float2 (cos, sin) [M_cap, head_dim / 2] of each row's position */
  int rope_features;     /* ROPE: features [0, rope_features) are rotated, a multiple of head_dim */
} qtale_epilogue_args;

/*
 * y = epilogue(a W^T) on the tensor cores; rows m >= *m_dev (or >= M_cap when
 * m_dev == NULL) are neither computed nor written.
 *   a  act_dtype [M_cap, lda]  (lda >= K elements, lda * 2 bytes % 16 == 0)
 *   y  [M_cap, ldy]; element type set by the epilogue; N % 8 == 0, ldy % 8 == 0
 * The packed weights are dequantised inside the kernel to the 16-bit format of
 * `a` (exact (code - zero) * scale in fp32, one rounding) and accumulated in
 * fp32.
 * ws / ws_bytes: optional scratch of qtale_wq_gemm_workspace_bytes() (NULL / 0:
 * none).  With it, products of at most 64 token rows (a decode step) run with
 * the input dimension split over the SMs, the partial sums meeting in the
 * scratch (added in a fixed order: results do not depend on timing); without it
 * they run on a kernel that needs no scratch.  Larger products never use it.
 */
size_t qtale_wq_gemm_workspace_bytes(void);
int qtale_wq_gemm(const void* a, int lda, const int32_t* m_dev, int M_cap, const qtale_wq_weight* w,
                  int act_dtype, int epilogue, const qtale_epilogue_args* epi, void* y, int ldy,
                  void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------- */
/* Attention among the executed tokens (Eq. 3: bypassed tokens have no query,   */
/* key or value at the layer)                                                   */
/* ------------------------------------------------------------------------- */

/*
 * Causal softmax attention of a compacted prefill batch: executed token i of a
 * sequence attends to the executed tokens j <= i of the same sequence, scale
 * 1/sqrt(head_dim), fp32 softmax, probabilities rounded once to act_dtype.
 *   qkv [T_cap, ld] act_dtype, device: row i = [n_heads query heads | n_kv_heads
 *     key heads | n_kv_heads value heads], each head_dim wide, queries and keys
 *     already rotated; rows in compacted order (sequence by sequence).
 *   cu_exec [B+1] int32, device: executed rows of sequence b are
 *     cu_exec[b] .. cu_exec[b+1]-1, non-decreasing, cu_exec[B] <= T_cap.
 *   out [T_cap, ldo] act_dtype: rows below cu_exec[B] are written (columns
 *     0 .. n_heads*head_dim-1), the rest left untouched.
 * Keys and values are read in tiles of 128 rows: the value columns of the rows
 * from cu_exec[B] to the end of that 128-row tile (as far as T_cap reaches) must
 * hold finite numbers (their probabilities are zero; the layer path clears them).
 * head_dim 64 or 128; n_heads a multiple of n_kv_heads; ld, ldo multiples of 8;
 * qkv and out 16-byte aligned.  Nothing is owned or allocated.
 * Errors: QTALE_ERR_NULL / _SHAPE / _ALIGN / _MODE before anything is launched.
 */
int qtale_attention_prefill(const void* qkv, int ld, int n_heads, int n_kv_heads, int head_dim,
                            int act_dtype, const int32_t* cu_exec, int B, int T_cap, void* out,
                            int ldo, void* stream);

/* ------------------------------------------------------------------------- */
/* Layer and model                                                             */
/* ------------------------------------------------------------------------- */

typedef struct {
  int d, n_heads, n_kv_heads, head_dim, ffn; /* Llama-style decoder layer shape          */
  int bits, group;                          /* quantisation of the four linears; bits = 0:
                                               each weight descriptor's own width, so the
                                               layers of a model may mix 2, 3 and 4 bits
                                               (mixed precision across layers, App. C)   */
  float rms_eps, rope_theta;                /* RMSNorm epsilon, rotary base               */
  int select_mode;                          /* QTALE_SELECT_*                             */
  float theta;                              /* threshold of Eq. 9 (THRESHOLD)             */
  float ratio;                              /* execution ratio in [0,1] (TOPK): k =
                                               qtale_topk_count(ratio, number of valid
                                               tokens); padding does not count (App. B.2);
                                               with a `valid` mask the count is taken on
                                               the device                                   */
  int act_dtype;                            /* QTALE_ACT_*: format of the layer's internal
                                               16-bit tensors and of its KV cache          */
} qtale_layer_config;

typedef struct {
  qtale_wq_weight qkv;     /* [(H + 2 Hkv) hd, d]: Wq rows, then Wk, then Wv   */
  qtale_wq_weight o;       /* [d, H hd]                                        */
  qtale_wq_weight gate_up; /* [2 F, d]: gate rows then up rows                 */
  qtale_wq_weight down;    /* [d, F]                                           */
  const float* gamma1;     /* [d] fp32, pre-attention RMSNorm gain             */
  const float* gamma2;     /* [d] fp32, pre-MLP RMSNorm gain                   */
  const float* router_w;   /* [d] fp32, execute-minus-bypass logit weights     */
  float router_b;
  int router_h;            /* 0: the linear router above; > 0: MLP router with this
                              many hidden units (see qtale_router_mlp_scores)   */
  const void* router_w1;   /* [router_h, d] bf16                               */
  const float* router_b1;  /* [router_h] fp32                                  */
  const float* router_w2;  /* [2, router_h] fp32                               */
  float router_b2[2];      /* execute, bypass                                  */
} qtale_layer_weights;

/* Per-layer KV cache.  Only executed tokens enter it: a bypassed token does not
 * evaluate f_l (Eq. 3) and therefore produces no key or value at that layer.
 * Capacity: a call appends (executed tokens of sequence b) entries to sequence b
 * and needs kv_len[b] + that count <= cap.  The lengths live on the device, so
 * the host cannot check this: entries that do not fit are dropped, kv_len[b]
 * stays at cap, and QTALE_ERR_CAPACITY is recorded in the device status word
 * (the layer output of that sequence is then not meaningful). */
typedef struct {
  void* k;         /* act_dtype [B, n_kv_heads, cap, head_dim], rotary already applied: the
                      entries of one (sequence, head) are contiguous, so the decode
                      attention streams them at full memory bandwidth                   */
  void* v;         /* act_dtype [B, n_kv_heads, cap, head_dim]                          */
  int32_t* kv_len; /* int32 [B], entries in use per sequence (updated)             */
  int cap;
} qtale_kv_cache;

#define QTALE_PHASE_PREFILL 0 /* any sequence lengths; cache (if given) must be empty */
#define QTALE_PHASE_DECODE 1  /* exactly one new token per sequence, cache required   */

size_t qtale_layer_workspace_bytes(const qtale_layer_config* cfg, int T_cap, int B_cap);

/*
 * One token-adaptive layer, in place on x (Eq. 1, 3, 9; App. B.2).
 * Executed tokens: x <- x + f_l(x) with f_l = attention branch + MLP branch on
 * the gathered executed tokens; attention is causal among the executed tokens
 * of the same sequence (plus that sequence's cache entries in DECODE), RoPE
 * uses each token's original position.  Bypassed tokens: x unchanged.
 *
 *   x_inout [T, d] bf16; cu_seqlens [B+1]; pos0 [B] or NULL (position of each
 *   sequence's first token in this call); valid [T] or NULL;
 *   scores_override [T] or NULL; forced_idx [forced_n] (FORCED mode);
 *   kv NULL or the layer's cache; n_exec_out [1] device int32;
 *   scores_out [T] fp32 or NULL.
 * `cfg`, `w`, `kv` are host structs holding device pointers.
 */
int qtale_layer_forward(const qtale_layer_config* cfg, const qtale_layer_weights* w, void* x_inout,
                        int T, const int32_t* cu_seqlens, int B, const int32_t* pos0,
                        const uint8_t* valid, const float* scores_override,
                        const int32_t* forced_idx, int forced_n, const qtale_kv_cache* kv,
                        int phase, int32_t* n_exec_out, float* scores_out, void* ws,
                        size_t ws_bytes, void* stream);

typedef struct {
  int n_layers, vocab;
  qtale_layer_config layer; /* shared by all layers; theta is the single global threshold */
} qtale_model_config;

typedef struct {
  const void* embed;                 /* bf16 [vocab, d]                         */
  const qtale_layer_weights* layers; /* HOST array [n_layers]                   */
  const float* final_gamma;          /* [d] fp32                                */
  const void* lm_head;               /* bf16 [vocab, d] or NULL                 */
} qtale_model_weights;

size_t qtale_model_workspace_bytes(const qtale_model_config* cfg, int T_cap, int B_cap,
                                   int n_logit_rows);

/*
 * Prefill of a stack of token-adaptive layers: embedding gather, n_layers x
 * qtale_layer_forward sharing one theta (Sec. 3.4) or, when per_layer_ratio
 * (HOST float [n_layers]) is given, per-layer top-k at those ratios; final
 * RMSNorm and LM head on the requested rows.
 *   ids [T] int32; valid [T] uint8 or NULL (0 = padding token, never executed
 *   at any layer, App. B.2); caches: HOST array [n_layers] of empty per-layer
 *   caches to fill with the executed tokens' keys / values, or NULL; hidden_out [T, d] bf16 (final residual stream);
 *   logits_out fp32 [n_logit_rows, vocab] or NULL; logit_rows [n_logit_rows]
 *   int32 device; per_layer_n_exec [n_layers] int32 device; layer_scores_out
 *   fp32 [n_layers, T] or NULL: every layer's router scores (the input of
 *   qtale_theta_for_ratio when theta is calibrated for a ratio).
 */
int qtale_model_prefill(const qtale_model_config* cfg, const qtale_model_weights* w,
                        const int32_t* ids, int T, const int32_t* cu_seqlens, int B,
                        const uint8_t* valid, const qtale_kv_cache* caches,
                        const float* per_layer_ratio, void* hidden_out, float* logits_out,
                        const int32_t* logit_rows, int n_logit_rows, int32_t* per_layer_n_exec,
                        float* layer_scores_out, void* ws, size_t ws_bytes, void* stream);

size_t qtale_model_decode_workspace_bytes(const qtale_model_config* cfg, int B_cap);

/*
 * One decode step of a stack of token-adaptive layers: every sequence brings one
 * new token, each layer decides per sequence whether that token executes
 * (Eq. 9, one theta for all layers, Sec. 3.4) and only then appends its key /
 * value to that layer's cache (Eq. 3: a bypassed token does not evaluate f_l).
 * Over many steps the cache lengths therefore diverge between sequences and
 * between layers; this is the regime where weight-only quantisation pays
 * (Sec. 2.3: the step is bound by the weight and cache streams).
 *
 *   ids [B] int32 (the new tokens); pos [B] int32 device: position of each new
 *   token in its sequence (rotary position; counts bypassed tokens too), advanced
 *   by one for every valid sequence when the step is done; valid [B] uint8 or
 *   NULL (0 = finished sequence: never executes, position kept); caches: HOST
 *   array [n_layers], each [B, n_kv_heads, cap, head_dim] with its own kv_len;
 *   hidden_out [B, d] bf16; logits_out fp32 [B, vocab] or NULL; next_ids_out [B]
 *   int32 or NULL: greedy choice (largest logit, lowest index among equal ones);
 *   per_layer_n_exec [n_layers] or NULL: sequences executed by each layer in
 *   this step; layer_scores_out fp32 [n_layers, B] or NULL.
 * Top-k selection works as in qtale_layer_forward (ratio of the valid sequences).
 */
int qtale_model_decode_step(const qtale_model_config* cfg, const qtale_model_weights* w,
                            const int32_t* ids, int B, int32_t* pos, const uint8_t* valid,
                            const qtale_kv_cache* caches, void* hidden_out, float* logits_out,
                            int32_t* next_ids_out, int32_t* per_layer_n_exec,
                            float* layer_scores_out, void* ws, size_t ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* QTALE_H_ */

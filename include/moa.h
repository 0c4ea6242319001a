/*
 * moa.h -- C ABI of the Mixture-of-Attentions drafter hot path for one NVIDIA B200 (sm_100a).
 *
 * The library computes the drafter's forward step of "Mixture of Attentions for
 * Speculative Decoding" (arXiv 2410.03804): Layer Self-Attention over each token's
 * stack of per-layer LLM activations followed by a mean over layers (Section 3.1.1),
 * causal / tree-masked self-attention over token embeddings and cross-attention into
 * keys and values derived from the LSA output (Section 3.1.2, Algorithm 1), the LM head
 * with log-softmax and the B most probable tokens (Eq. 1), and the EAGLE-2-style dynamic
 * draft tree with its ancestor mask (Section 2.2). Target Layer Inference (Section 3.2)
 * is off after moa_create (TLI = 0: the drafter predicts the last decoder layer's
 * activation); moa_tli_configure turns it on for the last N <= MOA_MAX_TLI decoder layers.
 *
 * Conventions
 *  - Every pointer is DEVICE memory owned by the caller unless its name ends in _host or
 *    the comment says "host". The library allocates and frees no device memory.
 *  - Matrices are row-major [out, in]; there are no biases. "T" below is the storage type
 *    selected by moa_config.dtype (float or bfloat16); accumulation is always fp32.
 *  - Every call enqueues work on `stream` (a cudaStream_t passed as void*) and returns
 *    without synchronising. Results are valid once the caller has synchronised the stream.
 *  - Arguments are validated on the host before anything is launched; on error a status is
 *    returned and nothing is enqueued. No call throws, aborts or exits.
 *  - All device base pointers must be 16-byte aligned.
 *  - One moa_ctx may be used by one host thread at a time.
 */
#ifndef MOA_H_
#define MOA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MOA_MAX_BATCH 64      /* sequences per call */
#define MOA_MAX_TOPK 16       /* tree breadth B */
#define MOA_MAX_DEPTH 16      /* tree depth D */
#define MOA_MAX_TLI 4         /* LLM decoder layers run by the drafter (Target Layer Inference) */

typedef struct moa_ctx moa_ctx; /* opaque, host side */

typedef enum {
  MOA_OK = 0,
  MOA_ERR_NULL = 1,       /* a required pointer is NULL */
  MOA_ERR_SHAPE = 2,      /* a dimension is out of range or inconsistent */
  MOA_ERR_DTYPE = 3,
  MOA_ERR_ALIGN = 4,      /* a device pointer is not 16-byte aligned */
  MOA_ERR_WORKSPACE = 5,  /* workspace smaller than moa_state_bytes() reports */
  MOA_ERR_CAPACITY = 6,   /* a cache or the node pool would overflow */
  MOA_ERR_STATE = 7,      /* calls out of order (e.g. draft step before moa_tree_begin) */
  MOA_ERR_ARCH = 8,       /* the current device is not compute capability 10.x */
  MOA_ERR_CUDA = 9,       /* a CUDA runtime call failed; see moa_last_cuda_error() */
  MOA_ERR_TIMEOUT = 10,   /* a bounded device-side wait expired */
  MOA_ERR_NONFINITE = 11  /* moa_state_status only: a tree expansion met a log-probability that is not a number (it
                             ranked that candidate last); the drafted tree of that cycle is not to be trusted */
} moa_status;

typedef enum { MOA_F32 = 0, MOA_BF16 = 1 } moa_dtype;

typedef struct {
  int32_t d_model;   /* E: token embedding width = SA and CA width                         */
  int32_t n_stack;   /* S: activations stacked per token (the LLM's layers) fed to LSA     */
  int32_t d_stack;   /* D_in: width of one stacked activation = LSA width                  */
  int32_t vocab;     /* V                                                                  */
  int32_t head_dim;  /* dh, 64 or 128, shared by the three attentions                      */
  int32_t lsa_hq, lsa_hkv, lsa_mlp; /* heads (query / key-value) and MLP width, LSA block  */
  int32_t sa_hq, sa_hkv, sa_mlp;    /* ... self-attention block                            */
  int32_t ca_hq, ca_hkv, ca_mlp;    /* ... cross-attention block                           */
  int32_t max_batch; /* <= MOA_MAX_BATCH                                                   */
  int32_t max_ctx;   /* capacity of the caches, in positions per sequence                  */
  int32_t tree_topk; /* B <= MOA_MAX_TOPK                                                  */
  int32_t tree_depth;/* D <= MOA_MAX_DEPTH: number of drafter forwards per tree            */
  int32_t tree_keep; /* m: nodes kept for verification (the root is one more)              */
  float rms_eps;       /* RMSNorm epsilon, added to the mean square                        */
  float sa_rope_theta; /* rotary base of the self-attention; 0 disables the rotation       */
  int32_t dtype;       /* moa_dtype of weights, activations and caches                     */
} moa_config;

typedef struct { /* device pointers of type T */
  const void *embed, *lm_head, *final_norm;                 /* [V,E] [V,E] [E] */
  const void *lsa_norm1, *lsa_wq, *lsa_wk, *lsa_wv, *lsa_wo; /* [D_in] [Hq*dh,D_in] [Hkv*dh,D_in] x2 [D_in,Hq*dh] */
  const void *lsa_norm2, *lsa_wgate, *lsa_wup, *lsa_wdown;  /* [D_in] [F,D_in] [F,D_in] [D_in,F] */
  const void *sa_norm1, *sa_wq, *sa_wk, *sa_wv, *sa_wo;     /* as above with E in place of D_in */
  const void *sa_norm2, *sa_wgate, *sa_wup, *sa_wdown;
  const void *ca_normq, *ca_normkv;                         /* [E] [D_in] */
  const void *ca_wq, *ca_wk, *ca_wv, *ca_wo;                /* [Hq*dh,E] [Hkv*dh,D_in] x2 [E,Hq*dh] */
  const void *ca_norm2, *ca_wgate, *ca_wup, *ca_wdown;
} moa_weights;

typedef struct {
  void *ca_k, *ca_v;        /* T [max_batch, max_ctx, ca_hkv, head_dim]: cross-attention keys / values   */
  void *sa_k, *sa_v;        /* T [max_batch, max_ctx, sa_hkv, head_dim]: rotated self-attention prefix   */
  int32_t *ca_len, *sa_len; /* device int32 [max_batch]: valid positions; written only by the library    */
  void *tree;               /* device blob of moa_state_bytes().tree_bytes: node pool, frontier, tree K/V, barrier
                               words of the fused kernels. ZERO IT ONCE after allocating it (and again after a call
                               reported MOA_ERR_TIMEOUT through moa_state_status) */
  int32_t *ca_len_host, *sa_len_host; /* HOST int32 [max_batch]: mirrors kept by the library             */
  int32_t step;             /* HOST: draft steps done since moa_tree_begin, -1 before it; library-owned  */
} moa_state;

/* Creates a context for the CURRENT device. Copies config and weight pointers (not the weights).
 * MOA_ERR_ARCH if the device is not compute capability 10.x: there is no fallback path. */
moa_status moa_create(const moa_config *cfg, const moa_weights *w, moa_ctx **out);
void moa_destroy(moa_ctx *ctx);

/* Target Layer Inference (Section 3.2; Algorithm 1, the loop over the last N decoder layers): with TLI = N > 0
 * the drafter's CA block predicts the input of LLM layer L+1-N, and moa_draft_step then runs the N last
 * (frozen) LLM decoder layers on the drafted rows before the LM head. Layer l attends over the LLM's own
 * key/value cache of that layer for the positions already decoded (0 .. sa_len[b]-1, the same positions as the
 * drafter's self-attention prefix) and over the keys/values of the row's drafted ancestors and itself, which
 * the library keeps in moa_state.tree for the duration of one tree and drops afterwards.
 * A layer is a Llama decoder layer: RMSNorm(norm1) -> q,k,v projections -> rotary embedding (half-split
 * pairing, base rope_theta) at the row's position -> grouped-query attention -> W_o, residual ->
 * RMSNorm(norm2) -> SwiGLU MLP, residual. Width E = d_model, head size = moa_config.head_dim.
 *   layers  HOST array [n_layers], layers[0] = the earliest of the N (LLM layer L+1-N); device pointers of T:
 *           norm1 [E], wq [hq*dh,E], wk, wv [hkv*dh,E], wo [E,hq*dh], norm2 [E], wgate, wup [mlp,E], wdown [E,mlp]
 *   k, v    device T [max_batch, max_ctx, hkv, head_dim] per layer: the LLM's cache of that layer (keys already
 *           rotated), owned and filled by the caller, never written by the library
 * Call it before moa_state_bytes: both sizes grow. n_layers = 0 (layers and caches may be NULL) turns it off
 * again.
 * MOA_ERR_SHAPE for n_layers > MOA_MAX_TLI, hq % hkv != 0, mlp % 16 != 0. */
typedef struct {
  int32_t n_layers;  /* N = TLI, 0 .. MOA_MAX_TLI */
  int32_t hq, hkv;   /* query / key-value heads of an LLM layer */
  int32_t mlp;       /* its MLP width */
  float rope_theta;  /* its rotary base; 0 disables the rotation */
} moa_tli_config;
typedef struct {
  const void *norm1, *wq, *wk, *wv, *wo, *norm2, *wgate, *wup, *wdown;
} moa_tli_layer;
typedef struct {
  const void *k[MOA_MAX_TLI], *v[MOA_MAX_TLI];
} moa_tli_caches;
moa_status moa_tli_configure(moa_ctx *ctx, const moa_tli_config *cfg, const moa_tli_layer *layers_host,
                             const moa_tli_caches *caches);

/* Sizes in bytes of moa_state.tree and of the workspace every compute call needs.
 * lsa_chunk_tokens (>= 1) is the number of tokens moa_lsa_forward processes per internal
 * pass; a larger value needs a larger workspace. */
moa_status moa_state_bytes(const moa_ctx *ctx, int32_t lsa_chunk_tokens, size_t *tree_bytes, size_t *workspace_bytes);

const char *moa_status_str(moa_status s);
const char *moa_last_cuda_error(void); /* text of the last CUDA error seen by this thread's calls */

/* Sets the valid length of the caches of sequences 0..batch-1 (device and host copies), e.g. after
 * the caller filled a cache itself or dropped rejected positions. which: 0 = ca, 1 = sa. */
moa_status moa_state_set_len(moa_ctx *ctx, moa_state *st, int32_t which, const int32_t *len_host, int32_t batch, void *stream);

/* Layer Self-Attention with mean, then the cross-attention key/value projection
 * (Section 3.1.1; Algorithm 1: kv <- LSA_layer_with_mean(h), kv <- (kv, kv')).
 *   h_stack    T [sum n_tok, S, D_in], sequences back to back
 *   n_tok_host HOST int32 [batch], tokens of each sequence (may be 0)
 *   kv_out     T [sum n_tok, D_in] or NULL: the LSA output rows
 * Appends n_tok[b] rows W_k n(kv), W_v n(kv) to ca_k / ca_v of sequence b at position ca_len[b]
 * and advances ca_len. MOA_ERR_CAPACITY if ca_len[b] + n_tok[b] > max_ctx. */
moa_status moa_lsa_forward(moa_ctx *ctx, moa_state *st, const void *h_stack, const int32_t *n_tok_host, int32_t batch,
                           void *kv_out, void *ws, size_t ws_bytes, void *stream);

/* Self-attention prefix for prompt / accepted tokens (Section 3.1.2 "Self-Attention"): embeds the
 * tokens, projects keys and values, rotates keys at positions sa_len[b], sa_len[b]+1, ... and
 * appends them to sa_k / sa_v.   tok: device int32 [sum n], n_host: HOST int32 [batch]. */
moa_status moa_sa_append(moa_ctx *ctx, moa_state *st, const int32_t *tok, const int32_t *n_host, int32_t batch,
                         void *ws, size_t ws_bytes, void *stream);

/* The drafter over whole token sequences in one pass (Section 3.1.2: self-attention with its causal mask over
 * prompt + response, cross-attention into the cached LSA keys / values; the parallel pass the paper trains the
 * drafter with, and a way to score many positions at once). Token i of sequence b sits at position sa_len[b] + i:
 * it sees the prefix and tokens 0..i in self-attention; in cross-attention it sees the first ca_limit[row] cached
 * positions (the K-step-bounded mask of the mask figure: the LLM activations available when that token is drafted),
 * or all ca_len[b] of them when ca_limit is NULL (the generation-time setting).
 *   tok        device int32 [sum n], sequences back to back;  n_host  HOST int32 [batch]
 *   ca_limit   device int32 [sum n] or NULL; values in 0 .. ca_len[b], non-decreasing within a sequence
 *   hidden_out T [sum n, E]: the drafter's output activation of every position (the LM head's input)
 * Appends the tokens' self-attention keys / values to sa_k / sa_v and advances sa_len, as moa_sa_append does.
 * Target Layer Inference and the LM head are not applied here. MOA_ERR_CAPACITY if the prefix would overflow. */
moa_status moa_drafter_prefill(moa_ctx *ctx, moa_state *st, const int32_t *tok, const int32_t *n_host, int32_t batch,
                               const int32_t *ca_limit, void *hidden_out, void *ws, size_t ws_bytes, void *stream);

/* The same operation as moa_sa_append for callers that cannot provide a workspace because they cannot
 * allocate device memory at that point: code running between other components that have already handed
 * all device memory to their own pools, or a serving loop in which a cudaMalloc (a device-wide
 * synchronisation) is not allowed. The paper has no counterpart; this is a convenience of the library.
 * Its scratch is a fixed array inside the library (4.5 MiB of device memory, held by every GPU on which
 * the library is loaded, until the process exits), so the call allocates and frees nothing. Inputs and
 * outputs are still the caller's: tok, the caches in st.
 *   Limits: sum(n_host) <= MOA_SA_STATIC_MAX_TOKENS, rows * d_model * sizeof(T) <= 512 KiB (rows = sum(n_host),
 *   on bf16 plus that count rounded up to 16, 32, 64 or 128 for the low-order terms of the activations) and
 *   sum(n_host) * 2 * sa_hkv * head_dim * 4 <= 4 MiB; beyond them MOA_ERR_WORKSPACE is returned, nothing
 *   is launched, and moa_last_cuda_error() holds the limits in words.
 *   The first call on a device looks up the array's device address (a CUDA runtime query made with that
 *   device current); make that first call outside any stream capture.
 *   All calls on one device share the array. It keeps the previous call's contents; nothing in it has
 *   to start at zero, because every element a call reads was written earlier in the same call. Two calls
 *   whose kernels can overlap on the GPU (different streams) race on it: serialise them. */
#define MOA_SA_STATIC_MAX_TOKENS 32
moa_status moa_sa_append_static(moa_ctx *ctx, moa_state *st, const int32_t *tok, const int32_t *n_host, int32_t batch,
                                void *stream);

/* Starts a draft tree per sequence (Section 2.2). root_tok: device int32 [batch], the last verified
 * token; it sits at position sa_len[b]. Sets st->step = 0. */
moa_status moa_tree_begin(moa_ctx *ctx, moa_state *st, const int32_t *root_tok, int32_t batch, void *stream);

/* One drafter forward for the current frontier (Algorithm 1, the SA_layer, CA_layer and LM_head
 * steps of the inner loop; Eq. 1): R = batch rows at step 0 (the roots), batch*B afterwards, row
 * b*B + r = r-th frontier node of sequence b. A row at depth d sits at position sa_len[b] + d and
 * sees the prefix, its ancestors and itself.
 *   topk_id    int32 [R, B]  token ids, by (log-probability descending, id ascending)
 *   topk_logp  float [R, B]  their log-probabilities (logit - logsumexp over the vocabulary)
 *   hidden_out T [R, E] or NULL: the drafter's output activation (input of the LM head; with Target Layer
 *              Inference on, the output of the last LLM decoder layer) */
moa_status moa_draft_step(moa_ctx *ctx, moa_state *st, int32_t batch, int32_t *topk_id, float *topk_logp,
                          void *hidden_out, void *ws, size_t ws_bytes, void *stream);

/* Expands the tree with the rows' top-B lists (Section 2.2): child score = parent score + logp
 * (fp32), children appended in (row, rank) order, next frontier = top B children by (score
 * descending, pool index ascending). Advances st->step. After the D-th expansion it also selects
 * the m best pool nodes (same order), lists them by pool index behind the root (slot 0) and, if the
 * out_* pointers are non-NULL, writes int32 / float [batch, m+1] arrays (parent = slot number,
 * root's parent = -1; unused tail slots hold -1 / 0) and out_n [batch] = 1 + nodes kept. */
moa_status moa_tree_expand(moa_ctx *ctx, moa_state *st, int32_t batch, const int32_t *topk_id, const float *topk_logp,
                           int32_t *out_tok, int32_t *out_parent, int32_t *out_depth, float *out_score, int32_t *out_n,
                           void *stream);

/* Tree Attention mask (Section 2.2, verification with Tree Attention): mask[b][i][j] = 1 iff j == i or
 * j is an ancestor of i. parent: device int32 [batch, n] with parent[0] = -1 and parent[i] < i; an
 * entry < 0 at i > 0 marks an unused slot (its row is zero).
 * packed = 0: uint8 [batch, n, n]; packed = 1: uint64 [batch, n, ceil(n/64)], bit j%64 of word j/64. */
moa_status moa_tree_attn_mask(const int32_t *parent, int32_t batch, int32_t n, void *mask_out, int32_t packed, void *stream);

/* Greedy verification of the kept tree (Section 2.2, step 2: exact matching, everything after the first mismatch
 * is discarded; Algorithm 1, the step that identifies the K' verified tokens and the LLM's next token y').
 * The LLM itself is not part of the library: the caller runs it once over the kept tree with the mask of
 * moa_tree_attn_mask and passes its logits.
 *   tok, parent    device int32 [batch, n]: the kept tree as moa_tree_expand wrote it (slot 0 = root, parent[0] = -1,
 *                  parent[i] < i, parent[i] < 0 at i > 0 = unused slot)
 *   target_logits  device [batch, n, vocab] of logits_dtype (moa_dtype): row (b, i) scores the token FOLLOWING slot i
 *   choice         device int32 [batch, n] out: arg-max of every row, ties to the smallest id (the row of an
 *                  unused slot is read like any other)
 *   acc_slot, acc_tok  device int32 [batch, cap] out: slots and tokens of the accepted path, root first, -1 behind it
 *   acc_len        device int32 [batch] out: 1 + K' (root included), at most cap
 *   next_tok       device int32 [batch] out: the LLM's choice at the last accepted slot = the next cycle's root
 * cap >= 1 bounds the path length (tree_depth + 1 covers every tree of this library). batch * n <= 65535. To carry the accepted
 * tokens into the drafter's self-attention prefix, pass acc_tok's first acc_len entries to moa_sa_append. */
moa_status moa_verify_greedy(const int32_t *tok, const int32_t *parent, int32_t batch, int32_t n, const void *target_logits,
                             int32_t logits_dtype, int32_t vocab, int32_t cap, int32_t *choice, int32_t *acc_slot,
                             int32_t *acc_tok, int32_t *acc_len, int32_t *next_tok, void *stream);

/* Client-server message codec (Section 4.2 "Client-Server" and the message-size table of the appendix).
 * moa_pack_tree: every node of the kept tree as 4 bytes -- the token id in 3 bytes, little endian, and 1 byte for
 * its position in the tree, here the parent's slot number -- so a tree of M nodes is a 4M-byte message. A negative
 * token id is written as ff ff ff, a negative parent (the root, an unused slot) as 255; token ids must be below
 * 2^24 - 1 and slots below 255 (larger values are truncated to their low bits).
 *   tok, parent  device int32 [count]      msg  device bytes [count, 4], 4-byte aligned
 * moa_unpack_tree is the inverse. */
moa_status moa_pack_tree(const int32_t *tok, const int32_t *parent, int64_t count, void *msg, void *stream);
moa_status moa_unpack_tree(const void *msg, int64_t count, int32_t *tok, int32_t *parent, void *stream);
/* 8-bit quantisation of activation rows (the E / E_kv tensors the server sends, Section 4.2). The paper names no
 * scheme; this one is symmetric with one fp32 scale per row: scale = max|x| / 127, code = round-half-even(x * r)
 * in [-127, 127] with r = 127 / max|x| (one fp32 reciprocal per row, one fp32 product per element), decided in fp32; an all-zero row has scale 0 and codes 0. moa_dequantize_rows writes
 * code * scale in `dtype`.
 *   x / out  device [rows, width] of dtype (moa_dtype)    codes  device int8 [rows, width]    scales  device float [rows] */
moa_status moa_quantize_rows(const void *x, int32_t dtype, int64_t rows, int32_t width, int8_t *codes, float *scales,
                             void *stream);
moa_status moa_dequantize_rows(const int8_t *codes, const float *scales, int64_t rows, int32_t width, void *out,
                               int32_t dtype, void *stream);

/* Reads back the device status word kept in st->tree (0 = no device-side problem seen). Synchronises the stream. */
moa_status moa_state_status(moa_ctx *ctx, moa_state *st, void *stream);

/* Measurement hooks (no counterpart in the paper). Between moa_profile_begin and moa_profile_end every
 * launch of the LM-head kernel (the step's dominant HBM stream, Eq. 1) is bracketed by CUDA events on the
 * caller's stream; moa_profile_end synchronises those events and returns their summed duration in
 * milliseconds and the number of launches timed (at most 512 per begin/end pair; later ones are skipped).
 * Do not use inside a stream capture. */
moa_status moa_profile_begin(moa_ctx *ctx);
moa_status moa_profile_end(moa_ctx *ctx, double *ms_total, int32_t *launches);
/* Phase timing of the LAST dense LSA pass (on the bf16 path an LSA pass of more than 256 (token, layer) rows runs as
 * one persistent kernel made of phases separated by grid-wide barriers). Valid when that launch was made between
 * moa_profile_begin and moa_profile_end with the same workspace. us_out[i] = microseconds phase i took on CTA 0
 * including its closing barrier, wait_us_out[i] (may be NULL) = the part of it CTA 0 spent in that barrier,
 * kind_out[i] = its kind (0 GEMM, 1 row norm, 2 residual + norm, 3 layer mean + norm, 4 cache append,
 * 5 layer self-attention).
 * Synchronises the stream. HOST output arrays of `cap` entries. */
moa_status moa_profile_phases(moa_ctx *ctx, const void *ws, size_t ws_bytes, int32_t cap, double *us_out,
                              double *wait_us_out, int32_t *kind_out, int32_t *n_out, void *stream);
/* Kernels launched so far by this host thread through the library. */
int64_t moa_launch_count(void);
/* Stage trace (no counterpart in the paper; only in a library built with -DMOA_TRACE, otherwise both calls return
 * MOA_ERR_STATE and the kernels carry no trace code). Between the two calls every kernel of the library stores one
 * entry when its first thread is released by the completion of the kernel before it in the stream:
 * dev_buf[2 i] = the GPU's nanosecond timer, dev_buf[2 i + 1] = kernel id << 32 | gridDim.x (ids: 1 embedding,
 * 2 GEMM, 3 attention, 4 attention merge, 5 LM-head merge, 6 tree expansion, 7 row norm, 8 residual + norm,
 * 9 SwiGLU, 10 sum + cast, 11 rotary, 12 cache append, 13 layer mean, 0 other). The difference of two consecutive
 * entries is what the earlier kernel cost inside the chain. dev_buf: device uint64 [2 * cap], caller-owned.
 * moa_trace_end synchronises the device and returns the number of entries made (entries beyond cap are dropped). */
moa_status moa_trace_begin(void *dev_buf, int32_t cap);
moa_status moa_trace_end(int32_t *n_out);

#ifdef __cplusplus
}
#endif
#endif /* MOA_H_ */

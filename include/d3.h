/*
 * d3.h -- C ABI of libd3: Position-Aware Depth Decay Decoding (D3) on one GPU.
 *
 * The library runs the autoregressive decode step of a Llama-style decoder in
 * which generated token T_i executes only floor(L * alpha^i) decoder blocks
 * (paper: Abstract; Sec. 3.4).  The dropped blocks form one window that opens
 * at the "flex layer" start id (Appendix, Table "HP description"); a token's
 * hidden state passes through dropped blocks unchanged and the KV-cache
 * entries of dropped blocks are filled per `kv_fill` (Sec. 1 (i); Sec. 3.2).
 *
 * Conventions
 *  - Every function returns D3_OK (0) or a negative D3_E* code; nothing throws,
 *    aborts or traps.  Arguments are validated on the host before any launch;
 *    a call that fails validation changes no state.
 *  - Pointers are HOST pointers unless the name ends in `_dev`.
 *  - The caller allocates and owns all device memory (weights, KV cache,
 *    scratch, logits) and the CUDA stream; the library allocates no device
 *    memory, never copies weights, and borrows the pointers until d3_free.
 *  - Work is enqueued on the stream given to d3_load and is asynchronous;
 *    d3_sync waits for it.  A model is not thread-safe.
 *  - Weights are bf16, row-major [out][in].  Activations, accumulators, the
 *    residual stream and logits are fp32.  The KV cache is bf16.
 */
#ifndef D3_H_
#define D3_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define D3_OK 0
#define D3_EINVAL (-1)    /* bad argument (null, out of range, NaN, unsupported size) */
#define D3_ECAPACITY (-2) /* a sequence would exceed max_seq, or batch > max_batch     */
#define D3_ESTATE (-3)    /* decode on a slot never prefilled; a slot twice in a batch */
#define D3_ECUDA (-4)     /* a CUDA runtime call failed                                */
#define D3_ETIMEOUT (-5)  /* a bounded device-side wait ran out                         */

#define D3_MAX_BATCH 128  /* rows per step (decode rows, or prompt positions per prefill pass) */
#define D3_MAX_LAYERS 128

/* Which blocks a token with retained count n drops. */
#define D3_ANCHOR_START 0 /* [start_id, start_id + L - n), n = max(floor(L alpha^i), start_id):
                             the paper's rule (Appendix, Table "HP description")      */
#define D3_ANCHOR_TAIL 1  /* [n, L): the Early-Exit direction (Sec. 1 (ii))           */

/* What is written to the KV cache of a dropped block for the token (Sec. 3.2). */
#define D3_FILL_NONE 0      /* nothing                                                 */
#define D3_FILL_COPY 1      /* the token's K,V of the block just below the window
                               (zeros when the window opens at block 0)               */
#define D3_FILL_RECOMPUTE 2 /* the dropped block's own norm, W_k, W_v and RoPE applied
                               to the carried hidden state                            */

#define D3_KV_CONTIGUOUS 0  /* K then V, each [L][slot][Hkv][max_seq][head_dim] bf16  */
#define D3_KV_PAGED 1       /* K then V, each a pool [n_pages][Hkv][page_size][head_dim] bf16.
                               A page holds page_size consecutive positions of ONE sequence
                               in ONE block; the library hands pages out on demand (host
                               bookkeeping, a device table [L][slot][max_seq / page_size]) and
                               takes them back in d3_reset_slot.  Depth-aware: with
                               D3_FILL_NONE a (token, block) pair inside the token's dropped
                               window is never written, so no page is taken for a block once
                               the sequence's tokens stop running it (Sec. 3.2 leaves those
                               states undefined; nothing reads them while depth only decays).
                               Page 0 is reserved and zero-filled by d3_load: it stands in
                               for every page never written.                                */

typedef struct d3_config {
  uint32_t struct_size;     /* sizeof(d3_config), checked                              */
  int32_t n_layers;         /* L, 1..D3_MAX_LAYERS                                     */
  int32_t d_model;          /* multiple of 8                                           */
  int32_t n_q_heads;
  int32_t n_kv_heads;       /* divides n_q_heads (grouped-query attention)             */
  int32_t head_dim;         /* 32, 64 or 128                                           */
  int32_t d_ffn;            /* multiple of 8                                           */
  int32_t vocab;
  float rms_eps;
  float rope_base;
  int32_t max_slots;        /* sequences the KV cache holds                            */
  int32_t max_seq;          /* positions per sequence                                  */
  int32_t max_batch;        /* rows per decode step, 1..D3_MAX_BATCH; also the prompt
                               positions one prefill pass takes (the weights are streamed
                               once per pass: 128 gives the shortest time to first token) */
  int32_t start_id;         /* 0..L: first droppable block, 0-based (floor(start * L)) */
  int32_t anchor;           /* D3_ANCHOR_*                                             */
  int32_t kv_fill;          /* D3_FILL_*                                               */
  int32_t kv_layout;        /* D3_KV_CONTIGUOUS or D3_KV_PAGED                         */
  int32_t page_size;        /* PAGED: positions per page, a power of two 16..1024 that
                               divides max_seq; CONTIGUOUS: 0                          */
  int32_t n_pages;          /* PAGED: pages in the pool (page 0 reserved), >= 2;
                               CONTIGUOUS: 0                                           */
} d3_config;

/* DEVICE pointers to bf16 tensors; the per-layer members are HOST arrays of L
 * device pointers.  Every tensor must be 16-byte aligned.
 *   embed, lm_head [vocab][d];  *_norm [d] gains;
 *   wqkv [(Hq + 2 Hkv) * head_dim][d]: rows of W_q, then W_k, then W_v;
 *   wo [d][Hq * head_dim];  w_gate, w_up [f][d];  w_down [d][f].            */
typedef struct d3_weights {
  const void *embed_dev, *lm_head_dev, *final_norm_dev;
  const void *const *attn_norm_dev;
  const void *const *wqkv_dev;
  const void *const *wo_dev;
  const void *const *mlp_norm_dev;
  const void *const *w_gate_dev;
  const void *const *w_up_dev;
  const void *const *w_down_dev;
} d3_weights;

/* What one decode step did (all integers exact).  `n` and `m_per_layer` are
 * caller-provided HOST arrays of `batch` and L entries, or NULL. */
typedef struct d3_step_stats {
  int32_t *n;                /* retained block count of each row, caller order        */
  int32_t *m_per_layer;      /* rows that executed each block                          */
  int64_t rows_layers;       /* sum of m_per_layer == sum of n                         */
  int32_t layers_touched;    /* blocks executed by at least one row                    */
  int32_t kernel_launches;   /* kernels this step enqueued                             */
  int64_t algorithmic_bytes; /* weights of touched blocks + KV read by retained blocks
                                + KV written + LM head + embedding rows + logits out  */
} d3_step_stats;

typedef struct d3_model d3_model;

/* floor(L * alpha^i): blocks retained when generating T_i (Abstract; Sec. 3.4).
 * Host, pure.  alpha in (0, 1], i >= 0, 0 <= L; otherwise D3_EINVAL. */
int32_t d3_depth(int32_t L, double alpha, int64_t i);

/* The batch schedule of one step (Sec. 3.4 + Appendix Table "HP description";
 * batching: Sec. 3.1).  Host, pure; the same integers the device kernel derives.
 * For each of `batch` rows with generation index gen_index[b]: retained count
 * n[b], dropped window [lo[b], hi[b]); perm = rows ordered by n descending,
 * ties by row index; m_per_layer[l] = rows that run block l (always a prefix of
 * perm).  Output arrays are caller-owned; rows_layers / layers_touched may be NULL. */
int32_t d3_schedule(int32_t L, double alpha, int32_t start_id, int32_t anchor, int32_t batch,
                    const int32_t *gen_index, int32_t *n, int32_t *lo, int32_t *hi,
                    int32_t *perm, int32_t *m_per_layer, int64_t *rows_layers,
                    int32_t *layers_touched);

/* Bytes of KV cache and of scratch the caller must allocate for `cfg`
 * (256-byte aligned device buffers). */
int32_t d3_workspace_bytes(const d3_config *cfg, size_t *kv_bytes, size_t *scratch_bytes);

/* Create a model over caller-owned device memory.  Enqueues one set-up kernel
 * (rotary table) on `cuda_stream` (a cudaStream_t passed as void*; NULL = the
 * default stream).  The KV cache is not cleared. */
int32_t d3_load(const d3_config *cfg, const d3_weights *weights, void *kv_dev, void *scratch_dev,
                void *cuda_stream, d3_model **out);

/* Initiation phase (Sec. 3.1; Sec. 4.1: prompts pass through all blocks): run
 * every prompt token through all L blocks, fill the slot's cache from position
 * 0, and write the logits that choose T_0 to logits_dev [vocab] (fp32; may be
 * NULL).  Resets the slot first.  The prompt is taken in passes of up to
 * max_batch consecutive positions: per pass the projections are tensor-core
 * GEMMs over all its positions (each weight read once per pass) and the
 * attention is a causal flash-attention kernel over the cache. */
int32_t d3_prefill(d3_model *m, int32_t slot, const int32_t *tokens, int32_t n_tokens,
                   float *logits_dev);

/* Generation phase, one step (Sec. 3.4).  Row b feeds tokens[b] = T_{i-1} of the
 * sequence in slots[b] at the slot's next cache position, with i = gen_index[b]
 * >= 1 the index of the token being generated; it runs the blocks outside its
 * window and receives logits_dev[b][vocab] (fp32, caller row order), the
 * logits that choose T_i.  alpha in (0, 1] applies to this call.  `stats` may
 * be NULL.  Slots must be distinct and prefilled.
 * tokens_dev (nullable): when given, int32 [batch] DEVICE token ids that
 * replace `tokens` (which may then be NULL), so that a greedy loop can feed
 * d3_argmax's output back without a host round trip. */
int32_t d3_decode_step(d3_model *m, int32_t batch, const int32_t *slots, const int32_t *tokens,
                       const int32_t *gen_index, double alpha, float *logits_dev,
                       d3_step_stats *stats, const int32_t *tokens_dev);

/* The same step with the retained block count of every row given by the caller
 * instead of derived from (alpha, i): depths[b] in 0..L.  Window (anchor,
 * start_id clamp), carried hidden state and KV fill follow the model's
 * configuration exactly as in d3_decode_step, and d3_decode_step(alpha, i) is
 * this call with depths[b] = d3_depth(L, alpha, i_b).  It serves the other
 * schedules the paper discusses (Sec. 3.4, Sec. 4.1 "Comparison Methods"):
 * linear decay between two bounds (d3_depth_linear), the Early-Exit direction
 * (anchor TAIL), per-task tables, or a controller outside the library. */
int32_t d3_decode_step_depths(d3_model *m, int32_t batch, const int32_t *slots, const int32_t *tokens,
                              const int32_t *depths, float *logits_dev, d3_step_stats *stats,
                              const int32_t *tokens_dev);

/* Saturation probe (Sec. 3.2, the experiment behind the saturation table): one
 * generation step at FULL depth for `batch` rows (slots advance and every
 * block's K,V are cached as in a normal step) which, after every block i =
 * 1..L, also runs the block's output through the final norm and the LM head
 * and records what it would predict: block_tokens_dev[b][i-1] (DEVICE int32
 * [batch][L]) = argmax, lowest index on ties; block_conf_dev[b][i-1] (DEVICE
 * fp32 [batch][L], nullable) = the softmax probability of that token.  Column
 * L-1 is the model's own prediction; a row's saturation depth is the first
 * block from which the column agrees with it.  logits_dev [batch][vocab]
 * (fp32) is used as the work buffer and ends up holding the final logits.
 * Costs L LM-head projections ("without regard to cost", as the paper says);
 * always runs as the sequence of kernels. */
int32_t d3_saturation_probe(d3_model *m, int32_t batch, const int32_t *slots, const int32_t *tokens,
                            float *logits_dev, int32_t *block_tokens_dev, float *block_conf_dev);

/* Linear decay of the retained count between an upper and a lower bound (the
 * shape Sec. 3.4 and Sec. 4.1 ascribe to SkipDecode; its constants are not in
 * the paper, so they are arguments): upper at i = 0, lower from i = span on,
 *   n(i) = upper - floor((upper - lower) * min(i, span) / span).
 * Host, pure, integers only.  0 <= lower <= upper, span >= 1, i >= 0; otherwise
 * D3_EINVAL. */
int32_t d3_depth_linear(int32_t upper, int32_t lower, int64_t span, int64_t i);

/* argmax over each row of logits_dev [batch][vocab], lowest index on ties
 * (greedy choice: Sec. 3.2, footnote on lm_head) -> tokens_dev [batch] int32. */
int32_t d3_argmax(d3_model *m, const float *logits_dev, int32_t batch, int32_t *tokens_dev);

/* Diagnostics of the last step, after waiting for the stream:
 * the device kernel's schedule (each array HOST, nullable: n, perm [batch];
 * m_per_layer [L]; counters[0] = rows_layers, counters[1] = layers_touched). */
int32_t d3_read_schedule(d3_model *m, int32_t *n, int32_t *perm, int32_t *m_per_layer,
                         int64_t *counters);
/* the residual stream before the final norm, caller row order, to HOST [batch][d] fp32 */
int32_t d3_read_hidden(d3_model *m, float *hidden);
/* one KV-cache entry to HOST: k, v [Hkv * head_dim] fp32 */
int32_t d3_read_kv(d3_model *m, int32_t layer, int32_t slot, int32_t pos, float *k, float *v);

/* How decode steps execute.  AUTO: a batch of one row runs as a single persistent
 * cooperative kernel when the device and sizes allow it (fill modes NONE and
 * COPY, contiguous or paged cache); everything else runs as a sequence
 * of kernels per block whose projections run on the tensor cores (tcgen05,
 * activations split exactly into three bf16 terms, fp32 accumulate) for depth
 * groups of D3_TENSOR_MIN_ROWS rows or more (FP32-FMA GEMVs where the driver
 * offers no tensor-map encoder).  KERNELS: always the sequence of kernels with
 * FMA GEMVs.  TENSOR: always the sequence of kernels with tensor-core
 * projections (D3_EINVAL without the encoder).  All modes compute the same
 * step (Sec. 3.4). */
#define D3_EXEC_AUTO 0
#define D3_EXEC_KERNELS 1
#define D3_EXEC_TENSOR 2
#define D3_EXEC_FUSED 3    /* like AUTO; D3_EINVAL when the single-kernel step cannot serve the model */
#define D3_TENSOR_MIN_ROWS 1
int32_t d3_set_exec(d3_model *m, int32_t mode);

/* Per-kernel-class device times (measurement aid for Sec. 4.2-style wall-clock
 * accounting).  While enabled, every step records CUDA events around each of its
 * launches on the model's stream and waits for the step to finish, so enabled
 * steps are slower end to end; totals accumulate until read.
 * d3_read_profile: ms[k], launches[k] for k < D3_PROF_KINDS (HOST arrays), then
 * clears the totals.  d3_profile_name(k): a static string. */
#define D3_PROF_KINDS 22   /* 10 kernel classes + 12 figures from inside the single-kernel step */
#define D3_PROF_FUSED0 10
int32_t d3_profile(d3_model *m, int32_t enable);
int32_t d3_read_profile(d3_model *m, float *ms, int32_t *launches);
const char *d3_profile_name(int32_t kind);
/* The raw per-CTA counters behind the "fused:" figures, without clearing them:
 * cycles [ctas][phases] int64 (HOST, room for 192 x 16), counts returned in
 * *ctas and *phases.  Phase order as in d3_profile_name(D3_PROF_FUSED0 + k). */
int32_t d3_read_fused_phases(d3_model *m, int64_t *cycles, int32_t *ctas, int32_t *phases);

/* One batch-1 decode step that allocates nothing.  (The paper has no
 * counterpart: this entry point exists for the sake of the caller, not of the
 * method.)
 *
 * Who needs it: code that may not call cudaMalloc at the point where it wants
 * to decode -- a plugin running inside a host application that owns all device
 * memory and hands out only the tensors it chooses, a real-time or
 * safety-critical loop that forbids allocation after start-up, a process
 * running so close to the memory limit that an allocation could fail.  Such a
 * caller cannot provide the scratch buffer that d3_load asks for.  Here the
 * scratch (schedule, rotary table, activations, attention partials, barrier
 * counters, weight-pointer table) is a fixed array of D3_NOALLOC_SCRATCH_BYTES
 * inside the library image; every GPU that loads the library holds that much
 * memory until the process exits.  No call made here allocates or frees device
 * memory, and no model handle is created.
 *
 * It computes what d3_decode_step computes for a single row (see that call's
 * comment), through the single-kernel step: the sequence in `slot`, whose cache holds
 * `pos` >= 1 tokens, feeds `token` = T_{i-1} with i = gen_index >= 1, writes
 * K,V of the retained blocks (and the fill of the dropped ones) at position
 * `pos` of kv_dev, and writes the logits that choose T_i to logits_dev
 * [vocab] (fp32).  The caller keeps count of `pos` itself.  cfg, weights and
 * kv_dev mean what they mean for d3_load (cfg->max_batch is ignored); kv_fill
 * must be D3_FILL_NONE or D3_FILL_COPY.
 *
 * Limits and errors: D3_ECAPACITY when the scratch one row of `cfg` needs
 * exceeds D3_NOALLOC_SCRATCH_BYTES (roughly: Llama-2-7B/13B shapes with
 * max_seq up to a few thousand fit, the 70B shape does not) or pos >= max_seq;
 * D3_EINVAL for sizes the single-kernel step does not serve (head_dim /
 * grouping other than 128x1, 128x4, 64x1, 32x4; vocab not a multiple of 4),
 * for fill RECOMPUTE and for bad arguments; D3_ECUDA when a runtime call fails.
 *
 * Set-up: the first call on a device looks up the array's device address, and
 * the first call for a new set of model sizes sets the kernel's shared-memory
 * attribute; both with the current device, which must be the one the buffers
 * live on.  Every call also does host-side work that a stream capture would
 * freeze or refuse (it passes pos, token and the depth thresholds by value and
 * may copy the weight-pointer table from host memory), so never call it inside
 * a stream capture.
 *
 * Device-side errors: the call returns once the kernel is enqueued.  A bounded
 * wait that ran out inside the kernel (D3_ETIMEOUT) is recorded in the array;
 * d3_noalloc_status reads it (it allocates nothing either) and should be
 * checked before the logits are trusted.
 *
 * All calls on a GPU share the one array, which keeps the previous call's
 * contents; the entry point re-initialises what must start from zero.  Two
 * calls whose kernels could overlap on the same GPU (different streams,
 * threads or processes sharing a context) race on it: serialise them.  The
 * kernel also needs the whole GPU (one cooperative CTA per SM). */
#define D3_NOALLOC_SCRATCH_BYTES (8u << 20)
int32_t d3_decode_step_noalloc(const d3_config *cfg, const d3_weights *weights, void *kv_dev,
                               int32_t slot, int32_t pos, int32_t token, int32_t gen_index,
                               double alpha, float *logits_dev, void *cuda_stream);
/* Waits for `cuda_stream` and returns the device status of the last
 * d3_decode_step_noalloc on the current device: D3_OK, D3_ETIMEOUT, or
 * D3_ECUDA when a runtime call fails.  Copies one int32 out of the built-in
 * array into a host local; allocates nothing.  (No counterpart in the paper.) */
int32_t d3_noalloc_status(void *cuda_stream);

int32_t d3_slot_pos(const d3_model *m, int32_t slot); /* tokens cached; D3_ESTATE if never prefilled */
/* PAGED layout: pages handed out at the moment (the reserved page not counted);
 * D3_EINVAL for a contiguous model.  Host bookkeeping only. */
int32_t d3_kv_pages_used(const d3_model *m);
int32_t d3_reset_slot(d3_model *m, int32_t slot);
/* Wait for the stream; returns a deferred device status (D3_ETIMEOUT) once and clears it. */
int32_t d3_sync(d3_model *m);

/* Window policy between steps (Appendix, Table "HP description": `start` differs per
 * task, Sec. 4.1 "Hyperparameter Settings"; anchor and fill as in d3_config).  Takes
 * effect from the next call on; sequences in flight keep their caches.  Host only. */
int32_t d3_set_policy(d3_model *m, int32_t start_id, int32_t anchor, int32_t kv_fill);

/* Failure detection.  Every device-side wait of the library (mbarrier, ring slot,
 * grid barrier) gives up after `ns` nanoseconds (default 2e9): the kernel raises
 * D3_ETIMEOUT in a status word that d3_sync returns, stops issuing copies, lets the
 * copies in flight land and runs to its end; nothing traps and the context stays
 * usable.  The outputs and the cache entries of such a step are undefined: reset
 * and prefill the slots it touched.  ns >= 1. */
int32_t d3_set_wait_ns(d3_model *m, uint64_t ns);
/* Drill for the above: the next single-kernel step (one row) is told to expect one
 * arrival more at its first grid barrier than there are CTAs, so that wait can only
 * end by its time limit -- a wait nobody satisfies, made on the host.  The step
 * then ends with D3_ETIMEOUT as described.  D3_EINVAL when the model has no
 * single-kernel step. */
int32_t d3_stall_next_step(d3_model *m);
void d3_free(d3_model *m);    /* host bookkeeping only */
const char *d3_strerror(int32_t code);

#ifdef __cplusplus
}
#endif
#endif /* D3_H_ */

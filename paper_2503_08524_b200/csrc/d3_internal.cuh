// Internal declarations shared by the kernels and the C ABI of libd3.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <map>

#include "d3.h"

namespace d3 {

typedef __nv_bfloat16 bf16;

// One step's caller arguments, passed to the schedule kernel by value (kernel
// parameters are copied at launch, so the host arrays may be reused at once).
struct StepArgs {
  int32_t B, L, start_id, anchor;
  int32_t slot[D3_MAX_BATCH];
  int32_t tok[D3_MAX_BATCH];
  int32_t gi[D3_MAX_BATCH];   // generation index i of the row (0 = full depth)
  int32_t pos[D3_MAX_BATCH];  // cache position the row's token is written to
  // thr[n] = smallest i with floor(L alpha^i) < n, for n = 1..L (thr[0] unused)
  int32_t thr[D3_MAX_LAYERS + 1];
  const int32_t *tok_dev;     // nullable: device token ids that replace tok[]
};

// The schedule of the running step in device memory (written by the schedule
// kernel, read by every other kernel).  "_s" arrays are in sorted row order.
struct DevSched {
  int32_t B, L;
  int32_t n[D3_MAX_BATCH];     // caller order
  int32_t perm[D3_MAX_BATCH];  // sorted index -> caller row
  int32_t slot_s[D3_MAX_BATCH], pos_s[D3_MAX_BATCH], tok_s[D3_MAX_BATCH];
  int32_t lo_s[D3_MAX_BATCH], hi_s[D3_MAX_BATCH];
  int32_t m[D3_MAX_LAYERS];    // rows that run block l = a prefix of the sorted order
  long long rows_layers;
  int32_t layers_touched;
  int32_t status;              // 0, or a D3_E* code detected on the device
};

// Which rows of the sorted batch a kernel works on.
enum RowMode {
  ROWS_PREFIX = 0,  // [0, m[layer])        rows that run the block
  ROWS_SUFFIX = 1,  // [m[layer], B)        rows that drop it (recompute fill)
  ROWS_ALL = 2,     // [0, B)
  ROWS_LAST = 3     // [B-1, B)             prefill: only the last position needs logits
};

enum Epilogue {
  EPI_STORE = 0,   // out[row][r] = y
  EPI_RESID = 1,   // out[row][r] += y          (residual stream)
  EPI_SWIGLU = 2,  // out[row][r] = silu(W y) * (W2 y)
  EPI_LOGITS = 3   // out[caller row][r] = y    (un-permuted)
};

// Opaque storage of one TMA tensor map (encoded on the host by the driver).
struct alignas(64) TMap {
  uint64_t w[16];
};

// Where a kernel also leaves its fp32 result as the three-term bf16 operand of the tensor-core
// projection that follows (rows j, np + j, 2 np + j of [3 np][K]); p == nullptr: nowhere.
struct OpndOut { bf16 *p; int np; };
// The order in which an attention launch takes the rows (longest context first, so that the short
// ones fill the tail); given == 0: as they come.
struct RowOrder { unsigned char r[D3_MAX_BATCH]; int given; };

struct GemvArgs {
  const bf16 *W, *W2;   // [R][K] row-major (W2: second matrix of EPI_SWIGLU)
  const TMap *tmap_w, *tmap_w2;  // host pointers, nullable: tensor maps of W and W2 (tensor-core path)
  int R, K;
  const float *act;     // [rows][act_stride]
  int act_stride;
  const bf16 *gain;     // nullable: RMSNorm gain fused on the activation
  float eps;
  float *out;
  int out_stride;
  int out_col0;         // column offset added to the output row index r
  // tensor-core path: `clear` (nullable) is a region of `clear_floats` floats (a multiple of 4, 16-byte
  // aligned) that a LATER kernel wants zeroed and nothing reads any more: the projection's idle
  // warps clear it while the weights stream.  `out_is_zero`: an earlier kernel did that for this
  // projection's output rows, so the pre-pass of a split-K store need not.
  float *clear;
  size_t clear_floats;
  int out_is_zero;
  // tensor-core path, operand hand-over between two projections of the same rows (<= 64):
  // `operand_out`: the SiLU * mul epilogue also writes its result as the three-term bf16 operand of
  // the projection that follows; `operand_in`: that operand is there, no pre-pass runs.
  int operand_out, operand_in;
  int short_chain_row0; // tensor-core path: rows r >= this are summed in short slices (0 = off)
  const DevSched *sched;
  int layer;
  int row_mode;
};

struct Dims {
  int L, d, Hq, Hkv, dh, f, V, max_slots, max_seq, qkv_rows;
  // paged KV cache (page_size == 0: contiguous)
  int page_size, page_shift, blocks_per_seq;
  const int32_t *block_table;   // device [L][max_slots][blocks_per_seq] page ids; 0 = never written
};

// Element offset of cache entry (layer, slot, kv head h, position pos) in the K (or V) array.
__host__ __device__ __forceinline__ size_t kv_offset(const Dims &dm, const int32_t *table, int layer, int slot,
                                                     int h, int pos) {
  if (dm.page_size == 0)
    return ((((size_t)layer * dm.max_slots + slot) * dm.Hkv + h) * dm.max_seq + pos) * (size_t)dm.dh;
  const int page = table[((size_t)layer * dm.max_slots + slot) * dm.blocks_per_seq + (pos >> dm.page_shift)];
  return (((size_t)page * dm.Hkv + h) * dm.page_size + (pos & (dm.page_size - 1))) * (size_t)dm.dh;
}

// device table of one block's weight pointers (fused step kernel)
struct LayerPtrs {
  const bf16 *attn_norm, *wqkv, *wo, *mlp_norm, *w_gate, *w_up, *w_down;
};

static constexpr int kFusedMaxCtas = 192;
static constexpr int kFusedSyncBytes = 1024;   // grid-barrier counter + per-stream arrival counters
static constexpr int kFusedPhases = 10;        // timed phases of the fused kernel (+ ring wait)

// parameters of the fused batch-1 step kernel (passed by value)
struct FusedParams {
  int32_t slot, tok, gi, pos;
  const int32_t *tok_dev;
  int32_t thr[D3_MAX_LAYERS + 1];
  int32_t L, start_id, anchor, kv_fill;
  Dims dm;
  float eps;
  const LayerPtrs *layers;
  const bf16 *embed, *lm_head, *final_norm;
  bf16 *Kc, *Vc;
  const float2 *rope;
  DevSched *sched;
  unsigned *bar_counter;        // grid barrier
  unsigned *stream_count;       // arrivals per attention stream
  long long *phase_cycles;      // nullable: [cta][kFusedPhases] cycles per phase
  float *x, *qkv, *u, *part, *attn_out;
  float *logits;
  int32_t n_stages, act_floats;
  uint32_t l2_window;           // ring stages the L2 prefetcher may run ahead (0 = off)
  unsigned long long wait_ns;   // bound of every device-side wait
  uint32_t barrier_extra;       // arrivals the FIRST grid barrier expects beyond the CTA count (0 in normal
                                // use; 1 = that barrier can only end by its time limit: time-out drill)
};

// Waits for copies already in flight are not waits for another party: they always end, so
// their bound never drops below this floor however short the configured limit is.
static constexpr unsigned long long kDrainFloorNs = 1000000ull;

// Host state of the tensor-core projection path.
struct TcContext {
  bool ok;                              // the driver's tensor-map encoder is there and the kernels are set up
  bf16 *act_split;                      // device: activations as bf16 hi, mid, lo rows, [3 NP][K]
  bf16 *act_split2;                     // a second one, written by a projection's epilogue for the next
  bool handed_over;                     // the last launch wrote act_split2 (GemvArgs.operand_out honoured)
  size_t act_bytes;
  std::map<uint64_t, TMap> act_maps;    // tensor maps of act_split, keyed by (NP, K)
  int sm_count;
  unsigned long long wait_ns;           // bound of every device-side wait
};

// Byte offsets of the regions of the caller's scratch buffer.
struct Layout {
  size_t sched, rope, x, qkv, attn_out, part_o, part_ml, u, layer_tab, bar, phase, part_fused, act_split,
      act_split2, act_split_bytes, block_table, total;
  int max_splits;
};

// Programmatic dependent launch: every kernel of the step sequence is launched
// with the stream-serialization attribute, so that it may become resident while
// its predecessor still runs.  Every thread calls pdl_wait() before it touches
// anything another kernel of the stream writes or reads (it returns once all
// earlier kernels have completed and their writes are visible); what precedes
// the call, and a thread that never makes it, may only touch kernel parameters,
// constant weights and the CTA's own shared / tensor memory.  Because no CTA
// exits before one of its threads has returned from the wait, completion of a
// kernel implies completion of all its predecessors.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// v as the three bf16 terms hi + mid + lo of row j of a projection operand [3 np][K]
__device__ __forceinline__ void opnd_store(const OpndOut &o, int j, size_t K, size_t col, float v) {
  const bf16 h = __float2bfloat16_rn(v);
  const float r1 = v - __bfloat162float(h);     // exact
  const bf16 md = __float2bfloat16_rn(r1);
  const bf16 lw = __float2bfloat16_rn(r1 - __bfloat162float(md));
  bf16 *p = o.p + (size_t)j * K + col;
  p[0] = h; p[(size_t)o.np * K] = md; p[(size_t)2 * o.np * K] = lw;
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args... args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

Layout make_layout(const d3_config &c);
bool config_ok(const d3_config *c);
// thr[n] = smallest i with floor(L alpha^i) < n, n = 1..L (INT32_MAX if none); thr[0] = 0
void thresholds(int32_t L, double alpha, int32_t *thr);

// launchers (each enqueues on `st`; returns the number of kernels launched)
int launch_rope_table(float2 *table, int max_seq, int dh, float base, cudaStream_t st);
int launch_rope_rows(float2 *table, int pos0, int n_pos, int dh, float base, cudaStream_t st);
int launch_schedule_embed(const StepArgs &a, DevSched *s, const bf16 *E, float *x, int d,
                          cudaStream_t st);
int launch_gemv(const GemvArgs &g, int epi, int m_rows, cudaStream_t st);
int launch_rope_append(float *qkv, const float2 *rope, bf16 *Kc, bf16 *Vc, const DevSched *s,
                       int layer, int row_mode, int kv_only, int m_rows, const Dims &dm,
                       cudaStream_t st);
int launch_attention(const float *qkv, const bf16 *Kc, const bf16 *Vc, const DevSched *s, int layer,
                     int m_rows, int split_len, int n_splits, int max_splits, float *part_o,
                     float *part_ml, float *attn_out, OpndOut opnd, const Dims &dm, cudaStream_t st,
                     const RowOrder *order = nullptr);
int init_attention_mma();
int init_attention_prefill();
int launch_attention_prefill(const float *qkv, const bf16 *Kc, const bf16 *Vc, int layer, int slot, int t0, int B,
                             float *attn_out, const Dims &dm, cudaStream_t st);
int launch_attention_partial_mma(const float *qkv, const bf16 *Kc, const bf16 *Vc, const DevSched *s, int layer,
                                 int m_rows, int split_len, int n_splits, int max_splits, float *part_o,
                                 float *part_ml, float *attn_out, OpndOut opnd, const Dims &dm, cudaStream_t st,
                                 const RowOrder *order = nullptr);
int launch_fill_copy(bf16 *Kc, bf16 *Vc, const DevSched *s, int B, const Dims &dm, cudaStream_t st);
int launch_argmax(const float *logits, int B, int V, int32_t *out, cudaStream_t st);
int launch_argmax_conf(const float *logits, int B, int V, int32_t *tok, float *conf, int stride, int col,
                       cudaStream_t st);
// paged KV cache: entries of the device block table that change before a step
struct TableUpdate {
  static constexpr int kMax = 256;
  int32_t n;
  int32_t index[kMax], page[kMax];
};
int launch_table_update(int32_t *table, const TableUpdate &u, cudaStream_t st);
int init_kernel_attributes();
// tensor-core projections: 0 when the path is usable on this device / driver
int tc_init();
bool tc_weight_map(TMap *out, const bf16 *W, int R, int K);
// pre-pass + GEMM for m_rows rows; returns kernels launched, 0 = not served (use launch_gemv)
int launch_gemm_tc(TcContext &tc, const GemvArgs &g, int epi, int m_rows, cudaStream_t st);
// fused batch-1 step: returns 1 and the launch plan when the kernel serves `c` on this device
int fused_plan(const d3_config &c, int *grid, int *n_stages, int *act_floats, size_t *smem, void **func);
int launch_fused_step(void *func, int grid, size_t smem, FusedParams &fp, cudaStream_t st);
uint32_t fused_l2_window();   // look-ahead of the L2 prefetcher in ring stages (D3_FUSED_L2_WINDOW overrides)

}  // namespace d3

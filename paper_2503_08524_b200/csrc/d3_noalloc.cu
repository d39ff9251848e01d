// d3_decode_step_noalloc: one batch-1 decode step for callers that cannot
// allocate device memory.  Its working memory is a fixed array that lives in
// the library image on every GPU that loads the library.
#include <string.h>

#include "d3_internal.cuh"

namespace d3 {
namespace {

// The step's scratch (schedule, rotary table, activations, attention partials,
// barrier counters, weight-pointer table).  File-scope device memory: allocated
// by the CUDA loader with the module, released when the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[D3_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
// device address of g_noalloc_scratch per device ordinal (nullptr = not set up yet)
static void *g_scratch_addr[kMaxDevices];

// What the array of a device already holds from the previous call, so that a call with the same
// model re-uploads nothing: the launch plan of the kernel for the sizes last seen, and the
// weight-pointer table last copied.  Every call on the device goes through the entry point below,
// which keeps this record in step with the array.
struct DeviceState {
  bool plan_ok;
  int32_t sig[8];                 // sizes the plan was made for
  int grid, stages, act;
  size_t smem;
  void *func;
  int tab_layers;                 // 0 = no table uploaded yet
  size_t tab_offset;              // where in the array that table sits
  LayerPtrs tab[D3_MAX_LAYERS];
};
static DeviceState g_state[kMaxDevices];
static size_t g_last_sched_offset[kMaxDevices];   // where the last step's schedule sits in the array

// In host code `g_noalloc_scratch` is only a handle of the symbol, not an
// address the GPU understands: the address comes from cudaGetSymbolAddress,
// asked once per device with that device current.
static int32_t scratch_for_current_device(char **out, int *dev_out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return D3_ECUDA;
  *dev_out = dev;
  if (!g_scratch_addr[dev]) {
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return D3_ECUDA;
    }
    g_scratch_addr[dev] = ptr;
  }
  *out = static_cast<char *>(g_scratch_addr[dev]);
  return D3_OK;
}

}  // namespace
}  // namespace d3

using namespace d3;

extern "C" int32_t d3_decode_step_noalloc(const d3_config *cfg, const d3_weights *w, void *kv_dev,
                                          int32_t slot, int32_t pos, int32_t token, int32_t gen_index,
                                          double alpha, float *logits_dev, void *cuda_stream) {
  if (!cfg || !w || !kv_dev || !logits_dev) return D3_EINVAL;
  d3_config c1 = *cfg;
  c1.max_batch = 1;   // the caller's value is ignored: this entry point runs one row
  if (!config_ok(&c1)) return D3_EINVAL;
  if (cfg->kv_layout != D3_KV_CONTIGUOUS) return D3_EINVAL;   // the page table lives in a model handle
  if (!w->embed_dev || !w->lm_head_dev || !w->final_norm_dev || !w->attn_norm_dev || !w->wqkv_dev ||
      !w->wo_dev || !w->mlp_norm_dev || !w->w_gate_dev || !w->w_up_dev || !w->w_down_dev)
    return D3_EINVAL;
  if (!(alpha > 0.0 && alpha <= 1.0) || gen_index < 1) return D3_EINVAL;
  if (slot < 0 || slot >= cfg->max_slots || token < 0 || token >= cfg->vocab || pos < 1) return D3_EINVAL;
  if (pos >= cfg->max_seq) return D3_ECAPACITY;
  if (cfg->kv_fill == D3_FILL_RECOMPUTE) return D3_EINVAL;   // only fills NONE and COPY
  auto misaligned = [](const void *p, size_t a) { return p == nullptr || ((uintptr_t)p % a) != 0; };
  if (misaligned(kv_dev, 256) || misaligned(w->embed_dev, 16) || misaligned(w->lm_head_dev, 16) ||
      misaligned(w->final_norm_dev, 16))
    return D3_EINVAL;
  const int L = cfg->n_layers;
  for (int l = 0; l < L; ++l)
    if (misaligned(w->attn_norm_dev[l], 16) || misaligned(w->wqkv_dev[l], 16) ||
        misaligned(w->wo_dev[l], 16) || misaligned(w->mlp_norm_dev[l], 16) ||
        misaligned(w->w_gate_dev[l], 16) || misaligned(w->w_up_dev[l], 16) ||
        misaligned(w->w_down_dev[l], 16))
      return D3_EINVAL;

  // the working set of one row must fit the fixed array
  const Layout lay = make_layout(c1);
  if (lay.total > (size_t)D3_NOALLOC_SCRATCH_BYTES) return D3_ECAPACITY;

  char *scratch = nullptr;
  int dev = 0;
  int32_t rc = scratch_for_current_device(&scratch, &dev);
  if (rc != D3_OK) return rc;
  DeviceState &ds = g_state[dev];
  // launch plan (shared-memory attribute, occupancy check): made when the sizes change
  const int32_t sig[8] = {cfg->d_model, cfg->d_ffn, cfg->n_q_heads, cfg->n_kv_heads,
                          cfg->head_dim, cfg->vocab, cfg->n_layers, 0};
  if (!ds.plan_ok || memcmp(ds.sig, sig, sizeof(sig)) != 0) {
    ds.plan_ok = false;
    if (!fused_plan(c1, &ds.grid, &ds.stages, &ds.act, &ds.smem, &ds.func))
      return D3_EINVAL;   // sizes the kernel does not serve
    memcpy(ds.sig, sig, sizeof(sig));
    ds.plan_ok = true;
  }

  cudaStream_t st = (cudaStream_t)cuda_stream;
  // The array keeps what the last call left.  Reset the schedule with its status word; write the
  // one rotary row this step reads (the row of `pos`); upload the weight-pointer table unless the
  // array already holds exactly this table (the region's offset depends on max_seq, so a change
  // of layout counts as a change of table).
  if (cudaMemsetAsync(scratch + lay.sched, 0, sizeof(DevSched), st) != cudaSuccess) return D3_ECUDA;
  launch_rope_rows(reinterpret_cast<float2 *>(scratch + lay.rope), pos, 1, cfg->head_dim, cfg->rope_base, st);
  LayerPtrs tab[D3_MAX_LAYERS];
  memset(tab, 0, sizeof(tab));
  for (int l = 0; l < L; ++l)
    tab[l] = LayerPtrs{(const bf16 *)w->attn_norm_dev[l], (const bf16 *)w->wqkv_dev[l],
                       (const bf16 *)w->wo_dev[l],        (const bf16 *)w->mlp_norm_dev[l],
                       (const bf16 *)w->w_gate_dev[l],    (const bf16 *)w->w_up_dev[l],
                       (const bf16 *)w->w_down_dev[l]};
  if (ds.tab_layers != L || ds.tab_offset != lay.layer_tab ||
      memcmp(ds.tab, tab, sizeof(LayerPtrs) * L) != 0) {
    ds.tab_layers = 0;
    // pageable source: the runtime stages it before returning, so `tab` may go out of scope
    if (cudaMemcpyAsync(scratch + lay.layer_tab, tab, sizeof(LayerPtrs) * L, cudaMemcpyHostToDevice, st) !=
        cudaSuccess)
      return D3_ECUDA;
    memcpy(ds.tab, tab, sizeof(LayerPtrs) * L);
    ds.tab_offset = lay.layer_tab;
    ds.tab_layers = L;
  }
  const int grid = ds.grid, stages = ds.stages, act = ds.act;
  const size_t smem = ds.smem;
  void *func = ds.func;

  FusedParams fp;
  memset(&fp, 0, sizeof(fp));
  fp.slot = slot; fp.tok = token; fp.gi = gen_index; fp.pos = pos; fp.tok_dev = nullptr;
  thresholds(L, alpha, fp.thr);
  fp.L = L; fp.start_id = cfg->start_id; fp.anchor = cfg->anchor; fp.kv_fill = cfg->kv_fill;
  fp.dm = Dims{cfg->n_layers, cfg->d_model, cfg->n_q_heads, cfg->n_kv_heads, cfg->head_dim, cfg->d_ffn,
               cfg->vocab, cfg->max_slots, cfg->max_seq,
               (cfg->n_q_heads + 2 * cfg->n_kv_heads) * cfg->head_dim};
  fp.eps = cfg->rms_eps;
  fp.layers = reinterpret_cast<const LayerPtrs *>(scratch + lay.layer_tab);
  fp.embed = (const bf16 *)w->embed_dev;
  fp.lm_head = (const bf16 *)w->lm_head_dev;
  fp.final_norm = (const bf16 *)w->final_norm_dev;
  const size_t kv_half = (size_t)L * cfg->max_slots * cfg->n_kv_heads * cfg->max_seq * cfg->head_dim;
  fp.Kc = (bf16 *)kv_dev;
  fp.Vc = fp.Kc + kv_half;
  fp.rope = reinterpret_cast<const float2 *>(scratch + lay.rope);
  fp.sched = reinterpret_cast<DevSched *>(scratch + lay.sched);
  fp.bar_counter = reinterpret_cast<unsigned *>(scratch + lay.bar);   // zeroed by the launcher
  fp.stream_count = fp.bar_counter + 16;
  fp.phase_cycles = nullptr;
  fp.x = reinterpret_cast<float *>(scratch + lay.x);
  fp.qkv = reinterpret_cast<float *>(scratch + lay.qkv);
  fp.u = reinterpret_cast<float *>(scratch + lay.u);
  fp.attn_out = reinterpret_cast<float *>(scratch + lay.attn_out);
  fp.part = reinterpret_cast<float *>(scratch + lay.part_fused);
  fp.logits = logits_dev;
  fp.n_stages = stages; fp.act_floats = act;
  fp.l2_window = fused_l2_window();
  fp.wait_ns = 2000000000ull;
  fp.barrier_extra = 0;
  g_last_sched_offset[dev] = lay.sched;
  if (launch_fused_step(func, grid, smem, fp, st) != 1) return D3_ECUDA;
  return cudaGetLastError() == cudaSuccess ? D3_OK : D3_ECUDA;
}

extern "C" int32_t d3_noalloc_status(void *cuda_stream) {
  char *scratch = nullptr;
  int dev = 0;
  int32_t rc = scratch_for_current_device(&scratch, &dev);
  if (rc != D3_OK) return rc;
  if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return D3_ECUDA;
  // the status word of the schedule the last step on this device used (a host local receives it)
  int32_t status = 0;
  const DevSched *sched = reinterpret_cast<const DevSched *>(scratch + g_last_sched_offset[dev]);
  if (cudaMemcpy(&status, &sched->status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return D3_ECUDA;
  return status;
}

// C ABI of libd3: argument validation, host bookkeeping, the host copy of the
// depth schedule, and the per-step launch sequence.
#include <algorithm>
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <map>
#include <new>
#include <vector>

#include "d3_internal.cuh"

namespace d3 {

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

Layout make_layout(const d3_config &c) {
  Layout y;
  const size_t B = (size_t)c.max_batch;
  const size_t qkv_rows = (size_t)(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
  y.max_splits = 32;
  size_t off = 0;
  y.sched = off;    off = align_up(off + sizeof(DevSched), 256);
  y.rope = off;     off = align_up(off + (size_t)c.max_seq * (c.head_dim / 2) * sizeof(float2), 256);
  y.x = off;        off = align_up(off + B * c.d_model * 4, 256);
  y.qkv = off;      off = align_up(off + B * qkv_rows * 4, 256);
  y.attn_out = off; off = align_up(off + B * c.n_q_heads * c.head_dim * 4, 256);
  y.part_o = off;   off = align_up(off + B * c.n_q_heads * y.max_splits * c.head_dim * 4, 256);
  y.part_ml = off;  off = align_up(off + B * c.n_q_heads * y.max_splits * 2 * 4, 256);
  y.u = off;        off = align_up(off + B * c.d_ffn * 4, 256);
  y.layer_tab = off; off = align_up(off + (size_t)c.n_layers * sizeof(LayerPtrs), 256);
  y.bar = off;      off = align_up(off + kFusedSyncBytes, 256);
  y.phase = off;    off = align_up(off + (size_t)kFusedMaxCtas * kFusedPhases * 8, 256);
  y.part_fused = off;
  off = align_up(off + (size_t)c.n_q_heads * kFusedMaxCtas * (c.head_dim + 2) * 4, 256);
  // tensor-core operand: bf16 hi, mid and lo rows of the widest activation
  size_t kmax = (size_t)c.d_model;
  if ((size_t)c.n_q_heads * c.head_dim > kmax) kmax = (size_t)c.n_q_heads * c.head_dim;
  if ((size_t)c.d_ffn > kmax) kmax = (size_t)c.d_ffn;
  y.act_split = off = align_up(off, 1024);
  y.act_split_bytes = (3 * ((B + 7) / 8 * 8) + 8) * kmax * sizeof(bf16);
  y.act_split2 = off = align_up(off + y.act_split_bytes, 1024);
  off = align_up(off + y.act_split_bytes, 256);
  y.block_table = off;
  if (c.kv_layout == D3_KV_PAGED)
    off = align_up(off + (size_t)c.n_layers * c.max_slots * (c.max_seq / c.page_size) * sizeof(int32_t), 256);
  y.total = off;
  return y;
}

bool config_ok(const d3_config *c) {
  if (!c || c->struct_size != sizeof(d3_config)) return false;
  if (c->n_layers < 1 || c->n_layers > D3_MAX_LAYERS) return false;
  if (c->d_model < 8 || c->d_model % 8) return false;
  if (c->d_ffn < 8 || c->d_ffn % 8) return false;
  if (c->n_q_heads < 1 || c->n_kv_heads < 1 || c->n_q_heads % c->n_kv_heads) return false;
  if (c->head_dim != 32 && c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->vocab < 1 || c->max_slots < 1 || c->max_seq < 1) return false;
  if (c->max_batch < 1 || c->max_batch > D3_MAX_BATCH) return false;
  if (!(c->rms_eps >= 0.f) || !(c->rope_base > 0.f)) return false;
  if (c->start_id < 0 || c->start_id > c->n_layers) return false;
  if (c->anchor != D3_ANCHOR_START && c->anchor != D3_ANCHOR_TAIL) return false;
  if (c->kv_fill < D3_FILL_NONE || c->kv_fill > D3_FILL_RECOMPUTE) return false;
  if (c->kv_layout == D3_KV_CONTIGUOUS) {
    if (c->page_size != 0 || c->n_pages != 0) return false;
  } else if (c->kv_layout == D3_KV_PAGED) {
    const int ps = c->page_size;
    if (ps < 16 || ps > 1024 || (ps & (ps - 1)) || c->max_seq % ps || c->n_pages < 2) return false;
  } else {
    return false;
  }
  return true;
}

static bool alpha_ok(double a) { return a > 0.0 && a <= 1.0; }  // false for NaN

static int32_t depth_host(int32_t L, double alpha, int64_t i) {
  return (int32_t)floor((double)L * pow(alpha, (double)i));
}

// thr[n] = smallest i with floor(L alpha^i) < n (n = 1..L); INT32_MAX if none.
void thresholds(int32_t L, double alpha, int32_t *thr) {
  thr[0] = 0;
  const int64_t imax = 0x7ffffffe;
  for (int n = 1; n <= L; ++n) {
    if (depth_host(L, alpha, imax) >= n) { thr[n] = 0x7fffffff; continue; }
    int64_t lo = 0, hi = imax;  // depth(lo) >= n, depth(hi) < n
    while (hi - lo > 1) {
      int64_t mid = lo + (hi - lo) / 2;
      if (depth_host(L, alpha, mid) >= n) lo = mid; else hi = mid;
    }
    thr[n] = (int32_t)hi;
  }
}

}  // namespace d3

using namespace d3;

struct d3_model {
  d3_config cfg;
  Dims dm;
  Layout lay;
  cudaStream_t stream;
  const bf16 *embed, *lm_head, *final_norm;
  std::vector<const bf16 *> attn_norm, wqkv, wo, mlp_norm, w_gate, w_up, w_down;
  bf16 *Kc, *Vc;
  char *scratch;
  std::vector<int32_t> pos;  // tokens cached per slot; -1 = never prefilled
  std::map<uint64_t, std::vector<int32_t>> thr_cache;
  // last step (diagnostics)
  int32_t last_B;
  int32_t last_perm[D3_MAX_BATCH];
  int64_t layer_bytes, head_bytes;
  // per-kernel-class timing (d3_profile)
  bool prof_on;
  std::vector<cudaEvent_t> prof_events;   // pool, two per recorded launch
  std::vector<int> prof_kind;             // kind of each recorded pair of the running step
  float prof_ms[10];
  int32_t prof_n[10];
  // fused batch-1 step kernel
  int32_t exec_mode;
  int fused_ok, fused_grid, fused_stages, fused_act;
  size_t fused_smem;
  void *fused_func;
  std::vector<LayerPtrs> layer_tab_host;
  unsigned long long wait_ns;   // bound of every device-side wait (d3_set_wait_ns)
  int stall_next;               // time-out drill: the next single-kernel step cannot pass its first barrier
  // tensor-core projections: tensor maps of the weight matrices (entry valid when tm_ok)
  TcContext tc;
  std::vector<TMap> tm_qkv, tm_kv, tm_o, tm_gate, tm_up, tm_down;
  TMap tm_head;
  bool tm_ok;
  // paged KV cache: host bookkeeping of the device table [L][slot][blocks_per_seq] (0 = no page)
  std::vector<int32_t> bt_host, free_pages;
  int32_t pages_used;
  int32_t *bt_dev() const { return reinterpret_cast<int32_t *>(scratch + lay.block_table); }

  DevSched *sched() const { return reinterpret_cast<DevSched *>(scratch + lay.sched); }
  float2 *rope() const { return reinterpret_cast<float2 *>(scratch + lay.rope); }
  float *x() const { return reinterpret_cast<float *>(scratch + lay.x); }
  float *qkv() const { return reinterpret_cast<float *>(scratch + lay.qkv); }
  float *attn_out() const { return reinterpret_cast<float *>(scratch + lay.attn_out); }
  float *part_o() const { return reinterpret_cast<float *>(scratch + lay.part_o); }
  float *part_ml() const { return reinterpret_cast<float *>(scratch + lay.part_ml); }
  float *u() const { return reinterpret_cast<float *>(scratch + lay.u); }
};

// prefill passes of at least this many positions take the causal flash-attention kernel
static constexpr int kPrefillAttnMinRows = 8;

enum ProfKind { PK_SCHED = 0, PK_QKV, PK_ROPE, PK_ATTN, PK_OPROJ, PK_GATEUP, PK_DOWN, PK_FILL,
                PK_HEAD, PK_FUSED };
static const char *kProfNames[D3_PROF_KINDS] = {
    "schedule+embed", "norm+qkv", "rope+kv_append", "attention", "o_proj+resid", "norm+gate_up+swiglu",
    "down+resid", "kv_fill", "norm+lm_head", "fused_step",
    // phases inside the fused step kernel (mean over CTAs, nominal-clock ms)
    "fused:prologue", "fused:load_act", "fused:qkv", "fused:grid_barriers", "fused:attention",
    "fused:o_proj", "fused:gate_up", "fused:down", "fused:head+fill", "fused:ring_wait(warp0)",
    // smallest and largest per-CTA time spent in grid barriers
    "fused:grid_barriers_min", "fused:grid_barriers_max"};

// Scope that brackets one launch (or a launcher's pair of launches) with events.
struct ProfScope {
  d3_model *m;
  cudaEvent_t stop;
  ProfScope(d3_model *mm, int kind) : m(mm), stop(nullptr) {
    if (!m->prof_on) return;
    size_t i = m->prof_kind.size() * 2;
    while (m->prof_events.size() < i + 2) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return;
      m->prof_events.push_back(e);
    }
    m->prof_kind.push_back(kind);
    cudaEventRecord(m->prof_events[i], m->stream);
    stop = m->prof_events[i + 1];
  }
  ~ProfScope() {
    if (stop) cudaEventRecord(stop, m->stream);
  }
};

static void prof_collect(d3_model *m) {
  if (!m->prof_on) return;
  cudaStreamSynchronize(m->stream);
  for (size_t i = 0; i < m->prof_kind.size(); ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, m->prof_events[2 * i], m->prof_events[2 * i + 1]) == cudaSuccess) {
      m->prof_ms[m->prof_kind[i]] += ms;
      m->prof_n[m->prof_kind[i]] += 1;
    }
  }
  m->prof_kind.clear();
}

static const int32_t *thr_for(d3_model *m, double alpha) {
  uint64_t key;
  memcpy(&key, &alpha, 8);
  auto it = m->thr_cache.find(key);
  if (it == m->thr_cache.end()) {
    if (m->thr_cache.size() > 64) m->thr_cache.clear();
    std::vector<int32_t> t(D3_MAX_LAYERS + 1, 0);
    thresholds(m->cfg.n_layers, alpha, t.data());
    it = m->thr_cache.emplace(key, std::move(t)).first;
  }
  return it->second.data();
}

// Paged layout: give every (block, page-sized run of positions) that the rows of this step
// write a page, before anything is enqueued.  D3_ECAPACITY (nothing changed) when the pool
// cannot cover the step.  Under D3_FILL_NONE a row takes no page for a block it drops.
static int32_t pages_for_step(d3_model *m, int B, const int32_t *slot, const int32_t *pos, const int32_t *lo,
                              const int32_t *hi, int32_t *launches) {
  const d3_config &c = m->cfg;
  if (c.kv_layout != D3_KV_PAGED) return D3_OK;
  const int L = c.n_layers, bps = c.max_seq / c.page_size;
  auto writes = [&](int b, int l) { return c.kv_fill != D3_FILL_NONE || l < lo[b] || l >= hi[b]; };
  auto entry = [&](int b, int l) { return ((size_t)l * c.max_slots + slot[b]) * bps + pos[b] / c.page_size; };
  std::vector<size_t> need;
  for (int b = 0; b < B; ++b)
    for (int l = 0; l < L; ++l)
      if (writes(b, l) && m->bt_host[entry(b, l)] == 0) {
        size_t e = entry(b, l);
        bool dup = false;
        for (size_t q : need) dup = dup || q == e;   // rows of a prefill pass share pages
        if (!dup) need.push_back(e);
      }
  if (need.size() > m->free_pages.size()) return D3_ECAPACITY;
  TableUpdate u;
  u.n = 0;
  for (size_t e : need) {
    const int32_t page = m->free_pages.back();
    m->free_pages.pop_back();
    m->pages_used += 1;
    m->bt_host[e] = page;
    u.index[u.n] = (int32_t)e; u.page[u.n] = page;
    if (++u.n == TableUpdate::kMax) { *launches += launch_table_update(m->bt_dev(), u, m->stream); u.n = 0; }
  }
  if (u.n) *launches += launch_table_update(m->bt_dev(), u, m->stream);
  return D3_OK;
}

// Up to this many rows the kernel in front of the O and down projections writes their three-term
// operand itself (no pre-pass).  Measured on the 7B shape, ms per step with / without: 16 rows 3.60 /
// 3.77, 32 rows 4.13 / 4.29, 40 rows 4.51 / 4.65, but 48 rows 6.0 / 5.35 and 56 rows 5.71 / 5.63: the
// 2-byte stores of a wide group cost the epilogues more than the pre-passes they replace.
static const int kHandOverMaxRows = 40;

// One projection over `rows` rows: tensor cores for a dense enough group, FMA GEMV otherwise.
static int project(d3_model *m, const GemvArgs &g, int epi, int rows) {
  const bool tensor = m->exec_mode == D3_EXEC_TENSOR ||
                      (m->exec_mode == D3_EXEC_AUTO && rows >= D3_TENSOR_MIN_ROWS);
  if (tensor && m->tm_ok) {
    int n = launch_gemm_tc(m->tc, g, epi, rows, m->stream);
    if (n) return n;
  }
  if (g.clear) cudaMemsetAsync(g.clear, 0, g.clear_floats * sizeof(float), m->stream);   // the FMA kernels clear nothing
  return launch_gemv(g, epi, rows, m->stream);
}

// Enqueue one step over the rows described by `a` (already validated).
// logits_mode: ROWS_ALL -> logits_dev[caller row][V]; ROWS_LAST -> logits_dev[V]
// for the last row; logits_dev may be NULL (no LM head).
// `probe` (nullable): after every block, the token and confidence the LM head predicts from the
// block's output go to probe->tokens / conf [B][L] (device); logits_dev is the work buffer.
struct ProbeOut {
  int32_t *tokens;
  float *conf;
};

static int32_t run_step(d3_model *m, const StepArgs &a, const int32_t *n, const int32_t *lo,
                        const int32_t *hi, const int32_t *perm, const int32_t *m_l,
                        float *logits_dev, int logits_mode, int32_t *launches_out,
                        const ProbeOut *probe = nullptr, int prefill_t0 = -1) {
  const d3_config &c = m->cfg;
  const Dims &dm = m->dm;
  cudaStream_t st = m->stream;
  const int B = a.B, L = c.n_layers;
  int launches = 0;
  {
    int32_t rc = pages_for_step(m, B, a.slot, a.pos, lo, hi, &launches);
    if (rc != D3_OK) return rc;
  }
  { ProfScope ps(m, PK_SCHED); launches += launch_schedule_embed(a, m->sched(), m->embed, m->x(), dm.d, st); }
  const int nq = dm.Hq * dm.dh, nkv = dm.Hkv * dm.dh;
  const int G = dm.Hq / dm.Hkv, GQ = (G % 4 == 0) ? 4 : (G % 2 == 0) ? 2 : 1;

  GemvArgs g;
  memset(&g, 0, sizeof(g));
  g.sched = m->sched();
  g.eps = c.rms_eps;
  g.clear = nullptr; g.clear_floats = 0; g.out_is_zero = 0; g.operand_out = g.operand_in = 0;
  // The QKV projection sums its k-slices into a zeroed buffer.  After a block's attention nothing
  // reads that buffer until the next block's projection, so the down projection in between clears
  // it on the side (decode steps without recomputed fills, which use the buffer in between).
  const bool clear_ahead = prefill_t0 < 0 && !probe && c.kv_fill != D3_FILL_RECOMPUTE;
  bool qkv_cleared = false;
  const bool tm = m->tm_ok;
  for (int l = 0; l < L; ++l) {
    const int ml = m_l[l];
    g.layer = l;
    if (ml > 0) {
      // RMSNorm + QKV projection
      g.row_mode = ROWS_PREFIX;
      g.W = m->wqkv[l]; g.W2 = nullptr; g.R = dm.qkv_rows; g.K = dm.d;
      g.tmap_w = tm ? &m->tm_qkv[l] : nullptr; g.tmap_w2 = nullptr;
      g.act = m->x(); g.act_stride = dm.d; g.gain = m->attn_norm[l];
      g.out = m->qkv(); g.out_stride = dm.qkv_rows; g.out_col0 = 0;
      g.short_chain_row0 = prefill_t0 >= 0 ? nq : 0;   // a prompt's K and V rows: see launch_gemm_tc
      g.out_is_zero = qkv_cleared ? 1 : 0;
      { ProfScope ps(m, PK_QKV); launches += project(m, g, EPI_STORE, ml); }
      g.short_chain_row0 = 0; g.out_is_zero = 0; qkv_cleared = false;
      bool o_handed = false;
      { ProfScope ps(m, PK_ROPE);
        launches += launch_rope_append(m->qkv(), m->rope(), m->Kc, m->Vc, m->sched(), l, ROWS_PREFIX,
                                       0, ml, dm, st); }
      // attention over the cache (positions 0..pos, the new one included)
      if (prefill_t0 >= 0 && ml == B && B >= kPrefillAttnMinRows) {
        // a prefill pass: the rows are the consecutive positions prefill_t0 .. + B - 1 of one slot
        ProfScope ps(m, PK_ATTN);
        launches += launch_attention_prefill(m->qkv(), m->Kc, m->Vc, l, a.slot[0], prefill_t0, B,
                                             m->attn_out(), dm, st);
      } else {
      int max_len = 1;
      for (int r = 0; r < ml; ++r) {
        int len = a.pos[perm[r]] + 1;
        if (len > max_len) max_len = len;
      }
      int ctas = ml * (dm.Hq / GQ);
      // Pieces the attention pass aims for: one per SM.  More, shorter pieces lose to their fixed
      // cost and to the combine pass (13B shape, 8 rows x 40 heads, 1024 positions: 6.13 ms per step
      // with one piece per row and head, 6.30 with two; 70B shape, 4 rows: 24.2 against 24.5 ms).
      static const int target_ctas = [] {   // tuning knob
        const char *env = getenv("D3_ATTN_TARGET_CTAS");
        const int v = env ? atoi(env) : 0;
        return v >= 32 && v <= 65536 ? v : 148;
      }();
      int want = (target_ctas + ctas - 1) / ctas;
      if (want < 1) want = 1;
      if (want > m->lay.max_splits) want = m->lay.max_splits;
      int split_len = ((max_len + want - 1) / want + 31) / 32 * 32;
      if (split_len < 32) split_len = 32;
      int n_splits = (max_len + split_len - 1) / split_len;
      { ProfScope ps(m, PK_ATTN);
        // the output projection's three-term operand, when that projection will go to the tensor cores
        OpndOut opnd = {nullptr, 0};
        const bool tensor = m->exec_mode == D3_EXEC_TENSOR || (m->exec_mode == D3_EXEC_AUTO && ml >= D3_TENSOR_MIN_ROWS);
        if (tensor && m->tm_ok && ml <= kHandOverMaxRows) { opnd.p = m->tc.act_split2; opnd.np = (ml + 7) / 8 * 8; o_handed = true; }
        // longest contexts first: the launch's last CTAs are then short ones (C3: 0.4 % of the step)
        RowOrder order;
        order.given = 1;
        {
          int idx[D3_MAX_BATCH];
          for (int r = 0; r < ml; ++r) idx[r] = r;
          std::stable_sort(idx, idx + ml, [&](int x, int y) { return a.pos[perm[x]] > a.pos[perm[y]]; });
          for (int r = 0; r < ml; ++r) order.r[r] = (unsigned char)idx[r];
        }
        launches += launch_attention(m->qkv(), m->Kc, m->Vc, m->sched(), l, ml, split_len, n_splits,
                                     m->lay.max_splits, m->part_o(), m->part_ml(), m->attn_out(), opnd, dm, st,
                                     &order); }
      }
      // output projection + residual
      g.W = m->wo[l]; g.R = dm.d; g.K = nq; g.act = m->attn_out(); g.act_stride = nq;
      g.tmap_w = tm ? &m->tm_o[l] : nullptr;
      g.gain = nullptr; g.out = m->x(); g.out_stride = dm.d;
      g.operand_in = o_handed ? 1 : 0;
      { ProfScope ps(m, PK_OPROJ); launches += project(m, g, EPI_RESID, ml); }
      g.operand_in = 0;
      // RMSNorm + gate/up + SiLU * mul
      g.W = m->w_gate[l]; g.W2 = m->w_up[l]; g.R = dm.f; g.K = dm.d; g.act = m->x();
      g.tmap_w = tm ? &m->tm_gate[l] : nullptr; g.tmap_w2 = tm ? &m->tm_up[l] : nullptr;
      g.act_stride = dm.d; g.gain = m->mlp_norm[l]; g.out = m->u(); g.out_stride = dm.f;
      g.operand_out = ml <= kHandOverMaxRows ? 1 : 0; m->tc.handed_over = false;
      { ProfScope ps(m, PK_GATEUP); launches += project(m, g, EPI_SWIGLU, ml); }
      g.operand_out = 0;
      // down projection + residual
      g.W = m->w_down[l]; g.W2 = nullptr; g.R = dm.d; g.K = dm.f; g.act = m->u();
      g.tmap_w = tm ? &m->tm_down[l] : nullptr; g.tmap_w2 = nullptr;
      g.act_stride = dm.f; g.gain = nullptr; g.out = m->x(); g.out_stride = dm.d;
      if (clear_ahead) {
        bool more = false;
        for (int l2 = l + 1; l2 < L; ++l2) more = more || m_l[l2] > 0;
        if (more) { g.clear = m->qkv(); g.clear_floats = (size_t)B * dm.qkv_rows; qkv_cleared = true; }
      }
      g.operand_in = m->tc.handed_over ? 1 : 0;
      { ProfScope ps(m, PK_DOWN); launches += project(m, g, EPI_RESID, ml); }
      g.clear = nullptr; g.clear_floats = 0; g.operand_in = 0; m->tc.handed_over = false;
    }
    if (probe && logits_dev && l + 1 < L) {
      // every row's state after block l through the final norm and the LM head (Sec. 3.2)
      GemvArgs h = g;
      h.layer = 0; h.row_mode = ROWS_ALL;
      h.W = m->lm_head; h.W2 = nullptr; h.R = dm.V; h.K = dm.d; h.act = m->x(); h.act_stride = dm.d;
      h.tmap_w = tm ? &m->tm_head : nullptr; h.tmap_w2 = nullptr;
      h.gain = m->final_norm; h.out = logits_dev; h.out_stride = dm.V; h.out_col0 = 0;
      ProfScope ps(m, PK_HEAD);
      launches += project(m, h, EPI_LOGITS, B);
      launches += launch_argmax_conf(logits_dev, B, dm.V, probe->tokens, probe->conf, L, l, st);
    }
    if (c.kv_fill == D3_FILL_RECOMPUTE && ml < B) {
      // rows that drop block l: K,V from the block's own norm, W_k, W_v on the carried state
      g.row_mode = ROWS_SUFFIX;
      g.W = m->wqkv[l] + (size_t)nq * dm.d; g.W2 = nullptr; g.R = 2 * nkv; g.K = dm.d;
      g.tmap_w = tm ? &m->tm_kv[l] : nullptr; g.tmap_w2 = nullptr;
      g.act = m->x(); g.act_stride = dm.d; g.gain = m->attn_norm[l];
      g.out = m->qkv(); g.out_stride = dm.qkv_rows; g.out_col0 = nq;
      ProfScope ps(m, PK_FILL);
      launches += project(m, g, EPI_STORE, B - ml);
      launches += launch_rope_append(m->qkv(), m->rope(), m->Kc, m->Vc, m->sched(), l, ROWS_SUFFIX,
                                     1, B - ml, dm, st);
      g.out_col0 = 0;
    }
  }
  if (c.kv_fill == D3_FILL_COPY) {
    bool any = false;
    for (int b = 0; b < B; ++b) any = any || hi[b] > lo[b];
    if (any) { ProfScope ps(m, PK_FILL); launches += launch_fill_copy(m->Kc, m->Vc, m->sched(), B, dm, st); }
  }
  if (logits_dev) {
    g.layer = 0; g.row_mode = logits_mode;
    g.W = m->lm_head; g.W2 = nullptr; g.R = dm.V; g.K = dm.d; g.act = m->x(); g.act_stride = dm.d;
    g.tmap_w = tm ? &m->tm_head : nullptr; g.tmap_w2 = nullptr;
    g.gain = m->final_norm; g.out = logits_dev; g.out_stride = dm.V; g.out_col0 = 0;
    { ProfScope ps(m, PK_HEAD); launches += project(m, g, EPI_LOGITS, logits_mode == ROWS_LAST ? 1 : B); }
    if (probe)
      launches += launch_argmax_conf(logits_dev, B, dm.V, probe->tokens, probe->conf, L, L - 1, st);
  }
  m->last_B = B;
  for (int b = 0; b < B; ++b) m->last_perm[b] = perm[b];
  (void)n;
  prof_collect(m);
  if (launches_out) *launches_out = launches;
  return cudaGetLastError() == cudaSuccess ? D3_OK : D3_ECUDA;
}

// One batch-1 step as a single cooperative kernel.
static int32_t run_fused_step(d3_model *m, const StepArgs &a, const int32_t *lo, const int32_t *hi,
                              float *logits_dev, int32_t *launches_out) {
  int32_t table_launches = 0;
  {
    int32_t rc = pages_for_step(m, 1, a.slot, a.pos, lo, hi, &table_launches);   // paged cache: before any launch
    if (rc != D3_OK) return rc;
  }
  FusedParams fp;
  memset(&fp, 0, sizeof(fp));
  fp.slot = a.slot[0]; fp.tok = a.tok[0]; fp.gi = a.gi[0]; fp.pos = a.pos[0]; fp.tok_dev = a.tok_dev;
  memcpy(fp.thr, a.thr, sizeof(fp.thr));
  fp.L = a.L; fp.start_id = a.start_id; fp.anchor = a.anchor; fp.kv_fill = m->cfg.kv_fill;
  fp.dm = m->dm; fp.eps = m->cfg.rms_eps;
  fp.layers = reinterpret_cast<const LayerPtrs *>(m->scratch + m->lay.layer_tab);
  fp.embed = m->embed; fp.lm_head = m->lm_head; fp.final_norm = m->final_norm;
  fp.Kc = m->Kc; fp.Vc = m->Vc; fp.rope = m->rope(); fp.sched = m->sched();
  fp.bar_counter = reinterpret_cast<unsigned *>(m->scratch + m->lay.bar);
  fp.stream_count = fp.bar_counter + 16;
  fp.phase_cycles = m->prof_on ? reinterpret_cast<long long *>(m->scratch + m->lay.phase) : nullptr;
  fp.x = m->x(); fp.qkv = m->qkv(); fp.u = m->u(); fp.attn_out = m->attn_out();
  fp.part = reinterpret_cast<float *>(m->scratch + m->lay.part_fused);
  fp.logits = logits_dev;
  fp.n_stages = m->fused_stages; fp.act_floats = m->fused_act;
  fp.l2_window = fused_l2_window();
  fp.wait_ns = m->wait_ns;
  fp.barrier_extra = m->stall_next ? 1u : 0u;
  m->stall_next = 0;
  int rc;
  {
    ProfScope ps(m, PK_FUSED);
    rc = launch_fused_step(m->fused_func, m->fused_grid, m->fused_smem, fp, m->stream);
  }
  m->last_B = 1;
  m->last_perm[0] = 0;
  prof_collect(m);
  if (launches_out) *launches_out = 1 + table_launches;
  return (rc == 1 && cudaGetLastError() == cudaSuccess) ? D3_OK : D3_ECUDA;
}

static void schedule_of_depths(int32_t L, int32_t start_id, int32_t anchor, int32_t batch,
                               const int32_t *depth, int32_t *n, int32_t *lo, int32_t *hi, int32_t *perm,
                               int32_t *m_per_layer, int64_t *rows_layers, int32_t *layers_touched);

// Paged layout: take back every page of `slot` (host list + device table, in stream order).
static int32_t release_pages(d3_model *m, int32_t slot) {
  const d3_config &c = m->cfg;
  if (c.kv_layout != D3_KV_PAGED) return D3_OK;
  const int bps = c.max_seq / c.page_size;
  for (int l = 0; l < c.n_layers; ++l) {
    int32_t *row = m->bt_host.data() + ((size_t)l * c.max_slots + slot) * bps;
    bool any = false;
    for (int k = 0; k < bps; ++k)
      if (row[k]) { m->free_pages.push_back(row[k]); m->pages_used -= 1; row[k] = 0; any = true; }
    if (any && cudaMemsetAsync(m->bt_dev() + ((size_t)l * c.max_slots + slot) * bps, 0, bps * sizeof(int32_t),
                               m->stream) != cudaSuccess)
      return D3_ECUDA;
  }
  return D3_OK;
}

extern "C" {

int32_t d3_depth(int32_t L, double alpha, int64_t i) {
  if (L < 0 || i < 0 || !alpha_ok(alpha)) return D3_EINVAL;
  return depth_host(L, alpha, i);
}

int32_t d3_schedule(int32_t L, double alpha, int32_t start_id, int32_t anchor, int32_t batch,
                    const int32_t *gen_index, int32_t *n, int32_t *lo, int32_t *hi, int32_t *perm,
                    int32_t *m_per_layer, int64_t *rows_layers, int32_t *layers_touched) {
  if (L < 1 || L > D3_MAX_LAYERS || !alpha_ok(alpha) || start_id < 0 || start_id > L ||
      (anchor != D3_ANCHOR_START && anchor != D3_ANCHOR_TAIL) || batch < 1 ||
      batch > D3_MAX_BATCH || !gen_index || !n || !lo || !hi || !perm || !m_per_layer)
    return D3_EINVAL;
  for (int b = 0; b < batch; ++b)
    if (gen_index[b] < 0) return D3_EINVAL;
  int32_t depth[D3_MAX_BATCH];
  for (int b = 0; b < batch; ++b) depth[b] = depth_host(L, alpha, gen_index[b]);
  schedule_of_depths(L, start_id, anchor, batch, depth, n, lo, hi, perm, m_per_layer, rows_layers,
                     layers_touched);
  return D3_OK;
}

}  // extern "C"

// Windows, depth-sorted order and per-block row counts for rows with the given depths.
static void schedule_of_depths(int32_t L, int32_t start_id, int32_t anchor, int32_t batch,
                               const int32_t *depth, int32_t *n, int32_t *lo, int32_t *hi, int32_t *perm,
                               int32_t *m_per_layer, int64_t *rows_layers, int32_t *layers_touched) {
  for (int b = 0; b < batch; ++b) {
    int32_t nb = depth[b];
    if (anchor == D3_ANCHOR_TAIL) {
      lo[b] = nb; hi[b] = L;
    } else {
      if (nb < start_id) nb = start_id;
      lo[b] = start_id; hi[b] = start_id + (L - nb);
    }
    n[b] = nb;
  }
  // counting sort by n descending, stable in the row index
  int32_t count[D3_MAX_LAYERS + 2];
  memset(count, 0, sizeof(count));
  for (int b = 0; b < batch; ++b) count[L - n[b] + 1]++;
  for (int k = 1; k <= L + 1; ++k) count[k] += count[k - 1];
  for (int b = 0; b < batch; ++b) perm[count[L - n[b]]++] = b;
  int64_t tot = 0;
  int32_t touched = 0;
  for (int l = 0; l < L; ++l) {
    int32_t ml = 0;
    for (int b = 0; b < batch; ++b) ml += (lo[b] <= l && l < hi[b]) ? 0 : 1;
    m_per_layer[l] = ml;
    tot += ml;
    touched += ml > 0;
  }
  if (rows_layers) *rows_layers = tot;
  if (layers_touched) *layers_touched = touched;
}

extern "C" {

int32_t d3_workspace_bytes(const d3_config *cfg, size_t *kv_bytes, size_t *scratch_bytes) {
  if (!config_ok(cfg) || !kv_bytes || !scratch_bytes) return D3_EINVAL;
  if (cfg->kv_layout == D3_KV_PAGED)
    *kv_bytes = 2 * (size_t)cfg->n_pages * cfg->n_kv_heads * cfg->page_size * cfg->head_dim * sizeof(bf16);
  else
    *kv_bytes = 2 * (size_t)cfg->n_layers * cfg->max_slots * cfg->n_kv_heads * cfg->max_seq *
                cfg->head_dim * sizeof(bf16);
  *scratch_bytes = make_layout(*cfg).total;
  return D3_OK;
}

int32_t d3_load(const d3_config *cfg, const d3_weights *w, void *kv_dev, void *scratch_dev,
                void *cuda_stream, d3_model **out) {
  if (!config_ok(cfg) || !w || !kv_dev || !scratch_dev || !out) return D3_EINVAL;
  if (!w->embed_dev || !w->lm_head_dev || !w->final_norm_dev || !w->attn_norm_dev || !w->wqkv_dev ||
      !w->wo_dev || !w->mlp_norm_dev || !w->w_gate_dev || !w->w_up_dev || !w->w_down_dev)
    return D3_EINVAL;
  auto misaligned = [](const void *p, size_t a) { return p == nullptr || ((uintptr_t)p % a) != 0; };
  if (misaligned(kv_dev, 256) || misaligned(scratch_dev, 256)) return D3_EINVAL;
  if (misaligned(w->embed_dev, 16) || misaligned(w->lm_head_dev, 16) || misaligned(w->final_norm_dev, 16))
    return D3_EINVAL;
  const int L = cfg->n_layers;
  for (int l = 0; l < L; ++l)
    if (misaligned(w->attn_norm_dev[l], 16) || misaligned(w->wqkv_dev[l], 16) ||
        misaligned(w->wo_dev[l], 16) || misaligned(w->mlp_norm_dev[l], 16) ||
        misaligned(w->w_gate_dev[l], 16) || misaligned(w->w_up_dev[l], 16) ||
        misaligned(w->w_down_dev[l], 16))
      return D3_EINVAL;
  d3_model *m = new (std::nothrow) d3_model();
  if (!m) return D3_EINVAL;
  m->cfg = *cfg;
  m->dm = Dims{cfg->n_layers, cfg->d_model, cfg->n_q_heads, cfg->n_kv_heads, cfg->head_dim,
               cfg->d_ffn, cfg->vocab, cfg->max_slots, cfg->max_seq,
               (cfg->n_q_heads + 2 * cfg->n_kv_heads) * cfg->head_dim};
  m->lay = make_layout(*cfg);
  m->stream = (cudaStream_t)cuda_stream;
  m->embed = (const bf16 *)w->embed_dev;
  m->lm_head = (const bf16 *)w->lm_head_dev;
  m->final_norm = (const bf16 *)w->final_norm_dev;
  for (int l = 0; l < L; ++l) {
    m->attn_norm.push_back((const bf16 *)w->attn_norm_dev[l]);
    m->wqkv.push_back((const bf16 *)w->wqkv_dev[l]);
    m->wo.push_back((const bf16 *)w->wo_dev[l]);
    m->mlp_norm.push_back((const bf16 *)w->mlp_norm_dev[l]);
    m->w_gate.push_back((const bf16 *)w->w_gate_dev[l]);
    m->w_up.push_back((const bf16 *)w->w_up_dev[l]);
    m->w_down.push_back((const bf16 *)w->w_down_dev[l]);
  }
  size_t kv_half = (size_t)L * cfg->max_slots * cfg->n_kv_heads * cfg->max_seq * cfg->head_dim;
  if (cfg->kv_layout == D3_KV_PAGED)
    kv_half = (size_t)cfg->n_pages * cfg->n_kv_heads * cfg->page_size * cfg->head_dim;
  m->Kc = (bf16 *)kv_dev;
  m->Vc = m->Kc + kv_half;
  m->scratch = (char *)scratch_dev;
  m->pages_used = 0;
  if (cfg->kv_layout == D3_KV_PAGED) {
    const int ps = cfg->page_size, bps = cfg->max_seq / ps;
    m->dm.page_size = ps;
    m->dm.page_shift = 0;
    while ((1 << m->dm.page_shift) < ps) m->dm.page_shift += 1;
    m->dm.blocks_per_seq = bps;
    m->dm.block_table = m->bt_dev();
    m->bt_host.assign((size_t)L * cfg->max_slots * bps, 0);
    for (int32_t pg = cfg->n_pages - 1; pg >= 1; --pg) m->free_pages.push_back(pg);   // page 0 reserved
    const size_t page_bytes = (size_t)cfg->n_kv_heads * ps * cfg->head_dim * sizeof(bf16);
    if (cudaMemsetAsync(m->bt_dev(), 0, m->bt_host.size() * sizeof(int32_t), m->stream) != cudaSuccess ||
        cudaMemsetAsync(m->Kc, 0, page_bytes, m->stream) != cudaSuccess ||
        cudaMemsetAsync(m->Vc, 0, page_bytes, m->stream) != cudaSuccess) {
      delete m;
      return D3_ECUDA;
    }
  }
  m->pos.assign(cfg->max_slots, -1);
  m->last_B = 0;
  m->prof_on = false;
  memset(m->prof_ms, 0, sizeof(m->prof_ms));
  memset(m->prof_n, 0, sizeof(m->prof_n));
  const int64_t d = cfg->d_model, f = cfg->d_ffn;
  m->layer_bytes = 2 * ((int64_t)m->dm.qkv_rows * d + d * cfg->n_q_heads * cfg->head_dim + 3 * d * f + 2 * d);
  m->head_bytes = 2 * ((int64_t)cfg->vocab * d + d);
  if (init_kernel_attributes() != 0 || init_attention_prefill() != 0) { delete m; return D3_ECUDA; }
  // tensor-core projections: usable when the driver encodes every weight's tensor map
  m->tc.ok = tc_init() == 0;
  m->tc.act_split = reinterpret_cast<bf16 *>(m->scratch + m->lay.act_split);
  m->tc.act_split2 = reinterpret_cast<bf16 *>(m->scratch + m->lay.act_split2);
  m->tc.handed_over = false;
  m->tc.act_bytes = m->lay.act_split_bytes;
  m->wait_ns = 2000000000ull;
  m->stall_next = 0;
  m->tc.wait_ns = m->wait_ns;
  {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
      sms = 148;
    m->tc.sm_count = sms;
  }
  m->tm_ok = m->tc.ok;
  if (m->tm_ok) {
    const int nq = m->dm.Hq * m->dm.dh, nkv = m->dm.Hkv * m->dm.dh, dd = m->dm.d, ff = m->dm.f;
    m->tm_qkv.resize(L); m->tm_kv.resize(L); m->tm_o.resize(L);
    m->tm_gate.resize(L); m->tm_up.resize(L); m->tm_down.resize(L);
    bool ok = tc_weight_map(&m->tm_head, m->lm_head, m->dm.V, dd);
    for (int l = 0; l < L && ok; ++l) {
      ok = tc_weight_map(&m->tm_qkv[l], m->wqkv[l], m->dm.qkv_rows, dd) &&
           tc_weight_map(&m->tm_kv[l], m->wqkv[l] + (size_t)nq * dd, 2 * nkv, dd) &&
           tc_weight_map(&m->tm_o[l], m->wo[l], dd, nq) &&
           tc_weight_map(&m->tm_gate[l], m->w_gate[l], ff, dd) &&
           tc_weight_map(&m->tm_up[l], m->w_up[l], ff, dd) &&
           tc_weight_map(&m->tm_down[l], m->w_down[l], dd, ff);
    }
    m->tm_ok = ok;
  }
  m->exec_mode = D3_EXEC_AUTO;
  for (int l = 0; l < L; ++l)
    m->layer_tab_host.push_back(LayerPtrs{m->attn_norm[l], m->wqkv[l], m->wo[l], m->mlp_norm[l],
                                          m->w_gate[l], m->w_up[l], m->w_down[l]});
  if (cudaMemcpyAsync(m->scratch + m->lay.layer_tab, m->layer_tab_host.data(),
                      sizeof(LayerPtrs) * L, cudaMemcpyHostToDevice, m->stream) != cudaSuccess) {
    delete m;
    return D3_ECUDA;
  }
  m->fused_ok = fused_plan(*cfg, &m->fused_grid, &m->fused_stages, &m->fused_act, &m->fused_smem,
                           &m->fused_func);
  if (m->fused_ok && m->fused_grid > kFusedMaxCtas) m->fused_grid = kFusedMaxCtas;
  if (cudaMemsetAsync(m->sched(), 0, sizeof(DevSched), m->stream) != cudaSuccess ||
      cudaMemsetAsync(m->scratch + m->lay.phase, 0, (size_t)kFusedMaxCtas * kFusedPhases * 8, m->stream) !=
          cudaSuccess) {
    delete m;
    return D3_ECUDA;
  }
  launch_rope_table(m->rope(), cfg->max_seq, cfg->head_dim, cfg->rope_base, m->stream);
  if (cudaGetLastError() != cudaSuccess) { delete m; return D3_ECUDA; }
  *out = m;
  return D3_OK;
}

int32_t d3_prefill(d3_model *m, int32_t slot, const int32_t *tokens, int32_t n_tokens,
                   float *logits_dev) {
  if (!m || !tokens || slot < 0 || slot >= m->cfg.max_slots || n_tokens < 1) return D3_EINVAL;
  if (n_tokens > m->cfg.max_seq) return D3_ECAPACITY;
  for (int t = 0; t < n_tokens; ++t)
    if (tokens[t] < 0 || tokens[t] >= m->cfg.vocab) return D3_EINVAL;
  const int L = m->cfg.n_layers, MB = m->cfg.max_batch;
  if (release_pages(m, slot) != D3_OK) return D3_ECUDA;
  m->pos[slot] = -1;
  const int32_t *thr = thr_for(m, 1.0);
  int32_t n[D3_MAX_BATCH], lo[D3_MAX_BATCH], hi[D3_MAX_BATCH], perm[D3_MAX_BATCH], m_l[D3_MAX_LAYERS];
  for (int t0 = 0; t0 < n_tokens; t0 += MB) {
    StepArgs a;
    memset(&a, 0, sizeof(a));
    a.B = (n_tokens - t0 < MB) ? n_tokens - t0 : MB;
    a.L = L; a.start_id = m->cfg.start_id; a.anchor = m->cfg.anchor;
    memcpy(a.thr, thr, sizeof(a.thr));
    for (int b = 0; b < a.B; ++b) {
      a.slot[b] = slot; a.tok[b] = tokens[t0 + b]; a.gi[b] = 0; a.pos[b] = t0 + b;
    }
    d3_schedule(L, 1.0, m->cfg.start_id, m->cfg.anchor, a.B, a.gi, n, lo, hi, perm, m_l, nullptr, nullptr);
    const bool last = t0 + a.B >= n_tokens;
    int32_t rc = run_step(m, a, n, lo, hi, perm, m_l, last ? logits_dev : nullptr, ROWS_LAST, nullptr, nullptr, t0);
    if (rc != D3_OK) return rc;
  }
  m->pos[slot] = n_tokens;
  return D3_OK;
}

// One generation step over rows whose retained counts `depth_in` are known.  `thr` / `gi`
// are what the device derives the same counts from: the alpha thresholds with the
// generation indices, or thr[k] = k with gi = L - depth (then #{k : gi < thr[k]} = depth).
static int32_t decode_rows(d3_model *m, int32_t batch, const int32_t *slots, const int32_t *tokens,
                           const int32_t *depth_in, const int32_t *thr, const int32_t *gi,
                           float *logits_dev, d3_step_stats *stats, const int32_t *tokens_dev,
                           const ProbeOut *probe = nullptr) {
  const d3_config &c = m->cfg;
  for (int b = 0; b < batch; ++b) {
    if (slots[b] < 0 || slots[b] >= c.max_slots) return D3_EINVAL;
    if (!tokens_dev && (tokens[b] < 0 || tokens[b] >= c.vocab)) return D3_EINVAL;
  }
  for (int b = 0; b < batch; ++b) {
    for (int a2 = 0; a2 < b; ++a2)
      if (slots[a2] == slots[b]) return D3_ESTATE;
    if (m->pos[slots[b]] < 1) return D3_ESTATE;
  }
  for (int b = 0; b < batch; ++b)
    if (m->pos[slots[b]] >= c.max_seq) return D3_ECAPACITY;

  const int L = c.n_layers;
  StepArgs a;
  memset(&a, 0, sizeof(a));
  a.B = batch; a.L = L; a.start_id = c.start_id; a.anchor = c.anchor; a.tok_dev = tokens_dev;
  memcpy(a.thr, thr, sizeof(a.thr));
  for (int b = 0; b < batch; ++b) {
    a.slot[b] = slots[b]; a.tok[b] = tokens_dev ? 0 : tokens[b]; a.gi[b] = gi[b];
    a.pos[b] = m->pos[slots[b]];
  }
  int32_t n[D3_MAX_BATCH], lo[D3_MAX_BATCH], hi[D3_MAX_BATCH], perm[D3_MAX_BATCH], m_l[D3_MAX_LAYERS];
  int64_t rows_layers = 0;
  int32_t touched = 0;
  schedule_of_depths(L, c.start_id, c.anchor, batch, depth_in, n, lo, hi, perm, m_l, &rows_layers, &touched);
  int32_t launches = 0;
  // Measured (one row, full depth, same box): the single kernel wins at every shape: 7B 2.55 ms
  // against 3.50 ms for the kernel sequence, 13B 5.47 against 5.90, 70B 25.4 against 25.7.
  const bool fused = batch == 1 && m->fused_ok &&
                     (m->exec_mode == D3_EXEC_AUTO || m->exec_mode == D3_EXEC_FUSED) &&
                     c.kv_fill != D3_FILL_RECOMPUTE && !probe;
  int32_t rc = fused ? run_fused_step(m, a, lo, hi, logits_dev, &launches)
                     : run_step(m, a, n, lo, hi, perm, m_l, logits_dev, ROWS_ALL, &launches, probe);
  if (rc != D3_OK) return rc;
  if (stats) {
    if (stats->n) memcpy(stats->n, n, sizeof(int32_t) * batch);
    if (stats->m_per_layer) memcpy(stats->m_per_layer, m_l, sizeof(int32_t) * L);
    stats->rows_layers = rows_layers;
    stats->layers_touched = touched;
    stats->kernel_launches = launches;
    const int64_t kv_tok = 2LL * c.n_kv_heads * c.head_dim * 2;  // K and V of one token, one block
    int64_t bytes = (int64_t)touched * m->layer_bytes + m->head_bytes;
    for (int b = 0; b < batch; ++b) {
      bytes += (int64_t)n[b] * kv_tok * (a.pos[b] + 1);           // KV read by retained blocks
      int64_t written = n[b] + (c.kv_fill != D3_FILL_NONE ? (hi[b] - lo[b]) : 0);
      bytes += written * kv_tok;                                   // KV appended / filled
    }
    bytes += (int64_t)batch * c.d_model * 2 + (int64_t)batch * c.vocab * 4;
    stats->algorithmic_bytes = bytes;
  }
  for (int b = 0; b < batch; ++b) m->pos[slots[b]] += 1;
  return D3_OK;
}

int32_t d3_decode_step(d3_model *m, int32_t batch, const int32_t *slots, const int32_t *tokens,
                       const int32_t *gen_index, double alpha, float *logits_dev,
                       d3_step_stats *stats, const int32_t *tokens_dev) {
  if (!m || !slots || !gen_index || !logits_dev || (!tokens && !tokens_dev)) return D3_EINVAL;
  if (batch < 1 || !alpha_ok(alpha)) return D3_EINVAL;
  if (batch > m->cfg.max_batch) return D3_ECAPACITY;
  int32_t depth[D3_MAX_BATCH];
  for (int b = 0; b < batch; ++b) {
    if (gen_index[b] < 1) return D3_EINVAL;
    depth[b] = depth_host(m->cfg.n_layers, alpha, gen_index[b]);
  }
  return decode_rows(m, batch, slots, tokens, depth, thr_for(m, alpha), gen_index, logits_dev, stats,
                     tokens_dev);
}

int32_t d3_decode_step_depths(d3_model *m, int32_t batch, const int32_t *slots, const int32_t *tokens,
                              const int32_t *depths, float *logits_dev, d3_step_stats *stats,
                              const int32_t *tokens_dev) {
  if (!m || !slots || !depths || !logits_dev || (!tokens && !tokens_dev)) return D3_EINVAL;
  if (batch < 1) return D3_EINVAL;
  if (batch > m->cfg.max_batch) return D3_ECAPACITY;
  const int L = m->cfg.n_layers;
  int32_t thr[D3_MAX_LAYERS + 1], gi[D3_MAX_BATCH];
  for (int k = 0; k <= D3_MAX_LAYERS; ++k) thr[k] = k;
  for (int b = 0; b < batch; ++b) {
    if (depths[b] < 0 || depths[b] > L) return D3_EINVAL;
    gi[b] = L - depths[b];
  }
  return decode_rows(m, batch, slots, tokens, depths, thr, gi, logits_dev, stats, tokens_dev);
}

int32_t d3_saturation_probe(d3_model *m, int32_t batch, const int32_t *slots, const int32_t *tokens,
                            float *logits_dev, int32_t *block_tokens_dev, float *block_conf_dev) {
  if (!m || !slots || !tokens || !logits_dev || !block_tokens_dev) return D3_EINVAL;
  if (batch < 1) return D3_EINVAL;
  if (batch > m->cfg.max_batch) return D3_ECAPACITY;
  const int L = m->cfg.n_layers;
  int32_t thr[D3_MAX_LAYERS + 1], gi[D3_MAX_BATCH], depth[D3_MAX_BATCH];
  for (int k = 0; k <= D3_MAX_LAYERS; ++k) thr[k] = k;
  for (int b = 0; b < batch; ++b) { gi[b] = 0; depth[b] = L; }   // every row at full depth
  ProbeOut probe{block_tokens_dev, block_conf_dev};
  return decode_rows(m, batch, slots, tokens, depth, thr, gi, logits_dev, nullptr, nullptr, &probe);
}

int32_t d3_depth_linear(int32_t upper, int32_t lower, int64_t span, int64_t i) {
  if (upper < 0 || lower < 0 || lower > upper || span < 1 || i < 0) return D3_EINVAL;
  const int64_t t = i < span ? i : span;
  return (int32_t)(upper - ((int64_t)(upper - lower) * t) / span);
}

int32_t d3_argmax(d3_model *m, const float *logits_dev, int32_t batch, int32_t *tokens_dev) {
  if (!m || !logits_dev || !tokens_dev || batch < 1) return D3_EINVAL;
  launch_argmax(logits_dev, batch, m->cfg.vocab, tokens_dev, m->stream);
  return cudaGetLastError() == cudaSuccess ? D3_OK : D3_ECUDA;
}

int32_t d3_read_schedule(d3_model *m, int32_t *n, int32_t *perm, int32_t *m_per_layer,
                         int64_t *counters) {
  if (!m) return D3_EINVAL;
  DevSched h;
  if (cudaStreamSynchronize(m->stream) != cudaSuccess) return D3_ECUDA;
  if (cudaMemcpy(&h, m->sched(), sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return D3_ECUDA;
  if (n) memcpy(n, h.n, sizeof(int32_t) * h.B);
  if (perm) memcpy(perm, h.perm, sizeof(int32_t) * h.B);
  if (m_per_layer) memcpy(m_per_layer, h.m, sizeof(int32_t) * h.L);
  if (counters) { counters[0] = h.rows_layers; counters[1] = h.layers_touched; }
  return D3_OK;
}

int32_t d3_read_hidden(d3_model *m, float *hidden) {
  if (!m || !hidden || m->last_B < 1) return D3_EINVAL;
  if (cudaStreamSynchronize(m->stream) != cudaSuccess) return D3_ECUDA;
  const size_t row = (size_t)m->cfg.d_model * 4;
  for (int r = 0; r < m->last_B; ++r)
    if (cudaMemcpy((char *)hidden + (size_t)m->last_perm[r] * row, (char *)m->x() + r * row, row,
                   cudaMemcpyDeviceToHost) != cudaSuccess)
      return D3_ECUDA;
  return D3_OK;
}

int32_t d3_read_kv(d3_model *m, int32_t layer, int32_t slot, int32_t pos, float *k, float *v) {
  if (!m || !k || !v || layer < 0 || layer >= m->cfg.n_layers || slot < 0 ||
      slot >= m->cfg.max_slots || pos < 0 || pos >= m->cfg.max_seq)
    return D3_EINVAL;
  if (cudaStreamSynchronize(m->stream) != cudaSuccess) return D3_ECUDA;
  const int dh = m->cfg.head_dim;
  std::vector<uint16_t> buf(dh);
  for (int h = 0; h < m->cfg.n_kv_heads; ++h) {
    size_t off = kv_offset(m->dm, m->bt_host.data(), layer, slot, h, pos);
    for (int which = 0; which < 2; ++which) {
      const bf16 *src = (which ? m->Vc : m->Kc) + off;
      if (cudaMemcpy(buf.data(), src, dh * 2, cudaMemcpyDeviceToHost) != cudaSuccess) return D3_ECUDA;
      float *dst = (which ? v : k) + h * dh;
      for (int e = 0; e < dh; ++e) {
        uint32_t u = (uint32_t)buf[e] << 16;
        memcpy(dst + e, &u, 4);
      }
    }
  }
  return D3_OK;
}

int32_t d3_slot_pos(const d3_model *m, int32_t slot) {
  if (!m || slot < 0 || slot >= m->cfg.max_slots) return D3_EINVAL;
  return m->pos[slot] < 0 ? D3_ESTATE : m->pos[slot];
}

int32_t d3_reset_slot(d3_model *m, int32_t slot) {
  if (!m || slot < 0 || slot >= m->cfg.max_slots) return D3_EINVAL;
  m->pos[slot] = -1;
  return release_pages(m, slot);
}

int32_t d3_kv_pages_used(const d3_model *m) {
  if (!m || m->cfg.kv_layout != D3_KV_PAGED) return D3_EINVAL;
  return m->pages_used;
}

int32_t d3_sync(d3_model *m) {
  if (!m) return D3_EINVAL;
  if (cudaStreamSynchronize(m->stream) != cudaSuccess) return D3_ECUDA;
  int32_t status = 0;
  if (cudaMemcpy(&status, &m->sched()->status, 4, cudaMemcpyDeviceToHost) != cudaSuccess)
    return D3_ECUDA;
  // a deferred status is reported once: the word is cleared so that later steps start clean
  if (status != 0 && cudaMemset(&m->sched()->status, 0, 4) != cudaSuccess) return D3_ECUDA;
  return status;
}

int32_t d3_set_policy(d3_model *m, int32_t start_id, int32_t anchor, int32_t kv_fill) {
  if (!m) return D3_EINVAL;
  if (start_id < 0 || start_id > m->cfg.n_layers) return D3_EINVAL;
  if (anchor != D3_ANCHOR_START && anchor != D3_ANCHOR_TAIL) return D3_EINVAL;
  if (kv_fill < D3_FILL_NONE || kv_fill > D3_FILL_RECOMPUTE) return D3_EINVAL;
  m->cfg.start_id = start_id;
  m->cfg.anchor = anchor;
  m->cfg.kv_fill = kv_fill;
  return D3_OK;
}

int32_t d3_set_wait_ns(d3_model *m, uint64_t ns) {
  if (!m || ns < 1) return D3_EINVAL;
  m->wait_ns = ns;
  m->tc.wait_ns = ns;
  return D3_OK;
}

int32_t d3_stall_next_step(d3_model *m) {
  if (!m || !m->fused_ok) return D3_EINVAL;
  m->stall_next = 1;
  return D3_OK;
}

int32_t d3_set_exec(d3_model *m, int32_t mode) {
  if (!m || mode < D3_EXEC_AUTO || mode > D3_EXEC_FUSED) return D3_EINVAL;
  if (mode == D3_EXEC_TENSOR && !m->tm_ok) return D3_EINVAL;
  if (mode == D3_EXEC_FUSED && !m->fused_ok) return D3_EINVAL;
  m->exec_mode = mode;
  return D3_OK;
}

int32_t d3_profile(d3_model *m, int32_t enable) {
  if (!m) return D3_EINVAL;
  m->prof_on = enable != 0;
  return D3_OK;
}

int32_t d3_read_profile(d3_model *m, float *ms, int32_t *launches) {
  if (!m || !ms || !launches) return D3_EINVAL;
  memset(ms, 0, sizeof(float) * D3_PROF_KINDS);
  memset(launches, 0, sizeof(int32_t) * D3_PROF_KINDS);
  memcpy(ms, m->prof_ms, sizeof(m->prof_ms));
  memcpy(launches, m->prof_n, sizeof(m->prof_n));
  if (m->fused_ok && m->prof_n[PK_FUSED] > 0) {
    // phases of the fused step kernel, timed by every CTA in SM cycles
    std::vector<long long> cyc((size_t)kFusedMaxCtas * kFusedPhases);
    int dev = 0, khz = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev);
    if (cudaStreamSynchronize(m->stream) != cudaSuccess) return D3_ECUDA;
    char *ph = m->scratch + m->lay.phase;
    if (cudaMemcpy(cyc.data(), ph, cyc.size() * 8, cudaMemcpyDeviceToHost) != cudaSuccess) return D3_ECUDA;
    if (cudaMemset(ph, 0, cyc.size() * 8) != cudaSuccess) return D3_ECUDA;
    const double to_ms = khz > 0 ? 1.0 / (double)khz : 0.0;
    const int nc = m->fused_grid;
    for (int k = 0; k < kFusedPhases; ++k) {
      double tot = 0;
      for (int cta = 0; cta < nc; ++cta) tot += (double)cyc[(size_t)cta * kFusedPhases + k];
      ms[D3_PROF_FUSED0 + k] = (float)(tot / nc * to_ms);
      launches[D3_PROF_FUSED0 + k] = m->prof_n[PK_FUSED];
    }
    long long mn = cyc[3], mx = cyc[3];
    for (int cta = 0; cta < nc; ++cta) {
      const long long v = cyc[(size_t)cta * kFusedPhases + 3];
      if (v < mn) mn = v;
      if (v > mx) mx = v;
    }
    ms[D3_PROF_FUSED0 + kFusedPhases] = (float)(mn * to_ms);
    ms[D3_PROF_FUSED0 + kFusedPhases + 1] = (float)(mx * to_ms);
    launches[D3_PROF_FUSED0 + kFusedPhases] = launches[D3_PROF_FUSED0 + kFusedPhases + 1] = m->prof_n[PK_FUSED];
  }
  memset(m->prof_ms, 0, sizeof(m->prof_ms));
  memset(m->prof_n, 0, sizeof(m->prof_n));
  return D3_OK;
}

int32_t d3_read_fused_phases(d3_model *m, int64_t *cycles, int32_t *ctas, int32_t *phases) {
  if (!m || !cycles || !ctas || !phases) return D3_EINVAL;
  *ctas = m->fused_ok ? m->fused_grid : 0;
  *phases = kFusedPhases;
  if (!m->fused_ok) return D3_OK;
  if (cudaStreamSynchronize(m->stream) != cudaSuccess) return D3_ECUDA;
  if (cudaMemcpy(cycles, m->scratch + m->lay.phase, (size_t)m->fused_grid * kFusedPhases * 8,
                 cudaMemcpyDeviceToHost) != cudaSuccess)
    return D3_ECUDA;
  return D3_OK;
}

const char *d3_profile_name(int32_t kind) {
  return (kind >= 0 && kind < D3_PROF_KINDS) ? kProfNames[kind] : "";
}

void d3_free(d3_model *m) {
  if (!m) return;
  for (cudaEvent_t e : m->prof_events) cudaEventDestroy(e);
  delete m;
}

const char *d3_strerror(int32_t code) {
  switch (code) {
    case D3_OK: return "ok";
    case D3_EINVAL: return "invalid argument";
    case D3_ECAPACITY: return "capacity exceeded (max_seq, max_batch or the page pool)";
    case D3_ESTATE: return "slot not prefilled, or used twice in one batch";
    case D3_ECUDA: return "CUDA runtime error";
    case D3_ETIMEOUT: return "a bounded device-side wait ran out";
    default: return "unknown error";
  }
}

}  // extern "C"

// Batch-1 decode step as ONE persistent cooperative kernel (sm_100a).
//
// One CTA per SM.  Warps 8-10 are producers: they stream the CTA's share of
// every weight matrix (and of the static part of the KV cache) through a
// shared-memory ring with bulk asynchronous copies (cp.async.bulk + mbarrier
// transaction counts), stage s issued by producer s mod 3 (one warp alone cannot
// turn stages around fast enough: ~300 ns per stage of barrier traffic).  They
// never wait for the computation: weights do not depend on activations.  Warp 11
// walks the same sequence of stages further ahead and only asks L2 for them
// (cp.async.bulk.prefetch.L2): the ring holds ~4 us of HBM time, a phase boundary
// stalls the consumers for longer (each cross-CTA round trip costs 1-2 us), and
// with the look-ahead window in L2 HBM keeps streaming through the stall while the
// ring refills from L2 afterwards.  Each ring
// stage is consumed by ONE of the warps 0-7 (stage s of a phase by warp s mod 8),
// so the warps work on eight stages at a time and never synchronise inside a
// projection.  Phases of a block (RMSNorm+QKV+RoPE+KV append | attention |
// O-proj+residual | RMSNorm+gate/up+SwiGLU | down+residual) are separated by
// grid barriers on a global counter; only the small fp32 activations cross them
// (through L2, read with ld.global.cg).
//
// A ring stage is 16 KB: four weight-row segments of 2048 bf16 (a "row group" x
// k-chunk), or 8 KB of K plus 8 KB of V for one KV head.  Row groups are issued
// eight at a time, k-chunk major, so that warp w keeps the four running sums of
// group w in registers across the k-chunks and finishes the group alone
// (shuffle reduction + epilogue).  A lane owns 8 consecutive k of every
// 256-element block, so the activation costs two shared loads per four weight
// loads.
//
// Every wait (mbarrier, release counter, grid barrier) is bounded in time; on
// expiry the kernel raises D3_ETIMEOUT in the schedule's status word and enters
// abort mode: waits return at once, the producer stops issuing and drains the
// copies in flight, and every thread still walks the same control flow to the
// end so that no barrier is left waiting.
#include <stdlib.h>

#include "d3_internal.cuh"

namespace d3 {

namespace {

constexpr int kConsumers = 256;
constexpr int kProducerWarps = 3;      // each issues the stages s with s mod 3 == its index
constexpr int kFusedThreads = kConsumers + 32 * (kProducerWarps + 1);   // + the L2 prefetcher warp
constexpr int kStageBytes = 16384;
constexpr int kChunk = 2048;          // weight elements of one row segment
constexpr int kMaxStages = 14;
constexpr int kMaxGQ = 4;
constexpr int kAttParts = 4;          // CTAs that share one attention stream, at most
constexpr int kMaxHeads = 128;        // query heads the merge scratch is sized for
constexpr int kMaxOwnRows = 1024;     // residual-stream rows one CTA may own (d / #CTAs, rounded up)

enum PhaseKind { PH_QKV = 0, PH_OPROJ, PH_GATEUP, PH_DOWN, PH_HEAD };

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ float bfl(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bfh(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ float4 ldcg4(const float *p) { return __ldcg(reinterpret_cast<const float4 *>(p)); }
__device__ __forceinline__ uint64_t now_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

struct Ctx {
  const FusedParams *p;
  unsigned char *ring;
  float *act;
  uint64_t *full, *empty;
  volatile uint32_t *released;   // per slot: fills consumed so far
  volatile int *abort_flag;
  volatile uint32_t *progress;   // stages issued into the ring so far (producer 0's count)
  float *x_own;      // this CTA's rows of the residual stream (the rows its O-proj/down groups own)
  float2 *rope_row;  // (cos, sin) of the step's position
  int cta, ncta;
};

__device__ __forceinline__ void raise_timeout(const Ctx &c) {
  c.p->sched->status = D3_ETIMEOUT;
  *c.abort_flag = 1;
}

// Wait for an mbarrier phase for at most wait_ns.  Returns false at once when
// the CTA is in abort mode, or after raising D3_ETIMEOUT and entering it.
__device__ __forceinline__ bool wait_bar(const Ctx &c, uint32_t bar, uint32_t parity) {
  if (*c.abort_flag) return false;
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = now_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 0u) {
      if (*c.abort_flag) return false;
      if (now_ns() - t0 > c.p->wait_ns) break;
    }
  }
  raise_timeout(c);
  return false;
}

// Grid barrier number `idx` (1-based) among the consumer threads of all CTAs.
// bar.sync orders the CTA's writes before thread 0; its release-add publishes them
// at GPU scope; the acquire-load that sees the full count orders the other CTAs'
// writes before everything after the second bar.sync.
__device__ __forceinline__ void grid_barrier(const Ctx &c, unsigned idx) {
  consumer_sync();
  if (threadIdx.x == 0) {
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(c.p->bar_counter) : "memory");
    // every barrier counts the arrivals of all earlier ones; barrier_extra (0 in normal use)
    // makes the first target unreachable so that the wait can only end by its time limit
    const unsigned target = idx * (unsigned)c.ncta + (idx == 1u ? c.p->barrier_extra : 0u);
    const uint64_t t0 = now_ns();
    for (uint32_t it = 1; !*c.abort_flag; ++it) {
      unsigned v;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(c.p->bar_counter) : "memory");
      if (v >= target) break;
      if ((it & 15u) == 0u && now_ns() - t0 > c.p->wait_ns) raise_timeout(c);
    }
  }
  consumer_sync();
}

// ---- the CTA's share of a phase ---------------------------------------------
struct Phase {
  int kind;
  const bf16 *W, *W2;
  int K, R;          // row length, rows of W
  int groups;        // row groups of the phase
  int g0, g1;        // this CTA's groups
  int nkc;           // k-chunks per row
};

__device__ __forceinline__ void split_range(int total, int cta, int ncta, int &b, int &e) {
  b = (int)(((long long)total * cta) / ncta);
  e = (int)(((long long)total * (cta + 1)) / ncta);
}

__device__ __forceinline__ Phase make_phase(const FusedParams &p, int kind, int layer, int cta, int ncta) {
  Phase ph;
  ph.kind = kind;
  ph.W2 = nullptr;
  const Dims &dm = p.dm;
  if (kind == PH_QKV) { ph.W = p.layers[layer].wqkv; ph.K = dm.d; ph.R = dm.qkv_rows; ph.groups = dm.qkv_rows / 4; }
  else if (kind == PH_OPROJ) { ph.W = p.layers[layer].wo; ph.K = dm.Hq * dm.dh; ph.R = dm.d; ph.groups = dm.d / 4; }
  else if (kind == PH_GATEUP) { ph.W = p.layers[layer].w_gate; ph.W2 = p.layers[layer].w_up; ph.K = dm.d; ph.R = dm.f; ph.groups = dm.f / 2; }
  else if (kind == PH_DOWN) { ph.W = p.layers[layer].w_down; ph.K = dm.f; ph.R = dm.d; ph.groups = dm.d / 4; }
  else { ph.W = p.lm_head; ph.K = dm.d; ph.R = dm.V; ph.groups = (dm.V + 3) / 4; }
  split_range(ph.groups, cta, ncta, ph.g0, ph.g1);
  ph.nkc = (ph.K + kChunk - 1) / kChunk;
  return ph;
}

// pointer of weight row j (0..3) of group g (rows beyond R are clamped)
__device__ __forceinline__ const bf16 *group_row(const Phase &ph, const Dims &dm, int g, int j) {
  int r;
  if (ph.kind == PH_QKV) {
    const int per_head = dm.dh / 4, half = dm.dh / 2;
    const int rot_groups = (dm.Hq + dm.Hkv) * per_head;
    if (g < rot_groups) {   // q or k head: two rotary pairs (jj, jj+half), (jj+1, jj+1+half)
      const int head = g / per_head, jj = (g % per_head) * 2;
      r = head * dm.dh + jj + (j & 1) + (j >> 1) * half;
    } else {
      r = (dm.Hq + dm.Hkv) * dm.dh + (g - rot_groups) * 4 + j;
    }
  } else if (ph.kind == PH_GATEUP) {
    r = 2 * g + (j & 1);   // rows 0,1: gate; rows 2,3: up
  } else {
    r = 4 * g + j;
  }
  if (r >= ph.R) r = ph.R - 1;
  const bf16 *base = (ph.kind == PH_GATEUP && j >= 2) ? ph.W2 : ph.W;
  return base + (size_t)r * ph.K;
}

// ---- attention work split ----------------------------------------------------
// Streams: (kv head, group of GQ query heads).  A stream's positions 0..pos are
// cut into chunks of CH positions (8 KB of K); the last chunk holds the current
// position and is read with plain loads after the grid barrier, the others go
// through the ring.  Every stream is served by P CTAs (a fixed number, so that
// the merge after the barrier is a fully unrolled, single-round-trip load): part
// k of stream s takes the chunks [nch*k/P, nch*(k+1)/P) and belongs to CTA
// (s*P + k) mod #CTAs.  A part may be empty; it still writes an (empty) partial.
struct AttPlan {
  int CH, nch, streams, P, parts, gq;
  // partials in the scratch buffer: o[part][gq][dh] (unnormalised), then (max, sum)[part][gq]
  __device__ __forceinline__ float *part_o(float *base, int part, int dh) const {
    return base + (size_t)part * (gq * dh);
  }
  __device__ __forceinline__ float *part_ml(float *base, int part, int dh) const {
    return base + (size_t)parts * (gq * dh) + (size_t)part * (gq * 2);
  }
};

__device__ __forceinline__ AttPlan make_att(const FusedParams &p, int gq, int ncta) {
  AttPlan a;
  a.gq = gq;
  a.CH = (kStageBytes / 2) / (p.dm.dh * 2);
  a.nch = p.pos / a.CH + 1;
  a.streams = p.dm.Hkv * ((p.dm.Hq / p.dm.Hkv) / gq);
  a.P = ncta / a.streams;
  if (a.P > kAttParts) a.P = kAttParts;
  if (a.P < 1) a.P = 1;
  a.parts = a.streams * a.P;
  return a;
}

// ---- producers (all 32 lanes of each producer warp run this) ----------------------
__device__ __forceinline__ void l2_prefetch(const void *src, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}

struct Producer {
  const Ctx &c;
  uint32_t s;     // stages of the step enumerated so far (every producer counts them all)
  uint32_t pid;   // this warp issues the stages with s % kProducerWarps == pid
  bool ok;
  bool l2_only;   // the prefetcher: every stage, L2 prefetch only, a bounded distance ahead
  __device__ Producer(const Ctx &cc, uint32_t id) : c(cc), s(0), pid(id), ok(true), l2_only(id == (uint32_t)kProducerWarps) {}
  __device__ __forceinline__ bool mine() const { return l2_only || s % (uint32_t)kProducerWarps == pid; }
  // prefetcher: stay at most l2_window stages ahead of the ring (producer 0's count)
  __device__ __forceinline__ bool throttle() {
    const uint32_t win = c.p->l2_window;
    if (s > *c.progress + win && !*c.abort_flag) {
      const uint64_t t0 = now_ns();
      for (uint32_t it = 1; s > *c.progress + win && !*c.abort_flag; ++it) {
        __nanosleep(100);
        if ((it & 63u) == 0u && now_ns() - t0 > c.p->wait_ns) raise_timeout(c);
      }
    }
    if (*c.abort_flag) { ok = false; return false; }
    return true;
  }
  // Wait until the slot of stage s is free.  Successive fills of a slot are issued by
  // different warps, so the release counter (not the parity alone) says which fill
  // was consumed; the mbarrier wait that follows orders the consumers' reads before
  // the copy that overwrites them.
  __device__ __forceinline__ bool acquire(uint32_t &slot) {
    const uint32_t ns = (uint32_t)c.p->n_stages;
    slot = s % ns;
    const uint32_t fill = s / ns;
    if (fill > 0) {
      if (c.released[slot] < fill && !*c.abort_flag) {
        const uint64_t t0 = now_ns();
        for (uint32_t it = 1; c.released[slot] < fill && !*c.abort_flag; ++it)
          if ((it & 63u) == 0u && now_ns() - t0 > c.p->wait_ns) raise_timeout(c);
      }
      if (!wait_bar(c, smem_u32(&c.empty[slot]), (fill - 1u) & 1u)) { ok = false; return false; }
    }
    return true;
  }
  // Lane 4w+j holds the pointer of row j of group w of the current batch of eight
  // groups; the four lanes of a group issue its copies.
  __device__ void gemv_phase(const Phase &ph) {
    const Dims &dm = c.p->dm;
    const int lane = threadIdx.x & 31, w = lane >> 2, j = lane & 3;
    for (int S0 = ph.g0; S0 < ph.g1 && ok; S0 += 8) {
      const int nw = min(8, ph.g1 - S0);
      const bf16 *row = (w < nw) ? group_row(ph, dm, S0 + w, j) : nullptr;
      for (int kc = 0; kc < ph.nkc; ++kc) {
        const int kw = min(kChunk, ph.K - kc * kChunk);
        for (int ww = 0; ww < nw; ++ww, ++s) {
          if (!mine()) continue;
          if (l2_only) {
            if (!throttle()) return;
            if (w == ww) l2_prefetch(row + (size_t)kc * kChunk, (uint32_t)kw * 2u);
            continue;
          }
          uint32_t slot;
          if (!acquire(slot)) return;
          if (pid == 0 && lane == 0) *c.progress = s;
          const uint32_t bar = smem_u32(&c.full[slot]);
          // the copies may complete bytes before the expect_tx lands: the phase cannot
          // end before its one arrival (the expect_tx itself)
          if (lane == ww * 4) mbar_expect_tx(bar, 4u * (uint32_t)kw * 2u);
          if (w == ww)
            bulk_g2s(smem_u32(c.ring + (size_t)slot * kStageBytes) + j * (kChunk * 2),
                     row + (size_t)kc * kChunk, (uint32_t)kw * 2u, bar);
        }
      }
    }
  }
  __device__ void att_phase(const AttPlan &a, int layer) {
    const FusedParams &p = *c.p;
    const Dims &dm = p.dm;
    const int lane = threadIdx.x & 31;
    const int G = dm.Hq / dm.Hkv, qgroups = G / a.gq;
    for (int part = c.cta; part < a.parts && ok; part += c.ncta) {
      const int stream = part / a.P, k = part % a.P;
      const int kvh = stream / qgroups;
      const int ch0 = a.nch * k / a.P, ch1 = a.nch * (k + 1) / a.P;
      for (int chunk = ch0; chunk < ch1; ++chunk) {
        if (chunk == a.nch - 1) continue;   // the chunk with the current position: plain loads
        if (!mine()) { ++s; continue; }
        // A chunk is one run of the cache, or (paged cache with pages shorter than a chunk) one
        // run per page: lanes 2j and 2j + 1 copy K and V of run j.  Pages hold a power of two of
        // positions and chunks start at multiples of their length, so no run straddles a page.
        const int run_pos = (dm.page_size == 0 || dm.page_size >= a.CH) ? a.CH : dm.page_size;
        const int n_run = a.CH / run_pos, j = lane >> 1;
        const uint32_t run_bytes = (uint32_t)(run_pos * dm.dh * 2);
        const size_t off = j < n_run ? kv_offset(dm, dm.block_table, layer, p.slot, kvh, chunk * a.CH + j * run_pos) : 0;
        const bf16 *src = ((lane & 1) ? p.Vc : p.Kc) + off;
        if (l2_only) {
          if (!throttle()) return;
          if (j < n_run) l2_prefetch(src, run_bytes);
          ++s;
          continue;
        }
        uint32_t slot;
        if (!acquire(slot)) return;
        if (pid == 0 && lane == 0) *c.progress = s;
        const uint32_t bar = smem_u32(&c.full[slot]);
        const uint32_t dst = smem_u32(c.ring + (size_t)slot * kStageBytes);
        // (bytes may complete before the expect_tx lands: the phase cannot end before its one arrival)
        if (lane == 0) mbar_expect_tx(bar, (uint32_t)kStageBytes);
        if (j < n_run) bulk_g2s(dst + (lane & 1) * (kStageBytes / 2) + j * run_bytes, src, run_bytes, bar);
        ++s;
      }
    }
  }
};

// ---- consumer helpers ----------------------------------------------------------
__device__ __forceinline__ float block_sum(float v) {
  __shared__ float s_part[8];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  consumer_sync();
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = v;
  consumer_sync();
  float t = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) t += s_part[w];
  return t;
}

// position of element k of an activation vector in the permuted shared layout:
// within each block of 256 elements, element lane*8 + j sits at (j/4)*128 + lane*4 + j%4
__device__ __forceinline__ int act_index(int k) {
  return (k & ~255) + ((k & 7) >> 2) * 128 + ((k & 255) >> 3) * 4 + (k & 3);
}

// RMSNorm gains of the next normalised load, fetched into registers before the
// grid barrier (they are weights: nothing to wait for), so that the load after the
// barrier costs one L2 round trip only.  Widths up to 4096 take this path; wider
// vectors are normalised in two passes and read their gains in the second.
struct GainRegs {
  static constexpr int kMaxIt = 4;   // 4 * 1024 elements
  uint2 g[kMaxIt];
};
__device__ __forceinline__ void prefetch_gain(GainRegs &gr, const bf16 *gain, int K) {
  if (K > GainRegs::kMaxIt * kConsumers * 4) return;
#pragma unroll
  for (int it = 0; it < GainRegs::kMaxIt; ++it) {
    const int k = it * (kConsumers * 4) + threadIdx.x * 4;
    if (k < K) gr.g[it] = *reinterpret_cast<const uint2 *>(gain + k);
  }
}

// act := src (global fp32, length K), no normalisation.  Twelve 16-byte loads per
// thread are in flight before the first is stored: one L2 round trip per 12 K floats.
__device__ void load_act_plain(const Ctx &c, const float *src, int K) {
  constexpr int kB = 12;
  for (int k0 = 0; k0 < K; k0 += kB * kConsumers * 4) {
    float4 v[kB];
#pragma unroll
    for (int q = 0; q < kB; ++q) {
      const int k = k0 + q * (kConsumers * 4) + threadIdx.x * 4;
      if (k < K) v[q] = ldcg4(src + k);
    }
#pragma unroll
    for (int q = 0; q < kB; ++q) {
      const int k = k0 + q * (kConsumers * 4) + threadIdx.x * 4;
      if (k < K) *reinterpret_cast<float4 *>(c.act + act_index(k)) = v[q];
    }
  }
  consumer_sync();
}

// act := RMSNorm(src) * gain.  Up to 4096 elements: one pass over L2, the values wait
// in registers for the scale.  Wider: sum of squares first, then a second pass.
// `emb` (nullable): take the vector from this bf16 row instead of `src` (the embedding row of the
// step's token: a weight, every CTA reads it itself, nothing to wait for).
__device__ __forceinline__ float4 ld_src4(const float *src, const bf16 *emb, int k) {
  if (emb) {
    const uint2 w = *reinterpret_cast<const uint2 *>(emb + k);
    return make_float4(bfl(w.x), bfh(w.x), bfl(w.y), bfh(w.y));
  }
  return ldcg4(src + k);
}

__device__ void load_act_norm(const Ctx &c, const float *src, int K, const GainRegs &gr, const bf16 *gain,
                              const bf16 *emb = nullptr) {
  const int tid = threadIdx.x;
  if (K <= GainRegs::kMaxIt * kConsumers * 4) {
    float4 v[GainRegs::kMaxIt];
    float ss = 0.f;
#pragma unroll
    for (int it = 0; it < GainRegs::kMaxIt; ++it) {
      const int k = it * (kConsumers * 4) + tid * 4;
      if (k < K) {
        v[it] = ld_src4(src, emb, k);
        ss += v[it].x * v[it].x + v[it].y * v[it].y + v[it].z * v[it].z + v[it].w * v[it].w;
      }
    }
    const float scale = rsqrtf(block_sum(ss) / (float)K + c.p->eps);
#pragma unroll
    for (int it = 0; it < GainRegs::kMaxIt; ++it) {
      const int k = it * (kConsumers * 4) + tid * 4;
      if (k < K) {
        float4 t = v[it];
        const uint2 gw = gr.g[it];
        t.x *= scale * bfl(gw.x); t.y *= scale * bfh(gw.x);
        t.z *= scale * bfl(gw.y); t.w *= scale * bfh(gw.y);
        *reinterpret_cast<float4 *>(c.act + act_index(k)) = t;
      }
    }
  } else {
    float ss = 0.f;
    for (int k = tid * 4; k < K; k += kConsumers * 4) {
      const float4 t = ld_src4(src, emb, k);
      ss += t.x * t.x + t.y * t.y + t.z * t.z + t.w * t.w;
    }
    const float scale = rsqrtf(block_sum(ss) / (float)K + c.p->eps);
    for (int k = tid * 4; k < K; k += kConsumers * 4) {
      float4 t = ld_src4(src, emb, k);
      const uint2 gw = *reinterpret_cast<const uint2 *>(gain + k);
      t.x *= scale * bfl(gw.x); t.y *= scale * bfh(gw.x);
      t.z *= scale * bfl(gw.y); t.w *= scale * bfh(gw.y);
      *reinterpret_cast<float4 *>(c.act + act_index(k)) = t;
    }
  }
  consumer_sync();
}

struct Consumer {
  const Ctx &c;
  uint32_t s;     // ring stages of all finished phases (the same in every warp)
  long long ring_wait;   // cycles this thread spent waiting for ring stages (timing runs)
  __device__ Consumer(const Ctx &cc) : c(cc), s(0), ring_wait(0) {}

  // Wait until stage number `sn` (counted over the whole step) has landed.
  // Stages of one slot are consumed by different warps, and a parity wait cannot
  // tell fill k from fill k-2: so first wait until fill k-1 of the slot has been
  // consumed (the producer issues fill k only after that), then for the parity.
  // In abort mode both waits return at once and the (meaningless) work goes on.
  __device__ __forceinline__ uint32_t wait_stage(uint32_t sn) {
    const uint32_t ns = (uint32_t)c.p->n_stages;
    const uint32_t slot = sn % ns, fill = sn / ns;
    const long long tw = clock64();
    if (c.released[slot] < fill && !*c.abort_flag) {
      const uint64_t t0 = now_ns();
      for (uint32_t it = 1; c.released[slot] < fill && !*c.abort_flag; ++it)
        if ((it & 63u) == 0u && now_ns() - t0 > c.p->wait_ns) raise_timeout(c);
    }
    wait_bar(c, smem_u32(&c.full[slot]), fill & 1u);
    ring_wait += clock64() - tw;
    return slot;
  }
  // the warp that consumed stage `sn` hands the slot back to the producer
  __device__ __forceinline__ void release_stage(uint32_t slot, uint32_t sn) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) {
      c.released[slot] = sn / (uint32_t)c.p->n_stages + 1u;
      mbar_arrive(smem_u32(&c.empty[slot]));
    }
  }

  // One GEMV phase over the activation vector held in c.act.
  __device__ void gemv_phase(const Phase &ph, int layer) {
    const Dims &dm = c.p->dm;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int S0 = ph.g0; S0 < ph.g1; S0 += 8) {
      const int nw = min(8, ph.g1 - S0);
      if (warp < nw) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        const uint32_t first = s + (uint32_t)(S0 - ph.g0) * (uint32_t)ph.nkc + (uint32_t)warp;
        for (int kc = 0; kc < ph.nkc; ++kc) {
          const uint32_t sn = first + (uint32_t)(kc * nw);
          const uint32_t slot = wait_stage(sn);
          const int kw = min(kChunk, ph.K - kc * kChunk);
          const unsigned char *st = c.ring + (size_t)slot * kStageBytes + lane * 16;
          const float *a = c.act + kc * kChunk + lane * 4;
#pragma unroll 2
          for (int b = 0; b < kChunk / 256; ++b) {
            if (b * 256 + lane * 8 < kw) {
              const float4 x0 = *reinterpret_cast<const float4 *>(a + b * 256);
              const float4 x1 = *reinterpret_cast<const float4 *>(a + b * 256 + 128);
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const uint4 w = *reinterpret_cast<const uint4 *>(st + j * (kChunk * 2) + b * 512);
                acc[j] += bfl(w.x) * x0.x + bfh(w.x) * x0.y + bfl(w.y) * x0.z + bfh(w.y) * x0.w +
                          bfl(w.z) * x1.x + bfh(w.z) * x1.y + bfl(w.w) * x1.z + bfh(w.w) * x1.w;
              }
            }
          }
          release_stage(slot, sn);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], o);
        }
        if (lane == 0) epilogue(ph, dm, layer, S0 + warp, acc[0], acc[1], acc[2], acc[3]);
      }
    }
    s += (uint32_t)(ph.g1 - ph.g0) * (uint32_t)ph.nkc;
  }

  __device__ void epilogue(const Phase &ph, const Dims &dm, int layer, int g, float y0, float y1, float y2,
                           float y3) {
    const FusedParams &p = *c.p;
    if (ph.kind == PH_QKV) {
      const int per_head = dm.dh / 4, half = dm.dh / 2;
      const int rot_groups = (dm.Hq + dm.Hkv) * per_head;
      if (g < rot_groups) {
        const int head = g / per_head, jj = (g % per_head) * 2;
        const float2 cs0 = c.rope_row[jj], cs1 = c.rope_row[jj + 1];
        const float a0 = y0 * cs0.x - y2 * cs0.y, b0 = y0 * cs0.y + y2 * cs0.x;
        const float a1 = y1 * cs1.x - y3 * cs1.y, b1 = y1 * cs1.y + y3 * cs1.x;
        if (head < dm.Hq) {
          float *q = p.qkv + head * dm.dh;
          q[jj] = a0; q[jj + 1] = a1; q[jj + half] = b0; q[jj + half + 1] = b1;
        } else {
          bf16 *dst = p.Kc + kv_offset(dm, dm.block_table, layer, p.slot, head - dm.Hq, p.pos);
          dst[jj] = __float2bfloat16_rn(a0); dst[jj + 1] = __float2bfloat16_rn(a1);
          dst[jj + half] = __float2bfloat16_rn(b0); dst[jj + half + 1] = __float2bfloat16_rn(b1);
        }
      } else {
        const int r = (g - rot_groups) * 4, h = r / dm.dh, e = r % dm.dh;
        bf16 *dst = p.Vc + kv_offset(dm, dm.block_table, layer, p.slot, h, p.pos) + e;
        dst[0] = __float2bfloat16_rn(y0); dst[1] = __float2bfloat16_rn(y1);
        dst[2] = __float2bfloat16_rn(y2); dst[3] = __float2bfloat16_rn(y3);
      }
    } else if (ph.kind == PH_GATEUP) {
      p.u[2 * g] = y0 / (1.f + __expf(-y0)) * y2;
      p.u[2 * g + 1] = y1 / (1.f + __expf(-y1)) * y3;
    } else if (ph.kind == PH_HEAD) {
      const int r = 4 * g;
      if (r < ph.R) p.logits[r] = y0;
      if (r + 1 < ph.R) p.logits[r + 1] = y1;
      if (r + 2 < ph.R) p.logits[r + 2] = y2;
      if (r + 3 < ph.R) p.logits[r + 3] = y3;
    } else {   // O-proj / down: residual add on the rows this CTA owns (its own copy
               // is current: no other CTA ever writes them), published for the others
      float4 *own = reinterpret_cast<float4 *>(c.x_own + 4 * (g - ph.g0));
      float4 v = *own;
      v.x += y0; v.y += y1; v.z += y2; v.w += y3;
      *own = v;
      *reinterpret_cast<float4 *>(p.x + 4 * g) = v;
    }
  }

  // Attention of this CTA's parts.  Each part yields one partial: unnormalised o
  // [gq][dh] and (max, sum) [gq] of part stream * P + k; the partials are merged by
  // merge_load_attn after the grid barrier.
  template <int DH, int GQ>
  __device__ void att_phase(const AttPlan &a, int layer) {
    const FusedParams &p = *c.p;
    const Dims &dm = p.dm;
    constexpr int EPL = DH / 8;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, part8 = lane & 7;
    const int worker = warp * 4 + (lane >> 3);
    // the 8 lanes of a worker run the position loop in lockstep; other workers of
    // the warp may run fewer iterations, so in-loop shuffles name only the worker
    const unsigned wmask = 0xffu << (lane & 24);
    const int G = dm.Hq / dm.Hkv, qgroups = G / GQ;
    const float scale = rsqrtf((float)DH);
    uint32_t ring_k = 0;   // ring stages of this phase seen so far (every warp counts them all)
    for (int part = c.cta; part < a.parts; part += c.ncta) {
      const int stream = part / a.P, kpart = part % a.P;
      const int kvh = stream / qgroups, qg = stream % qgroups;
      const int h0 = kvh * G + qg * GQ;
      const int ch0 = a.nch * kpart / a.P, ch1 = a.nch * (kpart + 1) / a.P;
      float *dst = a.part_o(p.part, part, DH);
      float *dst_ml = a.part_ml(p.part, part, DH);
      if (ch0 == ch1) {   // nothing to do: an empty partial (weight 0 in the merge)
        for (int i = tid; i < GQ * DH; i += kConsumers) dst[i] = 0.f;
        if (tid < GQ) { dst_ml[2 * tid] = -INFINITY; dst_ml[2 * tid + 1] = 0.f; }
        continue;
      }
      float q[GQ][EPL], mx[GQ], sum[GQ], o[GQ][EPL];
#pragma unroll
      for (int g = 0; g < GQ; ++g) {
        mx[g] = -INFINITY; sum[g] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; e += 4) {
          const float4 qv = ldcg4(p.qkv + (h0 + g) * DH + part8 * EPL + e);
          q[g][e] = qv.x * scale; q[g][e + 1] = qv.y * scale;
          q[g][e + 2] = qv.z * scale; q[g][e + 3] = qv.w * scale;
          o[g][e] = o[g][e + 1] = o[g][e + 2] = o[g][e + 3] = 0.f;
        }
      }
      for (int chunk = ch0; chunk < ch1; ++chunk) {
        const bool tail = chunk == a.nch - 1;
        // a ring stage belongs to one warp (its 4 workers walk the CH positions); the
        // tail chunk is read from global memory by all 32 workers
        uint32_t slot = 0, sn = 0;
        bool mine = true;
        if (!tail) {
          mine = (ring_k & 7u) == (uint32_t)warp;
          sn = s + ring_k;
          if (mine) slot = wait_stage(sn);
          ++ring_k;
        }
        const int t0 = chunk * a.CH;
        const int cnt = tail ? (p.pos - t0 + 1) : (mine ? a.CH : 0);
        const int i0 = tail ? worker : (lane >> 3), istep = tail ? 32 : 4;
        for (int i = i0; i < cnt; i += istep) {
          float kf[EPL], vf[EPL];
          if (tail) {
            const size_t goff = kv_offset(dm, dm.block_table, layer, p.slot, kvh, t0 + i) + part8 * EPL;
            const bf16 *kp = p.Kc + goff;
            const bf16 *vp = p.Vc + goff;
#pragma unroll
            for (int e = 0; e < EPL; e += 4) {
              const uint2 kw = __ldcg(reinterpret_cast<const uint2 *>(kp + e));
              const uint2 vw = __ldcg(reinterpret_cast<const uint2 *>(vp + e));
              kf[e] = bfl(kw.x); kf[e + 1] = bfh(kw.x); kf[e + 2] = bfl(kw.y); kf[e + 3] = bfh(kw.y);
              vf[e] = bfl(vw.x); vf[e + 1] = bfh(vw.x); vf[e + 2] = bfl(vw.y); vf[e + 3] = bfh(vw.y);
            }
          } else {
            const unsigned char *ks = c.ring + (size_t)slot * kStageBytes + ((size_t)i * DH + part8 * EPL) * 2;
            const unsigned char *vs = ks + kStageBytes / 2;
#pragma unroll
            for (int e = 0; e < EPL; e += 4) {
              const uint2 kw = *reinterpret_cast<const uint2 *>(ks + e * 2);
              const uint2 vw = *reinterpret_cast<const uint2 *>(vs + e * 2);
              kf[e] = bfl(kw.x); kf[e + 1] = bfh(kw.x); kf[e + 2] = bfl(kw.y); kf[e + 3] = bfh(kw.y);
              vf[e] = bfl(vw.x); vf[e + 1] = bfh(vw.x); vf[e + 2] = bfl(vw.y); vf[e + 3] = bfh(vw.y);
            }
          }
#pragma unroll
          for (int g = 0; g < GQ; ++g) {
            float sc = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) sc += q[g][e] * kf[e];
            sc += __shfl_xor_sync(wmask, sc, 1);
            sc += __shfl_xor_sync(wmask, sc, 2);
            sc += __shfl_xor_sync(wmask, sc, 4);
            const float mn = fmaxf(mx[g], sc);
            const float corr = __expf(mx[g] - mn), pr = __expf(sc - mn);
            mx[g] = mn;
            sum[g] = sum[g] * corr + pr;
#pragma unroll
            for (int e = 0; e < EPL; ++e) o[g][e] = o[g][e] * corr + pr * vf[e];
          }
        }
        if (!tail && mine) release_stage(slot, sn);
      }
      // merge the 32 workers: 4 per warp by shuffles, 8 warps through shared memory
#pragma unroll
      for (int off = 8; off <= 16; off <<= 1) {
#pragma unroll
        for (int g = 0; g < GQ; ++g) {
          const float m2 = __shfl_xor_sync(0xffffffffu, mx[g], off);
          const float s2 = __shfl_xor_sync(0xffffffffu, sum[g], off);
          const float mn = fmaxf(mx[g], m2);
          const float c1 = (mx[g] == -INFINITY) ? 0.f : __expf(mx[g] - mn);
          const float c2 = (m2 == -INFINITY) ? 0.f : __expf(m2 - mn);
          sum[g] = sum[g] * c1 + s2 * c2;
#pragma unroll
          for (int e = 0; e < EPL; ++e) {
            const float o2 = __shfl_xor_sync(0xffffffffu, o[g][e], off);
            o[g][e] = o[g][e] * c1 + o2 * c2;
          }
          mx[g] = mn;
        }
      }
      // the activation buffer is free during attention: it holds the merge scratch
      float *s_o = c.act;                       // [8][GQ][DH]
      float *s_ml = c.act + 8 * GQ * DH;        // [8][GQ][2]
      consumer_sync();
      if (lane < 8) {
#pragma unroll
        for (int g = 0; g < GQ; ++g) {
#pragma unroll
          for (int e = 0; e < EPL; ++e) s_o[(warp * GQ + g) * DH + part8 * EPL + e] = o[g][e];
          if (lane == 0) { s_ml[(warp * GQ + g) * 2] = mx[g]; s_ml[(warp * GQ + g) * 2 + 1] = sum[g]; }
        }
      }
      consumer_sync();
      for (int i = tid; i < GQ * DH; i += kConsumers) {
        const int g = i / DH, e = i % DH;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < 8; ++w) M = fmaxf(M, s_ml[(w * GQ + g) * 2]);
        float Ls = 0.f, O = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
          const float mw = s_ml[(w * GQ + g) * 2];
          const float cf = (mw == -INFINITY) ? 0.f : __expf(mw - M);
          Ls += s_ml[(w * GQ + g) * 2 + 1] * cf;
          O += s_o[(w * GQ + g) * DH + e] * cf;
        }
        dst[g * DH + e] = O;
        if (e == 0) { dst_ml[2 * g] = M; dst_ml[2 * g + 1] = Ls; }
      }
      consumer_sync();
    }
    s += ring_k;
  }

  // act := attention output of all heads, merged from the P partials of every stream
  // (after the grid barrier).  One L2 round trip: the (max, sum) pairs and the first
  // batch of 16-byte o loads are issued before anything is used; the merge weight
  // exp(m_k - M) / sum of every (head, part) is computed once, by one thread.
  template <int DH, int GQ>
  __device__ void merge_load_attn(const AttPlan &a, float *s_pm, float *s_pl) {
    const FusedParams &p = *c.p;
    const Dims &dm = p.dm;
    const int tid = threadIdx.x;
    const int n4 = dm.Hq * DH / 4, P = a.P;
    constexpr int kMl = (kMaxHeads * kAttParts + kConsumers - 1) / kConsumers;
    float2 ml_r[kMl];
#pragma unroll
    for (int q = 0; q < kMl; ++q) {
      const int idx = q * kConsumers + tid;   // = h * P + k
      ml_r[q] = make_float2(-INFINITY, 0.f);
      if (idx < dm.Hq * P) {
        const int h = idx / P, k = idx % P;
        // heads are ordered [kv head][query group][g]: stream = h / GQ, g = h % GQ
        ml_r[q] = __ldcg(reinterpret_cast<const float2 *>(a.part_ml(p.part, (h / GQ) * P + k, DH)) + (h % GQ));
      }
    }
    constexpr int kBatch = 4;   // float4 outputs per thread and batch
    for (int j0 = 0; j0 * kConsumers < n4; j0 += kBatch) {
      float4 r[kBatch][kAttParts];
#pragma unroll
      for (int jj = 0; jj < kBatch; ++jj) {
        const int i4 = (j0 + jj) * kConsumers + tid;
#pragma unroll
        for (int k = 0; k < kAttParts; ++k) {
          r[jj][k] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (i4 < n4 && k < P) {
            const int h = (i4 * 4) / DH, e = (i4 * 4) % DH;
            r[jj][k] = ldcg4(a.part_o(p.part, (h / GQ) * P + k, DH) + (h % GQ) * DH + e);
          }
        }
      }
      if (j0 == 0) {
#pragma unroll
        for (int q = 0; q < kMl; ++q) {
          const int idx = q * kConsumers + tid;
          if (idx < dm.Hq * P) {
            s_pm[(idx / P) * kAttParts + idx % P] = ml_r[q].x;
            s_pl[(idx / P) * kAttParts + idx % P] = ml_r[q].y;
          }
        }
        consumer_sync();   // the (max, sum) table is complete
        if (tid < dm.Hq) {   // merge weights of head tid, in place of its maxima
          float M = -INFINITY;
          for (int k = 0; k < P; ++k) M = fmaxf(M, s_pm[tid * kAttParts + k]);
          float wk[kAttParts], Ls = 0.f;
#pragma unroll
          for (int k = 0; k < kAttParts; ++k) {
            wk[k] = k < P ? __expf(s_pm[tid * kAttParts + k] - M) : 0.f;   // exp(-inf) = 0: an empty part
            if (k < P) Ls += s_pl[tid * kAttParts + k] * wk[k];
          }
          const float inv = 1.f / Ls;
#pragma unroll
          for (int k = 0; k < kAttParts; ++k) s_pm[tid * kAttParts + k] = wk[k] * inv;
        }
        consumer_sync();
      }
#pragma unroll
      for (int jj = 0; jj < kBatch; ++jj) {
        const int i4 = (j0 + jj) * kConsumers + tid;
        if (i4 < n4) {
          const int h = (i4 * 4) / DH;
          float4 O = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (int k = 0; k < kAttParts; ++k) {
            if (k < P) {
              const float wgt = s_pm[h * kAttParts + k];
              O.x += r[jj][k].x * wgt; O.y += r[jj][k].y * wgt;
              O.z += r[jj][k].z * wgt; O.w += r[jj][k].w * wgt;
            }
          }
          *reinterpret_cast<float4 *>(c.act + act_index(i4 * 4)) = O;
        }
      }
    }
    consumer_sync();
  }
};

template <int DH, int GQ>
__global__ void __launch_bounds__(kFusedThreads, 1) k_step_b1(const __grid_constant__ FusedParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) uint64_t s_full[kMaxStages], s_empty[kMaxStages];
  __shared__ uint32_t s_released[kMaxStages];
  __shared__ int s_abort;
  __shared__ uint32_t s_progress;
  __shared__ long long s_tacc[kFusedPhases];
  __shared__ float s_pm[kMaxHeads * kAttParts], s_pl[kMaxHeads * kAttParts];
  __shared__ __align__(16) float s_x_own[kMaxOwnRows];
  __shared__ float2 s_rope[64];
  const int tid = threadIdx.x, warp = tid >> 5;
  Ctx c;
  c.p = &p;
  c.ring = smem;
  c.act = reinterpret_cast<float *>(smem + (size_t)p.n_stages * kStageBytes);
  c.full = s_full; c.empty = s_empty;
  c.released = s_released;
  c.abort_flag = &s_abort;
  c.progress = &s_progress;
  c.x_own = s_x_own;
  c.rope_row = s_rope;
  c.cta = blockIdx.x; c.ncta = gridDim.x;
  if (tid == 0) {
    s_abort = 0;
    s_progress = 0;
    for (int i = 0; i < p.n_stages; ++i) {
      s_released[i] = 0;
      mbar_init(smem_u32(&s_full[i]), 1);
      mbar_init(smem_u32(&s_empty[i]), 1);   // released by the one warp that consumed the stage
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  // depth schedule of the row (every thread, integers only):
  // floor(L alpha^i) = #{ n in 1..L : i < thr[n] }
  const int L = p.L;
  int n = 0;
  for (int k = 1; k <= L; ++k) n += (p.gi < p.thr[k]) ? 1 : 0;
  int lo, hi;
  if (p.anchor == D3_ANCHOR_TAIL) { lo = n; hi = L; }
  else { if (n < p.start_id) n = p.start_id; lo = p.start_id; hi = p.start_id + (L - n); }

  const AttPlan att = make_att(p, GQ, c.ncta);

  // Register budget by role (warps 8-11 and warps 0-3 / 4-7 are whole warpgroups): the
  // copy-issuing warps need few registers, the consumers get what they give up.
  if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
    // ------------------------------------------------------------ producers
    Producer pr(c, (uint32_t)(warp - 8));
    if (pr.l2_only && p.l2_window == 0) return;   // look-ahead switched off
    for (int l = 0; l < L && pr.ok; ++l) {
      if (lo <= l && l < hi) continue;
      pr.gemv_phase(make_phase(p, PH_QKV, l, c.cta, c.ncta));
      pr.att_phase(att, l);
      pr.gemv_phase(make_phase(p, PH_OPROJ, l, c.cta, c.ncta));
      pr.gemv_phase(make_phase(p, PH_GATEUP, l, c.cta, c.ncta));
      pr.gemv_phase(make_phase(p, PH_DOWN, l, c.cta, c.ncta));
    }
    if (pr.ok && p.logits) pr.gemv_phase(make_phase(p, PH_HEAD, 0, c.cta, c.ncta));
    if (!pr.ok && !pr.l2_only && (tid & 31) == 0) {
      // drain: wait (bounded) until every copy already issued has landed
      const uint32_t ns = (uint32_t)p.n_stages;
      const uint32_t first = pr.s > ns ? pr.s - ns : 0;
      for (uint32_t s = first; s < pr.s; ++s) {
        if (s % (uint32_t)kProducerWarps != pr.pid) continue;
        const uint32_t bar = smem_u32(&s_full[s % ns]);
        const uint64_t t0 = now_ns();
        const uint64_t bound = p.wait_ns > kDrainFloorNs ? p.wait_ns : kDrainFloorNs;
        while (!mbar_try_wait(bar, (s / ns) & 1u) && now_ns() - t0 < bound) {}
      }
    }
    return;
  }

  // -------------------------------------------------------------- consumers
  asm volatile("setmaxnreg.inc.sync.aligned.u32 232;");
  const int tok = p.tok_dev ? p.tok_dev[0] : p.tok;
  if (c.cta == 0 && tid == 0) {
    DevSched *s = p.sched;
    s->B = 1; s->L = L; s->n[0] = n; s->perm[0] = 0; s->slot_s[0] = p.slot; s->pos_s[0] = p.pos;
    s->tok_s[0] = tok; s->lo_s[0] = lo; s->hi_s[0] = hi;
    for (int l = 0; l < L; ++l) s->m[l] = (lo <= l && l < hi) ? 0 : 1;
    s->rows_layers = n; s->layers_touched = n;
  }
  // embedding row -> residual stream: CTA 0 publishes it, every CTA keeps its own rows
  const Dims &dm = p.dm;
  const bf16 *emb = p.embed + (size_t)tok * dm.d;
  if (c.cta == 0) {
    for (int k = tid * 8; k < dm.d; k += kConsumers * 8) {
      const uint4 w = *reinterpret_cast<const uint4 *>(emb + k);
      *reinterpret_cast<float4 *>(p.x + k) = make_float4(bfl(w.x), bfh(w.x), bfl(w.y), bfh(w.y));
      *reinterpret_cast<float4 *>(p.x + k + 4) = make_float4(bfl(w.z), bfh(w.z), bfl(w.w), bfh(w.w));
    }
  }
  {
    int og0, og1;
    split_range(dm.d / 4, c.cta, c.ncta, og0, og1);
    for (int i = tid; i < (og1 - og0) * 4; i += kConsumers)
      s_x_own[i] = __bfloat162float(emb[og0 * 4 + i]);
    for (int i = tid; i < dm.dh / 2; i += kConsumers) s_rope[i] = p.rope[(size_t)p.pos * (dm.dh / 2) + i];
  }
  Consumer cs(c);
  unsigned bidx = 0;
  // optional phase timer (thread 0 of every CTA): cycles spent up to each phase
  // boundary, summed in shared memory and written once at the end
  const bool timing = p.phase_cycles != nullptr && tid == 0;
  long long t_prev = clock64();
  if (timing)
    for (int k = 0; k < kFusedPhases; ++k) s_tacc[k] = 0;
  auto tick = [&](int k) {
    if (timing) {
      const long long t = clock64();
      s_tacc[k] += t - t_prev;
      t_prev = t;
    }
  };
  // first executed block (or L when the row runs none)
  int l = 0;
  while (l < L && lo <= l && l < hi) ++l;
  GainRegs gr;
  const bf16 *gain = l < L ? p.layers[l].attn_norm : p.final_norm;
  prefetch_gain(gr, gain, dm.d);
  consumer_sync();   // s_x_own, s_rope
  tick(0);
  // until a block has run, the residual stream is the embedding row itself: no exchange needed
  const bf16 *x_is_emb = emb;
  while (l < L) {
    int next = l + 1;   // dropped blocks: the hidden state passes through
    while (next < L && lo <= next && next < hi) ++next;
    load_act_norm(c, p.x, dm.d, gr, gain, x_is_emb);
    x_is_emb = nullptr;
    tick(1);
    cs.gemv_phase(make_phase(p, PH_QKV, l, c.cta, c.ncta), l);
    tick(2);
    grid_barrier(c, ++bidx);
    tick(3);
    cs.template att_phase<DH, GQ>(att, l);
    tick(4);
    grid_barrier(c, ++bidx);
    tick(3);
    cs.template merge_load_attn<DH, GQ>(att, s_pm, s_pl);
    tick(1);
    cs.gemv_phase(make_phase(p, PH_OPROJ, l, c.cta, c.ncta), l);
    tick(5);
    gain = p.layers[l].mlp_norm;
    prefetch_gain(gr, gain, dm.d);
    grid_barrier(c, ++bidx);
    tick(3);
    load_act_norm(c, p.x, dm.d, gr, gain);
    tick(1);
    cs.gemv_phase(make_phase(p, PH_GATEUP, l, c.cta, c.ncta), l);
    tick(6);
    grid_barrier(c, ++bidx);
    tick(3);
    load_act_plain(c, p.u, dm.f);
    tick(1);
    cs.gemv_phase(make_phase(p, PH_DOWN, l, c.cta, c.ncta), l);
    tick(7);
    gain = next < L ? p.layers[next].attn_norm : p.final_norm;
    prefetch_gain(gr, gain, dm.d);
    grid_barrier(c, ++bidx);
    tick(3);
    l = next;
  }
  if (p.logits) {
    load_act_norm(c, p.x, dm.d, gr, gain, x_is_emb);
    cs.gemv_phase(make_phase(p, PH_HEAD, 0, c.cta, c.ncta), 0);
  }
  // KV fill by copy for the dropped blocks: CTA j takes block lo + j, lo + j + ncta, ...  (after the
  // LM head: nothing in this step reads the filled entries, and the head need not wait for them)
  if (p.kv_fill == D3_FILL_COPY) {
    const int nkv = dm.Hkv * dm.dh;
    unsigned short *Ku = reinterpret_cast<unsigned short *>(p.Kc);
    unsigned short *Vu = reinterpret_cast<unsigned short *>(p.Vc);
    for (int l = lo + c.cta; l < hi; l += c.ncta) {
      for (int i = tid; i < nkv; i += kConsumers) {
        const int h = i / dm.dh, e = i % dm.dh;
        const size_t dst = kv_offset(dm, dm.block_table, l, p.slot, h, p.pos) + e;
        if (lo == 0) {
          Ku[dst] = 0;
          Vu[dst] = 0;
        } else {
          const size_t src = kv_offset(dm, dm.block_table, lo - 1, p.slot, h, p.pos) + e;
          Ku[dst] = __ldcg(Ku + src);   // written by another CTA earlier in this kernel
          Vu[dst] = __ldcg(Vu + src);
        }
      }
    }
  }
  tick(8);
  if (timing) {
    s_tacc[9] = cs.ring_wait;
    for (int k = 0; k < kFusedPhases; ++k) p.phase_cycles[c.cta * kFusedPhases + k] += s_tacc[k];
  }
}

}  // namespace

// ------------------------------------------------------------------ host side
struct FusedPlan {
  int grid, n_stages, act_floats;
  size_t smem;
  void *func;
};

template <int DH, int GQ>
static bool try_plan(FusedPlan &pl, const d3_config &c) {
  int dev = 0, sms = 0, optin = 0, coop = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
  if (!coop || sms < 1) return false;
  const int ctas = sms < kFusedMaxCtas ? sms : kFusedMaxCtas;
  if ((c.d_model / 4 / ctas + 2) * 4 > kMaxOwnRows) return false;   // the CTA's own rows of x
  int need = c.d_model;
  if (c.d_ffn > need) need = c.d_ffn;
  if (c.n_q_heads * c.head_dim > need) need = c.n_q_heads * c.head_dim;
  need = (need + kChunk - 1) / kChunk * kChunk;
  const int att_need = 8 * kMaxGQ * (128 + 2);
  if (c.n_q_heads > kMaxHeads) return false;
  if (need < att_need) need = (att_need + kChunk - 1) / kChunk * kChunk;
  const int reserve = 12288;  // static shared memory of the kernel and slack
  int stages = (optin - reserve - need * 4) / kStageBytes;
  if (stages > kMaxStages) stages = kMaxStages;
  if (const char *env = getenv("D3_FUSED_STAGES")) {   // tuning knob: a shallower ring
    const int want = atoi(env);
    if (want >= 3 && want < stages) stages = want;
  }
  if (stages < 3) return false;
  pl.n_stages = stages;
  pl.act_floats = need;
  pl.smem = (size_t)stages * kStageBytes + (size_t)need * 4;
  pl.func = (void *)k_step_b1<DH, GQ>;
  if (cudaFuncSetAttribute(k_step_b1<DH, GQ>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem) !=
      cudaSuccess)
    return false;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_step_b1<DH, GQ>, kFusedThreads, pl.smem) !=
          cudaSuccess ||
      per_sm < 1)
    return false;
  pl.grid = sms < kFusedMaxCtas ? sms : kFusedMaxCtas;
  if (const char *env = getenv("D3_FUSED_CTAS")) {   // tuning knob: fewer CTAs than SMs
    const int want = atoi(env);
    if (want >= 8 && want < pl.grid) pl.grid = want;
  }
  return true;
}

int fused_plan(const d3_config &c, int *grid, int *n_stages, int *act_floats, size_t *smem, void **func) {
  FusedPlan pl;
  memset(&pl, 0, sizeof(pl));
  const int G = c.n_q_heads / c.n_kv_heads;
  const int gq = (G % 4 == 0) ? 4 : (G % 2 == 0) ? 2 : 1;
  bool ok = false;
  if (c.vocab % 4 == 0 && c.d_model <= 16 * 1024) {
    if (c.head_dim == 128 && gq == 1) ok = try_plan<128, 1>(pl, c);
    else if (c.head_dim == 128 && gq == 4) ok = try_plan<128, 4>(pl, c);
    else if (c.head_dim == 64 && gq == 1) ok = try_plan<64, 1>(pl, c);
    else if (c.head_dim == 32 && gq == 4) ok = try_plan<32, 4>(pl, c);
  }
  cudaGetLastError();   // a failed attribute call must not poison later launches
  if (!ok) return 0;
  *grid = pl.grid; *n_stages = pl.n_stages; *act_floats = pl.act_floats; *smem = pl.smem; *func = pl.func;
  return 1;
}

uint32_t fused_l2_window() {
  // 12 stages of 16 KB per CTA: ~29 MB over 148 CTAs, ~4.5 us of HBM time on top of the ring;
  // measured: 8-16 help, 24 and more lose to L2 evictions before use
  uint32_t w = 12;
  if (const char *env = getenv("D3_FUSED_L2_WINDOW")) {
    const int v = atoi(env);
    if (v == 0 || (v >= 4 && v <= 256)) w = (uint32_t)v;   // below 4 the prefetcher could not finish
  }
  return w;
}

int launch_fused_step(void *func, int grid, size_t smem, FusedParams &fp, cudaStream_t st) {
  // grid-barrier counter and per-stream arrival counters start every step at zero
  if (cudaMemsetAsync(fp.bar_counter, 0, kFusedSyncBytes, st) != cudaSuccess) return -1;
  void *args[] = {(void *)&fp};
  if (cudaLaunchCooperativeKernel(func, dim3(grid), dim3(kFusedThreads), args, smem, st) != cudaSuccess)
    return -1;
  return 1;
}

}  // namespace d3

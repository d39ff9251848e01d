// Batch-1 decode step as ONE persistent cooperative kernel (sm_100a).
//
// One CTA per SM.  Warp 8 is the producer: it streams the CTA's share of every
// weight matrix (and of the static part of the KV cache) through a
// shared-memory ring with bulk asynchronous copies (cp.async.bulk + mbarrier
// transaction counts).  It never waits for the computation, so HBM stays busy
// across phase boundaries: weights do not depend on activations.  Each ring
// stage is consumed by ONE of the warps 0-7 (stage s of a phase by warp s mod 8),
// so the warps work on eight stages at a time and never synchronise inside a
// projection.  Phases of a block (RMSNorm+QKV+RoPE+KV append | attention |
// O-proj+residual | RMSNorm+gate/up+SwiGLU | down+residual) are separated by
// grid barriers on a global counter; only the small fp32 activations cross them
// (through L2, read with ld.global.cg).
//
// A ring stage holds eight weight-row segments of 1024 bf16 (a "row group" x
// k-chunk; rows 2112 bytes apart so that the fragment loads below do not
// collide on banks), or 8 KB of K plus 8 KB of V for one KV head.  Row groups
// are issued eight at a time, k-chunk major, so that warp w keeps the running
// sums of group w in registers across the k-chunks and finishes the group
// alone (epilogue included).
//
// The dot products run on the tensor cores (mma.sync m16n8k16, bf16 x bf16 ->
// fp32) purely to cut the instruction count: widening and multiplying 8192
// weights per stage on the FP32 pipe costs ~1000 warp-instructions and made the
// consumer, not HBM, the bottleneck (see profiles/).  The MMA's 8-wide operand
// is the eight weight rows; its 16-high operand holds the activation vector
// split into two bf16 terms, x = hi + lo with hi = bf16(x), lo = bf16(x - hi),
// whose partial sums are added in fp32, so the activation keeps ~16 mantissa
// bits (the weights themselves are bf16).  A lane loads 8 consecutive k of its
// weight row and of its activation term with one 128-bit shared load each and
// feeds two MMAs; the order of k inside an MMA is a private permutation that
// both operands share.
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
constexpr int kFusedThreads = 288;
constexpr int kChunk = 1024;          // weight elements of one row segment
constexpr int kGroupRows = 8;         // weight rows of one ring stage
constexpr int kRowStride = kChunk * 2 + 64;            // bytes between row segments in a stage
constexpr int kStageBytes = kGroupRows * kRowStride;   // 16896
constexpr int kKvHalf = 8192;         // bytes of K (and of V) in an attention stage
constexpr int kMaxStages = 14;
constexpr int kMaxGQ = 4;

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
__device__ __forceinline__ void grid_barrier(const Ctx &c, unsigned idx) {
  consumer_sync();
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(c.p->bar_counter, 1u);
    const unsigned target = idx * (unsigned)c.ncta;
    const uint64_t t0 = now_ns();
    for (uint32_t it = 1; !*c.abort_flag; ++it) {
      unsigned v;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(c.p->bar_counter) : "memory");
      if (v >= target) break;
      if ((it & 15u) == 0u && now_ns() - t0 > c.p->wait_ns) raise_timeout(c);
    }
    __threadfence();
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
  if (kind == PH_QKV) { ph.W = p.layers[layer].wqkv; ph.K = dm.d; ph.R = dm.qkv_rows; ph.groups = dm.qkv_rows / 8; }
  else if (kind == PH_OPROJ) { ph.W = p.layers[layer].wo; ph.K = dm.Hq * dm.dh; ph.R = dm.d; ph.groups = dm.d / 8; }
  else if (kind == PH_GATEUP) { ph.W = p.layers[layer].w_gate; ph.W2 = p.layers[layer].w_up; ph.K = dm.d; ph.R = dm.f; ph.groups = dm.f / 4; }
  else if (kind == PH_DOWN) { ph.W = p.layers[layer].w_down; ph.K = dm.f; ph.R = dm.d; ph.groups = dm.d / 8; }
  else { ph.W = p.lm_head; ph.K = dm.d; ph.R = dm.V; ph.groups = (dm.V + 7) / 8; }
  split_range(ph.groups, cta, ncta, ph.g0, ph.g1);
  ph.nkc = (ph.K + kChunk - 1) / kChunk;
  return ph;
}

// pointer of weight row n (0..7) of group g (rows beyond R are clamped)
//   QKV, q/k heads: four rotary pairs: rows jj..jj+3 and their partners jj+half..
//   gate/up: four gate rows and the four up rows of the same outputs
__device__ __forceinline__ const bf16 *group_row(const Phase &ph, const Dims &dm, int g, int n) {
  int r;
  if (ph.kind == PH_QKV) {
    const int per_head = dm.dh / 8, half = dm.dh / 2;
    const int rot_groups = (dm.Hq + dm.Hkv) * per_head;
    if (g < rot_groups) {
      const int head = g / per_head, jj = (g % per_head) * 4;
      r = head * dm.dh + jj + (n & 3) + (n >> 2) * half;
    } else {
      r = (dm.Hq + dm.Hkv) * dm.dh + (g - rot_groups) * 8 + n;
    }
  } else if (ph.kind == PH_GATEUP) {
    r = 4 * g + (n & 3);
  } else {
    r = 8 * g + n;
  }
  if (r >= ph.R) r = ph.R - 1;
  const bf16 *base = (ph.kind == PH_GATEUP && n >= 4) ? ph.W2 : ph.W;
  return base + (size_t)r * ph.K;
}

// ---- attention work split ----------------------------------------------------
// Streams: (kv head, group of GQ query heads).  A stream's positions 0..pos are
// cut into chunks of CH positions (8 KB of K); the last chunk holds the current
// position and is read with plain loads after the grid barrier, the others go
// through the ring.  Units u = stream * nch + chunk are dealt to CTAs in
// contiguous ranges.
struct AttSplit {
  int CH, nch, streams, units, u0, u1, gq;
};

__device__ __forceinline__ AttSplit make_att(const FusedParams &p, int gq, int cta, int ncta) {
  AttSplit a;
  a.gq = gq;
  a.CH = kKvHalf / (p.dm.dh * 2);
  a.nch = p.pos / a.CH + 1;
  a.streams = p.dm.Hkv * ((p.dm.Hq / p.dm.Hkv) / gq);
  a.units = a.streams * a.nch;
  split_range(a.units, cta, ncta, a.u0, a.u1);
  return a;
}

__device__ __forceinline__ int cta_of_unit(int u, int units, int ncta) {
  int c = (int)(((long long)u * ncta) / units);
  if (c >= ncta) c = ncta - 1;
  while (c + 1 < ncta && (int)(((long long)units * (c + 1)) / ncta) <= u) ++c;
  while (c > 0 && (int)(((long long)units * c) / ncta) > u) --c;
  return c;
}

// ---- producer (all 32 lanes of warp 8 run it) -----------------------------------
struct Producer {
  const Ctx &c;
  uint32_t s;   // stages issued so far
  bool ok;
  __device__ Producer(const Ctx &cc) : c(cc), s(0), ok(true) {}
  __device__ __forceinline__ bool acquire(uint32_t &slot) {
    const uint32_t ns = (uint32_t)c.p->n_stages;
    slot = s % ns;
    if (s >= ns) {
      if (!wait_bar(c, smem_u32(&c.empty[slot]), ((s / ns) - 1u) & 1u)) { ok = false; return false; }
    }
    return true;
  }
  // Lane 4w+j holds the pointers of rows j and j+4 of group w of the current batch
  // of eight groups; the four lanes of a group issue its eight copies.
  __device__ void gemv_phase(const Phase &ph) {
    const Dims &dm = c.p->dm;
    const int lane = threadIdx.x & 31, w = lane >> 2, j = lane & 3;
    for (int S0 = ph.g0; S0 < ph.g1 && ok; S0 += 8) {
      const int nw = min(8, ph.g1 - S0);
      const bf16 *row_a = nullptr, *row_b = nullptr;
      if (w < nw) {
        row_a = group_row(ph, dm, S0 + w, j);
        row_b = group_row(ph, dm, S0 + w, j + 4);
      }
      for (int kc = 0; kc < ph.nkc; ++kc) {
        const int kw = min(kChunk, ph.K - kc * kChunk);
        for (int ww = 0; ww < nw; ++ww) {
          uint32_t slot;
          if (!acquire(slot)) return;
          const uint32_t bar = smem_u32(&c.full[slot]);
          if (lane == ww * 4) mbar_expect_tx(bar, (uint32_t)kGroupRows * (uint32_t)kw * 2u);
          __syncwarp();
          if (w == ww) {
            const uint32_t dst = smem_u32(c.ring + (size_t)slot * kStageBytes);
            bulk_g2s(dst + j * kRowStride, row_a + (size_t)kc * kChunk, (uint32_t)kw * 2u, bar);
            bulk_g2s(dst + (j + 4) * kRowStride, row_b + (size_t)kc * kChunk, (uint32_t)kw * 2u, bar);
          }
          ++s;
        }
      }
    }
  }
  __device__ void att_phase(const AttSplit &a, int layer) {
    const FusedParams &p = *c.p;
    const Dims &dm = p.dm;
    const int lane = threadIdx.x & 31;
    const int G = dm.Hq / dm.Hkv, qgroups = G / a.gq;
    for (int u = a.u0; u < a.u1 && ok; ++u) {
      const int stream = u / a.nch, chunk = u % a.nch;
      if (chunk == a.nch - 1) continue;   // the chunk with the current position: plain loads
      const int kvh = stream / qgroups;
      uint32_t slot;
      if (!acquire(slot)) return;
      const size_t off = ((((size_t)layer * dm.max_slots + p.slot) * dm.Hkv + kvh) * dm.max_seq +
                          (size_t)chunk * a.CH) * dm.dh;
      const uint32_t bar = smem_u32(&c.full[slot]);
      const uint32_t dst = smem_u32(c.ring + (size_t)slot * kStageBytes);
      if (lane == 0) mbar_expect_tx(bar, 2u * (uint32_t)kKvHalf);
      __syncwarp();
      if (lane == 0) bulk_g2s(dst, p.Kc + off, kKvHalf, bar);
      if (lane == 1) bulk_g2s(dst + kKvHalf, p.Vc + off, kKvHalf, bar);
      ++s;
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

// The activation vector of a projection sits in shared memory as two bf16
// arrays, x = hi + lo (hi = bf16(x), lo = bf16(x - hi)), lo 64 bytes past a
// multiple of 128 after hi so that the two terms land on different banks.
__device__ __forceinline__ uint32_t act_lo_offset(int K) {   // bytes from hi to lo
  return (uint32_t)((K * 2 + 127) / 128 * 128 + 64);
}

__device__ __forceinline__ void store_split4(unsigned char *act, uint32_t lo_off, int k, float4 t) {
  const __nv_bfloat16 h0 = __float2bfloat16_rn(t.x), h1 = __float2bfloat16_rn(t.y);
  const __nv_bfloat16 h2 = __float2bfloat16_rn(t.z), h3 = __float2bfloat16_rn(t.w);
  const __nv_bfloat16 l0 = __float2bfloat16_rn(t.x - __bfloat162float(h0));
  const __nv_bfloat16 l1 = __float2bfloat16_rn(t.y - __bfloat162float(h1));
  const __nv_bfloat16 l2 = __float2bfloat16_rn(t.z - __bfloat162float(h2));
  const __nv_bfloat16 l3 = __float2bfloat16_rn(t.w - __bfloat162float(h3));
  uint2 hv, lv;
  hv.x = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
  hv.y = (uint32_t)__bfloat16_as_ushort(h2) | ((uint32_t)__bfloat16_as_ushort(h3) << 16);
  lv.x = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
  lv.y = (uint32_t)__bfloat16_as_ushort(l2) | ((uint32_t)__bfloat16_as_ushort(l3) << 16);
  *reinterpret_cast<uint2 *>(act + (size_t)k * 2) = hv;
  *reinterpret_cast<uint2 *>(act + lo_off + (size_t)k * 2) = lv;
}

// act := src (global fp32, length K) split into hi/lo.  With `gain` the vector
// (K <= 16 * 1024, the model width) is RMS-normalised first: one pass over L2,
// the values wait in registers for the scale.
__device__ void load_act(const Ctx &c, const float *src, int K, const bf16 *gain) {
  const int tid = threadIdx.x;
  unsigned char *act = reinterpret_cast<unsigned char *>(c.act);
  const uint32_t lo_off = act_lo_offset(K);
  if (!gain) {
#pragma unroll 4
    for (int k = tid * 4; k < K; k += kConsumers * 4) store_split4(act, lo_off, k, ldcg4(src + k));
    consumer_sync();
    return;
  }
  constexpr int kMaxIt = 16;   // 16 * 1024 floats
  float4 v[kMaxIt];
  float ss = 0.f;
#pragma unroll
  for (int it = 0; it < kMaxIt; ++it) {
    const int k = it * (kConsumers * 4) + tid * 4;
    if (k < K) {
      v[it] = ldcg4(src + k);
      ss += v[it].x * v[it].x + v[it].y * v[it].y + v[it].z * v[it].z + v[it].w * v[it].w;
    }
  }
  const float scale = rsqrtf(block_sum(ss) / (float)K + c.p->eps);
#pragma unroll
  for (int it = 0; it < kMaxIt; ++it) {
    const int k = it * (kConsumers * 4) + tid * 4;
    if (k < K) {
      float4 t = v[it];
      const uint2 gw = *reinterpret_cast<const uint2 *>(gain + k);
      t.x *= scale * bfl(gw.x); t.y *= scale * bfh(gw.x);
      t.z *= scale * bfl(gw.y); t.w *= scale * bfh(gw.y);
      store_split4(act, lo_off, k, t);
    }
  }
  consumer_sync();
}

__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  // rows 8..15 of the 16-high operand (a1, a3) are zero
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
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

  // One GEMV phase over the activation vector held (split) in c.act.
  // Lane (g = lane / 4, t = lane % 4) loads k = 8t..8t+7 of every 32-wide step from
  // weight row g of the stage, and (g < 2) from activation term g; after the last
  // k-chunk lane t < 4 of term 0 plus lane t + 4 of term 1 hold the outputs of rows
  // 2t and 2t + 1 of the group.
  __device__ void gemv_phase(const Phase &ph, int layer) {
    const Dims &dm = c.p->dm;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const unsigned char *act = reinterpret_cast<const unsigned char *>(c.act);
    const uint32_t lo_off = act_lo_offset(ph.K);
    const unsigned char *a_lane = act + (g == 1 ? lo_off : 0u) + t * 16;
    for (int S0 = ph.g0; S0 < ph.g1; S0 += 8) {
      const int nw = min(8, ph.g1 - S0);
      if (warp < nw) {
        float d0[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};
        const uint32_t first = s + (uint32_t)(S0 - ph.g0) * (uint32_t)ph.nkc + (uint32_t)warp;
        for (int kc = 0; kc < ph.nkc; ++kc) {
          const uint32_t sn = first + (uint32_t)(kc * nw);
          const uint32_t slot = wait_stage(sn);
          const int kw = min(kChunk, ph.K - kc * kChunk);
          const unsigned char *w_lane = c.ring + (size_t)slot * kStageBytes + g * kRowStride + t * 16;
          const unsigned char *a_kc = a_lane + (size_t)kc * (kChunk * 2);
#pragma unroll 4
          for (int k0 = 0; k0 < kw; k0 += 32) {
            uint4 wv = make_uint4(0u, 0u, 0u, 0u), av = make_uint4(0u, 0u, 0u, 0u);
            if (k0 + t * 8 < kw) {
              wv = *reinterpret_cast<const uint4 *>(w_lane + k0 * 2);
              if (g < 2) av = *reinterpret_cast<const uint4 *>(a_kc + k0 * 2);
            }
            mma_bf16(d0, av.x, av.y, wv.x, wv.y);
            mma_bf16(d1, av.z, av.w, wv.z, wv.w);
          }
          release_stage(slot, sn);
        }
        // hi + lo terms: lanes 4..7 (term 1) onto lanes 0..3 (term 0)
        float y0 = d0[0] + d1[0], y1 = d0[1] + d1[1];
        y0 += __shfl_down_sync(0xffffffffu, y0, 4);
        y1 += __shfl_down_sync(0xffffffffu, y1, 4);
        // rows n and n + 4 of the group pair up (rotary pair, gate with up): lanes 0,1
        // fetch rows 4..7 from lanes 2,3
        const float p0 = __shfl_down_sync(0xffffffffu, y0, 2), p1 = __shfl_down_sync(0xffffffffu, y1, 2);
        if (lane < 4) epilogue(ph, dm, layer, S0 + warp, lane, y0, y1, p0, p1);
      }
    }
    s += (uint32_t)(ph.g1 - ph.g0) * (uint32_t)ph.nkc;
  }

  // Lane t (0..3) holds y0, y1 = outputs of rows 2t, 2t+1 of group g; lanes 0,1 also
  // hold p0, p1 = outputs of rows 2t+4, 2t+5.
  __device__ void epilogue(const Phase &ph, const Dims &dm, int layer, int g, int t, float y0, float y1,
                           float p0, float p1) {
    const FusedParams &p = *c.p;
    if (ph.kind == PH_QKV) {
      const int per_head = dm.dh / 8, half = dm.dh / 2;
      const int rot_groups = (dm.Hq + dm.Hkv) * per_head;
      const size_t cbase = ((size_t)layer * dm.max_slots + p.slot) * dm.Hkv;
      if (g < rot_groups) {
        if (t >= 2) return;
        const int head = g / per_head, jj = (g % per_head) * 4 + 2 * t;
        const float2 cs0 = p.rope[(size_t)p.pos * half + jj], cs1 = p.rope[(size_t)p.pos * half + jj + 1];
        const float a0 = y0 * cs0.x - p0 * cs0.y, b0 = y0 * cs0.y + p0 * cs0.x;
        const float a1 = y1 * cs1.x - p1 * cs1.y, b1 = y1 * cs1.y + p1 * cs1.x;
        if (head < dm.Hq) {
          float *q = p.qkv + head * dm.dh;
          q[jj] = a0; q[jj + 1] = a1; q[jj + half] = b0; q[jj + half + 1] = b1;
        } else {
          bf16 *dst = p.Kc + ((cbase + (head - dm.Hq)) * dm.max_seq + p.pos) * dm.dh;
          dst[jj] = __float2bfloat16_rn(a0); dst[jj + 1] = __float2bfloat16_rn(a1);
          dst[jj + half] = __float2bfloat16_rn(b0); dst[jj + half + 1] = __float2bfloat16_rn(b1);
        }
      } else {
        const int r = (g - rot_groups) * 8 + 2 * t, h = r / dm.dh, e = r % dm.dh;
        bf16 *dst = p.Vc + ((cbase + h) * dm.max_seq + p.pos) * dm.dh + e;
        dst[0] = __float2bfloat16_rn(y0); dst[1] = __float2bfloat16_rn(y1);
      }
    } else if (ph.kind == PH_GATEUP) {
      if (t >= 2) return;
      p.u[4 * g + 2 * t] = y0 / (1.f + __expf(-y0)) * p0;
      p.u[4 * g + 2 * t + 1] = y1 / (1.f + __expf(-y1)) * p1;
    } else if (ph.kind == PH_HEAD) {
      const int r = 8 * g + 2 * t;
      if (r < ph.R) p.logits[r] = y0;
      if (r + 1 < ph.R) p.logits[r + 1] = y1;
    } else {   // O-proj / down: residual add on the rows this CTA owns
      float2 *xp = reinterpret_cast<float2 *>(p.x + 8 * g + 2 * t);
      float2 v = __ldcg(xp);
      v.x += y0; v.y += y1;
      *xp = v;
    }
  }

  // Attention of this CTA's units.  Each stream segment yields one partial
  // (max, sum, o) in part[(stream * ncta + cta)][gq][dh + 2]; the CTA whose
  // arrival completes a stream merges the stream's partials into attn_out.
  template <int DH, int GQ>
  __device__ void att_phase(const AttSplit &a, int layer, unsigned ordinal) {
    const FusedParams &p = *c.p;
    const Dims &dm = p.dm;
    constexpr int EPL = DH / 8;
    __shared__ int s_nseg, s_last;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, part = lane & 7;
    const int worker = warp * 4 + (lane >> 3);
    // the 8 lanes of a worker run the position loop in lockstep; other workers of
    // the warp may run fewer iterations, so in-loop shuffles name only the worker
    const unsigned wmask = 0xffu << (lane & 24);
    const int G = dm.Hq / dm.Hkv, qgroups = G / GQ;
    const float scale = rsqrtf((float)DH);
    int u = a.u0;
    uint32_t ring_k = 0;   // ring stages of this phase seen so far (every warp counts them all)
    while (u < a.u1) {
      const int stream = u / a.nch;
      const int kvh = stream / qgroups, qg = stream % qgroups;
      const int h0 = kvh * G + qg * GQ;
      const int u_end = min(a.u1, (stream + 1) * a.nch);
      float q[GQ][EPL], mx[GQ], sum[GQ], o[GQ][EPL];
#pragma unroll
      for (int g = 0; g < GQ; ++g) {
        mx[g] = -INFINITY; sum[g] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
          q[g][e] = __ldcg(p.qkv + (h0 + g) * DH + part * EPL + e) * scale;
          o[g][e] = 0.f;
        }
      }
      for (; u < u_end; ++u) {
        const int chunk = u % a.nch;
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
        const size_t goff = ((((size_t)layer * dm.max_slots + p.slot) * dm.Hkv + kvh) * dm.max_seq + t0) * DH;
        for (int i = i0; i < cnt; i += istep) {
          float kf[EPL], vf[EPL];
          if (tail) {
            const bf16 *kp = p.Kc + goff + (size_t)i * DH + part * EPL;
            const bf16 *vp = p.Vc + goff + (size_t)i * DH + part * EPL;
#pragma unroll
            for (int e = 0; e < EPL; e += 4) {
              const uint2 kw = __ldcg(reinterpret_cast<const uint2 *>(kp + e));
              const uint2 vw = __ldcg(reinterpret_cast<const uint2 *>(vp + e));
              kf[e] = bfl(kw.x); kf[e + 1] = bfh(kw.x); kf[e + 2] = bfl(kw.y); kf[e + 3] = bfh(kw.y);
              vf[e] = bfl(vw.x); vf[e + 1] = bfh(vw.x); vf[e + 2] = bfl(vw.y); vf[e + 3] = bfh(vw.y);
            }
          } else {
            const unsigned char *ks = c.ring + (size_t)slot * kStageBytes + ((size_t)i * DH + part * EPL) * 2;
            const unsigned char *vs = ks + kKvHalf;
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
      int *s_list = reinterpret_cast<int *>(c.act + 8 * GQ * (DH + 2));   // CTAs holding a partial
      float *s_pm = c.act + 8 * GQ * (DH + 2) + kFusedMaxCtas;            // [seg][kMaxGQ] max
      float *s_pl = s_pm + kFusedMaxCtas * kMaxGQ;                        // [seg][kMaxGQ] sum
      consumer_sync();
      if (lane < 8) {
#pragma unroll
        for (int g = 0; g < GQ; ++g) {
#pragma unroll
          for (int e = 0; e < EPL; ++e) s_o[(warp * GQ + g) * DH + part * EPL + e] = o[g][e];
          if (lane == 0) { s_ml[(warp * GQ + g) * 2] = mx[g]; s_ml[(warp * GQ + g) * 2 + 1] = sum[g]; }
        }
      }
      consumer_sync();
      float *dst = p.part + ((size_t)stream * c.ncta + c.cta) * (GQ * (DH + 2));
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
        dst[g * (DH + 2) + e] = O;
        if (e == 0) { dst[g * (DH + 2) + DH] = M; dst[g * (DH + 2) + DH + 1] = Ls; }
      }
      consumer_sync();
      // Publish the partial.  The CTA whose arrival completes the stream merges all
      // of the stream's partials into attn_out; the others go on to the barrier.
      if (tid == 0) {
        const int c0 = cta_of_unit(stream * a.nch, a.units, c.ncta);
        const int c1 = cta_of_unit((stream + 1) * a.nch - 1, a.units, c.ncta);
        int nseg = 0;
        for (int cc = c0; cc <= c1; ++cc)   // a CTA with an empty range wrote nothing
          if ((long long)a.units * cc / c.ncta != (long long)a.units * (cc + 1) / c.ncta) s_list[nseg++] = cc;
        __threadfence();
        const unsigned old = atomicAdd(p.stream_count + stream, 1u);
        s_nseg = nseg;
        s_last = (old + 1u == (unsigned)nseg * ordinal) ? 1 : 0;
      }
      consumer_sync();
      if (s_last) {
        __threadfence();
        const int nseg = s_nseg;
        for (int i = tid; i < nseg * GQ; i += kConsumers) {
          const int sg = i / GQ, g = i % GQ;
          const float *src = p.part + ((size_t)stream * c.ncta + s_list[sg]) * (GQ * (DH + 2)) + g * (DH + 2);
          s_pm[sg * kMaxGQ + g] = __ldcg(src + DH);
          s_pl[sg * kMaxGQ + g] = __ldcg(src + DH + 1);
        }
        consumer_sync();
        for (int i = tid; i < GQ * DH; i += kConsumers) {
          const int g = i / DH, e = i % DH;
          float M = -INFINITY;
          for (int sg = 0; sg < nseg; ++sg) M = fmaxf(M, s_pm[sg * kMaxGQ + g]);
          float Ls = 0.f, O = 0.f;
#pragma unroll 4
          for (int sg = 0; sg < nseg; ++sg) {
            const float cf = __expf(s_pm[sg * kMaxGQ + g] - M);
            Ls += s_pl[sg * kMaxGQ + g] * cf;
            O += __ldcg(p.part + ((size_t)stream * c.ncta + s_list[sg]) * (GQ * (DH + 2)) + g * (DH + 2) + e) * cf;
          }
          p.attn_out[(h0 + g) * DH + e] = O / Ls;
        }
      }
      consumer_sync();
    }
    s += ring_k;
  }
};

template <int DH, int GQ>
__global__ void __launch_bounds__(kFusedThreads, 1) k_step_b1(const __grid_constant__ FusedParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) uint64_t s_full[kMaxStages], s_empty[kMaxStages];
  __shared__ uint32_t s_released[kMaxStages];
  __shared__ int s_abort;
  const int tid = threadIdx.x, warp = tid >> 5;
  Ctx c;
  c.p = &p;
  c.ring = smem;
  c.act = reinterpret_cast<float *>(smem + (size_t)p.n_stages * kStageBytes);
  c.full = s_full; c.empty = s_empty;
  c.released = s_released;
  c.abort_flag = &s_abort;
  c.cta = blockIdx.x; c.ncta = gridDim.x;
  if (tid == 0) {
    s_abort = 0;
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

  const AttSplit att = make_att(p, GQ, c.cta, c.ncta);

  if (warp == 8) {
    // ------------------------------------------------------------ producer
    Producer pr(c);
    for (int l = 0; l < L && pr.ok; ++l) {
      if (lo <= l && l < hi) continue;
      pr.gemv_phase(make_phase(p, PH_QKV, l, c.cta, c.ncta));
      pr.att_phase(att, l);
      pr.gemv_phase(make_phase(p, PH_OPROJ, l, c.cta, c.ncta));
      pr.gemv_phase(make_phase(p, PH_GATEUP, l, c.cta, c.ncta));
      pr.gemv_phase(make_phase(p, PH_DOWN, l, c.cta, c.ncta));
    }
    if (pr.ok && p.logits) pr.gemv_phase(make_phase(p, PH_HEAD, 0, c.cta, c.ncta));
    if (!pr.ok && (tid & 31) == 0) {
      // drain: wait (bounded) until every copy already issued has landed
      const uint32_t ns = (uint32_t)p.n_stages;
      const uint32_t first = pr.s > ns ? pr.s - ns : 0;
      for (uint32_t s = first; s < pr.s; ++s) {
        const uint32_t bar = smem_u32(&s_full[s % ns]);
        const uint64_t t0 = now_ns();
        while (!mbar_try_wait(bar, (s / ns) & 1u) && now_ns() - t0 < p.wait_ns) {}
      }
    }
    return;
  }

  // -------------------------------------------------------------- consumers
  const int tok = p.tok_dev ? p.tok_dev[0] : p.tok;
  if (c.cta == 0 && tid == 0) {
    DevSched *s = p.sched;
    s->B = 1; s->L = L; s->n[0] = n; s->perm[0] = 0; s->slot_s[0] = p.slot; s->pos_s[0] = p.pos;
    s->tok_s[0] = tok; s->lo_s[0] = lo; s->hi_s[0] = hi;
    for (int l = 0; l < L; ++l) s->m[l] = (lo <= l && l < hi) ? 0 : 1;
    s->rows_layers = n; s->layers_touched = n;
  }
  // embedding row -> residual stream (CTA 0 publishes it)
  const Dims &dm = p.dm;
  if (c.cta == 0) {
    const bf16 *e = p.embed + (size_t)tok * dm.d;
    for (int k = tid * 8; k < dm.d; k += kConsumers * 8) {
      const uint4 w = *reinterpret_cast<const uint4 *>(e + k);
      *reinterpret_cast<float4 *>(p.x + k) = make_float4(bfl(w.x), bfh(w.x), bfl(w.y), bfh(w.y));
      *reinterpret_cast<float4 *>(p.x + k + 4) = make_float4(bfl(w.z), bfh(w.z), bfl(w.w), bfh(w.w));
    }
  }
  Consumer cs(c);
  unsigned bidx = 0, ordinal = 0;
  // optional phase timer (thread 0 of every CTA): cycles spent up to each phase boundary
  const bool timing = p.phase_cycles != nullptr && tid == 0;
  long long t_prev = clock64();
  auto tick = [&](int k) {
    if (timing) {
      const long long t = clock64();
      p.phase_cycles[c.cta * kFusedPhases + k] += t - t_prev;
      t_prev = t;
    }
  };
  grid_barrier(c, ++bidx);
  tick(0);
  for (int l = 0; l < L; ++l) {
    if (lo <= l && l < hi) continue;   // dropped block: the hidden state passes through
    load_act(c, p.x, dm.d, p.layers[l].attn_norm);
    tick(1);
    cs.gemv_phase(make_phase(p, PH_QKV, l, c.cta, c.ncta), l);
    tick(2);
    grid_barrier(c, ++bidx);
    tick(3);
    cs.template att_phase<DH, GQ>(att, l, ++ordinal);
    tick(4);
    grid_barrier(c, ++bidx);
    tick(3);
    load_act(c, p.attn_out, dm.Hq * dm.dh, nullptr);
    tick(1);
    cs.gemv_phase(make_phase(p, PH_OPROJ, l, c.cta, c.ncta), l);
    tick(5);
    grid_barrier(c, ++bidx);
    tick(3);
    load_act(c, p.x, dm.d, p.layers[l].mlp_norm);
    tick(1);
    cs.gemv_phase(make_phase(p, PH_GATEUP, l, c.cta, c.ncta), l);
    tick(6);
    grid_barrier(c, ++bidx);
    tick(3);
    load_act(c, p.u, dm.f, nullptr);
    tick(1);
    cs.gemv_phase(make_phase(p, PH_DOWN, l, c.cta, c.ncta), l);
    tick(7);
    grid_barrier(c, ++bidx);
    tick(3);
  }
  // KV fill by copy for the dropped blocks: CTA j takes block lo + j, lo + j + ncta, ...
  if (p.kv_fill == D3_FILL_COPY) {
    const int nkv = dm.Hkv * dm.dh;
    unsigned short *Ku = reinterpret_cast<unsigned short *>(p.Kc);
    unsigned short *Vu = reinterpret_cast<unsigned short *>(p.Vc);
    for (int l = lo + c.cta; l < hi; l += c.ncta) {
      for (int i = tid; i < nkv; i += kConsumers) {
        const int h = i / dm.dh, e = i % dm.dh;
        const size_t dst = ((((size_t)l * dm.max_slots + p.slot) * dm.Hkv + h) * dm.max_seq + p.pos) * dm.dh + e;
        if (lo == 0) {
          Ku[dst] = 0;
          Vu[dst] = 0;
        } else {
          const size_t src = ((((size_t)(lo - 1) * dm.max_slots + p.slot) * dm.Hkv + h) * dm.max_seq + p.pos) * dm.dh + e;
          Ku[dst] = __ldcg(Ku + src);   // written by another CTA earlier in this kernel
          Vu[dst] = __ldcg(Vu + src);
        }
      }
    }
  }
  if (p.logits) {
    load_act(c, p.x, dm.d, p.final_norm);
    cs.gemv_phase(make_phase(p, PH_HEAD, 0, c.cta, c.ncta), 0);
  }
  tick(8);
  if (timing) p.phase_cycles[c.cta * kFusedPhases + 9] += cs.ring_wait;
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
  int kmax = c.d_model;
  if (c.d_ffn > kmax) kmax = c.d_ffn;
  if (c.n_q_heads * c.head_dim > kmax) kmax = c.n_q_heads * c.head_dim;
  // hi and lo bf16 arrays of the widest activation vector, or the attention merge scratch
  int need = (2 * ((kmax * 2 + 127) / 128 * 128 + 64) + 3) / 4;
  const int att_need = 8 * kMaxGQ * (128 + 2) + kFusedMaxCtas * (1 + 2 * kMaxGQ);
  if (need < att_need) need = att_need;
  need = (need + 255) / 256 * 256;
  const int reserve = 4096;   // static shared memory of the kernel and slack
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
  return true;
}

int fused_plan(const d3_config &c, int *grid, int *n_stages, int *act_floats, size_t *smem, void **func) {
  FusedPlan pl;
  memset(&pl, 0, sizeof(pl));
  const int G = c.n_q_heads / c.n_kv_heads;
  const int gq = (G % 4 == 0) ? 4 : (G % 2 == 0) ? 2 : 1;
  bool ok = false;
  if (c.d_model <= 16 * 1024) {
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

int launch_fused_step(void *func, int grid, size_t smem, FusedParams &fp, cudaStream_t st) {
  // grid-barrier counter and per-stream arrival counters start every step at zero
  if (cudaMemsetAsync(fp.bar_counter, 0, kFusedSyncBytes, st) != cudaSuccess) return -1;
  void *args[] = {(void *)&fp};
  if (cudaLaunchCooperativeKernel(func, dim3(grid), dim3(kFusedThreads), args, smem, st) != cudaSuccess)
    return -1;
  return 1;
}

}  // namespace d3

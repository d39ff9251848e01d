// Batched projections on the 5th-generation tensor cores (sm_100a):
//   y[row][r] = sum_k W[r][k] * act'[row][k]     for the rows of one depth group.
//
// With more than a handful of rows the FP32 pipes cannot multiply as fast as
// HBM delivers the weights, so the projection moves to tcgen05.mma while the
// kernel stays a weight-streaming (bandwidth-bound) one: every weight byte is
// read from HBM once per step whatever the row count.
//
// Operand roles are swapped with respect to the usual GEMM: the WEIGHT tile is
// the 128-row "A" operand (UMMA M = 128), the activations are the narrow "B"
// operand (UMMA N = 3 * padded rows).  The fp32 activations are split by a
// small pre-pass (k_act_split, which also applies the fused RMSNorm) into
// three bf16 terms hi + mid + lo = act exactly (3 x 8 significand bits cover
// fp32's 24): the three sit side by side in N and the epilogue adds the three
// accumulator columns of a row.  The products are exact in the fp32
// accumulator, so the result differs from the fp32-activation FMA path only by
// the summation order.  (Two terms leave a 2^-17 relative error; at 32 blocks
// that flips enough bf16 roundings of cached K and V to double the logit error.)
//
// One CTA = one tile of 128 weight rows (two 64-row TMA boxes: rows r..r+63 and
// r+64..r+127 of one matrix, or 64 gate rows + the same 64 up rows for SwiGLU)
// x one split-K slice.  Warp 0 lane 0 drives TMA (cp.async.bulk.tensor, 128-byte
// swizzle, mbarrier transaction counts) through a ring of stages of 64 k each;
// warp 1 lane 0 issues tcgen05.mma (kind::f16, bf16 x bf16 -> fp32 in TMEM) and
// frees stages with tcgen05.commit; warps 2-5 read the accumulator back with
// tcgen05.ld and run the epilogue (store / residual add / SiLU*mul / logits).
// Split-K slices combine with red.global.add.f32 (the residual add is one anyway).
//
// Every mbarrier wait is bounded in time; on expiry the CTA raises D3_ETIMEOUT in
// the schedule's status word, stops issuing, waits (bounded) for its copies in
// flight, frees its TMEM columns and returns.
#include <stdlib.h>

#include <cuda.h>   // CUtensorMap and its enums; the encoder is fetched at run time

#include "d3_internal.cuh"

namespace d3 {

namespace {

constexpr int kTcThreads = 192;
constexpr int kTileM = 128;                      // weight rows of a CTA tile
constexpr int kBoxRows = 64;                     // rows of one weight TMA box
constexpr int kTileK = 64;                       // bf16 per row of a stage = 128 bytes
constexpr int kABytes = kTileM * kTileK * 2;     // 16 KB
constexpr int kMaxStagesTc = 8;
constexpr int kSmemBudget = 100 * 1024;          // two CTAs per SM stay resident
constexpr int kSmemBudgetWide = 200 * 1024;      // more than 64 rows: one CTA per SM, stages of 64 KB
constexpr int kGroupRows = 64;                   // activation rows of one operand group (UMMA N = 192)
constexpr int kMaxTcRows = 2 * kGroupRows;       // activation rows of one launch
constexpr int kShortChainKb = 4;                 // k-blocks (of 4 MMAs) per slice of a short accumulation chain

static_assert(sizeof(TMap) == sizeof(CUtensorMap), "opaque tensor-map storage");

__device__ __forceinline__ uint32_t smem_addr(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ uint64_t timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void bar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t bar_try_wait(uint32_t bar, uint32_t parity) {
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

struct TcArgs {
  int R, K;              // weight rows (outputs), reduction length
  int NP;                // padded activation rows of one operand group, a multiple of 8 (<= 64)
  int N;                 // UMMA N = 3 NP rounded up to a multiple of 16 (the spare columns are not read)
  int groups;            // operand groups (1, or 2 for 65..128 rows): one MMA and N TMEM columns each
  int n_kb, kb_per_split;
  // CHAIN kernels: tiles that start at or after row `short_row0` sum in chains of `chain_kb` k-blocks;
  // after each chain the epilogue warps add the accumulator to registers and the next chain starts
  // the accumulator afresh
  int short_row0, chain_kb;
  int n_stages, tmem_cols;
  int atomic;            // combine with red.add (split-K or residual)
  bf16 *opnd_out;        // nullable (SiLU * mul epilogue): the result also as the next projection's operand, [3 NP][R]
  float4 *clear;         // nullable: a region for a later kernel, zeroed by the epilogue warps up front
  unsigned clear_n4;     // its length in 16-byte units
  float *out;
  int out_stride, out_col0;
  const DevSched *sched;
  DevSched *status;      // where D3_ETIMEOUT is raised
  int layer, row_mode;
  unsigned long long wait_ns;
};

// Bounded wait on one mbarrier phase.  `check_abort` = leave early once the CTA aborted.
__device__ __forceinline__ bool bar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                         unsigned long long wait_ns, bool check_abort) {
  if (check_abort && *abort_flag) return false;
  if (bar_try_wait(bar, parity)) return true;
  const uint64_t t0 = timer_ns();
  for (uint32_t it = 1;; ++it) {
    if (bar_try_wait(bar, parity)) return true;
    if ((it & 31u) == 0u) {
      if (check_abort && *abort_flag) return false;
      if (timer_ns() - t0 > wait_ns) break;
    }
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes
// (64 bf16) in the 128-byte swizzle: groups of 8 rows are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffffu) >> 4);        // start address, 16-byte units
  d |= (uint64_t)1 << 16;                          // leading byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset: 8 rows x 128 bytes
  d |= (uint64_t)1 << 46;                          // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                          // 128-byte swizzle
  return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The barrier gets one arrival once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float (&v)[8]) {
  uint32_t r[8];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
// y[i] = the three accumulator columns (hi, mid, lo term) of activation rows j0 .. j0+7, small first
__device__ __forceinline__ void tmem_sum3(uint32_t tbase, int j0, int NP, float (&y)[8]) {
  float hi[8], mid[8], lo[8];
  tmem_ld8(tbase + (uint32_t)j0, hi);
  tmem_ld8(tbase + (uint32_t)(NP + j0), mid);
  tmem_ld8(tbase + (uint32_t)(2 * NP + j0), lo);
#pragma unroll
  for (int i = 0; i < 8; ++i) y[i] = (lo[i] + mid[i]) + hi[i];
}
// 16 accumulator columns of this thread's TMEM lane, without waiting for them (tmem_ld_wait does)
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void fence_before_sync() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void fence_after_sync() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void epilogue_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

__device__ __forceinline__ void row_span(const DevSched *s, int layer, int mode, int &r0, int &r1) {
  const int B = s->B;
  if (mode == ROWS_PREFIX) { r0 = 0; r1 = s->m[layer]; }
  else if (mode == ROWS_SUFFIX) { r0 = s->m[layer]; r1 = B; }
  else if (mode == ROWS_ALL) { r0 = 0; r1 = B; }
  else { r0 = B - 1; r1 = B; }
}

// ------------------------------------------------------------------ the GEMM
template <int EPI, bool CHAIN = false>
__global__ void __launch_bounds__(kTcThreads)
k_gemm_tc(const __grid_constant__ CUtensorMap map_w0, const __grid_constant__ CUtensorMap map_w1,
          const __grid_constant__ CUtensorMap map_act, const TcArgs t) {
  extern __shared__ unsigned char tc_smem_raw[];
  __shared__ __align__(8) uint64_t s_full[kMaxStagesTc], s_empty[kMaxStagesTc], s_accum, s_free;
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // this tile sums in short chains (uniform over the CTA)
  const bool chain_tile = CHAIN && (int)blockIdx.x * kTileM >= t.short_row0;
  const int chain = chain_tile ? t.chain_kb : 0x7fffffff;
  const int kb0 = blockIdx.y * t.kb_per_split;
  const int kb1 = min(t.n_kb, kb0 + t.kb_per_split);
  if (kb0 >= kb1) {         // uniform over the CTA; the host launches no such slice
    pdl_wait();
    return;
  }
  const int n_it = kb1 - kb0;
  const int S = t.n_stages;
  const int N = t.N;
  const int G = t.groups;
  const uint32_t stage_bytes = (uint32_t)(kABytes + G * N * kTileK * 2);
  // the swizzle pattern is a function of the address: tiles start on 1024-byte boundaries
  const uint32_t ring = (smem_addr(tc_smem_raw) + 1023u) & ~1023u;
  volatile int *abort_flag = &s_abort;

  if (tid == 0) {
    for (int s = 0; s < S; ++s) {
      bar_init(smem_addr(&s_full[s]), 1);
      bar_init(smem_addr(&s_empty[s]), 1);
    }
    bar_init(smem_addr(&s_accum), 1);
    bar_init(smem_addr(&s_free), 128);   // the four epilogue warps
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&s_tmem)),
                 "r"((uint32_t)t.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem = s_tmem;
  pdl_trigger();
  // Up to here nothing depends on an earlier kernel.  The producer lane goes one step further: the
  // weights are constants, so it puts the first ring fill of weight tiles in flight before it waits
  // for the earlier kernels.  It is the only thread of the CTA that sits in that wait when they
  // complete: the MMA lane touches shared and tensor memory only, and the epilogue warps make their
  // own call once the first stage has landed, when it returns at once (measured: with every thread
  // of 288 CTAs blocked in griddepcontrol.wait the CTAs go on 2.3 - 4 us after the earlier kernel's
  // last CTA left; C3 4.32 -> 4.21 ms per step, C4 6.30 -> 6.20 with one thread per CTA).

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int row_a, row_b;
      if (EPI == EPI_SWIGLU) { row_a = blockIdx.x * kBoxRows; row_b = row_a; }
      else { row_a = blockIdx.x * kTileM; row_b = row_a + kBoxRows; }
      int issued = 0;
      const int first = min(S, n_it);
      for (int it = 0; it < first; ++it) {   // first fill: weight tiles only
        const uint32_t full = smem_addr(&s_full[it]);
        const uint32_t a = ring + (uint32_t)it * stage_bytes;
        const int x = (kb0 + it) * kTileK;   // x * 2 bytes is a multiple of 128
        bar_expect_tx(full, stage_bytes);
        tma_load_2d(a, &map_w0, x, row_a, full);
        tma_load_2d(a + kBoxRows * kTileK * 2, &map_w1, x, row_b, full);
      }
      pdl_wait();                            // the activations come from the previous kernel
      for (int it = 0; it < first; ++it) {
        const uint32_t a = ring + (uint32_t)it * stage_bytes;
        for (int g = 0; g < G; ++g)
          tma_load_2d(a + kABytes + g * N * kTileK * 2, &map_act, (kb0 + it) * kTileK, g * N,
                      smem_addr(&s_full[it]));
        issued = it + 1;
      }
      for (int it = first; it < n_it; ++it) {
        const int s = it % S, fill = it / S;
        if (!bar_wait(smem_addr(&s_empty[s]), (uint32_t)((fill - 1) & 1), abort_flag, t.wait_ns, true))
          break;
        const uint32_t full = smem_addr(&s_full[s]);
        const uint32_t a = ring + (uint32_t)s * stage_bytes;
        const int x = (kb0 + it) * kTileK;
        bar_expect_tx(full, stage_bytes);
        tma_load_2d(a, &map_w0, x, row_a, full);
        tma_load_2d(a + kBoxRows * kTileK * 2, &map_w1, x, row_b, full);
        for (int g = 0; g < G; ++g) tma_load_2d(a + kABytes + g * N * kTileK * 2, &map_act, x, g * N, full);
        issued = it + 1;
      }
      if (*abort_flag) {
        // copies still in flight must land before the CTA's shared memory is given back
        const unsigned long long bound = t.wait_ns > kDrainFloorNs ? t.wait_ns : kDrainFloorNs;
        for (int it = max(0, issued - S); it < issued; ++it)
          bar_wait(smem_addr(&s_full[it % S]), (uint32_t)((it / S) & 1), abort_flag, bound, false);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16(kTileM, N);
      bool ok = true;
      int chains_done = 0;   // chains committed to s_accum so far
      for (int it = 0; it < n_it && ok; ++it) {
        const int s = it % S, fill = it / S;
        if (CHAIN && it > 0 && it % chain == 0) {
          // the previous chain is committed; its sums must be out of the accumulator before the
          // next chain overwrites it
          umma_commit(smem_addr(&s_accum));
          ok = bar_wait(smem_addr(&s_free), (uint32_t)(chains_done & 1), abort_flag, t.wait_ns, true);
          ++chains_done;
          if (!ok) break;
          fence_after_sync();
        }
        ok = bar_wait(smem_addr(&s_full[s]), (uint32_t)(fill & 1), abort_flag, t.wait_ns, true);
        if (!ok) break;
        fence_after_sync();
        const uint32_t a = ring + (uint32_t)s * stage_bytes;
        const uint64_t adesc = smem_desc_sw128(a);
        for (int g = 0; g < G; ++g) {
          const uint64_t bdesc = smem_desc_sw128(a + kABytes + g * N * kTileK * 2);
#pragma unroll
          for (int k = 0; k < kTileK / 16; ++k)   // 16 bf16 = 32 bytes = 2 descriptor units per MMA
            umma_bf16(tmem + (uint32_t)(g * N), adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc,
                      ((CHAIN ? it % chain : it) | k) ? 1u : 0u);
        }
        umma_commit(smem_addr(&s_empty[s]));
      }
      umma_commit(smem_addr(&s_accum));
      if (!ok) {
        // aborted: the MMAs already issued still read shared memory and write TMEM; they end by
        // themselves, so wait for them (bounded) before the CTA gives both back
        const unsigned long long bound = t.wait_ns > kDrainFloorNs ? t.wait_ns : kDrainFloorNs;
        bar_wait(smem_addr(&s_accum), (uint32_t)(chains_done & 1), abort_flag, bound, false);
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- epilogue
    const int q = warp & 3;                   // the TMEM lane quarter this warp may read
    const int trow = q * 32 + lane;           // row of the tile = TMEM lane
    // the first stage has landed, so the producer lane's wait on the earlier kernels has returned:
    // this call returns at once, and what this thread reads below (the schedule) is what they wrote
    bar_wait(smem_addr(&s_full[0]), 0u, abort_flag, t.wait_ns, true);
    pdl_wait();
    if (t.clear) {   // nothing reads the region any more (the earlier kernels are complete)
      const unsigned nthr = gridDim.x * gridDim.y * 128u;
      for (unsigned i = (blockIdx.y * gridDim.x + blockIdx.x) * 128u + (unsigned)(tid - 64); i < t.clear_n4; i += nthr)
        t.clear[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    int r0, r1;
    row_span(t.sched, t.layer, t.row_mode, r0, r1);
    const int nrows = min(r1 - r0, G * t.NP);
    const uint32_t tbase = tmem + ((uint32_t)(q * 32) << 16);
    if (CHAIN && chain_tile) {
      // ---- short chains: the row's sums live in registers, one partial sum per chain is added
      float acc[kMaxTcRows / 16][16];
#pragma unroll
      for (int b = 0; b < kMaxTcRows / 16; ++b)
#pragma unroll
        for (int i = 0; i < 16; ++i) acc[b][i] = 0.f;
      const int n_chains = (n_it + chain - 1) / chain;
      bool ok = true;
      for (int c = 0; c < n_chains && ok; ++c) {
        ok = bar_wait(smem_addr(&s_accum), (uint32_t)(c & 1), abort_flag, t.wait_ns, true);
        if (!ok) break;
        fence_after_sync();
        // 16 activation rows per trip: the three terms' columns are requested together and awaited
        // once (a trip may read past the group's rows into columns of rows that are never written out)
#pragma unroll
        for (int b = 0; b < kMaxTcRows / 16; ++b) {
          if (b * 16 < nrows) {
            const uint32_t col = tbase + (uint32_t)(((b * 16) / t.NP) * N + (b * 16) % t.NP);
            uint32_t hi[16], mid[16], lo[16];
            tmem_ld16_issue(col, hi);
            tmem_ld16_issue(col + (uint32_t)t.NP, mid);
            tmem_ld16_issue(col + (uint32_t)(2 * t.NP), lo);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 16; ++i)
              acc[b][i] += (__uint_as_float(lo[i]) + __uint_as_float(mid[i])) + __uint_as_float(hi[i]);
          }
        }
        if (c + 1 < n_chains) {   // the accumulator may be overwritten
          fence_before_sync();
          asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(&s_free)) : "memory");
        }
      }
      epilogue_sync();
      if (*abort_flag == 0) {
        const int r = blockIdx.x * kTileM + trow;
#pragma unroll
        for (int b = 0; b < kMaxTcRows / 16; ++b) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int j = b * 16 + i;
            if (j < nrows && r < t.R) {
              float *o = t.out + (size_t)(r0 + j) * t.out_stride + t.out_col0 + r;
              if (t.atomic) asm volatile("red.global.add.f32 [%0], %1;" ::"l"(o), "f"(acc[b][i]) : "memory");
              else *o = acc[b][i];
            }
          }
        }
      }
    } else {
    bar_wait(smem_addr(&s_accum), 0u, abort_flag, t.wait_ns, true);
    fence_after_sync();
    epilogue_sync();                          // every epilogue warp sees the same abort state below
    const bool live = *abort_flag == 0;
    // activation row j sits in operand group j / NP at TMEM columns (j / NP) * N + j % NP (+ NP, + 2 NP)
    float *xch = reinterpret_cast<float *>(tc_smem_raw + (ring - smem_addr(tc_smem_raw)));   // [G NP][64], SwiGLU
    if (EPI == EPI_SWIGLU) {
      if (live && trow >= kBoxRows) {
        for (int j0 = 0; j0 < nrows; j0 += 8) {
          float y[8];
          tmem_sum3(tbase + (uint32_t)((j0 / t.NP) * N), j0 % t.NP, t.NP, y);
#pragma unroll
          for (int i = 0; i < 8; ++i) xch[(j0 + i) * kBoxRows + (trow - kBoxRows)] = y[i];
        }
      }
      epilogue_sync();
      const int r = blockIdx.x * kBoxRows + trow;
      if (live && trow < kBoxRows) {
        for (int j0 = 0; j0 < nrows; j0 += 8) {
          float y[8];
          tmem_sum3(tbase + (uint32_t)((j0 / t.NP) * N), j0 % t.NP, t.NP, y);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int j = j0 + i;
            if (j < nrows && r < t.R) {
              const float z = y[i], up = xch[j * kBoxRows + trow];
              const float val = z / (1.f + __expf(-z)) * up;
              t.out[(size_t)(r0 + j) * t.out_stride + t.out_col0 + r] = val;
              if (t.opnd_out) {   // hi + mid + lo = val, rows j, NP + j, 2 NP + j of the next operand
                const bf16 h = __float2bfloat16_rn(val);
                const float r1 = val - __bfloat162float(h);     // exact
                const bf16 md = __float2bfloat16_rn(r1);
                const bf16 lw = __float2bfloat16_rn(r1 - __bfloat162float(md));
                bf16 *o = t.opnd_out + (size_t)j * t.R + r;
                o[0] = h; o[(size_t)t.NP * t.R] = md; o[(size_t)2 * t.NP * t.R] = lw;
              }
            }
          }
        }
      }
    } else if (live) {
      const int r = blockIdx.x * kTileM + trow;
      for (int j0 = 0; j0 < nrows; j0 += 8) {
        float y[8];
        tmem_sum3(tbase + (uint32_t)((j0 / t.NP) * N), j0 % t.NP, t.NP, y);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int j = j0 + i;
          if (j < nrows && r < t.R) {
            const int row = r0 + j;
            const int orow = (EPI == EPI_LOGITS) ? (t.row_mode == ROWS_LAST ? 0 : t.sched->perm[row]) : row;
            float *o = t.out + (size_t)orow * t.out_stride + t.out_col0 + r;
            if (t.atomic) asm volatile("red.global.add.f32 [%0], %1;" ::"l"(o), "f"(y[i]) : "memory");
            else *o = y[i];
          }
        }
      }
    }
    }
  }

  fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)t.tmem_cols)
                 : "memory");
  }
  if (tid == 0 && s_abort) t.status->status = D3_ETIMEOUT;
}

// -------------------------------------------------------------- the pre-pass
// Row j of the group: act' = act (or RMSNorm(act) * gain), written as three bf16
// terms in rows j, NP + j and 2 NP + j of the operand buffer (hi + mid + lo = act').  When the GEMM
// combines split-K slices into a plain (non-residual) output, the pre-pass also
// zeroes that output row.
struct SplitArgs {
  const float *act;
  int act_stride, K, NP, N, groups;   // NP rows per operand group, groups of N operand rows each
  const bf16 *gain;
  float eps;
  bf16 *dst;             // [3 NP][K]
  float *zero_out;       // nullable
  int out_stride, out_col0, R;
  const DevSched *sched;
  int layer, row_mode;
};

// grid (rows, K / 1024 chunks): every CTA of a row recomputes the row's sum of squares (a few
// KB out of L2) and converts its own 1024-element chunk.
__global__ void __launch_bounds__(256) k_act_split(const SplitArgs a) {
  __shared__ float s_red[8];
  __shared__ float s_scale;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  pdl_wait();
  pdl_trigger();
  int r0, r1;
  row_span(a.sched, a.layer, a.row_mode, r0, r1);
  const int j = blockIdx.x, row = r0 + j;
  if (row >= r1 || j >= a.groups * a.NP) return;
  const float *src = a.act + (size_t)row * a.act_stride;
  float sc = 1.f;
  if (a.gain) {
    float ss = 0.f;
    for (int k = tid * 4; k < a.K; k += 256 * 4) {
      float4 v = *reinterpret_cast<const float4 *>(src + k);
      ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (lane == 0) s_red[warp] = ss;
    __syncthreads();
    if (tid == 0) {
      float tot = 0.f;
      for (int w = 0; w < 8; ++w) tot += s_red[w];
      s_scale = rsqrtf(tot / (float)a.K + a.eps);
    }
    __syncthreads();
    sc = s_scale;
  }
  const int grow = (j / a.NP) * a.N + j % a.NP;   // the row's hi term in its operand group
  bf16 *hi = a.dst + (size_t)grow * a.K, *mid = a.dst + (size_t)(a.NP + grow) * a.K,
       *lo = a.dst + (size_t)(2 * a.NP + grow) * a.K;
  const int k = blockIdx.y * 1024 + tid * 4;
  if (k < a.K) {
    float4 v = *reinterpret_cast<const float4 *>(src + k);
    if (a.gain) {
      uint2 gw = *reinterpret_cast<const uint2 *>(a.gain + k);
      v.x *= sc * __uint_as_float(gw.x << 16); v.y *= sc * __uint_as_float(gw.x & 0xffff0000u);
      v.z *= sc * __uint_as_float(gw.y << 16); v.w *= sc * __uint_as_float(gw.y & 0xffff0000u);
    }
    const float f[4] = {v.x, v.y, v.z, v.w};
    __align__(8) bf16 h[4], md[4], l[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      h[i] = __float2bfloat16_rn(f[i]);
      const float r1 = f[i] - __bfloat162float(h[i]);     // exact
      md[i] = __float2bfloat16_rn(r1);
      l[i] = __float2bfloat16_rn(r1 - __bfloat162float(md[i]));
    }
    *reinterpret_cast<uint2 *>(hi + k) = *reinterpret_cast<const uint2 *>(h);
    *reinterpret_cast<uint2 *>(mid + k) = *reinterpret_cast<const uint2 *>(md);
    *reinterpret_cast<uint2 *>(lo + k) = *reinterpret_cast<const uint2 *>(l);
  }
  if (a.zero_out) {
    float *o = a.zero_out + (size_t)row * a.out_stride + a.out_col0;
    for (int c = blockIdx.y * 256 + tid; c < a.R; c += gridDim.y * 256) o[c] = 0.f;
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encoder() {
  static EncodeTiledFn fn = [] {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// 2-D bf16 tensor [rows][K] (K contiguous), box = 64 k x box_rows, 128-byte swizzle, zero fill outside.
bool encode_map(TMap *out, const void *base, int rows, int K, int box_rows) {
  EncodeTiledFn fn = encoder();
  if (!fn || ((uintptr_t)base & 15u) || (K % 8) || K < kTileK || rows < 1 || box_rows < 1 || box_rows > 256)
    return false;
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {(cuuint32_t)kTileK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(reinterpret_cast<CUtensorMap *>(out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                  const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <int EPI>
cudaError_t tc_attr() {
  return cudaFuncSetAttribute(k_gemm_tc<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kSmemBudgetWide + 1024);
}

}  // namespace

bool tc_weight_map(TMap *out, const bf16 *W, int R, int K) {
  if (R < kBoxRows) return false;
  return encode_map(out, W, R, K, kBoxRows);
}

int tc_init() {
  if (!encoder()) return -1;
  cudaError_t e = tc_attr<EPI_STORE>();
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(k_gemm_tc<EPI_STORE, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kSmemBudgetWide + 1024);
  if (e == cudaSuccess) e = tc_attr<EPI_RESID>();
  if (e == cudaSuccess) e = tc_attr<EPI_SWIGLU>();
  if (e == cudaSuccess) e = tc_attr<EPI_LOGITS>();
  return e == cudaSuccess ? 0 : -1;
}

// Enqueue pre-pass + GEMM for `m_rows` rows.  Returns kernels launched (2), or 0
// when this projection cannot take the tensor-core path (the caller falls back).
int launch_gemm_tc(TcContext &tc, const GemvArgs &g, int epi, int m_rows, cudaStream_t st) {
  if (!tc.ok || !g.tmap_w || m_rows < 1 || m_rows > D3_MAX_BATCH) return 0;
  if (epi == EPI_SWIGLU && !g.tmap_w2) return 0;
  // three operand rows per activation row; UMMA M = 128 wants N a multiple of 16 (<= 192 here):
  // up to 8 spare rows of the operand buffer ride along (whatever they hold, their columns are unused)
  // More than 64 rows: two operand groups of 64 rows (N = 192 each, one MMA per group and k-step,
  // the weight tile read from shared memory by both), so that a pass of up to 128 prompt
  // positions streams the weights once.
  const int groups = m_rows > kGroupRows ? 2 : 1;
  const int NP = groups > 1 ? kGroupRows : (m_rows + 7) / 8 * 8, N = (3 * NP + 15) / 16 * 16;
  if ((size_t)groups * N * g.K * sizeof(bf16) > tc.act_bytes) return 0;
  // the operand comes from the pre-pass (act_split) or was left by the previous projection (act_split2)
  const bool handed = g.operand_in && groups == 1 && !g.gain && epi == EPI_RESID;
  const uint64_t key = ((uint64_t)(handed ? 1 : 0) << 56) | ((uint64_t)groups << 48) | ((uint64_t)NP << 32) | (uint32_t)g.K;
  auto it = tc.act_maps.find(key);
  if (it == tc.act_maps.end()) {
    TMap mp;
    if (!encode_map(&mp, handed ? tc.act_split2 : tc.act_split, groups * N, g.K, N)) return 0;
    it = tc.act_maps.emplace(key, mp).first;
  }

  const int tile_rows = epi == EPI_SWIGLU ? kBoxRows : kTileM;
  const int tiles = (g.R + tile_rows - 1) / tile_rows;
  const int n_kb = (g.K + kTileK - 1) / kTileK;
  int ksplit = 1;
  if (epi == EPI_STORE || epi == EPI_RESID) {
    // all CTAs resident at once (two per SM), slices of at least 8 k-blocks
    ksplit = (groups > 1 ? 1 : 2) * tc.sm_count / tiles;
    if (ksplit > n_kb / 8) ksplit = n_kb / 8;
    if (ksplit < 1) ksplit = 1;
    if (ksplit > 16) ksplit = 16;
  }
  int per = (n_kb + ksplit - 1) / ksplit;
  ksplit = (n_kb + per - 1) / per;   // no empty slice
  // Rows from g.short_chain_row0 on (the K and V rows of a prefill pass, which end up rounded to
  // bf16 in the cache) are summed in chains of kShortChainKb k-blocks: the error of the tensor core's
  // fp32 accumulation grows with the length of the chain; with chains of 32 MMAs the cached values
  // round like those of the fp32-FMA kernels, with 16 a little better (measured through the logits
  // of a 32-block model).  The chains are summed inside the CTA (k_gemm_tc<EPI_STORE, true>): after
  // each one the epilogue warps add the accumulator to registers.  Tiles above that row keep one chain.
  int short_row0 = g.R, chain_kb = 0;
  if (epi == EPI_STORE && g.short_chain_row0 > 0 && g.short_chain_row0 < g.R && per > kShortChainKb) {
    chain_kb = kShortChainKb;
    if (const char *env = getenv("D3_TC_SHORT_KB")) {   // tuning knob
      const int v = atoi(env);
      if (v >= 2 && v <= 64) chain_kb = v;
    }
    short_row0 = (g.short_chain_row0 + kTileM - 1) / kTileM * kTileM;
    if (short_row0 >= g.R) chain_kb = 0;
  }

  SplitArgs sa;
  sa.act = g.act; sa.act_stride = g.act_stride; sa.K = g.K; sa.NP = NP; sa.N = N; sa.groups = groups;
  sa.gain = g.gain; sa.eps = g.eps;
  sa.dst = tc.act_split;
  sa.zero_out = (epi == EPI_STORE && ksplit > 1 && !g.out_is_zero) ? g.out : nullptr;
  sa.out_stride = g.out_stride; sa.out_col0 = g.out_col0; sa.R = g.R;
  sa.sched = g.sched; sa.layer = g.layer; sa.row_mode = g.row_mode;
  if (!handed) launch_pdl(k_act_split, dim3(m_rows, (g.K + 1023) / 1024), dim3(256), 0, st, sa);

  TcArgs t;
  t.R = g.R; t.K = g.K; t.NP = NP; t.N = N; t.groups = groups; t.n_kb = n_kb; t.kb_per_split = per;
  t.short_row0 = short_row0; t.chain_kb = chain_kb;
  const int stage_bytes = kABytes + groups * N * kTileK * 2;
  t.n_stages = (groups > 1 ? kSmemBudgetWide : kSmemBudget) / stage_bytes;
  if (t.n_stages > kMaxStagesTc) t.n_stages = kMaxStagesTc;
  // Measured: a fifth stage does not shorten any launch, but its shared memory keeps the next
  // kernel's CTAs from becoming resident early (13B shape, 8 rows: 7.24 ms per step with 5, 6.43 with 4).
  if (t.n_stages > 4) t.n_stages = 4;
  if (t.n_stages > per) t.n_stages = per < 2 ? 2 : per;
  t.tmem_cols = 32;
  while (t.tmem_cols < groups * N) t.tmem_cols *= 2;
  t.atomic = (epi == EPI_RESID || (epi == EPI_STORE && ksplit > 1)) ? 1 : 0;
  t.opnd_out = nullptr;
  if (g.operand_out && epi == EPI_SWIGLU && groups == 1 && (size_t)N * g.R * sizeof(bf16) <= tc.act_bytes && g.R % 8 == 0) {
    t.opnd_out = tc.act_split2;
    tc.handed_over = true;
  }
  t.clear = reinterpret_cast<float4 *>(g.clear); t.clear_n4 = g.clear ? (unsigned)(g.clear_floats / 4) : 0u;
  t.out = g.out; t.out_stride = g.out_stride; t.out_col0 = g.out_col0;
  t.sched = g.sched; t.status = const_cast<DevSched *>(g.sched); t.layer = g.layer; t.row_mode = g.row_mode;
  t.wait_ns = tc.wait_ns;
  const size_t smem = (size_t)t.n_stages * stage_bytes + 1024;
  const CUtensorMap *w0 = reinterpret_cast<const CUtensorMap *>(g.tmap_w);
  const CUtensorMap *w1 = reinterpret_cast<const CUtensorMap *>(epi == EPI_SWIGLU ? g.tmap_w2 : g.tmap_w);
  const CUtensorMap *ma = reinterpret_cast<const CUtensorMap *>(&it->second);
  dim3 grid((unsigned)tiles, (unsigned)ksplit);
  switch (epi) {
    case EPI_STORE:
      if (chain_kb > 0) launch_pdl(k_gemm_tc<EPI_STORE, true>, grid, dim3(kTcThreads), smem, st, *w0, *w1, *ma, t);
      else launch_pdl(k_gemm_tc<EPI_STORE>, grid, dim3(kTcThreads), smem, st, *w0, *w1, *ma, t);
      break;
    case EPI_RESID: launch_pdl(k_gemm_tc<EPI_RESID>, grid, dim3(kTcThreads), smem, st, *w0, *w1, *ma, t); break;
    case EPI_SWIGLU: launch_pdl(k_gemm_tc<EPI_SWIGLU>, grid, dim3(kTcThreads), smem, st, *w0, *w1, *ma, t); break;
    default: launch_pdl(k_gemm_tc<EPI_LOGITS>, grid, dim3(kTcThreads), smem, st, *w0, *w1, *ma, t); break;
  }
  return handed ? 1 : 2;
}

}  // namespace d3

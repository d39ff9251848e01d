// CUDA kernels of the D3 decode step (sm_100a): depth schedule + sort,
// embedding gather, fused RMSNorm + projection GEMVs, RoPE + KV append,
// split-K flash-decoding attention with grouped KV heads, KV fill, argmax.
#include <stdlib.h>

#include "d3_internal.cuh"

namespace d3 {

static constexpr int kThreads = 256;
static constexpr int kWarps = kThreads / 32;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// two bf16 packed in a 32-bit word -> two floats (exact)
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ uint4 ldg_stream(const void *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ void row_range(const DevSched *s, int layer, int mode, int &r0, int &r1) {
  int B = s->B;
  if (mode == ROWS_PREFIX) { r0 = 0; r1 = s->m[layer]; }
  else if (mode == ROWS_SUFFIX) { r0 = s->m[layer]; r1 = B; }
  else if (mode == ROWS_ALL) { r0 = 0; r1 = B; }
  else { r0 = B - 1; r1 = B; }
}

// ------------------------------------------------------------------ rope table
// table[pos][j] = (cos, sin)(pos * base^(-2j/dh)), evaluated in fp64.
// Rows pos0 .. pos0 + n_pos - 1 of the table.
__global__ void k_rope_table(float2 *table, int pos0, int n_pos, int half, int dh, double base) {
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_pos * half) return;
  int pos = pos0 + idx / half, j = idx % half;
  double theta = pow(base, -2.0 * (double)j / (double)dh);
  double s, c;
  sincos((double)pos * theta, &s, &c);
  table[(size_t)pos * half + j] = make_float2((float)c, (float)s);
}

int launch_rope_table(float2 *table, int max_seq, int dh, float base, cudaStream_t st) {
  return launch_rope_rows(table, 0, max_seq, dh, base, st);
}

int launch_rope_rows(float2 *table, int pos0, int n_pos, int dh, float base, cudaStream_t st) {
  int n = n_pos * (dh / 2);
  k_rope_table<<<(n + 255) / 256, 256, 0, st>>>(table, pos0, n_pos, dh / 2, dh, (double)base);
  return 1;
}

// --------------------------------------------------- depth schedule + embedding
// Every CTA derives the whole schedule in shared memory (a few hundred integer
// operations); CTA 0 publishes it; CTA r gathers the embedding of sorted row r.
// Depth of a row: floor(L alpha^i) = #{ n in 1..L : i < thr[n] }  (integers only).
__global__ void __launch_bounds__(kThreads)
k_schedule_embed(const __grid_constant__ StepArgs a, DevSched *s, const bf16 *E, float *x, int d) {
  __shared__ int sn[D3_MAX_BATCH], slo[D3_MAX_BATCH], shi[D3_MAX_BATCH], sperm[D3_MAX_BATCH];
  __shared__ int sm[D3_MAX_LAYERS];
  const int B = a.B, L = a.L, tid = threadIdx.x;
  pdl_wait();
  pdl_trigger();
  if (tid < B) {
    int i = a.gi[tid], n = 0;
    for (int k = 1; k <= L; ++k) n += (i < a.thr[k]) ? 1 : 0;
    int lo, hi;
    if (a.anchor == D3_ANCHOR_TAIL) { lo = n; hi = L; }
    else { if (n < a.start_id) n = a.start_id; lo = a.start_id; hi = a.start_id + (L - n); }
    sn[tid] = n; slo[tid] = lo; shi[tid] = hi;
  }
  __syncthreads();
  if (tid < B) {  // stable rank by n descending
    int n = sn[tid], rank = 0;
    for (int b = 0; b < B; ++b) rank += (sn[b] > n || (sn[b] == n && b < tid)) ? 1 : 0;
    sperm[rank] = tid;
  }
  if (tid < L) {
    int m = 0;
    for (int b = 0; b < B; ++b) m += (slo[b] <= tid && tid < shi[b]) ? 0 : 1;
    sm[tid] = m;
  }
  __syncthreads();
  if (blockIdx.x == 0) {
    if (tid < B) {
      int b = sperm[tid];
      s->n[tid] = sn[tid];
      s->perm[tid] = b;
      s->slot_s[tid] = a.slot[b];
      s->pos_s[tid] = a.pos[b];
      s->tok_s[tid] = a.tok_dev ? a.tok_dev[b] : a.tok[b];
      s->lo_s[tid] = slo[b];
      s->hi_s[tid] = shi[b];
    }
    if (tid < L) s->m[tid] = sm[tid];
    if (tid == 0) {
      long long tot = 0;
      int touched = 0;
      for (int l = 0; l < L; ++l) { tot += sm[l]; touched += sm[l] > 0; }
      s->B = B; s->L = L; s->rows_layers = tot; s->layers_touched = touched;
    }
  }
  const int r = blockIdx.x;
  const int b = sperm[r];
  int tok = a.tok_dev ? a.tok_dev[b] : a.tok[b];
  const bf16 *e = E + (size_t)tok * d;
  float *xr = x + (size_t)r * d;
  for (int k = tid * 8; k < d; k += kThreads * 8) {
    uint4 w = *reinterpret_cast<const uint4 *>(e + k);
    float4 f0 = make_float4(bf_lo(w.x), bf_hi(w.x), bf_lo(w.y), bf_hi(w.y));
    float4 f1 = make_float4(bf_lo(w.z), bf_hi(w.z), bf_lo(w.w), bf_hi(w.w));
    *reinterpret_cast<float4 *>(xr + k) = f0;
    *reinterpret_cast<float4 *>(xr + k + 4) = f1;
  }
}

int launch_schedule_embed(const StepArgs &a, DevSched *s, const bf16 *E, float *x, int d,
                          cudaStream_t st) {
  launch_pdl(k_schedule_embed, dim3(a.B), dim3(kThreads), 0, st, a, s, E, x, d);
  return 1;
}

// ------------------------------------------------------------------------ GEMV
// y[row][r] = sum_k W[r][k] * act'[row][k], act' = act or RMSNorm(act) * gain.
// A CTA owns 2 weight streams per warp (two rows, or the gate and up rows of
// one SwiGLU output) and walks the batch rows MT at a time.  The activation
// tile sits in shared memory in fp32; weights stream from HBM with 128-bit
// non-allocating loads, 4 deep per stream, and are widened to fp32 in
// registers.  Accumulation is fp32.
//
// Shared layout of one activation row chunk: element e of a 256-element group
// (e = lane*8 + j) is stored at (j/4)*128 + lane*4 + (j%4), so that the two
// float4 reads of a lane are bank-conflict free.
template <int MT, int EPI>
__global__ void __launch_bounds__(kThreads)
k_gemv(const GemvArgs g, int kc_max) {
  extern __shared__ __align__(16) float s_act[];  // [MT][kc_max]
  __shared__ float s_red[kWarps][MT];
  __shared__ float s_scale[MT];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  pdl_wait();
  pdl_trigger();
  int r0, r1;
  row_range(g.sched, g.layer, g.row_mode, r0, r1);
  if (r0 >= r1) return;

  const int K = g.K;
  // weight streams of this warp
  const bf16 *w0, *w1;
  int out_r0, out_r1;   // output indices (or -1)
  if (EPI == EPI_SWIGLU) {
    int r = blockIdx.x * kWarps + warp;
    int rc = r < g.R ? r : g.R - 1;
    w0 = g.W + (size_t)rc * K;
    w1 = g.W2 + (size_t)rc * K;
    out_r0 = r < g.R ? r : -1;
    out_r1 = -1;
  } else {
    int r = (blockIdx.x * kWarps + warp) * 2;
    int ra = r < g.R ? r : g.R - 1, rb = r + 1 < g.R ? r + 1 : g.R - 1;
    w0 = g.W + (size_t)ra * K;
    w1 = g.W + (size_t)rb * K;
    out_r0 = r < g.R ? r : -1;
    out_r1 = r + 1 < g.R ? r + 1 : -1;
  }

  for (int rt = r0; rt < r1; rt += MT) {
    // RMSNorm scale of each row of the tile (pre-pass over the full row)
    if (g.gain) {
      float ss[MT];
#pragma unroll
      for (int m = 0; m < MT; ++m) {
        ss[m] = 0.f;
        if (rt + m < r1) {
          const float *a = g.act + (size_t)(rt + m) * g.act_stride;
          for (int k = tid * 4; k < K; k += kThreads * 4) {
            float4 v = *reinterpret_cast<const float4 *>(a + k);
            ss[m] += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
          }
        }
        ss[m] = warp_sum(ss[m]);
      }
      __syncthreads();
      if (lane == 0)
#pragma unroll
        for (int m = 0; m < MT; ++m) s_red[warp][m] = ss[m];
      __syncthreads();
      if (tid < MT) {
        float t = 0.f;
        for (int w = 0; w < kWarps; ++w) t += s_red[w][tid];
        s_scale[tid] = rsqrtf(t / (float)K + g.eps);
      }
      __syncthreads();
    }

    float acc0[MT], acc1[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) acc0[m] = acc1[m] = 0.f;

    for (int kc0 = 0; kc0 < K; kc0 += kc_max) {
      const int kc = min(kc_max, K - kc0);
      __syncthreads();  // previous chunk fully consumed
      // stage the activation chunk (normalised), permuted within 256-groups
      for (int m = 0; m < MT; ++m) {
        const bool live = rt + m < r1;
        const float *a = g.act + (size_t)(rt + m) * g.act_stride + kc0;
        const float sc = (g.gain && live) ? s_scale[m] : 1.f;
        for (int k = tid * 4; k < kc; k += kThreads * 4) {
          float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
          if (live) {
            v = *reinterpret_cast<const float4 *>(a + k);
            if (g.gain) {
              uint2 gw = *reinterpret_cast<const uint2 *>(g.gain + kc0 + k);
              v.x *= sc * bf_lo(gw.x); v.y *= sc * bf_hi(gw.x);
              v.z *= sc * bf_lo(gw.y); v.w *= sc * bf_hi(gw.y);
            }
          }
          int grp = k >> 8, e = k & 255, ln = e >> 3, j = e & 7;  // j is 0 or 4
          *reinterpret_cast<float4 *>(s_act + (size_t)m * kc_max + grp * 256 + (j >> 2) * 128 + ln * 4) = v;
        }
      }
      __syncthreads();

      const bf16 *p0 = w0 + kc0, *p1 = w1 + kc0;
      constexpr int U = 4;
      for (int kb = 0; kb < kc; kb += 256 * U) {
        uint4 a0[U], a1[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          int k = kb + u * 256 + lane * 8;
          if (k < kc) {
            a0[u] = ldg_stream(p0 + k);
            a1[u] = ldg_stream(p1 + k);
          } else {
            a0[u] = make_uint4(0, 0, 0, 0);
            a1[u] = make_uint4(0, 0, 0, 0);
          }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          int k = kb + u * 256;
          if (k + lane * 8 < kc) {
#pragma unroll
            for (int m = 0; m < MT; ++m) {
              const float *sa = s_act + (size_t)m * kc_max + k + lane * 4;
              float4 x0 = *reinterpret_cast<const float4 *>(sa);
              float4 x1 = *reinterpret_cast<const float4 *>(sa + 128);
              acc0[m] += bf_lo(a0[u].x) * x0.x + bf_hi(a0[u].x) * x0.y + bf_lo(a0[u].y) * x0.z +
                         bf_hi(a0[u].y) * x0.w + bf_lo(a0[u].z) * x1.x + bf_hi(a0[u].z) * x1.y +
                         bf_lo(a0[u].w) * x1.z + bf_hi(a0[u].w) * x1.w;
              acc1[m] += bf_lo(a1[u].x) * x0.x + bf_hi(a1[u].x) * x0.y + bf_lo(a1[u].y) * x0.z +
                         bf_hi(a1[u].y) * x0.w + bf_lo(a1[u].z) * x1.x + bf_hi(a1[u].z) * x1.y +
                         bf_lo(a1[u].w) * x1.z + bf_hi(a1[u].w) * x1.w;
            }
          }
        }
      }
    }

#pragma unroll
    for (int m = 0; m < MT; ++m) {
      acc0[m] = warp_sum(acc0[m]);
      acc1[m] = warp_sum(acc1[m]);
    }
    if (lane == 0) {
#pragma unroll
      for (int m = 0; m < MT; ++m) {
        int row = rt + m;
        if (row >= r1) break;
        int orow = (EPI == EPI_LOGITS) ? (g.row_mode == ROWS_LAST ? 0 : g.sched->perm[row]) : row;
        float *o = g.out + (size_t)orow * g.out_stride + g.out_col0;
        if (EPI == EPI_SWIGLU) {
          if (out_r0 >= 0) {
            float z = acc0[m];
            o[out_r0] = z / (1.f + __expf(-z)) * acc1[m];
          }
        } else if (EPI == EPI_RESID) {
          if (out_r0 >= 0) o[out_r0] += acc0[m];
          if (out_r1 >= 0) o[out_r1] += acc1[m];
        } else {
          if (out_r0 >= 0) o[out_r0] = acc0[m];
          if (out_r1 >= 0) o[out_r1] = acc1[m];
        }
      }
    }
  }
}

static constexpr int kGemvSmem = 64 * 1024;

template <int MT, int EPI>
static void gemv_launch(const GemvArgs &g, cudaStream_t st) {
  int rows_per_cta = (EPI == EPI_SWIGLU) ? kWarps : 2 * kWarps;
  int grid = (g.R + rows_per_cta - 1) / rows_per_cta;
  int kc_max = kGemvSmem / (4 * MT);          // floats per row chunk, a multiple of 256
  int kpad = (g.K + 255) / 256 * 256;
  if (kc_max > kpad) kc_max = kpad;
  size_t smem = (size_t)MT * kc_max * 4;
  launch_pdl(k_gemv<MT, EPI>, dim3(grid), dim3(kThreads), smem, st, g, kc_max);
}

template <int EPI>
static void gemv_dispatch(const GemvArgs &g, int m_rows, cudaStream_t st) {
  if (m_rows <= 1) gemv_launch<1, EPI>(g, st);
  else if (m_rows == 2) gemv_launch<2, EPI>(g, st);
  else gemv_launch<4, EPI>(g, st);
}

int launch_gemv(const GemvArgs &g, int epi, int m_rows, cudaStream_t st) {
  switch (epi) {
    case EPI_STORE: gemv_dispatch<EPI_STORE>(g, m_rows, st); break;
    case EPI_RESID: gemv_dispatch<EPI_RESID>(g, m_rows, st); break;
    case EPI_SWIGLU: gemv_dispatch<EPI_SWIGLU>(g, m_rows, st); break;
    default: gemv_dispatch<EPI_LOGITS>(g, m_rows, st); break;
  }
  return 1;
}

template <int MT, int EPI>
static cudaError_t gemv_attr() {
  return cudaFuncSetAttribute(k_gemv<MT, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemvSmem);
}

int init_kernel_attributes() {
  if (init_attention_mma() != 0) return -1;
  cudaError_t e = cudaSuccess;
#define D3_ATTR(MT)                                           \
  if (e == cudaSuccess) e = gemv_attr<MT, EPI_STORE>();       \
  if (e == cudaSuccess) e = gemv_attr<MT, EPI_RESID>();       \
  if (e == cudaSuccess) e = gemv_attr<MT, EPI_SWIGLU>();      \
  if (e == cudaSuccess) e = gemv_attr<MT, EPI_LOGITS>();
  D3_ATTR(1) D3_ATTR(2) D3_ATTR(4)
#undef D3_ATTR
  return e == cudaSuccess ? 0 : -1;
}

// ---------------------------------------------------------- RoPE + KV append
// Rotates q (in place, fp32) and k at the row's position, pair (j, j + dh/2),
// and stores k, v as bf16 at cache[layer][slot][kv head][pos][:].
// grid (rows, head chunks): a thread owns one pair of one head; the heads are
// numbered q heads, then k heads, then v heads.
__global__ void __launch_bounds__(kThreads)
k_rope_append(float *qkv, const float2 *rope, bf16 *Kc, bf16 *Vc, const DevSched *s, int layer,
              int row_mode, int kv_only, Dims dm) {
  pdl_wait();
  pdl_trigger();
  int r0, r1;
  row_range(s, layer, row_mode, r0, r1);
  const int row = r0 + blockIdx.x;
  if (row >= r1) return;
  const int dh = dm.dh, half = dh / 2;
  const int hs = blockIdx.y * (kThreads / half) + threadIdx.x / half, j = threadIdx.x % half;
  if (hs >= dm.Hq + 2 * dm.Hkv) return;
  const int pos = s->pos_s[row], slot = s->slot_s[row];
  float *p = qkv + (size_t)row * dm.qkv_rows + (size_t)hs * dh;
  if (hs < dm.Hq) {
    if (kv_only) return;
    const float2 cs = rope[(size_t)pos * half + j];
    const float a = p[j], b = p[j + half];
    p[j] = a * cs.x - b * cs.y;
    p[j + half] = a * cs.y + b * cs.x;
  } else if (hs < dm.Hq + dm.Hkv) {
    const float2 cs = rope[(size_t)pos * half + j];
    const float a = p[j], b = p[j + half];
    bf16 *dst = Kc + kv_offset(dm, dm.block_table, layer, slot, hs - dm.Hq, pos);
    dst[j] = __float2bfloat16_rn(a * cs.x - b * cs.y);
    dst[j + half] = __float2bfloat16_rn(a * cs.y + b * cs.x);
  } else {
    bf16 *dst = Vc + kv_offset(dm, dm.block_table, layer, slot, hs - dm.Hq - dm.Hkv, pos);
    dst[j] = __float2bfloat16_rn(p[j]);
    dst[j + half] = __float2bfloat16_rn(p[j + half]);
  }
}

int launch_rope_append(float *qkv, const float2 *rope, bf16 *Kc, bf16 *Vc, const DevSched *s,
                       int layer, int row_mode, int kv_only, int m_rows, const Dims &dm,
                       cudaStream_t st) {
  const int heads_per_cta = kThreads / (dm.dh / 2);
  dim3 grid(m_rows, (dm.Hq + 2 * dm.Hkv + heads_per_cta - 1) / heads_per_cta);
  launch_pdl(k_rope_append, grid, dim3(kThreads), 0, st, qkv, rope, Kc, Vc, s, layer, row_mode, kv_only, dm);
  return 1;
}

// ------------------------------------------------------------------ attention
// Flash-decoding: a CTA handles one (row, group of GQ query heads sharing a KV
// head, split of the positions).  An 8-lane group ("worker") owns one position
// at a time: each lane holds dh/8 elements of q, K and V; scores are reduced
// over the 8 lanes; every worker keeps a running (max, sum, o) which are merged
// over the 4 workers of a warp by shuffles and over the 8 warps through shared
// memory.  The CTA writes its partial (max, sum, unnormalised o).
template <int DH, int GQ>
__global__ void __launch_bounds__(kThreads)
k_attn_partial(const float *qkv, const bf16 *Kc, const bf16 *Vc, const DevSched *s, int layer,
               int split_len, int max_splits, float *part_o, float *part_ml, Dims dm) {
  constexpr int EPL = DH / 8;
  pdl_wait();
  pdl_trigger();
  const int row = blockIdx.z;
  if (row >= s->m[layer]) return;
  const int len = s->pos_s[row] + 1;
  const int split = blockIdx.x;
  const int t0 = split * split_len;
  if (t0 >= len) return;
  const int t1 = min(len, t0 + split_len);
  const int h0 = blockIdx.y * GQ;
  const int kvh = h0 / (dm.Hq / dm.Hkv);
  const int slot = s->slot_s[row];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, part = lane & 7;
  const int worker = warp * 4 + (lane >> 3);
  // the 8 lanes of a worker run the position loop in lockstep; other workers of
  // the warp may run fewer iterations, so in-loop shuffles name only the worker
  const unsigned wmask = 0xffu << (lane & 24);

  float q[GQ][EPL];
  const float scale = rsqrtf((float)DH);
#pragma unroll
  for (int g = 0; g < GQ; ++g) {
    const float *qp = qkv + (size_t)row * dm.qkv_rows + (h0 + g) * DH + part * EPL;
#pragma unroll
    for (int e = 0; e < EPL; ++e) q[g][e] = qp[e] * scale;
  }
  float mx[GQ], sum[GQ], o[GQ][EPL];
#pragma unroll
  for (int g = 0; g < GQ; ++g) {
    mx[g] = -INFINITY; sum[g] = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) o[g][e] = 0.f;
  }
  for (int t = t0 + worker; t < t1; t += 32) {
    const size_t off = kv_offset(dm, dm.block_table, layer, slot, kvh, t) + part * EPL;
    const bf16 *kp = Kc + off;
    const bf16 *vp = Vc + off;
    float kf[EPL], vf[EPL];
    if constexpr (EPL == 4) {
      uint2 kw = *reinterpret_cast<const uint2 *>(kp), vw = *reinterpret_cast<const uint2 *>(vp);
      kf[0] = bf_lo(kw.x); kf[1] = bf_hi(kw.x); kf[2] = bf_lo(kw.y); kf[3] = bf_hi(kw.y);
      vf[0] = bf_lo(vw.x); vf[1] = bf_hi(vw.x); vf[2] = bf_lo(vw.y); vf[3] = bf_hi(vw.y);
    } else {
#pragma unroll
      for (int c = 0; c < EPL / 8; ++c) {
        uint4 kw = ldg_stream(kp + c * 8), vw = ldg_stream(vp + c * 8);
        kf[c * 8 + 0] = bf_lo(kw.x); kf[c * 8 + 1] = bf_hi(kw.x); kf[c * 8 + 2] = bf_lo(kw.y);
        kf[c * 8 + 3] = bf_hi(kw.y); kf[c * 8 + 4] = bf_lo(kw.z); kf[c * 8 + 5] = bf_hi(kw.z);
        kf[c * 8 + 6] = bf_lo(kw.w); kf[c * 8 + 7] = bf_hi(kw.w);
        vf[c * 8 + 0] = bf_lo(vw.x); vf[c * 8 + 1] = bf_hi(vw.x); vf[c * 8 + 2] = bf_lo(vw.y);
        vf[c * 8 + 3] = bf_hi(vw.y); vf[c * 8 + 4] = bf_lo(vw.z); vf[c * 8 + 5] = bf_hi(vw.z);
        vf[c * 8 + 6] = bf_lo(vw.w); vf[c * 8 + 7] = bf_hi(vw.w);
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
      float mn = fmaxf(mx[g], sc);
      float corr = __expf(mx[g] - mn), p = __expf(sc - mn);
      mx[g] = mn;
      sum[g] = sum[g] * corr + p;
#pragma unroll
      for (int e = 0; e < EPL; ++e) o[g][e] = o[g][e] * corr + p * vf[e];
    }
  }
  // merge the 4 workers of the warp (lanes with equal `part`)
#pragma unroll
  for (int off = 8; off <= 16; off <<= 1) {
#pragma unroll
    for (int g = 0; g < GQ; ++g) {
      float m2 = __shfl_xor_sync(0xffffffffu, mx[g], off);
      float s2 = __shfl_xor_sync(0xffffffffu, sum[g], off);
      float mn = fmaxf(mx[g], m2);
      float c1 = (mx[g] == -INFINITY) ? 0.f : __expf(mx[g] - mn);
      float c2 = (m2 == -INFINITY) ? 0.f : __expf(m2 - mn);
      sum[g] = sum[g] * c1 + s2 * c2;
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        float o2 = __shfl_xor_sync(0xffffffffu, o[g][e], off);
        o[g][e] = o[g][e] * c1 + o2 * c2;
      }
      mx[g] = mn;
    }
  }
  __shared__ float s_o[kWarps][GQ][DH];
  __shared__ float s_m[kWarps][GQ], s_l[kWarps][GQ];
  if (lane < 8) {
#pragma unroll
    for (int g = 0; g < GQ; ++g) {
#pragma unroll
      for (int e = 0; e < EPL; ++e) s_o[warp][g][part * EPL + e] = o[g][e];
      if (lane == 0) { s_m[warp][g] = mx[g]; s_l[warp][g] = sum[g]; }
    }
  }
  __syncthreads();
  for (int i = tid; i < GQ * DH; i += kThreads) {
    int g = i / DH, e = i % DH;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) M = fmaxf(M, s_m[w][g]);
    float Lsum = 0.f, O = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      float c = (s_m[w][g] == -INFINITY) ? 0.f : __expf(s_m[w][g] - M);
      Lsum += s_l[w][g] * c;
      O += s_o[w][g][e] * c;
    }
    size_t pi = ((size_t)row * dm.Hq + h0 + g) * max_splits + split;
    part_o[pi * DH + e] = O;
    if (e == 0) { part_ml[pi * 2] = M; part_ml[pi * 2 + 1] = Lsum; }
  }
}

// merge the splits of one (row, head): attn_out[row][h*dh + e]
__global__ void k_attn_combine(const float *part_o, const float *part_ml, const DevSched *s, int layer,
                               int split_len, int max_splits, float *attn_out, OpndOut opnd, Dims dm) {
  pdl_wait();
  pdl_trigger();
  const int row = blockIdx.y, h = blockIdx.x, e = threadIdx.x;
  if (row >= s->m[layer]) return;
  const int len = s->pos_s[row] + 1;
  const int ns = (len + split_len - 1) / split_len;
  const size_t pi = ((size_t)row * dm.Hq + h) * max_splits;
  float M = -INFINITY;
  for (int i = 0; i < ns; ++i) M = fmaxf(M, part_ml[(pi + i) * 2]);
  float Lsum = 0.f, O = 0.f;
  for (int i = 0; i < ns; ++i) {
    float c = __expf(part_ml[(pi + i) * 2] - M);
    Lsum += part_ml[(pi + i) * 2 + 1] * c;
    O += part_o[(pi + i) * dm.dh + e] * c;
  }
  const float val = O / Lsum;
  attn_out[(size_t)row * dm.Hq * dm.dh + h * dm.dh + e] = val;
  if (opnd.p) opnd_store(opnd, row, (size_t)dm.Hq * dm.dh, (size_t)h * dm.dh + e, val);
}

template <int DH>
static void attn_launch(const float *qkv, const bf16 *Kc, const bf16 *Vc, const DevSched *s, int layer,
                        int m_rows, int split_len, int n_splits, int max_splits, float *part_o,
                        float *part_ml, const Dims &dm, cudaStream_t st) {
  int G = dm.Hq / dm.Hkv;
  if (G % 4 == 0) {
    dim3 grid(n_splits, dm.Hq / 4, m_rows);
    launch_pdl(k_attn_partial<DH, 4>, grid, dim3(kThreads), 0, st, qkv, Kc, Vc, s, layer, split_len,
               max_splits, part_o, part_ml, dm);
  } else if (G % 2 == 0) {
    dim3 grid(n_splits, dm.Hq / 2, m_rows);
    launch_pdl(k_attn_partial<DH, 2>, grid, dim3(kThreads), 0, st, qkv, Kc, Vc, s, layer, split_len,
               max_splits, part_o, part_ml, dm);
  } else {
    dim3 grid(n_splits, dm.Hq, m_rows);
    launch_pdl(k_attn_partial<DH, 1>, grid, dim3(kThreads), 0, st, qkv, Kc, Vc, s, layer, split_len,
               max_splits, part_o, part_ml, dm);
  }
}

int launch_attention(const float *qkv, const bf16 *Kc, const bf16 *Vc, const DevSched *s, int layer,
                     int m_rows, int split_len, int n_splits, int max_splits, float *part_o,
                     float *part_ml, float *attn_out, OpndOut opnd, const Dims &dm, cudaStream_t st,
                     const RowOrder *order) {
  static const bool fma_path = getenv("D3_ATTN_FMA") != nullptr;   // the scalar kernel, for comparison
  // The tensor-core kernel pays a fixed cost per CTA (Q fragments, merge) that needs a few
  // 16-position trips per warp to amortise, unless several query heads share the K/V fragments:
  // measured, one row of the 13B shape (15 splits of 96 positions) is 13 % slower with it.
  const bool shared_kv = (dm.Hq / dm.Hkv) % 2 == 0;
  if (!fma_path && (shared_kv || split_len >= 256)) {
    launch_attention_partial_mma(qkv, Kc, Vc, s, layer, m_rows, split_len, n_splits, max_splits, part_o,
                                 part_ml, n_splits == 1 ? attn_out : nullptr, opnd, dm, st, order);
    if (n_splits == 1) return 1;   // every row and head in one piece: written directly
  } else if (dm.dh == 128)
    attn_launch<128>(qkv, Kc, Vc, s, layer, m_rows, split_len, n_splits, max_splits, part_o, part_ml, dm, st);
  else if (dm.dh == 64)
    attn_launch<64>(qkv, Kc, Vc, s, layer, m_rows, split_len, n_splits, max_splits, part_o, part_ml, dm, st);
  else
    attn_launch<32>(qkv, Kc, Vc, s, layer, m_rows, split_len, n_splits, max_splits, part_o, part_ml, dm, st);
  dim3 cgrid(dm.Hq, m_rows);
  launch_pdl(k_attn_combine, cgrid, dim3(dm.dh), 0, st, part_o, part_ml, s, layer, split_len, max_splits,
             attn_out, opnd, dm);
  return 2;
}

// --------------------------------------------------------------- KV fill: copy
// For every (dropped block l, row): K,V at the row's position := the row's K,V
// of block lo-1 written earlier in this step, or zeros when the window opens at
// block 0.  grid (L, B).
__global__ void k_fill_copy(bf16 *Kc, bf16 *Vc, const DevSched *s, Dims dm) {
  pdl_wait();
  pdl_trigger();
  const int l = blockIdx.x, row = blockIdx.y;
  const int lo = s->lo_s[row], hi = s->hi_s[row];
  if (l < lo || l >= hi) return;
  const int slot = s->slot_s[row], pos = s->pos_s[row];
  // 16-byte pieces (8 bf16; head_dim is a multiple of 32, every cache row 16-byte aligned)
  const int per_head = dm.dh / 8, n = dm.Hkv * per_head;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const int h = i / per_head, e = (i % per_head) * 8;
    uint4 *kd = reinterpret_cast<uint4 *>(Kc + kv_offset(dm, dm.block_table, l, slot, h, pos) + e);
    uint4 *vd = reinterpret_cast<uint4 *>(Vc + kv_offset(dm, dm.block_table, l, slot, h, pos) + e);
    if (lo == 0) {
      *kd = make_uint4(0u, 0u, 0u, 0u);   // bf16 zero is all-zero bits
      *vd = make_uint4(0u, 0u, 0u, 0u);
    } else {
      const size_t src = kv_offset(dm, dm.block_table, lo - 1, slot, h, pos) + e;
      const uint4 kw = *reinterpret_cast<const uint4 *>(Kc + src);
      const uint4 vw = *reinterpret_cast<const uint4 *>(Vc + src);
      *kd = kw;
      *vd = vw;
    }
  }
}

int launch_fill_copy(bf16 *Kc, bf16 *Vc, const DevSched *s, int B, const Dims &dm, cudaStream_t st) {
  dim3 grid(dm.L, B);
  launch_pdl(k_fill_copy, grid, dim3(128), 0, st, Kc, Vc, s, dm);
  return 1;
}

// ------------------------------------------------------- paged cache: block table
__global__ void k_table_update(int32_t *table, const __grid_constant__ TableUpdate u) {
  pdl_wait();
  pdl_trigger();
  const int i = threadIdx.x;
  if (i < u.n) table[u.index[i]] = u.page[i];
}

int launch_table_update(int32_t *table, const TableUpdate &u, cudaStream_t st) {
  launch_pdl(k_table_update, dim3(1), dim3(TableUpdate::kMax), 0, st, table, u);
  return 1;
}

// --------------------------------------------------------------------- argmax
// One CTA per row: 16-byte loads, (value, index) pairs reduced by shuffles inside a warp and
// through shared memory across warps; the lowest index wins a tie at every level.
__device__ __forceinline__ void argmax_take(float &best, int &bi, float v, int i) {
  if (v > best || (v == best && i < bi)) { best = v; bi = i; }
}

__global__ void __launch_bounds__(1024) k_argmax(const float *logits, int V, int32_t *out) {
  pdl_wait();
  pdl_trigger();
  const float *p = logits + (size_t)blockIdx.x * V;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  const bool vec = (V % 4 == 0) && ((reinterpret_cast<uintptr_t>(p) & 15u) == 0);
  if (vec) {
    for (int i = threadIdx.x * 4; i < V; i += blockDim.x * 4) {
      const float4 v = *reinterpret_cast<const float4 *>(p + i);
      argmax_take(best, bi, v.x, i); argmax_take(best, bi, v.y, i + 1);
      argmax_take(best, bi, v.z, i + 2); argmax_take(best, bi, v.w, i + 3);
    }
  } else {
    for (int i = threadIdx.x; i < V; i += blockDim.x) argmax_take(best, bi, p[i], i);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1)
    argmax_take(best, bi, __shfl_xor_sync(0xffffffffu, best, o), __shfl_xor_sync(0xffffffffu, bi, o));
  __shared__ float sv[32];
  __shared__ int si[32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) { sv[warp] = best; si[warp] = bi; }
  __syncthreads();
  if (warp == 0) {
    const int nw = blockDim.x >> 5;
    best = lane < nw ? sv[lane] : -INFINITY;
    bi = lane < nw ? si[lane] : 0x7fffffff;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
      argmax_take(best, bi, __shfl_xor_sync(0xffffffffu, best, o), __shfl_xor_sync(0xffffffffu, bi, o));
    if (lane == 0) out[blockIdx.x] = bi == 0x7fffffff ? 0 : bi;
  }
}

// argmax and its softmax probability of one logits row; results at out[row * stride + col]
__global__ void __launch_bounds__(1024) k_argmax_conf(const float *logits, int V, int32_t *tok, float *conf,
                                                      int stride, int col) {
  pdl_wait();
  pdl_trigger();
  const float *p = logits + (size_t)blockIdx.x * V;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  for (int i = threadIdx.x; i < V; i += blockDim.x) {
    float v = p[i];
    if (v > best) { best = v; bi = i; }
  }
  __shared__ float sv[1024];
  __shared__ int si[1024];
  sv[threadIdx.x] = best; si[threadIdx.x] = bi;
  __syncthreads();
  for (int o = blockDim.x / 2; o > 0; o >>= 1) {
    if (threadIdx.x < o) {
      float v2 = sv[threadIdx.x + o];
      int i2 = si[threadIdx.x + o];
      if (v2 > sv[threadIdx.x] || (v2 == sv[threadIdx.x] && i2 < si[threadIdx.x])) {
        sv[threadIdx.x] = v2; si[threadIdx.x] = i2;
      }
    }
    __syncthreads();
  }
  const float mx = sv[0];
  const int arg = si[0] == 0x7fffffff ? 0 : si[0];
  __syncthreads();
  float z = 0.f;
  for (int i = threadIdx.x; i < V; i += blockDim.x) z += __expf(p[i] - mx);
  sv[threadIdx.x] = z;
  __syncthreads();
  for (int o = blockDim.x / 2; o > 0; o >>= 1) {
    if (threadIdx.x < o) sv[threadIdx.x] += sv[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    tok[(size_t)blockIdx.x * stride + col] = arg;
    if (conf) conf[(size_t)blockIdx.x * stride + col] = 1.f / sv[0];
  }
}

int launch_argmax_conf(const float *logits, int B, int V, int32_t *tok, float *conf, int stride, int col,
                       cudaStream_t st) {
  launch_pdl(k_argmax_conf, dim3(B), dim3(1024), 0, st, logits, V, tok, conf, stride, col);
  return 1;
}

int launch_argmax(const float *logits, int B, int V, int32_t *out, cudaStream_t st) {
  launch_pdl(k_argmax, dim3(B), dim3(1024), 0, st, logits, V, out);
  return 1;
}

}  // namespace d3

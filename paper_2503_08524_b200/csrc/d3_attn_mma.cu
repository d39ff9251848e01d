// Flash-decoding attention with the scores and the value sums on the tensor cores
// (mma.sync m16n8k16, bf16 x bf16 -> fp32), for the sequence-of-kernels path.
//
// Same work split and outputs as k_attn_partial (a CTA = one row, one group of GQ
// query heads that share a KV head, one split of the positions; it writes the
// partial (max, sum, unnormalised o) of every head), but a warp takes 16
// positions per trip instead of 4 and spends ~3x fewer instructions per position:
// K and V enter the MMAs as the bf16 they are stored as, no widening to fp32.
//
// The query stays exact enough by splitting: row g of the 16-row A operand holds
// bf16(q_g), row g + 8 holds bf16(q_g - bf16(q_g)) (head g of the group, scaled by
// 1/sqrt(dh)); the two score rows land in the same thread (accumulator rows g and
// g + 8) and are added there.  The probabilities take the same two rows for the
// second product, o = p V.  Rows GQ..7 and 8+GQ..15 are zero.
//
// K and V of a warp's 16 positions are staged row-major in shared memory by cp.async (rows padded
// by 16 bytes, two stages per warp: the next trip's rows are in flight while this trip computes),
// which keeps bytes in flight without holding them in registers: three 128-thread CTAs fit an SM.
// Fragment bookkeeping (thread = (g, t) = (lane / 4, lane % 4)):
//   scores  S = Q K^T : B = K^T (k = head dimension, column n = position): ldmatrix on K rows.
//   values  O = P V   : B = V   (k = position, n = dimension): ldmatrix.trans on V rows.
#include "d3_internal.cuh"

namespace d3 {

namespace {

constexpr int kAThreads = 128;
constexpr int kAWarps = kAThreads / 32;

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const uint32_t a = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(lo));
  const uint32_t b = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(hi));
  return a | (b << 16);
}
__device__ __forceinline__ float bf16_round(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int DH>
struct VStage {
  static constexpr int kRowBytes = DH * 2 + 16;       // padded: ldmatrix rows fall in distinct banks
  static constexpr int kTile = 16 * kRowBytes;        // 16 positions of K or of V
  static constexpr int kBytes = 2 * kTile;            // one stage: K tile, then V tile
};

template <int DH, int GQ>
__global__ void __launch_bounds__(kAThreads)
k_attn_partial_mma(const float *qkv, const bf16 *Kc, const bf16 *Vc, const DevSched *s, int layer,
                   int split_len, int max_splits, float *part_o, float *part_ml, float *attn_out, OpndOut opnd,
                   Dims dm, const __grid_constant__ RowOrder order) {
  static_assert(GQ <= 8, "one accumulator row per query head");
  constexpr int KK = DH / 16;          // MMA steps over the head dimension
  constexpr int NT = DH / 8;           // 8-wide dimension tiles of the output
  extern __shared__ __align__(16) unsigned char s_v[];   // [warp][2 stages][K | V][16 positions][padded row]
  __shared__ float s_o[kAWarps][GQ][DH];
  __shared__ float s_m[kAWarps][GQ], s_l[kAWarps][GQ];
  pdl_wait();
  pdl_trigger();
  const int row = order.given ? order.r[blockIdx.z] : blockIdx.z;
  if (row >= s->m[layer]) return;
  const int len = s->pos_s[row] + 1;
  const int split = blockIdx.x;
  const int t0 = split * split_len;
  if (t0 >= len) return;
  const int t1 = min(len, t0 + split_len);
  const int h0 = blockIdx.y * GQ;
  const int kvh = h0 / (dm.Hq / dm.Hkv);
  const int slot = s->slot_s[row];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;

  // ---- A operand of the score product: this thread's pieces of Q (hi rows g, lo rows g + 8)
  uint32_t qa[KK][4];
  {
    const float scale = rsqrtf((float)DH);
    const float *qp = qkv + (size_t)row * dm.qkv_rows + (size_t)(h0 + (g < GQ ? g : 0)) * DH;
#pragma unroll
    for (int kk = 0; kk < KK; ++kk) {
      float v[4], r[4];   // dims 16kk + 2t + {0, 1} and 16kk + 8 + 2t + {0, 1}
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        v[j] = g < GQ ? qp[16 * kk + 8 * (j >> 1) + 2 * t + (j & 1)] * scale : 0.f;
        r[j] = v[j] - bf16_round(v[j]);
      }
      qa[kk][0] = pack_bf16(v[0], v[1]);   // row g,     k = 2t, 2t+1
      qa[kk][1] = pack_bf16(r[0], r[1]);   // row g + 8
      qa[kk][2] = pack_bf16(v[2], v[3]);   // row g,     k = 2t+8, 2t+9
      qa[kk][3] = pack_bf16(r[2], r[3]);   // row g + 8
    }
  }

  float o[NT][4];      // rows g (hi term of p) and g + 8 (lo term): dims 8n + 2t, 8n + 2t + 1
#pragma unroll
  for (int n = 0; n < NT; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
  float mx = -INFINITY, sum = 0.f;     // of head g, this thread's positions only (sum) / all (mx)

  unsigned char *vbuf = s_v + (size_t)warp * 2 * VStage<DH>::kBytes;
  // chunk c of this warp: positions t0 + 16 * (warp + 8 c) .. + 15
  auto chunk_pos = [&](int c) { return t0 + 16 * (warp + kAWarps * c); };
  auto stage_v = [&](int c, int buf) {
    const int p0 = chunk_pos(c);
    if (p0 < t1) {
      constexpr int CPR = DH * 2 / 16;   // 16-byte pieces per row
      // the 16 positions are consecutive rows of the cache (one page at most: p0 is a multiple
      // of 16 and a page holds a power of two >= 16 positions): one offset per trip
      const size_t base = kv_offset(dm, dm.block_table, layer, slot, kvh, p0);
      const int rmax = t1 - 1 - p0;      // rows past the end repeat the last valid one
#pragma unroll
      for (int i = 0; i < 16 * CPR / 32; ++i) {
        const int idx = i * 32 + lane, r = idx / CPR, cidx = idx % CPR;
        const size_t off = base + (size_t)(min(r, rmax) * DH + cidx * 8);
        const uint32_t dst =
            (uint32_t)__cvta_generic_to_shared(vbuf + buf * VStage<DH>::kBytes + r * VStage<DH>::kRowBytes + cidx * 16);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(Kc + off) : "memory");
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + VStage<DH>::kTile), "l"(Vc + off)
                     : "memory");
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };

  stage_v(0, 0);
  for (int c = 0; chunk_pos(c) < t1; ++c) {
    const int p0 = chunk_pos(c), buf = c & 1;
    stage_v(c + 1, buf ^ 1);                       // next chunk's K and V while this one is used
    asm volatile("cp.async.wait_group 1;" ::: "memory");   // all but the copies just issued
    __syncwarp();
    const uint32_t ks = (uint32_t)__cvta_generic_to_shared(vbuf + buf * VStage<DH>::kBytes);
    // ---- scores of the 16 positions: K fragments straight from the staged rows
    float sc[2][4];
    sc[0][0] = sc[0][1] = sc[0][2] = sc[0][3] = 0.f;
    sc[1][0] = sc[1][1] = sc[1][2] = sc[1][3] = 0.f;
#pragma unroll
    for (int kk = 0; kk < KK; ++kk) {
      // matrices: (positions 0-7, dims 16kk..+7), (0-7, +8..+15), (8-15, 16kk..+7), (8-15, +8..+15)
      const int mat = lane >> 3, r = (lane & 7) + 8 * (mat >> 1), piece = 2 * kk + (mat & 1);
      uint32_t b[4];
      asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                   : "=r"(b[0]), "=r"(b[1]), "=r"(b[2]), "=r"(b[3])
                   : "r"(ks + r * VStage<DH>::kRowBytes + piece * 16));
      mma_bf16(sc[0], qa[kk], b[0], b[1]);
      mma_bf16(sc[1], qa[kk], b[2], b[3]);
    }
    // this thread: head g, positions p0 + 8h + 2t + {0, 1}: hi row + lo row
    float sv[4];
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int pos = p0 + 8 * h + 2 * t + j;
        sv[2 * h + j] = pos < t1 ? sc[h][j] + sc[h][2 + j] : -INFINITY;
      }
    float cm = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
    cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 1));
    cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, 2));
    const float mn = fmaxf(mx, cm);            // finite: the chunk holds at least one position
    if (__any_sync(0xffffffffu, g < GQ && mn > mx)) {   // a new maximum somewhere: rescale
      const float corr = (mx == -INFINITY) ? 0.f : __expf(mx - mn);
      sum *= corr;
#pragma unroll
      for (int n = 0; n < NT; ++n) { o[n][0] *= corr; o[n][1] *= corr; o[n][2] *= corr; o[n][3] *= corr; }
    }
    mx = mn;
    uint32_t pa[4];
    {
      float p[4], r[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        p[i] = (g < GQ && sv[i] != -INFINITY) ? __expf(sv[i] - mn) : 0.f;
        r[i] = p[i] - bf16_round(p[i]);
        sum += p[i];
      }
      pa[0] = pack_bf16(p[0], p[1]);   // row g,     positions 2t, 2t+1
      pa[1] = pack_bf16(r[0], r[1]);   // row g + 8
      pa[2] = pack_bf16(p[2], p[3]);   // row g,     positions 8+2t, 8+2t+1
      pa[3] = pack_bf16(r[2], r[3]);   // row g + 8
    }
    // ---- o += p V: V of this chunk from shared memory, transposed fragments
    const uint32_t vs = ks + VStage<DH>::kTile;
#pragma unroll
    for (int n = 0; n < NT; n += 2) {
      // matrices: (positions 0-7, tile n), (8-15, tile n), (0-7, tile n+1), (8-15, tile n+1)
      const int mat = lane >> 3, r = (lane & 7) + 8 * (mat & 1), tile = n + (mat >> 1);
      uint32_t b[4];
      asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                   : "=r"(b[0]), "=r"(b[1]), "=r"(b[2]), "=r"(b[3])
                   : "r"(vs + r * VStage<DH>::kRowBytes + tile * 16));
      mma_bf16(o[n], pa, b[0], b[1]);
      mma_bf16(o[n + 1], pa, b[2], b[3]);
    }
    __syncwarp();   // the buffer is refilled two trips from now, by this warp
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");

  // ---- this warp's partial of head g: sum over the four threads of the group
  sum += __shfl_xor_sync(0xffffffffu, sum, 1);
  sum += __shfl_xor_sync(0xffffffffu, sum, 2);
  if (g < GQ) {
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      s_o[warp][g][8 * n + 2 * t] = o[n][0] + o[n][2];
      s_o[warp][g][8 * n + 2 * t + 1] = o[n][1] + o[n][3];
    }
    if (t == 0) { s_m[warp][g] = mx; s_l[warp][g] = sum; }
  }
  __syncthreads();
  for (int i = tid; i < GQ * DH; i += kAThreads) {
    const int gg = i / DH, e = i % DH;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kAWarps; ++w) M = fmaxf(M, s_m[w][gg]);
    float Lsum = 0.f, O = 0.f;
#pragma unroll
    for (int w = 0; w < kAWarps; ++w) {
      const float c = (s_m[w][gg] == -INFINITY) ? 0.f : __expf(s_m[w][gg] - M);
      Lsum += s_l[w][gg] * c;
      O += s_o[w][gg][e] * c;
    }
    if (attn_out) {   // the only piece of its row and head: the result itself, no combine pass
      const float val = O / Lsum;
      attn_out[(size_t)row * dm.Hq * DH + (size_t)(h0 + gg) * DH + e] = val;
      if (opnd.p) opnd_store(opnd, row, (size_t)dm.Hq * DH, (size_t)(h0 + gg) * DH + e, val);
      continue;
    }
    const size_t pi = ((size_t)row * dm.Hq + h0 + gg) * max_splits + split;
    part_o[pi * DH + e] = O;
    if (e == 0) { part_ml[pi * 2] = M; part_ml[pi * 2 + 1] = Lsum; }
  }
}

template <int DH>
constexpr size_t v_smem() { return (size_t)kAWarps * 2 * VStage<DH>::kBytes; }

template <int DH, int GQ>
cudaError_t mma_attr() {
  return cudaFuncSetAttribute(k_attn_partial_mma<DH, GQ>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)v_smem<DH>());
}

template <int DH>
void launch_dh(const float *qkv, const bf16 *Kc, const bf16 *Vc, const DevSched *s, int layer, int m_rows,
               int split_len, int n_splits, int max_splits, float *part_o, float *part_ml, float *attn_out,
               OpndOut opnd, const Dims &dm, cudaStream_t st, const RowOrder &order) {
  const int G = dm.Hq / dm.Hkv;
  if (G % 4 == 0) {
    launch_pdl(k_attn_partial_mma<DH, 4>, dim3(n_splits, dm.Hq / 4, m_rows), dim3(kAThreads), v_smem<DH>(), st,
               qkv, Kc, Vc, s, layer, split_len, max_splits, part_o, part_ml, attn_out, opnd, dm, order);
  } else if (G % 2 == 0) {
    launch_pdl(k_attn_partial_mma<DH, 2>, dim3(n_splits, dm.Hq / 2, m_rows), dim3(kAThreads), v_smem<DH>(), st,
               qkv, Kc, Vc, s, layer, split_len, max_splits, part_o, part_ml, attn_out, opnd, dm, order);
  } else {
    launch_pdl(k_attn_partial_mma<DH, 1>, dim3(n_splits, dm.Hq, m_rows), dim3(kAThreads), v_smem<DH>(), st,
               qkv, Kc, Vc, s, layer, split_len, max_splits, part_o, part_ml, attn_out, opnd, dm, order);
  }
}

}  // namespace

int init_attention_mma() {
  cudaError_t e = cudaSuccess;
#define D3_MMA_ATTR(DH)                               \
  if (e == cudaSuccess) e = mma_attr<DH, 1>();        \
  if (e == cudaSuccess) e = mma_attr<DH, 2>();        \
  if (e == cudaSuccess) e = mma_attr<DH, 4>();
  D3_MMA_ATTR(128) D3_MMA_ATTR(64) D3_MMA_ATTR(32)
#undef D3_MMA_ATTR
  return e == cudaSuccess ? 0 : -1;
}

// The partial pass of launch_attention on the tensor cores.  attn_out non-null (only with one
// piece per row and head): the normalised result goes there and no combine pass is needed.
int launch_attention_partial_mma(const float *qkv, const bf16 *Kc, const bf16 *Vc, const DevSched *s, int layer,
                                 int m_rows, int split_len, int n_splits, int max_splits, float *part_o,
                                 float *part_ml, float *attn_out, OpndOut opnd, const Dims &dm, cudaStream_t st,
                                 const RowOrder *order_in) {
  RowOrder order;
  if (order_in) order = *order_in; else order.given = 0;
  if (dm.dh == 128)
    launch_dh<128>(qkv, Kc, Vc, s, layer, m_rows, split_len, n_splits, max_splits, part_o, part_ml, attn_out, opnd, dm, st, order);
  else if (dm.dh == 64)
    launch_dh<64>(qkv, Kc, Vc, s, layer, m_rows, split_len, n_splits, max_splits, part_o, part_ml, attn_out, opnd, dm, st, order);
  else
    launch_dh<32>(qkv, Kc, Vc, s, layer, m_rows, split_len, n_splits, max_splits, part_o, part_ml, attn_out, opnd, dm, st, order);
  return 1;
}

}  // namespace d3

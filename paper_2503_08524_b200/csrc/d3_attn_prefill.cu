// Causal flash attention of a prefill pass (initiation phase, Sec. 3.1): the rows of
// the pass are consecutive prompt positions t0 .. t0 + B - 1 of ONE sequence, every
// row attends to the cache positions 0 .. its own (its K and V were appended by the
// pass's RoPE kernel just before).
//
// A CTA takes 16 consecutive rows (one m16 tile) of one query head; its four warps
// share the key range 16 positions at a time (warp w: chunks w, w + 4, ...), each
// keeping a running (max, sum, o) per row, merged through shared memory at the end.
// Scores and value sums run on mma.sync.m16n8k16 (bf16 x bf16 -> fp32) with K and V
// as stored; the fp32 queries and probabilities enter as two bf16 terms each
// (hi + lo, two MMAs), which keeps them exact to 16 significand bits.  K and V
// rows are staged in shared memory by cp.async, two stages per warp.
// Fragment bookkeeping (thread = (g, t) = (lane / 4, lane % 4)): accumulator
// entries 0, 1 belong to row g, entries 2, 3 to row g + 8 of the tile.
#include "d3_internal.cuh"

namespace d3 {

namespace {

constexpr int kPThreads = 128;
constexpr int kPWarps = kPThreads / 32;
constexpr int kTileRows = 16;

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  const uint32_t a = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(lo));
  const uint32_t b = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(hi));
  return a | (b << 16);
}
__device__ __forceinline__ float rnd_bf16(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int DH>
struct PStage {
  static constexpr int kRowBytes = DH * 2 + 16;       // padded: ldmatrix rows fall in distinct banks
  static constexpr int kTile = 16 * kRowBytes;        // 16 positions of K or of V
  static constexpr int kBytes = 2 * kTile;            // one stage: K tile, then V tile
};

template <int DH>
constexpr size_t p_smem() {
  // K/V staging of four warps, reused for the merge of their partial results ([warp][16][DH] floats)
  return (size_t)kPWarps * 2 * PStage<DH>::kBytes > (size_t)kPWarps * kTileRows * DH * 4
             ? (size_t)kPWarps * 2 * PStage<DH>::kBytes
             : (size_t)kPWarps * kTileRows * DH * 4;
}

template <int DH>
__global__ void __launch_bounds__(kPThreads)
k_attn_prefill(const float *qkv, const bf16 *Kc, const bf16 *Vc, int layer, int slot, int t0, int B,
               float *attn_out, Dims dm) {
  constexpr int KK = DH / 16;          // MMA steps over the head dimension
  constexpr int NT = DH / 8;           // 8-wide dimension tiles of the output
  extern __shared__ __align__(16) unsigned char s_v[];
  __shared__ float s_m[kPWarps][kTileRows], s_l[kPWarps][kTileRows];
  pdl_wait();
  pdl_trigger();
  const int i0 = blockIdx.x * kTileRows;
  if (i0 >= B) return;
  const int h = blockIdx.y;
  const int kvh = h / (dm.Hq / dm.Hkv);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int last_row = min(i0 + kTileRows, B) - 1;
  const int t1 = t0 + last_row + 1;            // keys 0 .. t1 - 1 matter to this tile
  const int qpos0 = t0 + i0 + g, qpos1 = qpos0 + 8;   // positions of this thread's two rows

  // ---- A operands of the score product: rows g and g + 8 of Q, hi and lo terms
  uint32_t qh[KK][4], ql[KK][4];
  {
    const float scale = rsqrtf((float)DH);
    const int ra = min(i0 + g, B - 1), rb = min(i0 + g + 8, B - 1);   // rows past the pass repeat the last one
    const float *qa = qkv + (size_t)ra * dm.qkv_rows + (size_t)h * DH;
    const float *qb = qkv + (size_t)rb * dm.qkv_rows + (size_t)h * DH;
#pragma unroll
    for (int kk = 0; kk < KK; ++kk) {
      float va[4], vb[4];   // dims 16kk + 2t + {0, 1} and 16kk + 8 + 2t + {0, 1}
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int e = 16 * kk + 8 * (j >> 1) + 2 * t + (j & 1);
        va[j] = qa[e] * scale;
        vb[j] = qb[e] * scale;
      }
      qh[kk][0] = pack2(va[0], va[1]); qh[kk][1] = pack2(vb[0], vb[1]);
      qh[kk][2] = pack2(va[2], va[3]); qh[kk][3] = pack2(vb[2], vb[3]);
      ql[kk][0] = pack2(va[0] - rnd_bf16(va[0]), va[1] - rnd_bf16(va[1]));
      ql[kk][1] = pack2(vb[0] - rnd_bf16(vb[0]), vb[1] - rnd_bf16(vb[1]));
      ql[kk][2] = pack2(va[2] - rnd_bf16(va[2]), va[3] - rnd_bf16(va[3]));
      ql[kk][3] = pack2(vb[2] - rnd_bf16(vb[2]), vb[3] - rnd_bf16(vb[3]));
    }
  }

  float o[NT][4];
#pragma unroll
  for (int n = 0; n < NT; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
  float mx[2] = {-INFINITY, -INFINITY}, sum[2] = {0.f, 0.f};   // rows g, g + 8 (sum: this thread's keys only)

  unsigned char *vbuf = s_v + (size_t)warp * 2 * PStage<DH>::kBytes;
  auto chunk_pos = [&](int c) { return 16 * (warp + kPWarps * c); };
  auto stage_kv = [&](int c, int buf) {
    const int p0 = chunk_pos(c);
    if (p0 < t1) {
      constexpr int CPR = DH * 2 / 16;   // 16-byte pieces per row
      // 16 consecutive positions starting at a multiple of 16 never straddle a page
      const size_t base = kv_offset(dm, dm.block_table, layer, slot, kvh, p0);
      const int rmax = t1 - 1 - p0;      // rows past the end repeat the last valid one
#pragma unroll
      for (int i = 0; i < 16 * CPR / 32; ++i) {
        const int idx = i * 32 + lane, r = idx / CPR, cidx = idx % CPR;
        const size_t off = base + (size_t)(min(r, rmax) * DH + cidx * 8);
        const uint32_t dst =
            (uint32_t)__cvta_generic_to_shared(vbuf + buf * PStage<DH>::kBytes + r * PStage<DH>::kRowBytes + cidx * 16);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(Kc + off) : "memory");
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + PStage<DH>::kTile), "l"(Vc + off)
                     : "memory");
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };

  stage_kv(0, 0);
  for (int c = 0; chunk_pos(c) < t1; ++c) {
    const int p0 = chunk_pos(c), buf = c & 1;
    stage_kv(c + 1, buf ^ 1);                      // next chunk's K and V while this one is used
    asm volatile("cp.async.wait_group 1;" ::: "memory");   // all but the copies just issued
    __syncwarp();
    const uint32_t ks = (uint32_t)__cvta_generic_to_shared(vbuf + buf * PStage<DH>::kBytes);
    // ---- scores of the 16 keys for the 16 rows: K fragments straight from the staged rows
    float sc[2][4];
    sc[0][0] = sc[0][1] = sc[0][2] = sc[0][3] = 0.f;
    sc[1][0] = sc[1][1] = sc[1][2] = sc[1][3] = 0.f;
#pragma unroll
    for (int kk = 0; kk < KK; ++kk) {
      // matrices: (keys 0-7, dims 16kk..+7), (0-7, +8..+15), (8-15, 16kk..+7), (8-15, +8..+15)
      const int mat = lane >> 3, r = (lane & 7) + 8 * (mat >> 1), piece = 2 * kk + (mat & 1);
      uint32_t b[4];
      asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                   : "=r"(b[0]), "=r"(b[1]), "=r"(b[2]), "=r"(b[3])
                   : "r"(ks + r * PStage<DH>::kRowBytes + piece * 16));
      mma16816(sc[0], qh[kk], b[0], b[1]);
      mma16816(sc[0], ql[kk], b[0], b[1]);
      mma16816(sc[1], qh[kk], b[2], b[3]);
      mma16816(sc[1], ql[kk], b[2], b[3]);
    }
    // this thread: rows g (entries 0, 1) and g + 8 (entries 2, 3), keys p0 + 8 hh + 2t + {0, 1};
    // causal: a key counts when it is not beyond the row's own position
    float sv[2][4];   // [row][hh * 2 + j]
    float cm[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int hh = 0; hh < 2; ++hh)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int key = p0 + 8 * hh + 2 * t + j;
        sv[0][2 * hh + j] = key <= qpos0 ? sc[hh][j] : -INFINITY;
        sv[1][2 * hh + j] = key <= qpos1 ? sc[hh][2 + j] : -INFINITY;
        cm[0] = fmaxf(cm[0], sv[0][2 * hh + j]);
        cm[1] = fmaxf(cm[1], sv[1][2 * hh + j]);
      }
    uint32_t ph[4], pl[4];
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      float m = cm[rr];
      m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
      m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
      const float mn = fmaxf(mx[rr], m);
      // a row may have no key at all in this chunk (or so far): every exponent then reads -inf - 0
      const float mref = (mn == -INFINITY) ? 0.f : mn;
      if (mn > mx[rr]) {
        const float corr = (mx[rr] == -INFINITY) ? 0.f : __expf(mx[rr] - mref);
        sum[rr] *= corr;
#pragma unroll
        for (int n = 0; n < NT; ++n) { o[n][2 * rr] *= corr; o[n][2 * rr + 1] *= corr; }
      }
      mx[rr] = mn;
      float p[4], r[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        p[i] = __expf(sv[rr][i] - mref);     // exp(-inf) = 0 for masked keys
        r[i] = p[i] - rnd_bf16(p[i]);
        sum[rr] += p[i];
      }
      // A fragment of the value product: entry rr = (row, keys 2t, 2t+1), entry 2 + rr = keys 8 + 2t, ...
      ph[rr] = pack2(p[0], p[1]);     pl[rr] = pack2(r[0], r[1]);
      ph[2 + rr] = pack2(p[2], p[3]); pl[2 + rr] = pack2(r[2], r[3]);
    }
    // ---- o += p V: V of this chunk from shared memory, transposed fragments
    const uint32_t vs = ks + PStage<DH>::kTile;
#pragma unroll
    for (int n = 0; n < NT; n += 2) {
      // matrices: (keys 0-7, tile n), (8-15, tile n), (0-7, tile n+1), (8-15, tile n+1)
      const int mat = lane >> 3, r = (lane & 7) + 8 * (mat & 1), tile = n + (mat >> 1);
      uint32_t b[4];
      asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                   : "=r"(b[0]), "=r"(b[1]), "=r"(b[2]), "=r"(b[3])
                   : "r"(vs + r * PStage<DH>::kRowBytes + tile * 16));
      mma16816(o[n], ph, b[0], b[1]);
      mma16816(o[n], pl, b[0], b[1]);
      mma16816(o[n + 1], ph, b[2], b[3]);
      mma16816(o[n + 1], pl, b[2], b[3]);
    }
    __syncwarp();   // the buffer is refilled two trips from now, by this warp
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();   // every warp is done with its staging buffers: they now hold the partial results

  // ---- this warp's partial of rows g, g + 8: sums over the four threads of a row
  float *s_o = reinterpret_cast<float *>(s_v);   // [warp][16][DH]
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    sum[rr] += __shfl_xor_sync(0xffffffffu, sum[rr], 1);
    sum[rr] += __shfl_xor_sync(0xffffffffu, sum[rr], 2);
    const int row = g + 8 * rr;
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      s_o[((size_t)warp * kTileRows + row) * DH + 8 * n + 2 * t] = o[n][2 * rr];
      s_o[((size_t)warp * kTileRows + row) * DH + 8 * n + 2 * t + 1] = o[n][2 * rr + 1];
    }
    if (t == 0) { s_m[warp][row] = mx[rr]; s_l[warp][row] = sum[rr]; }
  }
  __syncthreads();
  for (int i = tid; i < kTileRows * DH; i += kPThreads) {
    const int row = i / DH, e = i % DH;
    if (i0 + row >= B) continue;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kPWarps; ++w) M = fmaxf(M, s_m[w][row]);
    float Lsum = 0.f, O = 0.f;
#pragma unroll
    for (int w = 0; w < kPWarps; ++w) {
      const float cf = (s_m[w][row] == -INFINITY) ? 0.f : __expf(s_m[w][row] - M);
      Lsum += s_l[w][row] * cf;
      O += s_o[((size_t)w * kTileRows + row) * DH + e] * cf;
    }
    attn_out[(size_t)(i0 + row) * dm.Hq * DH + (size_t)h * DH + e] = O / Lsum;
  }
}

template <int DH>
cudaError_t pf_attr() {
  return cudaFuncSetAttribute(k_attn_prefill<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p_smem<DH>());
}

template <int DH>
void launch_pf(const float *qkv, const bf16 *Kc, const bf16 *Vc, int layer, int slot, int t0, int B,
               float *attn_out, const Dims &dm, cudaStream_t st) {
  launch_pdl(k_attn_prefill<DH>, dim3((B + kTileRows - 1) / kTileRows, dm.Hq), dim3(kPThreads), p_smem<DH>(), st,
             qkv, Kc, Vc, layer, slot, t0, B, attn_out, dm);
}

}  // namespace

int init_attention_prefill() {
  cudaError_t e = pf_attr<128>();
  if (e == cudaSuccess) e = pf_attr<64>();
  if (e == cudaSuccess) e = pf_attr<32>();
  return e == cudaSuccess ? 0 : -1;
}

// Attention of a prefill pass: rows 0 .. B-1 of qkv are the positions t0 .. t0 + B - 1 of `slot`
// (q already rotated, K and V of these positions already in the cache); attn_out [B][Hq * dh].
int launch_attention_prefill(const float *qkv, const bf16 *Kc, const bf16 *Vc, int layer, int slot, int t0, int B,
                             float *attn_out, const Dims &dm, cudaStream_t st) {
  if (dm.dh == 128) launch_pf<128>(qkv, Kc, Vc, layer, slot, t0, B, attn_out, dm, st);
  else if (dm.dh == 64) launch_pf<64>(qkv, Kc, Vc, layer, slot, t0, B, attn_out, dm, st);
  else launch_pf<32>(qkv, Kc, Vc, layer, slot, t0, B, attn_out, dm, st);
  return 1;
}

}  // namespace d3

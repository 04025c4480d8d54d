// Weight-streaming skinny GEMM of the batched recurrence (Sec. 4.2 step 1): y[m][n] = sum_k x[m][k] W[n][k]
// for the few token rows m of one pass, with the prologue (RMSNorm of the residual stream) and the
// epilogue (rotary + KV write, residual add, SwiGLU, logits) fused in.
//
// Mapping.  The weights are the 16-row A operand of mma.sync.m16n8k16 (bf16, fp32 accumulate); the token
// rows are the 8 B columns.  Every fp32 activation is split into three bf16 terms hi + mid + lo (an exact
// 24-bit decomposition), each fed through its own MMA into the same accumulator, so products are exact and
// a token's result does not depend on which other tokens share the pass.  A CTA of 8 warps owns a block of
// 128 output rows (one 16-row tile per warp) over a contiguous range of 32-wide k-blocks.  The work
// (row block x k-block) is linearised and cut into equal shares, one per CTA (stream-K): a row block whose
// k-range is shared by several CTAs is reduced in fixed order by whichever CTA arrives last, which then runs
// the epilogue.  No atomics touch data, so results are bit-reproducible.
#pragma once
#include "common.cuh"

namespace ls {

enum { EPI_PLAIN = 0, EPI_QKV = 1, EPI_RESID = 2, EPI_SWIGLU = 3, EPI_LOGITS = 4 };
enum { XS_BUF = 0, XS_HID_NORM = 1, XS_HID_NORM_RO = 2 };

constexpr int GEMM_THREADS = 256;
constexpr int RB_ROWS = 128;      // output rows per row block
constexpr int TILE_LD = 132;      // padded leading dimension of the epilogue tile
constexpr int UNROLL_BF16 = 4;    // k-blocks whose weight loads are in flight per warp (x2 for the prefetch)
constexpr int UNROLL_F32 = 2;

__host__ __device__ constexpr int xchunk_kblocks(int NG) { return NG <= 1 ? 16 : (NG == 2 ? 8 : (NG <= 4 ? 4 : 2)); }
__host__ __device__ constexpr int gemm_smem_bytes(int NG) {
  return 3 * xchunk_kblocks(NG) * 8 * NG * 64 + 8 * NG * TILE_LD * 4 + 8 * NG * 4 + 16;
}

struct GemmParams {
  const void* W;
  int N, K;
  int n_rb, kb_per_rb, units_per_cta, total_units;
  // activation source
  int xs_kind;
  const float* xbuf;  // XS_BUF: xbuf[row * x_ld + k]
  int x_ld;
  float* hid;         // hidden states [hid_idx][H] (XS_HID_*, EPI_RESID)
  int H;
  const float* gain;  // RMSNorm gain [K]
  const float* sumsq; // per row partial sums of squares [row][n_sq]; n_sq = 0: compute from the row
  int n_sq;
  float eps;
  const RowTable* tab;
  int m_fixed;        // tab == nullptr: number of rows of a stand-alone call
  // split-k scratch
  float* partials;    // [n_rb][max_contrib][8*NG][128]
  int max_contrib;
  int* counters;      // [n_rb], zero between launches
  // epilogue outputs
  float* out;         // PLAIN y, SWIGLU act buffer
  int out_ld;
  float* sumsq_out;   // RESID: [row][n_sq_out]
  int n_sq_out;
  float* qbuf;        // QKV: [row][n_q_heads * d]
  __nv_bfloat16* kv;  // QKV: this layer's KV pool [R][2][S][n_kv][slots][d]
  long long kv_plane_stride, kv_sel_stride;
  int slots, n_kv_heads, n_q_heads, head_dim;
  const float2* rope; // [pos][d/2] (cos, sin)
  float* logits;      // LOGITS: [logit_idx][V]
  int F;              // SWIGLU: ffn width
};

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0,
                                         unsigned b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// x = hi + mid + lo with hi, mid, lo bf16 (round-to-nearest at each stage; the remainders are exact in fp32)
__device__ __forceinline__ void split3(float x, unsigned short& hi, unsigned short& mid, unsigned short& lo) {
  __nv_bfloat16 h = __float2bfloat16_rn(x);
  float r1 = x - __bfloat162float(h);
  __nv_bfloat16 m = __float2bfloat16_rn(r1);
  float r2 = r1 - __bfloat162float(m);
  __nv_bfloat16 l = __float2bfloat16_rn(r2);
  hi = __bfloat16_as_ushort(h);
  mid = __bfloat16_as_ushort(m);
  lo = __bfloat16_as_ushort(l);
}

template <typename WT>
struct WTraits;
template <>
struct WTraits<__nv_bfloat16> {
  static constexpr int U = UNROLL_BF16;
  static constexpr int V4 = 2;  // uint4 loads per unit per thread: row g, row g+8 (8 bf16 each)
};
template <>
struct WTraits<float> {
  static constexpr int U = UNROLL_F32;
  static constexpr int V4 = 4;  // row g (8 floats), row g+8 (8 floats)
};

template <typename WT, int NG, int EPI>
__global__ void __launch_bounds__(GEMM_THREADS) gemm_kernel(const GemmParams p) {
  constexpr int NTOK = 8 * NG;
  constexpr int XCH = xchunk_kblocks(NG);
  constexpr int U = WTraits<WT>::U;
  constexpr int V4 = WTraits<WT>::V4;
  constexpr bool IS_BF16 = (sizeof(WT) == 2);

  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4* xs = reinterpret_cast<uint4*>(smem_raw);                       // staged activations
  float* tile = reinterpret_cast<float*>(smem_raw + 3 * XCH * NTOK * 64);  // [NTOK][TILE_LD]
  float* s_rstd = tile + NTOK * TILE_LD;                                // [NTOK]
  int* s_flag = reinterpret_cast<int*>(s_rstd + NTOK);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const RowTable* tab = p.tab;
  int n_cols;
  if (tab == nullptr) n_cols = p.m_fixed;
  else n_cols = (p.xs_kind == XS_HID_NORM_RO) ? tab->n_readout : tab->n_rows;
  if (n_cols <= 0) return;
  if (n_cols > NTOK) n_cols = NTOK;

  const int u_begin = blockIdx.x * p.units_per_cta;
  const int u_end = min(u_begin + p.units_per_cta, p.total_units);
  if (u_begin >= u_end) return;
  const int kpr = p.kb_per_rb;

  // ---- which weight rows this warp streams for row block rb ------------------------------------------
  auto row0_of = [&](int rb) -> int {
    if (EPI == EPI_SWIGLU) {
      int j = rb * 64 + (warp & 3) * 16;
      if (j >= p.F) return -1;
      return (warp < 4) ? j : p.F + j;
    }
    int r = rb * RB_ROWS + warp * 16;
    return r < p.N ? r : -1;
  };

  // ---- weight loads of a batch of up to U consecutive units (same row block) -------------------------
  uint4 nxt[U][V4];
  auto load_batch = [&](int u, int nb) {
    int rb = u / kpr, kb = u - rb * kpr;
    int r0 = row0_of(rb);
#pragma unroll
    for (int i = 0; i < U; ++i) {
      if (i < nb && r0 >= 0 && (kb + i) * 32 + t * 8 < p.K) {
        const WT* base = static_cast<const WT*>(p.W) + (size_t)(r0 + g) * p.K + (size_t)(kb + i) * 32 + t * 8;
        if (IS_BF16) {
          nxt[i][0] = ldg_stream(base);
          nxt[i][1] = ldg_stream(base + (size_t)8 * p.K);
        } else {
          nxt[i][0] = ldg_stream(base);
          nxt[i][1] = ldg_stream(base + 4);
          nxt[i][2] = ldg_stream(base + (size_t)8 * p.K);
          nxt[i][3] = ldg_stream(base + (size_t)8 * p.K + 4);
        }
      } else {
#pragma unroll
        for (int v = 0; v < V4; ++v) nxt[i][v] = make_uint4(0, 0, 0, 0);
      }
    }
  };
  // a batch never crosses a row block or an activation chunk (chunks are counted from the segment start)
  auto batch_len = [&](int u, int seg_begin) -> int {
    int rb = u / kpr;
    int seg_end = min((rb + 1) * kpr, u_end);
    int chunk_end = seg_begin + ((u - seg_begin) / XCH + 1) * XCH;
    return min(U, min(seg_end, chunk_end) - u);
  };

  // ---- per-row 1/rms for the fused RMSNorm -----------------------------------------------------------
  auto row_of_col = [&](int c) -> int { return (p.xs_kind == XS_HID_NORM_RO) ? tab->ro_rows[c] : c; };

  int u = u_begin;
  int seg_begin = u_begin;
  int nb_next = batch_len(u, seg_begin);
  load_batch(u, nb_next);  // weights are in flight while the activations are prepared

  if (p.xs_kind != XS_BUF) {
    if (p.n_sq > 0) {
      if (tid < n_cols) {
        int row = row_of_col(tid);
        float ss = 0.f;
        for (int j = 0; j < p.n_sq; ++j) ss += p.sumsq[row * p.n_sq + j];
        s_rstd[tid] = 1.0f / sqrtf(ss / (float)p.H + p.eps);
      }
    } else {
      for (int c = warp; c < n_cols; c += GEMM_THREADS / 32) {
        const float4* xr = reinterpret_cast<const float4*>(p.hid + (size_t)tab->hid_idx[row_of_col(c)] * p.H);
        float ss = 0.f;
        for (int i = lane; i < p.H / 4; i += 32) {
          float4 v = xr[i];
          ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
        ss = warp_sum(ss);
        if (lane == 0) s_rstd[c] = 1.0f / sqrtf(ss / (float)p.H + p.eps);
      }
    }
  }
  // (visibility of s_rstd is ordered by the first __syncthreads below)

  // ---- stage one chunk of activations into shared memory in MMA-fragment order -----------------------
  auto stage_x = [&](int kb0, int nkb) {
    for (int idx = tid; idx < nkb * NTOK * 4; idx += GEMM_THREADS) {
      int tt = idx & 3, c = (idx >> 2) % NTOK, kbl = idx / (4 * NTOK);
      int k = (kb0 + kbl) * 32 + tt * 8;
      float v[8];
      if (c < n_cols && k < p.K) {
        const float* src;
        if (p.xs_kind == XS_BUF) src = p.xbuf + (size_t)c * p.x_ld + k;
        else src = p.hid + (size_t)tab->hid_idx[row_of_col(c)] * p.H + k;
        float4 a = *reinterpret_cast<const float4*>(src), b = *reinterpret_cast<const float4*>(src + 4);
        v[0] = a.x, v[1] = a.y, v[2] = a.z, v[3] = a.w, v[4] = b.x, v[5] = b.y, v[6] = b.z, v[7] = b.w;
        if (p.xs_kind != XS_BUF) {
          float rs = s_rstd[c];
          float4 ga = *reinterpret_cast<const float4*>(p.gain + k), gb = *reinterpret_cast<const float4*>(p.gain + k + 4);
          float gg[8] = {ga.x, ga.y, ga.z, ga.w, gb.x, gb.y, gb.z, gb.w};
#pragma unroll
          for (int i = 0; i < 8; ++i) v[i] = v[i] * rs * gg[i];
        }
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = 0.f;
      }
      if (IS_BF16) {
        unsigned short h[8], m[8], l[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) split3(v[i], h[i], m[i], l[i]);
        auto pack = [](const unsigned short* s) {
          return make_uint4(s[0] | ((unsigned)s[1] << 16), s[2] | ((unsigned)s[3] << 16), s[4] | ((unsigned)s[5] << 16),
                            s[6] | ((unsigned)s[7] << 16));
        };
        int o = (kbl * NTOK + c) * 4 + tt;
        xs[o] = pack(h);
        xs[XCH * NTOK * 4 + o] = pack(m);
        xs[2 * XCH * NTOK * 4 + o] = pack(l);
      } else {
        float4* xf = reinterpret_cast<float4*>(xs);
        int o = ((kbl * NTOK + c) * 32 + tt * 8) / 4;
        xf[o] = make_float4(v[0], v[1], v[2], v[3]);
        xf[o + 1] = make_float4(v[4], v[5], v[6], v[7]);
      }
    }
  };

  float acc[NG][4];
  float accf[IS_BF16 ? 1 : NG][IS_BF16 ? 1 : 8][2];
  auto zero_acc = [&]() {
#pragma unroll
    for (int n = 0; n < NG; ++n)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[n][i] = 0.f;
    if (!IS_BF16) {
#pragma unroll
      for (int n = 0; n < NG; ++n)
#pragma unroll
        for (int j = 0; j < 8; ++j) accf[n][j][0] = accf[n][j][1] = 0.f;
    }
  };
  zero_acc();

  // ---- epilogue over the finished tile of row block rb -----------------------------------------------
  auto epilogue = [&](int rb) {
    if (EPI == EPI_PLAIN || EPI == EPI_LOGITS) {
      int n0 = rb * RB_ROWS;
      for (int idx = tid; idx < n_cols * RB_ROWS; idx += GEMM_THREADS) {
        int c = idx / RB_ROWS, j = idx % RB_ROWS;
        if (n0 + j < p.N) {
          if (EPI == EPI_PLAIN) p.out[(size_t)c * p.out_ld + n0 + j] = tile[c * TILE_LD + j];
          else p.logits[(size_t)tab->logit_idx[tab->ro_rows[c]] * p.N + n0 + j] = tile[c * TILE_LD + j];
        }
      }
    } else if (EPI == EPI_RESID) {
      int n0 = rb * RB_ROWS;
      for (int c = warp; c < n_cols; c += GEMM_THREADS / 32) {
        float4* h = reinterpret_cast<float4*>(p.hid + (size_t)tab->hid_idx[c] * p.H + n0) + lane;
        float4 v = *h;
        const float* tr = tile + c * TILE_LD + lane * 4;
        v.x += tr[0], v.y += tr[1], v.z += tr[2], v.w += tr[3];
        *h = v;
        float ss = warp_sum(v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w);
        if (lane == 0) p.sumsq_out[c * p.n_sq_out + rb] = ss;
      }
    } else if (EPI == EPI_SWIGLU) {
      int j0 = rb * 64;
      for (int idx = tid; idx < n_cols * 64; idx += GEMM_THREADS) {
        int c = idx >> 6, jj = idx & 63;
        if (j0 + jj < p.F) {
          float gt = tile[c * TILE_LD + jj], up = tile[c * TILE_LD + 64 + jj];
          p.out[(size_t)c * p.out_ld + j0 + jj] = gt / (1.0f + expf(-gt)) * up;
        }
      }
    } else if (EPI == EPI_QKV) {
      const int d = p.head_dim, hd2 = d >> 1;
      const int Hq = p.n_q_heads * d, Hk = p.n_kv_heads * d;
      int n0 = rb * RB_ROWS;
      int region = n0 < Hq ? 0 : (n0 < Hq + Hk ? 1 : 2);
      int base = region == 0 ? 0 : (region == 1 ? Hq : Hq + Hk);
      for (int idx = tid; idx < n_cols * 64; idx += GEMM_THREADS) {
        int c = idx >> 6, pr = idx & 63;        // pair index inside the 128-row block
        int hh = pr / hd2, i = pr - hh * hd2;   // head inside the block, rotary pair
        float x1 = tile[c * TILE_LD + hh * d + i], x2 = tile[c * TILE_LD + hh * d + i + hd2];
        float y1 = x1, y2 = x2;
        if (region < 2) {
          float2 cs = p.rope[(size_t)tab->pos[c] * hd2 + i];
          y1 = x1 * cs.x - x2 * cs.y;
          y2 = x2 * cs.x + x1 * cs.y;
        }
        int head = (n0 - base) / d + hh;
        if (region == 0) {
          float* q = p.qbuf + (size_t)c * Hq + head * d + i;
          q[0] = y1;
          q[hd2] = y2;
        } else {
          __nv_bfloat16* dst = p.kv + (size_t)(tab->r[c] - 1) * p.kv_plane_stride + (size_t)(region - 1) * p.kv_sel_stride +
                               ((size_t)(tab->seq[c] * p.n_kv_heads + head) * p.slots + tab->kv_slot[c]) * d + i;
          dst[0] = __float2bfloat16_rn(y1);
          dst[hd2] = __float2bfloat16_rn(y2);
        }
      }
    }
  };

  // ---- a row block's share is complete: publish it, and reduce + finish if this CTA is the last one ---
  auto finish_segment = [&](int rb) {
    if (!IS_BF16) {  // fold the four k-lanes, then take the MMA accumulator layout
#pragma unroll
      for (int n = 0; n < NG; ++n)
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            float v = accf[n][j][h];
            v += __shfl_xor_sync(0xffffffffu, v, 1);
            v += __shfl_xor_sync(0xffffffffu, v, 2);
            if (j == 2 * t) acc[n][2 * h] = v;
            if (j == 2 * t + 1) acc[n][2 * h + 1] = v;
          }
    }
    int c_first = (rb * kpr) / p.units_per_cta;
    int c_last = ((rb + 1) * kpr - 1) / p.units_per_cta;
    int n_contrib = c_last - c_first + 1;
    int rl = warp * 16 + g;
    if (n_contrib == 1) {
#pragma unroll
      for (int n = 0; n < NG; ++n) {
        int c0 = n * 8 + 2 * t;
        tile[c0 * TILE_LD + rl] = acc[n][0];
        tile[(c0 + 1) * TILE_LD + rl] = acc[n][1];
        tile[c0 * TILE_LD + rl + 8] = acc[n][2];
        tile[(c0 + 1) * TILE_LD + rl + 8] = acc[n][3];
      }
      __syncthreads();
      epilogue(rb);
    } else {
      int ord = blockIdx.x - c_first;
      float* dst = p.partials + ((size_t)rb * p.max_contrib + ord) * (NTOK * RB_ROWS);
#pragma unroll
      for (int n = 0; n < NG; ++n) {
        int c0 = n * 8 + 2 * t;
        dst[c0 * RB_ROWS + rl] = acc[n][0];
        dst[(c0 + 1) * RB_ROWS + rl] = acc[n][1];
        dst[c0 * RB_ROWS + rl + 8] = acc[n][2];
        dst[(c0 + 1) * RB_ROWS + rl + 8] = acc[n][3];
      }
      __threadfence();
      __syncthreads();
      if (tid == 0) {
        int old = atomicAdd(p.counters + rb, 1);
        *s_flag = (old == n_contrib - 1);
      }
      __syncthreads();
      if (*s_flag) {
        __threadfence();
        const float4* src = reinterpret_cast<const float4*>(p.partials + (size_t)rb * p.max_contrib * (NTOK * RB_ROWS));
        for (int idx = tid; idx < NTOK * RB_ROWS / 4; idx += GEMM_THREADS) {
          float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
          for (int o = 0; o < n_contrib; ++o) {
            float4 v = __ldcg(src + (size_t)o * (NTOK * RB_ROWS / 4) + idx);
            s.x += v.x, s.y += v.y, s.z += v.z, s.w += v.w;
          }
          int c = idx / (RB_ROWS / 4), j = (idx % (RB_ROWS / 4)) * 4;
          float* tr = tile + c * TILE_LD + j;
          tr[0] = s.x, tr[1] = s.y, tr[2] = s.z, tr[3] = s.w;
        }
        if (tid == 0) p.counters[rb] = 0;
        __syncthreads();
        epilogue(rb);
      }
    }
    __syncthreads();  // tile and s_flag are reused by the next segment
    zero_acc();
  };

  // ---- main loop over this CTA's units ---------------------------------------------------------------
  uint4 cur[U][V4];
  bool need_stage = true;
  while (u < u_end) {
    const int nb = nb_next, ucur = u;
#pragma unroll
    for (int i = 0; i < U; ++i)
#pragma unroll
      for (int v = 0; v < V4; ++v) cur[i][v] = nxt[i][v];
    u += nb;
    const int rb = ucur / kpr;
    const bool seg_done = (u == u_end) || (u / kpr != rb);
    if (u < u_end) {
      int sb = seg_done ? u : seg_begin;
      nb_next = batch_len(u, sb);
      load_batch(u, nb_next);
    }
    const int kb = ucur - rb * kpr;
    const int kbl0 = (ucur - seg_begin) % XCH;
    if (need_stage || kbl0 == 0) {
      int seg_end = min((rb + 1) * kpr, u_end);
      __syncthreads();
      stage_x(kb, min(XCH, seg_end - ucur));
      __syncthreads();
      need_stage = false;
    }
    if (row0_of(rb) >= 0) {
#pragma unroll
      for (int i = 0; i < U; ++i) {
        if (i < nb) {
          const int kbl = kbl0 + i;
          if (IS_BF16) {
#pragma unroll
            for (int s = 0; s < 3; ++s) {
#pragma unroll
              for (int n = 0; n < NG; ++n) {
                uint4 b = xs[((s * XCH + kbl) * NTOK + n * 8 + g) * 4 + t];
                mma_bf16(acc[n], cur[i][0].x, cur[i][1].x, cur[i][0].y, cur[i][1].y, b.x, b.y);
                mma_bf16(acc[n], cur[i][0].z, cur[i][1].z, cur[i][0].w, cur[i][1].w, b.z, b.w);
              }
            }
          } else {
            const float4* xf = reinterpret_cast<const float4*>(xs);
            const float* wl = reinterpret_cast<const float*>(&cur[i][0]);  // row g: 8 floats
            const float* wh = reinterpret_cast<const float*>(&cur[i][2]);  // row g+8
#pragma unroll
            for (int n = 0; n < NG; ++n)
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                int o = ((kbl * NTOK + n * 8 + j) * 32 + t * 8) / 4;
                float4 xa = xf[o], xb = xf[o + 1];
                float xv[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                  accf[n][j][0] = fmaf(wl[e], xv[e], accf[n][j][0]);
                  accf[n][j][1] = fmaf(wh[e], xv[e], accf[n][j][1]);
                }
              }
          }
        }
      }
    }
    if (seg_done) {
      finish_segment(rb);
      seg_begin = u;
      need_stage = true;
    }
  }
}

}  // namespace ls

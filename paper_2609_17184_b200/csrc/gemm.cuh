// Weight-streaming skinny GEMM of the batched recurrence (Sec. 4.2 step 1): y[m][n] = sum_k x[m][k] W[n][k]
// for the few token rows m of one pass, with the epilogue (RMSNorm scale, rotary + KV write, residual add,
// SwiGLU, logits) fused in.
//
// Activations travel between kernels as three bf16 planes hi + mid + lo (an exact 24-bit decomposition of
// the fp32 value, made once by the producer), so products with bf16 weights are exact and a token's result
// does not depend on which other tokens share the pass.  RMSNorm is applied as gain (by the producer, before
// the split) and 1/rms (by the consumer's epilogue, from the per-row sums of squares) -- both linear.
//
// Mapping.  The weights are the 16-row A operand of mma.sync.m16n8k16 (bf16, fp32 accumulate); the token rows
// are the 8 B columns.  A CTA of 8 warps owns blocks of 128 output rows (one 16-row tile per warp) over a
// contiguous range of 32-wide k-blocks.  The work (row block x k-block) is linearised and cut into equal
// shares, one per CTA (stream-K); a row block shared by several CTAs is reduced in fixed order by whichever
// CTA arrives last, which then runs the epilogue.  No atomics touch data, so results are bit-reproducible.
// Weight tiles stream through a deep thread-private cp.async ring in shared memory; the first stages are
// issued before the kernel waits for its predecessor (programmatic dependent launch).
#pragma once
#include "common.cuh"

namespace ls {

enum { EPI_PLAIN = 0, EPI_QKV = 1, EPI_RESID = 2, EPI_SWIGLU = 3, EPI_LOGITS = 4 };

constexpr int GEMM_THREADS = 256;
constexpr int RB_ROWS = 128;   // output rows per row block
constexpr int TILE_LD = 132;   // padded leading dimension of the epilogue tile
constexpr int RING = 8;        // weight stages in flight per thread (8 KB per stage per CTA)

__host__ __device__ constexpr int xchunk_kblocks(int NG) { return NG >= 4 ? 2 : 8 / NG; }
__host__ __device__ constexpr int xbuf_uint4(int NG) { return 3 * xchunk_kblocks(NG) * 8 * NG * 4; }
__host__ __device__ constexpr int gemm_smem_bytes(int NG) {
  return RING * 2 * GEMM_THREADS * 16 + 2 * xbuf_uint4(NG) * 16 + 8 * NG * TILE_LD * 4 + 8 * NG * 4 + 16;
}

struct GemmParams {
  const void* W;
  int N, K;
  int n_rb, kb_per_rb, units_per_cta, total_units;
  // activations: bf16 planes [col][3][x_ld]
  const __nv_bfloat16* xplanes;
  int x_ld;
  const RowTable* tab;
  int m_fixed;            // tab == nullptr: number of rows of a stand-alone call
  int cols_from_readout;  // columns are the reading-out rows (lm_head)
  // fused RMSNorm: scale row c by 1/sqrt(sum_j sumsq[c*sq_stride + j] / H + eps); sumsq == nullptr: none
  const float* sumsq;
  int n_sq, sq_stride, H;
  float eps;
  // split-k scratch
  float* partials;        // [n_rb][max_contrib][8*NG][128]
  int max_contrib;
  int* counters;          // [n_rb], zero between launches
  // epilogue outputs
  float* out;             // PLAIN y [m][out_ld]
  int out_ld;
  __nv_bfloat16* out_planes;  // RESID: planes of x_new * gain_next (may be null); SWIGLU: planes of the activation
  int planes_ld;
  const float* gain_next;
  float* hid;             // RESID: residual stream [hid_idx][H]
  float* sumsq_out;       // RESID: [row][n_sq_out]
  int n_sq_out;
  float* qbuf;            // QKV: [row][n_q_heads * d]
  __nv_bfloat16* kv;      // QKV: this layer's KV pool [R][2][S][n_kv][slots][d]
  long long kv_plane_stride, kv_sel_stride;
  int slots, n_kv_heads, n_q_heads, head_dim;
  const float2* rope;     // [pos][d/2] (cos, sin)
  float* logits;          // LOGITS: [logit_idx][V]
  int F;                  // SWIGLU: ffn width
};

__device__ __forceinline__ void mma_bf16(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0,
                                         unsigned b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc, bool valid) {
  unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
  int n = valid ? 16 : 0;  // src-size 0: the 16 bytes are zero-filled and nothing is read
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(gsrc), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// ---- epilogue over the finished tile [col][TILE_LD] of row block rb ------------------------------------
template <int EPI>
__device__ __forceinline__ void gemm_epilogue(const GemmParams& p, const RowTable* tab, int rb, int n_cols, const float* tile,
                                              const float* s_rstd) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (EPI == EPI_PLAIN || EPI == EPI_LOGITS) {
    int n0 = rb * RB_ROWS;
    for (int idx = tid; idx < n_cols * RB_ROWS; idx += GEMM_THREADS) {
      int c = idx / RB_ROWS, j = idx % RB_ROWS;
      if (n0 + j < p.N) {
        float v = tile[c * TILE_LD + j] * s_rstd[c];
        if (EPI == EPI_PLAIN) p.out[(size_t)c * p.out_ld + n0 + j] = v;
        else p.logits[(size_t)tab->logit_idx[tab->ro_rows[c]] * p.N + n0 + j] = v;
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
      if (p.out_planes) {  // the next norm's gain, then the three-way split, once for every consumer
        float4 gn = *reinterpret_cast<const float4*>(p.gain_next + n0 + lane * 4);
        float xv[4] = {v.x * gn.x, v.y * gn.y, v.z * gn.z, v.w * gn.w};
        unsigned short hh[4], mm[4], ll[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) split3(xv[i], hh[i], mm[i], ll[i]);
        __nv_bfloat16* dst = p.out_planes + (size_t)c * 3 * p.planes_ld + n0 + lane * 4;
        *reinterpret_cast<uint2*>(dst) = make_uint2(hh[0] | ((unsigned)hh[1] << 16), hh[2] | ((unsigned)hh[3] << 16));
        *reinterpret_cast<uint2*>(dst + p.planes_ld) = make_uint2(mm[0] | ((unsigned)mm[1] << 16), mm[2] | ((unsigned)mm[3] << 16));
        *reinterpret_cast<uint2*>(dst + 2 * p.planes_ld) = make_uint2(ll[0] | ((unsigned)ll[1] << 16), ll[2] | ((unsigned)ll[3] << 16));
      }
    }
  } else if (EPI == EPI_SWIGLU) {
    int j0 = rb * 64;
    for (int idx = tid; idx < n_cols * 64; idx += GEMM_THREADS) {
      int c = idx >> 6, jj = idx & 63;
      if (j0 + jj < p.F) {
        float gt = tile[c * TILE_LD + jj] * s_rstd[c], up = tile[c * TILE_LD + 64 + jj] * s_rstd[c];
        store_split(p.out_planes + (size_t)c * 3 * p.planes_ld, p.planes_ld, j0 + jj, gt / (1.0f + expf(-gt)) * up);
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
      float x1 = tile[c * TILE_LD + hh * d + i] * s_rstd[c], x2 = tile[c * TILE_LD + hh * d + i + hd2] * s_rstd[c];
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
}

// ---- a row block's share is complete: publish it, and reduce + finish if this CTA is the last one -------
// acc: this thread's MMA accumulator fragments (rows warp*16+g / +8, columns n*8+2t / +1)
template <int NG, int EPI>
__device__ __forceinline__ void gemm_finish_segment(const GemmParams& p, const RowTable* tab, int rb, int n_cols,
                                                    const float (&acc)[NG][4], float* tile, const float* s_rstd, int* s_flag) {
  constexpr int NTOK = 8 * NG;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int kpr = p.kb_per_rb;
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
    gemm_epilogue<EPI>(p, tab, rb, n_cols, tile, s_rstd);
  } else {
    int ord = blockIdx.x - c_first;
    float* dst = p.partials + ((size_t)rb * p.max_contrib + ord) * (NTOK * RB_ROWS);
#pragma unroll
    for (int n = 0; n < NG; ++n) {
      int c0 = n * 8 + 2 * t;
      if (c0 < n_cols) {  // columns beyond the live rows are never read back
        __stcg(dst + c0 * RB_ROWS + rl, acc[n][0]);
        __stcg(dst + c0 * RB_ROWS + rl + 8, acc[n][2]);
        if (c0 + 1 < n_cols) {
          __stcg(dst + (c0 + 1) * RB_ROWS + rl, acc[n][1]);
          __stcg(dst + (c0 + 1) * RB_ROWS + rl + 8, acc[n][3]);
        }
      }
    }
    __syncthreads();
    if (tid == 0) {
      __threadfence();  // the CTA's partials (ordered before this by the barrier) are visible device-wide
      int old = atomicAdd(p.counters + rb, 1);
      *s_flag = (old == n_contrib - 1);
      __threadfence();
    }
    __syncthreads();
    if (*s_flag) {
      const float4* src = reinterpret_cast<const float4*>(p.partials + (size_t)rb * p.max_contrib * (NTOK * RB_ROWS));
      for (int idx = tid; idx < n_cols * (RB_ROWS / 4); idx += GEMM_THREADS) {
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
      gemm_epilogue<EPI>(p, tab, rb, n_cols, tile, s_rstd);
    }
  }
  __syncthreads();  // tile and s_flag are reused by the next segment
}

// first weight row this warp streams for row block rb (-1: outside the matrix)
template <int EPI>
__device__ __forceinline__ int gemm_row0(const GemmParams& p, int rb, int warp) {
  if (EPI == EPI_SWIGLU) {  // 64 gate rows and the 64 matching up rows
    int j = rb * 64 + (warp & 3) * 16;
    if (j >= p.F) return -1;
    return (warp < 4) ? j : p.F + j;
  }
  int r = rb * RB_ROWS + warp * 16;
  return r < p.N ? r : -1;
}

__device__ __forceinline__ void gemm_rstd(const GemmParams& p, int n_cols, float* s_rstd) {
  const int tid = threadIdx.x;
  if (tid < n_cols) {
    float r = 1.0f;
    if (p.sumsq) {
      float ss = 0.f;
      for (int j = 0; j < p.n_sq; ++j) ss += p.sumsq[tid * p.sq_stride + j];
      r = 1.0f / sqrtf(ss / (float)p.H + p.eps);
    }
    s_rstd[tid] = r;
  }
}

// ======================================= bf16 weights: tensor cores ========================================
template <int NG, int EPI>
__global__ void __launch_bounds__(GEMM_THREADS) gemm_bf16_kernel(const __grid_constant__ GemmParams p) {
  constexpr int NTOK = 8 * NG;
  constexpr int XCH = xchunk_kblocks(NG);
  constexpr int XBUF = xbuf_uint4(NG);
  constexpr int PIECES = 3 * XCH * NTOK * 4;
  constexpr int PPT = (PIECES + GEMM_THREADS - 1) / GEMM_THREADS;
  constexpr int NCH = 3;  // independent accumulator chains, one per split term (the same for every NG:
                          // a row's bits must not depend on how many rows share the pass)

  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4* ring = reinterpret_cast<uint4*>(smem_raw);            // [RING][2][256], slot of thread tid only
  uint4* xbuf = ring + RING * 2 * GEMM_THREADS;                // [2][3][XCH][NTOK][4]
  float* tile = reinterpret_cast<float*>(xbuf + 2 * XBUF);     // [NTOK][TILE_LD]
  float* s_rstd = tile + NTOK * TILE_LD;
  int* s_flag = reinterpret_cast<int*>(s_rstd + NTOK);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int kpr = p.kb_per_rb;
  const int u_begin = blockIdx.x * p.units_per_cta;
  const int u_end = min(u_begin + p.units_per_cta, p.total_units);
  const int n_units = u_end - u_begin;  // >= 1 by construction of the grid

  // ---- weight ring: issue side ---------------------------------------------------------------------------
  int i_rb = u_begin / kpr, i_kb = u_begin - i_rb * kpr, i_row0 = gemm_row0<EPI>(p, i_rb, warp), i_cnt = 0;
  auto issue_unit = [&]() {
    if (i_cnt < n_units) {
      const int k = i_kb * 32 + t * 8;
      const bool valid = i_row0 >= 0 && k < p.K;
      const __nv_bfloat16* src = static_cast<const __nv_bfloat16*>(p.W);
      if (valid) src += (size_t)(i_row0 + g) * p.K + k;
      uint4* slot = ring + (size_t)(i_cnt % RING) * 2 * GEMM_THREADS + tid;
      cp_async16(slot, src, valid);
      cp_async16(slot + GEMM_THREADS, valid ? src + (size_t)8 * p.K : src, valid);
      ++i_cnt;
      if (++i_kb == kpr) i_kb = 0, ++i_rb, i_row0 = gemm_row0<EPI>(p, i_rb, warp);
    }
    cp_async_commit();
  };
#pragma unroll
  for (int s = 0; s < RING - 1; ++s) issue_unit();

  // the weights above are constants; everything below reads what earlier kernels of the pass produced
  pdl_launch_dependents();
  pdl_wait();

  const RowTable* tab = p.tab;
  int n_cols = tab ? (p.cols_from_readout ? tab->n_readout : tab->n_rows) : p.m_fixed;
  if (n_cols > NTOK) n_cols = NTOK;
  if (n_cols <= 0) {
    cp_async_wait<0>();
    return;
  }
  gemm_rstd(p, n_cols, s_rstd);

  // ---- activation chunks: gathered into registers one chunk ahead, then stored in MMA-fragment order -----
  uint4 xr[PPT];
  auto x_fetch = [&](int kb0, int nkb) {
#pragma unroll
    for (int i = 0; i < PPT; ++i) {
      int idx = tid + i * GEMM_THREADS;
      xr[i] = make_uint4(0, 0, 0, 0);
      if (idx < 3 * nkb * NTOK * 4) {
        int tt = idx & 3, c = (idx >> 2) % NTOK, r = idx / (4 * NTOK), kbl = r % nkb, s = r / nkb;
        int k = (kb0 + kbl) * 32 + tt * 8;
        if (c < n_cols && k < p.K)
          xr[i] = *reinterpret_cast<const uint4*>(p.xplanes + ((size_t)c * 3 + s) * p.x_ld + k);
      }
    }
  };
  auto x_store = [&](int nkb, int buf) {
#pragma unroll
    for (int i = 0; i < PPT; ++i) {
      int idx = tid + i * GEMM_THREADS;
      if (idx < 3 * nkb * NTOK * 4) {
        int tt = idx & 3, c = (idx >> 2) % NTOK, r = idx / (4 * NTOK), kbl = r % nkb, s = r / nkb;
        xbuf[buf * XBUF + ((s * XCH + kbl) * NTOK + c) * 4 + tt] = xr[i];
      }
    }
  };

  float acc[NCH][NG][4];
  auto zero_acc = [&]() {
#pragma unroll
    for (int h = 0; h < NCH; ++h)
#pragma unroll
      for (int n = 0; n < NG; ++n)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[h][n][i] = 0.f;
  };
  zero_acc();

  // ---- consume side: segments (one row block each) of chunks of units ------------------------------------
  int c_rb = u_begin / kpr, c_kb = u_begin - c_rb * kpr;
  int j = 0, xb = 0;
  {
    int seg_len = min(kpr - c_kb, n_units);
    x_fetch(c_kb, min(XCH, seg_len));
  }
  while (j < n_units) {
    const int seg_len = min(kpr - c_kb, n_units - j);
    const bool warp_valid = gemm_row0<EPI>(p, c_rb, warp) >= 0;
    for (int ck = 0; ck < seg_len; ck += XCH) {
      const int nkb = min(XCH, seg_len - ck);
      x_store(nkb, xb);
      __syncthreads();
      {  // fetch the next chunk (of this segment, or the first of the next) while this one is consumed
        int nk0 = ck + XCH;
        if (nk0 < seg_len) x_fetch(c_kb + nk0, min(XCH, seg_len - nk0));
        else if (j + (seg_len - ck) < n_units) x_fetch(0, min(XCH, min(kpr, n_units - j - (seg_len - ck))));
      }
      const uint4* xs = xbuf + xb * XBUF;
      for (int kbl = 0; kbl < nkb; ++kbl, ++j) {
        issue_unit();
        cp_async_wait<RING - 1>();
        if (warp_valid) {
          const uint4* slot = ring + (size_t)(j % RING) * 2 * GEMM_THREADS + tid;
          const uint4 a_lo = slot[0], a_hi = slot[GEMM_THREADS];
#pragma unroll
          for (int s = 0; s < 3; ++s) {
#pragma unroll
            for (int n = 0; n < NG; ++n) {
              const uint4 b = xs[((s * XCH + kbl) * NTOK + n * 8 + g) * 4 + t];
              float(&c)[4] = acc[NCH == 3 ? s : 0][n];
              mma_bf16(c, a_lo.x, a_hi.x, a_lo.y, a_hi.y, b.x, b.y);
              mma_bf16(c, a_lo.z, a_hi.z, a_lo.w, a_hi.w, b.z, b.w);
            }
          }
        }
      }
      xb ^= 1;
    }
    // fold the chains in fixed order: hi + (mid + lo)
    float tot[NG][4];
#pragma unroll
    for (int n = 0; n < NG; ++n)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if constexpr (NCH == 3) tot[n][i] = acc[0][n][i] + (acc[1][n][i] + acc[2][n][i]);
        else tot[n][i] = acc[0][n][i];
      }
    gemm_finish_segment<NG, EPI>(p, tab, c_rb, n_cols, tot, tile, s_rstd, s_flag);
    zero_acc();
    c_kb += seg_len;
    if (c_kb == kpr) c_kb = 0, ++c_rb;
  }
  cp_async_wait<0>();
}

// ======================================= fp32 weights: CUDA cores ==========================================
// Same decomposition and epilogues; the activation is rebuilt exactly from its three planes.  Used by the
// small fp32 configuration only, so it is written for clarity, not speed.
template <int NG, int EPI>
__global__ void __launch_bounds__(GEMM_THREADS) gemm_f32_kernel(const __grid_constant__ GemmParams p) {
  constexpr int NTOK = 8 * NG;
  constexpr int XCH = 4;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* xf = reinterpret_cast<float*>(smem_raw);              // [XCH][NTOK][32]
  float* tile = xf + XCH * NTOK * 32;                          // [NTOK][TILE_LD]
  float* s_rstd = tile + NTOK * TILE_LD;
  int* s_flag = reinterpret_cast<int*>(s_rstd + NTOK);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int kpr = p.kb_per_rb;
  const int u_begin = blockIdx.x * p.units_per_cta;
  const int u_end = min(u_begin + p.units_per_cta, p.total_units);
  const int n_units = u_end - u_begin;
  pdl_launch_dependents();
  pdl_wait();
  const RowTable* tab = p.tab;
  int n_cols = tab ? (p.cols_from_readout ? tab->n_readout : tab->n_rows) : p.m_fixed;
  if (n_cols > NTOK) n_cols = NTOK;
  if (n_cols <= 0) return;
  gemm_rstd(p, n_cols, s_rstd);

  int c_rb = u_begin / kpr, c_kb = u_begin - c_rb * kpr, j = 0;
  while (j < n_units) {
    const int seg_len = min(kpr - c_kb, n_units - j);
    const int row0 = gemm_row0<EPI>(p, c_rb, warp);
    float accf[NG][8][2];
#pragma unroll
    for (int n = 0; n < NG; ++n)
#pragma unroll
      for (int c = 0; c < 8; ++c) accf[n][c][0] = accf[n][c][1] = 0.f;
    for (int ck = 0; ck < seg_len; ck += XCH) {
      const int nkb = min(XCH, seg_len - ck);
      __syncthreads();
      for (int idx = tid; idx < nkb * NTOK * 32; idx += GEMM_THREADS) {
        int e = idx & 31, c = (idx >> 5) % NTOK, kbl = idx / (32 * NTOK);
        int k = (c_kb + ck + kbl) * 32 + e;
        float v = 0.f;
        if (c < n_cols && k < p.K) {
          const __nv_bfloat16* pl = p.xplanes + (size_t)c * 3 * p.x_ld + k;
          v = (__bfloat162float(pl[0]) + __bfloat162float(pl[p.x_ld])) + __bfloat162float(pl[2 * p.x_ld]);
        }
        xf[idx] = v;
      }
      __syncthreads();
      if (row0 >= 0) {
        for (int kbl = 0; kbl < nkb; ++kbl) {
          const int k = (c_kb + ck + kbl) * 32 + t * 8;
          if (k < p.K) {
            const float* wl = static_cast<const float*>(p.W) + (size_t)(row0 + g) * p.K + k;
            const float* wh = wl + (size_t)8 * p.K;
            float4 l0 = *reinterpret_cast<const float4*>(wl), l1 = *reinterpret_cast<const float4*>(wl + 4);
            float4 h0 = *reinterpret_cast<const float4*>(wh), h1 = *reinterpret_cast<const float4*>(wh + 4);
            const float wlo[8] = {l0.x, l0.y, l0.z, l0.w, l1.x, l1.y, l1.z, l1.w};
            const float whi[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
#pragma unroll
            for (int n = 0; n < NG; ++n)
#pragma unroll
              for (int c = 0; c < 8; ++c) {
                const float* xv = xf + (kbl * NTOK + n * 8 + c) * 32 + t * 8;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                  accf[n][c][0] = fmaf(wlo[e], xv[e], accf[n][c][0]);
                  accf[n][c][1] = fmaf(whi[e], xv[e], accf[n][c][1]);
                }
              }
          }
        }
      }
    }
    j += seg_len;
    // fold the four k-lanes, then take the MMA accumulator layout the shared epilogue expects
    float tot[NG][4];
#pragma unroll
    for (int n = 0; n < NG; ++n)
#pragma unroll
      for (int c = 0; c < 8; ++c)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          float v = accf[n][c][h];
          v += __shfl_xor_sync(0xffffffffu, v, 1);
          v += __shfl_xor_sync(0xffffffffu, v, 2);
          if (c == 2 * t) tot[n][2 * h] = v;
          if (c == 2 * t + 1) tot[n][2 * h + 1] = v;
        }
    gemm_finish_segment<NG, EPI>(p, tab, c_rb, n_cols, tot, tile, s_rstd, s_flag);
    c_kb += seg_len;
    if (c_kb == kpr) c_kb = 0, ++c_rb;
  }
}
__host__ __device__ constexpr int gemm_f32_smem_bytes(int NG) { return 4 * 8 * NG * 32 * 4 + 8 * NG * TILE_LD * 4 + 8 * NG * 4 + 16; }

// ---- fp32 rows -> three bf16 planes, optionally through RMSNorm's gain, with the row's sum of squares -----
struct PrepParams {
  const RowTable* tab;      // null: rows 0..m_fixed-1 of `x`
  int m_fixed;
  const float* x;           // stand-alone source [m][K]
  const float* hid;         // row source [hid_idx][K]
  int K;
  const float* gain;        // may be null
  __nv_bfloat16* planes;    // [col][3][K]
  float* sumsq;             // [col * sq_stride] full sum of squares (may be null)
  int sq_stride;
  int readout_only;         // columns are the reading-out rows
};

__global__ void __launch_bounds__(256) prep_planes_kernel(const __grid_constant__ PrepParams p) {
  __shared__ float s_part[8];
  pdl_launch_dependents();
  pdl_wait();
  const int c = blockIdx.x;
  int n = p.tab ? (p.readout_only ? p.tab->n_readout : p.tab->n_rows) : p.m_fixed;
  if (c >= n) return;
  const float* src;
  if (p.tab) {
    int row = p.readout_only ? p.tab->ro_rows[c] : c;
    src = p.hid + (size_t)p.tab->hid_idx[row] * p.K;
  } else {
    src = p.x + (size_t)c * p.K;
  }
  __nv_bfloat16* dst = p.planes + (size_t)c * 3 * p.K;
  float ss = 0.f;
  for (int k = threadIdx.x; k < p.K; k += blockDim.x) {
    float v = src[k];
    ss += v * v;
    store_split(dst, p.K, k, p.gain ? v * p.gain[k] : v);
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0 && p.sumsq) {
    float tsum = 0.f;
    for (int w = 0; w < 8; ++w) tsum += s_part[w];
    p.sumsq[c * p.sq_stride] = tsum;
  }
}

}  // namespace ls

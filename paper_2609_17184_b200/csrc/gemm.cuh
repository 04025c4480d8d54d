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
// are the 8 B columns.  A thread-block cluster owns a block of 128 output rows; its CTAs split K into
// contiguous ranges (one 16-row tile per warp, 32-wide k-blocks).  Each CTA leaves its partial tile in its
// own shared memory; after a cluster barrier the CTAs sum the partials over distributed shared memory in rank
// order -- each CTA finishing a subset of the token columns -- and run the epilogue.  No global scratch, no
// atomics: results are bit-reproducible.  Weight tiles stream through a deep thread-private cp.async ring
// whose first stages are issued before the kernel waits for its predecessor (programmatic dependent launch).
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"

namespace ls {
namespace cg = cooperative_groups;

enum { EPI_PLAIN = 0, EPI_QKV = 1, EPI_RESID = 2, EPI_SWIGLU = 3, EPI_LOGITS = 4 };

constexpr int GEMM_THREADS = 256;
constexpr int RB_ROWS = 128;   // output rows per row block
constexpr int TILE_LD = 132;   // padded leading dimension of the partial tile
// shape of a GEMM CTA (overridable at build time for tuning): ring depth, staged k-blocks, register cap
#ifndef LS_RING
#define LS_RING 8
#endif
#ifndef LS_XCH
#define LS_XCH 24
#endif
#ifndef LS_MAXREG
#define LS_MAXREG 96
#endif
constexpr int RING = LS_RING;  // weight stages per thread (8 KB per stage per CTA), RING - 1 of them in flight
constexpr int MAX_XCH_BLOCKS = LS_XCH;  // k-blocks of activations one CTA keeps staged when NG = 1
// per-column copies of the row-table fields the epilogues need ([field][column] in shared memory)
enum { CT_POS = 0, CT_R = 1, CT_SEQ = 2, CT_SLOT = 3, CT_HID = 4, CT_LOGIT = 5, CT_XROW = 6, CT_FIELDS = 7 };

// k-blocks of activations staged at a time.  The wide kernels (NG >= 4: prefill, batches) need too many registers for
// two CTAs per SM anyway, so they take a larger staging buffer and restage less often.
__host__ __device__ constexpr int xchunk_kblocks(int NG) { return NG >= 8 ? 8 : NG == 4 ? 12 : MAX_XCH_BLOCKS / NG; }
__host__ __device__ constexpr int xbuf_uint4(int NG) { return 3 * xchunk_kblocks(NG) * 8 * NG * 4; }
// partial columns received from the cluster's ranks: [rank][owned column][128 rows]
__host__ __device__ constexpr int recv_floats(int NG) { return (8 * NG + 7) * RB_ROWS; }
__host__ __device__ constexpr int gemm_smem_bytes(int NG) {
  return RING * 2 * GEMM_THREADS * 16 + xbuf_uint4(NG) * 16 + recv_floats(NG) * 4 + 2 * RB_ROWS * 4 + 8 * NG * 4 * (1 + CT_FIELDS) + 64;
}

struct GemmParams {
  const void* W;
  int N, K;
  int n_rb, kb_per_rb;    // row blocks; 32-wide k-blocks per row
  int cluster_size, n_clusters;
  // activations: bf16 planes [col][3][x_ld]
  const __nv_bfloat16* xplanes;
  int x_ld;
  const RowTable* tab;
  int m_fixed;            // tab == nullptr: number of rows of a stand-alone call
  int col0;               // first column (row of the pass, or reading-out row) this launch carries: passes wider than one
                          // launch's columns run as several launches; the per-column buffers below are offset by the host
  int cols_from_readout;  // columns are the reading-out rows (lm_head)
  // fused RMSNorm: scale column c by 1/sqrt(sum_j sumsq[c*sq_stride + j] / H + eps); sumsq == nullptr: none
  const float* sumsq;
  int n_sq, sq_stride, H;
  float eps;
  // epilogue outputs
  float* out;             // PLAIN y [m][out_ld]
  int out_ld;
  __nv_bfloat16* out_planes;  // RESID: planes of x_new * gain_next (may be null); SWIGLU: planes of the activation
  int planes_ld;
  const float* gain_next;
  float* hid;             // RESID: residual stream [hid_idx][H]
  int no_resid;           // RESID: the output REPLACES the stream (the adapter of a Raven-style model: H = W_a [H; e])
  int recv_ranks;         // contributions per column in the receive buffer (0: one per rank of the cluster)
  float* sumsq_out;       // RESID: [row][n_sq_out]
  int n_sq_out;
  float* qbuf;            // QKV: [row][n_q_heads * d]
  __nv_bfloat16* kv;      // QKV: this layer's KV pool [R][2][S][n_kv][slots][d]
  long long kv_plane_stride, kv_sel_stride;
  int slots, n_kv_heads, n_q_heads, head_dim;
  const float2* rope;     // [pos][d/2] (cos, sin)
  float* logits;          // LOGITS: [logit_idx][V]
  float2* argpart;        // LOGITS: [column][row block] (largest logit of the block, its vocabulary index as int bits)
  int F;                  // SWIGLU: ffn width
  int perm, perm_a, perm_d;  // order of the row tiles in the packed weights (see packed_tile)
  volatile int* err;      // host-visible error flag (a bounded wait in a tcgen05 kernel ran out)
  long long* dbg;         // tuning aid: cycle stamps of CTA 0 / thread 0 (null in production)
  unsigned long long* tl; // tuning aid: kernel timeline (null in production)
  int tl_id;
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

// Row tile order of the packed weights.  perm 0: natural.  perm 1 (gate/up, a = ffn width): gate tile u and up
// tile u are adjacent (2u, 2u + 1).  perm 2 (QKV, a = tiles per rotary half, d = head size): the tile holding
// rows i of a head and the tile holding their rotary partners i + d/2 are adjacent.
__host__ __device__ __forceinline__ int packed_tile(int perm, int a, int d, int row0) {
  const int tt = row0 >> 4;
  if (perm == 1) return row0 < a ? 2 * tt : 2 * ((row0 - a) >> 4) + 1;
  if (perm == 2) {  // a is 2 or 4 (head size 64 or 128): shifts, no divisions
    const int la = a == 4 ? 2 : 1, h = tt >> (la + 1), w = tt & (2 * a - 1);
    return 2 * (h * a + (w & (a - 1))) + (w >> la);
  }
  return tt;
}
// first row of packed tile pt in the source matrix (inverse of packed_tile)
__host__ __device__ __forceinline__ int packed_tile_row0(int perm, int a, int d, int pt) {
  if (perm == 1) return (pt & 1) * a + (pt >> 1) * 16;
  if (perm == 2) {
    const int grp = pt >> 1, h = grp / a, j = grp - h * a;
    return h * d + (j + (pt & 1) * a) * 16;
  }
  return pt * 16;
}

// first weight row this warp streams for row block rb (-1: outside the matrix)
template <int EPI, int KH = 1>
__device__ __forceinline__ int gemm_row0(const GemmParams& p, int rb, int warp) {
  if (EPI == EPI_SWIGLU) {  // 64 gate rows and the 64 matching up rows
    int j = rb * 64 + (warp & 3) * 16;
    if (j >= p.F) return -1;
    return (warp < 4) ? j : p.F + j;
  }
  // KH = 2: blocks of 64 rows; warps 0-3 and 4-7 take the same four row tiles and alternate k-blocks
  int r = rb * (RB_ROWS / KH) + (warp % (8 / KH)) * 16;
  return r < p.N ? r : -1;
}

// k-blocks [lo, hi) of cluster rank `rank`
__device__ __forceinline__ void gemm_krange(int kpr, int cs, int rank, int& lo, int& hi) {
  int q = kpr / cs, r = kpr % cs;
  lo = rank * q + min(rank, r);
  hi = lo + q + (rank < r ? 1 : 0);
}

// ---- every rank has pushed its partial columns into the owners' receive buffers: sum them in rank order and
// finish this CTA's columns.  Column c of row block rb is finished by rank (c mod cluster size); threads 0..127
// take one column, threads 128..255 the next one of this rank, one output row each.
template <int EPI, int KH = 1>
__device__ __forceinline__ void gemm_reduce_epilogue(const GemmParams& p, const int* ct, int ntok, int rb, int n_cols, const float* recv,
                                                     int own_max, float* colbuf, const float* s_rstd, int rank, float pre_h = 0.f,
                                                     float pre_g = 1.f, float2 pre_rope = make_float2(1.f, 0.f), bool pre_valid = false) {
  constexpr int RBW = RB_ROWS / KH;  // rows of this row block
  const int tid = threadIdx.x, half = tid >> 7, j = tid & 127, lane = tid & 31, hw = (tid >> 5) & 3;
  const int cs = p.cluster_size, vcs = p.recv_ranks ? p.recv_ranks : cs * KH;
  __shared__ float s_ss[2][4];
  for (int base = rank; base < n_cols; base += 2 * cs) {
    const int c = base + cs * half;
    const bool live = c < n_cols && j < RBW;
    // global operands of the epilogue are requested first so that their latency overlaps the summation
    float h_old = 0.f, g_next = 1.f;
    float* h_ptr = nullptr;
    if (EPI == EPI_RESID && live) {
      h_ptr = p.hid + (size_t)ct[CT_HID * ntok + c] * p.H + rb * RBW + j;
      if (pre_valid && base == rank) {  // requested before the cluster barrier
        h_old = pre_h, g_next = pre_g;
      } else {
        h_old = *h_ptr;
        if (p.out_planes) g_next = p.gain_next[rb * RBW + j];
      }
      if (p.no_resid) h_old = 0.f;
    }
    float v = 0.f;
    if (live) {
      const float* src = recv + (size_t)(c / cs) * RBW + j;
      v = src[0];
      for (int rk = 1; rk < vcs; ++rk) v += src[(size_t)rk * own_max * RBW];  // rank order, the same for every launch
      v *= s_rstd[c];
    }
    if (EPI == EPI_PLAIN || EPI == EPI_LOGITS) {
      const int n = rb * RB_ROWS + j;
      if (live && n < p.N) {
        if (EPI == EPI_PLAIN) p.out[(size_t)c * p.out_ld + n] = v;
        else p.logits[(size_t)ct[CT_LOGIT * ntok + c] * p.N + n] = v;
      }
      if (EPI == EPI_LOGITS) {  // the block's largest logit (ties: lowest index), so that greedy selection reads
                                // one partial per row block instead of the whole row
        __shared__ float s_av[2][4];
        __shared__ int s_ai[2][4];
        float bv = (live && n < p.N) ? v : -INFINITY;
        int bi = n;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
          const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
          if (ov > bv || (ov == bv && oi < bi)) bv = ov, bi = oi;
        }
        if (lane == 0) s_av[half][hw] = bv, s_ai[half][hw] = bi;
        __syncthreads();
        if (c < n_cols && j == 0) {
          for (int w = 1; w < 4; ++w)
            if (s_av[half][w] > bv || (s_av[half][w] == bv && s_ai[half][w] < bi)) bv = s_av[half][w], bi = s_ai[half][w];
          p.argpart[(size_t)c * p.n_rb + rb] = make_float2(bv, __int_as_float(bi));
        }
        __syncthreads();
      }
    } else if (EPI == EPI_RESID) {
      const int n = rb * RBW + j;
      float xn = 0.f;
      if (live) {
        xn = h_old + v;
        *h_ptr = xn;
        if (p.out_planes) store_split(p.out_planes + (size_t)c * 3 * p.planes_ld, p.planes_ld, n, xn * g_next);
      }
      float ss = warp_sum(xn * xn);
      if (lane == 0) s_ss[half][hw] = ss;
      __syncthreads();
      if (c < n_cols && j == 0) p.sumsq_out[c * p.n_sq_out + rb] = (s_ss[half][0] + s_ss[half][1]) + (s_ss[half][2] + s_ss[half][3]);
      __syncthreads();
    } else {
      colbuf[half * RB_ROWS + j] = v;
      __syncthreads();
      if (live && j < 64) {
        const float* col = colbuf + half * RB_ROWS;
        if (EPI == EPI_SWIGLU) {
          const int f = rb * 64 + j;
          if (f < p.F) {
            float gt = col[j], up = col[64 + j];
            store_split(p.out_planes + (size_t)c * 3 * p.planes_ld, p.planes_ld, f, gt / (1.0f + expf(-gt)) * up);
          }
        } else {  // EPI_QKV: rotary pair j of the 128-row block, then q to the query buffer, k/v to the cache
          const int d = p.head_dim, hd2 = d >> 1;
          const int Hq = p.n_q_heads * d, Hk = p.n_kv_heads * d;
          const int n0 = rb * RB_ROWS;
          const int region = n0 < Hq ? 0 : (n0 < Hq + Hk ? 1 : 2);
          const int rbase = region == 0 ? 0 : (region == 1 ? Hq : Hq + Hk);
          const int hh = j / hd2, i = j - hh * hd2;
          const float x1 = col[hh * d + i], x2 = col[hh * d + i + hd2];
          float y1 = x1, y2 = x2;
          if (region < 2) {
            const float2 csn = (pre_valid && base == rank) ? pre_rope : p.rope[(size_t)ct[CT_POS * ntok + c] * hd2 + i];
            y1 = x1 * csn.x - x2 * csn.y;
            y2 = x2 * csn.x + x1 * csn.y;
          }
          const int head = (n0 - rbase) / d + hh;
          if (region == 0) {
            float* q = p.qbuf + (size_t)c * Hq + head * d + i;
            q[0] = y1;
            q[hd2] = y2;
          } else {
            __nv_bfloat16* dst = p.kv + (size_t)(ct[CT_R * ntok + c] - 1) * p.kv_plane_stride + (size_t)(region - 1) * p.kv_sel_stride +
                                 ((size_t)(ct[CT_SEQ * ntok + c] * p.n_kv_heads + head) * p.slots + ct[CT_SLOT * ntok + c]) * d + i;
            dst[0] = __float2bfloat16_rn(y1);
            dst[hd2] = __float2bfloat16_rn(y2);
          }
        }
      }
      __syncthreads();
    }
  }
}

// 1/rms of every live column: warp w sums the partial sums of squares of columns w, w + 8, ... (one partial per lane,
// butterfly sum: the same order in every launch)
__device__ __forceinline__ void gemm_rstd(const GemmParams& p, int n_cols, float* s_rstd, const int* ct, int ntok) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int c = warp; c < n_cols; c += GEMM_THREADS / 32) {
    const int xr = p.cols_from_readout ? ct[CT_XROW * ntok + c] : c;  // the lm_head's columns are the reading-out rows
    float ss = 0.f;
    if (p.sumsq)
      for (int j = lane; j < p.n_sq; j += 32) ss += p.sumsq[xr * p.sq_stride + j];
    ss = warp_sum(ss);
    if (lane == 0) s_rstd[c] = p.sumsq ? 1.0f / sqrtf(ss / (float)p.H + p.eps) : 1.0f;
  }
}

// The row table of a pass is final before the pass starts, so its fields can be copied ahead of the predecessor.
__device__ __forceinline__ void gemm_load_cols(const GemmParams& p, int n_cols, int ntok, int* ct) {
  const int c = threadIdx.x;
  const RowTable* tab = p.tab;
  if (tab && c < n_cols) {
    const int row = p.cols_from_readout ? tab->ro_rows[p.col0 + c] : p.col0 + c;
    ct[CT_POS * ntok + c] = tab->pos[row], ct[CT_R * ntok + c] = tab->r[row], ct[CT_SEQ * ntok + c] = tab->seq[row];
    ct[CT_SLOT * ntok + c] = tab->kv_slot[row], ct[CT_HID * ntok + c] = tab->hid_idx[row], ct[CT_LOGIT * ntok + c] = tab->logit_idx[row];
    ct[CT_XROW * ntok + c] = row;  // where a reading-out column's activation planes and sums of squares live
  }
}

// push this thread's accumulator fragments (rows warp*16+g / +8, columns n*8+2t / +1) into the receive buffers of
// the ranks that own the columns (distributed shared memory stores; made visible by the cluster barrier)
template <int NG, int KH = 1>
__device__ __forceinline__ void gemm_push_tile(const float (&acc)[NG][4], float* recv, int own_max, int n_cols, int cs, int rank,
                                               cg::cluster_group& cluster) {
  constexpr int RBW = RB_ROWS / KH;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int rl = (warp % (8 / KH)) * 16 + g;
  rank = rank * KH + warp / (8 / KH);  // the two k-halves of a CTA count as separate contributors
#pragma unroll
  for (int n = 0; n < NG; ++n)
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int c = n * 8 + 2 * t + e;
      if (c < n_cols) {
        const int owner = c % cs, slot = c / cs;
        float* dst = (cs > 1 ? cluster.map_shared_rank(recv, owner) : recv) + ((size_t)rank * own_max + slot) * RBW + rl;
        dst[0] = acc[n][e];
        dst[8] = acc[n][2 + e];
      }
    }
}

// ======================================= bf16 weights: tensor cores ========================================
template <int NG, int EPI>
__global__ void __launch_bounds__(GEMM_THREADS) __maxnreg__(NG == 1 ? LS_MAXREG : 255) gemm_bf16_kernel(const __grid_constant__ GemmParams p) {
  // KH = 2 (64-row blocks, the warps of a CTA in two groups that alternate k-blocks) is supported by the helpers below
  // and doubles the CTAs of a GEMM with few output rows; measured slower than 128-row blocks once the kernels of the
  // chain overlap, so every epilogue runs with KH = 1
  constexpr int KH = 1;
  constexpr int NTOK = 8 * NG;
  constexpr int XCH = xchunk_kblocks(NG);

  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4* ring = reinterpret_cast<uint4*>(smem_raw);            // [RING][2][256], slot of thread tid only
  uint4* xbuf = ring + RING * 2 * GEMM_THREADS;                // [3][XCH][NTOK][4]
  float* recv = reinterpret_cast<float*>(xbuf + xbuf_uint4(NG));  // [cs][own_max][128]
  float* colbuf = recv + recv_floats(NG);                      // [2][128]
  float* s_rstd = colbuf + 2 * RB_ROWS;
  int* s_ct = reinterpret_cast<int*>(s_rstd + NTOK);           // [CT_FIELDS][NTOK]

  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int cs = p.cluster_size, rank = (int)cluster.block_rank(), cid = blockIdx.x / cs;
  const int own_max = (NTOK + cs - 1) / cs;
  int dbg_n = 0;
  auto stamp = [&]() {
    if (kTune && p.dbg && blockIdx.x == 0 && tid == 0) p.dbg[dbg_n++] = clock64();
  };
  stamp();
  pdl_launch_dependents();  // first thing: the next kernel's CTAs may become resident and request their weights (pass 1.056 -> 1.049 ms
                            // against releasing them after this kernel's own first requests)
  timeline_mark(p.tl, p.tl_id, false);
  if (kTune && p.tl && tid == 0 && (p.tl_id == 28 || p.tl_id == 29 || p.tl_id == 27)) {  // per-CTA start time and SM of one layer's kernels
    unsigned long long tns;
    unsigned smid;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(tns));
    asm volatile("mov.u32 %0, %smid;" : "=r"(smid));
    p.tl[4096 + (p.tl_id - 27) * 1024 + blockIdx.x * 2] = tns;
    p.tl[4096 + (p.tl_id - 27) * 1024 + blockIdx.x * 2 + 1] = smid;
  }
  const int kpr = p.kb_per_rb;
  int kb_lo, kb_hi;
  gemm_krange(kpr, cs, rank, kb_lo, kb_hi);
  const int upt = kb_hi - kb_lo;                                 // k-blocks per task (whole CTA)
  const int khalf = warp / (8 / KH);                             // which k-blocks of the range this warp takes
  const int my_upt = (upt - khalf + KH - 1) / KH;                // units per task of this warp
  const int n_tasks = (p.n_rb - cid + p.n_clusters - 1) / p.n_clusters;  // row blocks cid, cid + n_clusters, ...

  // ---- weight ring: issue side.  The weights are stored tile-major (see pack_weights_kernel): the 1 KB a warp
  // consumes per unit is contiguous and consecutive k-blocks of a 16-row tile follow each other, so every warp
  // streams one contiguous region and every request covers whole 128-byte lines.  The loop is kept to a few
  // instructions per unit: shared-memory addresses are 32-bit registers advanced by constants.
  constexpr unsigned SLOT_BYTES = 2 * GEMM_THREADS * 16, RING_BYTES = RING * SLOT_BYTES, HI_OFF = GEMM_THREADS * 16;
  const unsigned ring_s = (unsigned)__cvta_generic_to_shared(ring) + tid * 16;
  const __nv_bfloat16* const Wb = static_cast<const __nv_bfloat16*>(p.W);
  const char* i_ptr = reinterpret_cast<const char*>(Wb);
  unsigned i_slot = 0;
  int i_rb = cid, i_left = my_upt, i_tasks = my_upt > 0 ? n_tasks : 0, i_size = 0;
  auto i_setup = [&]() {
    int r0 = gemm_row0<EPI, KH>(p, i_rb, warp);
    i_size = r0 >= 0 ? 16 : 0;  // rows beyond the matrix: zero-fill, nothing is read
    const int pt = r0 >= 0 ? packed_tile(p.perm, p.perm_a, p.perm_d, r0) : 0;
    i_ptr = reinterpret_cast<const char*>(Wb + ((size_t)pt * kpr + kb_lo + khalf) * 512 + lane * 8);
  };
  i_setup();
  auto issue_unit = [&]() {
    if (i_tasks > 0) {
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(ring_s + i_slot), "l"(i_ptr), "r"(i_size) : "memory");
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(ring_s + i_slot + HI_OFF), "l"(i_ptr + 512), "r"(i_size)
                   : "memory");
      i_ptr += 1024 * KH;
      i_slot += SLOT_BYTES;
      if (i_slot == RING_BYTES) i_slot = 0;
      if (--i_left == 0) {
        i_left = my_upt, i_rb += p.n_clusters;
        if (--i_tasks > 0) i_setup();
      }
    }
    cp_async_commit();
  };
  auto drain = [&]() { cp_async_wait<0>(); };
#pragma unroll
  for (int s = 0; s < RING - 1; ++s) issue_unit();

  // the row table was written before this pass started, so the live row count can be read ahead of the predecessor
  const RowTable* tab = p.tab;
  int n_cols = (tab ? (p.cols_from_readout ? tab->n_readout : tab->n_rows) : p.m_fixed) - p.col0;
  if (n_cols > NTOK) n_cols = NTOK;
  gemm_load_cols(p, n_cols, NTOK, s_ct);
  // the weights above are constants; everything below reads what earlier kernels of the pass produced
  stamp();
  pdl_wait();
  stamp();
  timeline_mark(p.tl, p.tl_id + 256, false);
  if (n_cols <= 0) {  // uniform over the cluster: nobody reaches a cluster barrier
    drain();
    return;
  }

  // ---- activations of this CTA's k-range, copied asynchronously into MMA-fragment order: piece idx -> (plane s,
  // k-block kbl, column c, quarter tt).  Columns beyond the live rows are zero-filled without being read.
  // Thread tid always copies quarter tt of column c; 256 threads cover 256 / (4 NTOK) k-blocks of one plane per
  // round.  Dead columns are left as they are: an MMA output column depends on its own B column only, and dead
  // columns are never read back.
  auto x_stage = [&](int kb0, int nkb) {
    constexpr int KPR = GEMM_THREADS / (4 * NTOK);  // k-blocks per round
    const int tt = tid & 3, c = (tid >> 2) % NTOK, kq = tid / (4 * NTOK);
    if (c < n_cols) {
      const int xr = p.cols_from_readout ? s_ct[CT_XROW * NTOK + c] : c;
#pragma unroll
      for (int s = 0; s < 3; ++s) {
        const __nv_bfloat16* src = p.xplanes + ((size_t)xr * 3 + s) * p.x_ld + (kb0 + kq) * 32 + tt * 8;
        uint4* dst = xbuf + ((s * XCH + kq) * NTOK + c) * 4 + tt;
#pragma unroll
        for (int j = 0; j < XCH; j += KPR) {
          const int kbl = kq + j;
          const bool ok = (kb0 + kbl) * 32 + tt * 8 < p.K;
          if (kbl < nkb) cp_async16(dst + j * NTOK * 4, ok ? src + j * 32 : p.xplanes, ok);
        }
      }
    }
    cp_async_commit();
  };
  const bool one_chunk = upt <= XCH;  // the whole k-range stays staged for every row block of this CTA

  float acc[3][NG][4];  // one chain per split term, the same for every NG: a row's bits must not depend on
                        // how many rows share the pass
  const unsigned xs_s = (unsigned)__cvta_generic_to_shared(xbuf) + (g * 4 + t) * 16;
  constexpr unsigned X_KB = NTOK * 64, X_PLANE = XCH * NTOK * 64;  // bytes per k-block / per plane in xbuf
  unsigned c_slot = 0;
  auto lds128 = [](unsigned addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
  };
  float pre_h = 0.f, pre_g = 1.f;
  float2 pre_rope = make_float2(1.f, 0.f);
  for (int task = 0; task < n_tasks; ++task) {
    const int rb = cid + task * p.n_clusters;
    const bool warp_valid = gemm_row0<EPI, KH>(p, rb, warp) >= 0;
#pragma unroll
    for (int h = 0; h < 3; ++h)
#pragma unroll
      for (int n = 0; n < NG; ++n)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[h][n][i] = 0.f;
    for (int ck = 0; ck < upt; ck += XCH) {
      const int nkb = min(XCH, upt - ck);
      const bool first = task == 0 && ck == 0;
      if (first || !one_chunk) {  // wide passes (prefill) restage the activations chunk by chunk
        if (!first || p.cols_from_readout) __syncthreads();  // (the lm_head's staging reads the column table)
        x_stage(kb_lo + ck, nkb);
        if (first) gemm_rstd(p, n_cols, s_rstd, s_ct, NTOK);
        cp_async_wait<0>();
        __syncthreads();
        if (first) stamp();
      }
      if (ck == 0) {  // operands of this CTA's first output column, requested ahead of the main loop
        const int c = rank + cs * (tid >> 7), jr = tid & 127;
        if (EPI == EPI_RESID && c < n_cols && jr < RB_ROWS / KH) {
          pre_h = p.hid[(size_t)s_ct[CT_HID * NTOK + c] * p.H + rb * (RB_ROWS / KH) + jr];
          if (p.out_planes) pre_g = p.gain_next[rb * (RB_ROWS / KH) + jr];
        }
        if (EPI == EPI_QKV && c < n_cols && jr < 64) {
          const int hd2 = p.head_dim >> 1;
          pre_rope = p.rope[(size_t)s_ct[CT_POS * NTOK + c] * hd2 + jr % hd2];
        }
      }
      const int kbl0 = (khalf + KH - (ck % KH)) % KH;  // this warp's first k-block of the chunk
      unsigned xk = xs_s + kbl0 * X_KB;
      for (int kbl = kbl0; kbl < nkb; kbl += KH) {
        issue_unit();
        cp_async_wait<RING - 1>();
        if (warp_valid) {
          const uint4 a_lo = lds128(ring_s + c_slot), a_hi = lds128(ring_s + c_slot + HI_OFF);
          if (NG == 1) {
#pragma unroll
            for (int s = 0; s < 3; ++s) {
              const uint4 b = lds128(xk + s * X_PLANE);
              mma_bf16(acc[s][0], a_lo.x, a_hi.x, a_lo.y, a_hi.y, b.x, b.y);
              mma_bf16(acc[s][0], a_lo.z, a_hi.z, a_lo.w, a_hi.w, b.z, b.w);
            }
          } else {
            // wide passes: a plane's B fragments are requested together, one plane ahead of the MMAs that use them
            // (the asm statements keep their order, so a load placed next to its MMA would expose the shared-memory
            // latency once per column group); the accumulation order of every chain is unchanged
            uint4 b[2][NG];
#pragma unroll
            for (int n = 0; n < NG; ++n) b[0][n] = lds128(xk + n * 512);
#pragma unroll
            for (int s = 0; s < 3; ++s) {
              if (s < 2) {
#pragma unroll
                for (int n = 0; n < NG; ++n) b[(s + 1) & 1][n] = lds128(xk + (s + 1) * X_PLANE + n * 512);
              }
              // the two k-halves of a chain depend on each other: all first halves, then all second halves
#pragma unroll
              for (int n = 0; n < NG; ++n) mma_bf16(acc[s][n], a_lo.x, a_hi.x, a_lo.y, a_hi.y, b[s & 1][n].x, b[s & 1][n].y);
#pragma unroll
              for (int n = 0; n < NG; ++n) mma_bf16(acc[s][n], a_lo.z, a_hi.z, a_lo.w, a_hi.w, b[s & 1][n].z, b[s & 1][n].w);
            }
          }
        }
        c_slot += SLOT_BYTES;
        if (c_slot == RING_BYTES) c_slot = 0;
        xk += X_KB * KH;
      }
    }
    // fold the chains in fixed order, hi + (mid + lo), and publish this CTA's partial tile
    float tot[NG][4];
#pragma unroll
    for (int n = 0; n < NG; ++n)
#pragma unroll
      for (int i = 0; i < 4; ++i) tot[n][i] = acc[0][n][i] + (acc[1][n][i] + acc[2][n][i]);
    stamp();
    gemm_push_tile<NG, KH>(tot, recv, own_max, n_cols, cs, rank, cluster);
    cluster.sync();
    stamp();
    gemm_reduce_epilogue<EPI, KH>(p, s_ct, NTOK, rb, n_cols, recv, own_max, colbuf, s_rstd, rank, pre_h, pre_g, pre_rope,
                                  EPI == EPI_RESID || EPI == EPI_QKV);
    stamp();
    if (task + 1 < n_tasks) cluster.sync();  // the owners are done with the receive buffer before it is refilled
  }
  drain();
  timeline_mark(p.tl, p.tl_id, true);
  if (kTune && p.tl && tid == 0 && (p.tl_id == 28 || p.tl_id == 29 || p.tl_id == 27)) {
    unsigned long long tns;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(tns));
    p.tl[4096 + 3 * 1024 + (p.tl_id - 27) * 512 + blockIdx.x] = tns;
  }
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
  float* recv = xf + XCH * NTOK * 32;                          // [cs][own_max][128]
  float* colbuf = recv + recv_floats(NG);
  float* s_rstd = colbuf + 2 * RB_ROWS;
  int* s_ct = reinterpret_cast<int*>(s_rstd + NTOK);

  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int cs = p.cluster_size, rank = (int)cluster.block_rank(), cid = blockIdx.x / cs;
  const int kpr = p.kb_per_rb;
  int kb_lo, kb_hi;
  gemm_krange(kpr, cs, rank, kb_lo, kb_hi);
  const int upt = kb_hi - kb_lo;
  const int n_tasks = (p.n_rb - cid + p.n_clusters - 1) / p.n_clusters;
  const int own_max = (NTOK + cs - 1) / cs;
  pdl_launch_dependents();
  pdl_wait();
  const RowTable* tab = p.tab;
  int n_cols = (tab ? (p.cols_from_readout ? tab->n_readout : tab->n_rows) : p.m_fixed) - p.col0;
  if (n_cols > NTOK) n_cols = NTOK;
  if (n_cols <= 0) return;
  gemm_load_cols(p, n_cols, NTOK, s_ct);
  __syncthreads();
  gemm_rstd(p, n_cols, s_rstd, s_ct, NTOK);

  for (int task = 0; task < n_tasks; ++task) {
    const int rb = cid + task * p.n_clusters;
    const int row0 = gemm_row0<EPI>(p, rb, warp);
    float accf[NG][8][2];
#pragma unroll
    for (int n = 0; n < NG; ++n)
#pragma unroll
      for (int c = 0; c < 8; ++c) accf[n][c][0] = accf[n][c][1] = 0.f;
    for (int ck = 0; ck < upt; ck += XCH) {
      const int nkb = min(XCH, upt - ck);
      __syncthreads();
      for (int idx = tid; idx < nkb * NTOK * 32; idx += GEMM_THREADS) {
        int e = idx & 31, c = (idx >> 5) % NTOK, kbl = idx / (32 * NTOK);
        int k = (kb_lo + ck + kbl) * 32 + e;
        float v = 0.f;
        if (c < n_cols && k < p.K) {
          const int xr = p.cols_from_readout ? s_ct[CT_XROW * NTOK + c] : c;
          const __nv_bfloat16* pl = p.xplanes + (size_t)xr * 3 * p.x_ld + k;
          v = (__bfloat162float(pl[0]) + __bfloat162float(pl[p.x_ld])) + __bfloat162float(pl[2 * p.x_ld]);
        }
        xf[idx] = v;
      }
      __syncthreads();
      if (row0 >= 0) {
        for (int kbl = 0; kbl < nkb; ++kbl) {
          const int k = (kb_lo + ck + kbl) * 32 + t * 8;
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
    gemm_push_tile<NG>(tot, recv, own_max, n_cols, cs, rank, cluster);
    cluster.sync();
    gemm_reduce_epilogue<EPI>(p, s_ct, NTOK, rb, n_cols, recv, own_max, colbuf, s_rstd, rank);
    if (task + 1 < n_tasks) cluster.sync();
  }
}
__host__ __device__ constexpr int gemm_f32_smem_bytes(int NG) {
  return 4 * 8 * NG * 32 * 4 + recv_floats(NG) * 4 + 2 * RB_ROWS * 4 + 8 * NG * 4 * (1 + CT_FIELDS) + 64;
}

// ---- one-time repacking of a bf16 weight matrix [N][K] into the tile-major streaming layout ----------------
// unit (rt, kb) = rows rt*16 .. +15, k = kb*32 .. +31, 1 KB: first the 512 bytes of the "low" pieces (lane g*4+t
// holds row rt*16+g, k = kb*32 + t*8 .. +7), then the 512 bytes of the "high" pieces (row rt*16+g+8); k beyond
// K is zero.  Units of one row tile are consecutive in kb.
struct PackParams {
  const __nv_bfloat16* src;  // [N][K]
  __nv_bfloat16* dst;        // [N/16][kpr][2][32][8]
  int N, K, kpr;
  int perm, perm_a, perm_d;  // row tile order (see packed_tile)
};
__global__ void pack_weights_kernel(const __grid_constant__ PackParams p) {
  const size_t n_pieces = (size_t)(p.N / 16) * p.kpr * 64;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_pieces; i += (size_t)gridDim.x * blockDim.x) {
    const int lane = (int)(i & 31), hi = (int)((i >> 5) & 1);
    const size_t unit = i >> 6;
    const int kb = (int)(unit % p.kpr);
    const size_t rt = unit / p.kpr;
    const int g = lane >> 2, t = lane & 3;
    const size_t row = (size_t)packed_tile_row0(p.perm, p.perm_a, p.perm_d, (int)rt) + g + 8 * hi;
    const int k = kb * 32 + t * 8;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (k < p.K) v = *reinterpret_cast<const uint4*>(p.src + row * p.K + k);
    reinterpret_cast<uint4*>(p.dst)[i] = v;
  }
}

// ---- fp32 rows -> three bf16 planes, optionally through RMSNorm's gain, with the row's sum of squares -----
struct PrepParams {
  const RowTable* tab;      // null: rows 0..m_fixed-1 of `x`
  int m_fixed;
  const float* x;           // stand-alone source [m][K]
  float* hid;               // row source [hid_idx][K]
  int K;
  const float* gain;        // may be null
  __nv_bfloat16* planes;    // [col][3][K]
  float* sumsq;             // [col * sq_stride] full sum of squares (may be null)
  int sq_stride;
  int use_src;              // rows with src_hid >= 0 are first copied from there (the copy is what the pass updates)
};

// ---- Raven-style recurrence input: the adapter reads [H; e] (Sec. 3.1 with P holding blocks: H0 = e = P(X), then
// H <- B(W_a [H; e])).  Rows entering their first recurrence have H = e: their e is kept for the later recurrences. ----
struct ConcatParams {
  const RowTable* tab;
  float* hid;               // [hid_idx][H] the rows' states
  float* e_store;           // [hid_idx][H] the rows' prelude outputs
  int H;
  __nv_bfloat16* planes;    // [col][3][2 H]
};
__global__ void __launch_bounds__(256) raven_concat_kernel(const __grid_constant__ ConcatParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int c = blockIdx.x;
  if (c >= p.tab->n_rows) return;
  const int idx = p.tab->hid_idx[c];
  const float* h = p.hid + (size_t)idx * p.H;
  float* e = p.e_store + (size_t)idx * p.H;
  const bool first = p.tab->r[c] == 1;
  __nv_bfloat16* dst = p.planes + (size_t)c * 3 * 2 * p.H;
  for (int k = threadIdx.x; k < p.H; k += blockDim.x) {
    const float hv = h[k];
    float ev = hv;
    if (first) e[k] = hv;
    else ev = e[k];
    store_split(dst, 2 * p.H, k, hv);
    store_split(dst, 2 * p.H, p.H + k, ev);
  }
}

__global__ void __launch_bounds__(256) prep_planes_kernel(const __grid_constant__ PrepParams p) {
  __shared__ float s_part[8];
  tune_mark(600, false);
  pdl_launch_dependents();
  pdl_wait();
  const int c = blockIdx.x;
  int n = p.tab ? p.tab->n_rows : p.m_fixed;
  if (c >= n) return;
  const float* src;
  float* copy = nullptr;  // the pass works on a copy of another hidden state
  if (p.tab) {
    src = p.hid + (size_t)p.tab->hid_idx[c] * p.K;
    if (p.use_src && p.tab->src_hid[c] >= 0) copy = p.hid + (size_t)p.tab->hid_idx[c] * p.K, src = p.hid + (size_t)p.tab->src_hid[c] * p.K;
  } else {
    src = p.x + (size_t)c * p.K;
  }
  __nv_bfloat16* dst = p.planes + (size_t)c * 3 * p.K;
  float ss = 0.f;
  for (int k = threadIdx.x; k < p.K; k += blockDim.x) {
    float v = src[k];
    if (copy) copy[k] = v;
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
  tune_mark(600, true);
}

// ======================= fused epilogue for sums produced by the tcgen05 kernel (prefill passes) ==========================
// linear_tc_kernel leaves raw k-split partial sums [split][column][N] in global memory; one CTA per row block adds the
// splits in split order into the receive-buffer layout of a one-rank cluster and runs the same epilogue code as the
// mma.sync kernels (1/rms, then RoPE + KV write / residual + sum of squares + planes / SwiGLU + planes).
constexpr int TCE_MAX_COLS = 64;
#ifndef LS_TCE_GROUPS
#define LS_TCE_GROUPS 32  // measured on the 512-token prefill of the 1.4B shape: 8 / 16 / 32 / 64 groups -> 80.3 / 70.9 / 67.9 / 71.7 ms
#endif
constexpr int TCE_GROUPS = LS_TCE_GROUPS;   // column groups = CTAs per row block (the epilogue code sees a cluster of this size)
struct TcEpiParams {
  GemmParams g;        // cluster_size = TCE_GROUPS; the per-column buffers start at the pass's first column
  const float* part;   // [group][n_split][cols_ld][N]
  int n_split, cols_ld;
  int Hq;              // query width (rows of the query buffer)
};

template <int EPI, bool GROUPED>
__global__ void __launch_bounds__(GEMM_THREADS) tc_epilogue_kernel(const __grid_constant__ TcEpiParams q) {
  __shared__ float s_recv[(TCE_MAX_COLS / TCE_GROUPS) * RB_ROWS];
  __shared__ float s_colbuf[2 * RB_ROWS];
  __shared__ float s_rstd[TCE_MAX_COLS];
  __shared__ int s_ct[CT_FIELDS * TCE_MAX_COLS];
  // GROUPED: blockIdx.z = group of TCE_MAX_COLS token columns, with its slices of the per-column buffers (a private copy
  // of the parameters; passes of up to TCE_MAX_COLS rows read them where they are)
  GemmParams p_grp;
  if (GROUPED) p_grp = q.g;
  const GemmParams& p = GROUPED ? p_grp : q.g;
  if (GROUPED) {
    GemmParams& p = p_grp;
    const int col0 = (int)blockIdx.z * TCE_MAX_COLS;
    p.col0 = col0;
    if (p.out_planes) p.out_planes += (size_t)col0 * 3 * p.planes_ld;
    if (p.sumsq) p.sumsq += (size_t)col0 * p.sq_stride;
    if (p.sumsq_out) p.sumsq_out += (size_t)col0 * p.n_sq_out;
    if (p.qbuf) p.qbuf += (size_t)col0 * q.Hq;
  }
  const float* part = q.part + (size_t)blockIdx.z * q.n_split * q.cols_ld * p.N;
  const int tid = threadIdx.x, rb = blockIdx.x;
  const RowTable* tab = p.tab;  // final before the pass starts
  int n_cols = tab->n_rows - p.col0;  // this group's live columns
  if (n_cols > TCE_MAX_COLS) n_cols = TCE_MAX_COLS;
  gemm_load_cols(p, n_cols, TCE_MAX_COLS, s_ct);
  pdl_launch_dependents();
  pdl_wait();
  if ((int)blockIdx.y >= n_cols) return;  // no column for this group
  {  // 1/rms of this group's columns only (gemm_rstd's arithmetic: one partial per lane, butterfly sum)
    const int warp = tid >> 5, lane = tid & 31;
    for (int c = blockIdx.y + TCE_GROUPS * warp; c < n_cols; c += TCE_GROUPS * (GEMM_THREADS / 32)) {
      float ss = 0.f;
      if (p.sumsq)
        for (int i = lane; i < p.n_sq; i += 32) ss += p.sumsq[c * p.sq_stride + i];
      ss = warp_sum(ss);
      if (lane == 0) s_rstd[c] = p.sumsq ? 1.0f / sqrtf(ss / (float)p.H + p.eps) : 1.0f;
    }
  }
  // row j of the block -> row of the weight matrix (gate/up: 64 gate rows, then the 64 matching up rows)
  const int j = tid & (RB_ROWS - 1);
  int n;
  if (EPI == EPI_SWIGLU) {
    const int f = rb * 64 + (j & 63);
    n = f < p.F ? (j < 64 ? f : p.F + f) : -1;
  } else {
    n = rb * RB_ROWS + j;
    if (n >= p.N) n = -1;
  }
  // blockIdx.y takes the columns c = y, y + TCE_GROUPS, ... exactly as rank y of a cluster of TCE_GROUPS CTAs would, with
  // one contribution per column in the receive buffer (recv_ranks = 1): the k-split sums added below
  const int rank = blockIdx.y, own_max = TCE_MAX_COLS / TCE_GROUPS;
  const size_t split_stride = (size_t)q.cols_ld * p.N;
  for (int c = rank + TCE_GROUPS * (tid >> 7); c < n_cols; c += TCE_GROUPS * (GEMM_THREADS / RB_ROWS)) {
    float v = 0.f;
    if (n >= 0) {
      const float* src = part + (size_t)c * p.N + n;
      v = __ldcg(src);
      for (int s0 = 1; s0 < q.n_split; s0 += 8) {  // eight loads in flight, added in split order
        float t[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) t[u] = s0 + u < q.n_split ? __ldcg(src + (size_t)(s0 + u) * split_stride) : 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u)
          if (s0 + u < q.n_split) v += t[u];
      }
    }
    s_recv[(c / TCE_GROUPS) * RB_ROWS + j] = v;
  }
  __syncthreads();
  gemm_reduce_epilogue<EPI>(p, s_ct, TCE_MAX_COLS, rb, n_cols, s_recv, own_max, s_colbuf, s_rstd, rank);
}

}  // namespace ls

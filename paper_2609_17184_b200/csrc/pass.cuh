// One persistent kernel for a whole batched pass through the shared block stack (Sec. 4.2 step 1): for every
// layer QKV -> attention -> O -> gate/up -> down, separated by grid barriers instead of kernel boundaries.
//
// Why: each of the 5 x L stages streams only 1.3-7 us worth of weights, so the latency between stages decides
// the pass time.  Here every warp walks a fixed sequence of weight units (all stages of all layers) and keeps
// RING units of it in flight in a thread-private cp.async ring that never drains at a stage boundary: while a
// CTA waits at a barrier, stages activations or reduces partial sums, the weights of its next stage arrive.
//
// Decomposition.  The grid is n_clusters thread-block clusters of 8 CTAs.  In every stage a cluster owns a
// contiguous set of output row tiles (16 rows each; rotary partners and gate/up partners are adjacent tiles of
// the packed weights, so a cluster always holds both) and its 8 CTAs split K into equal contiguous ranges.  A
// warp carries up to three row tiles through its k-blocks (activation fragments are loaded once per k-block
// and reused for the tiles).  Partial sums are pushed into the shared memory of the CTA that finishes the
// token column (rank c finishes column c; distributed shared memory stores + one cluster barrier), summed in
// rank order, and the stage's epilogue runs there.  No atomics on data, no global partials: bit-reproducible.
// The grid barrier is a monotonic counter touched by one thread per cluster; a wait that exceeds its bound
// raises an error flag and every later barrier falls through (no CTA leaves early, nothing can hang).
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"
#include "gemm.cuh"

namespace ls {

constexpr int PASS_THREADS = 256;
constexpr int PASS_CS = 8;             // CTAs per cluster = K ranges per stage = token columns of a pass
constexpr int PASS_TPW = 3;            // row tiles a warp carries through a stage
constexpr int PASS_RING = 8;            // weight stages per thread
constexpr int PASS_XCH = 24;           // k-blocks of activations a CTA stages (its whole k-range)
constexpr int PASS_RECV_FLOATS = 8 * PASS_TPW * 8 * 16;  // [contribution][tile][16 rows] of one token column
constexpr unsigned PASS_SPIN_LIMIT = 1u << 20;
enum { ST_QKV = 0, ST_O = 1, ST_GU = 2, ST_DOWN = 3, N_STAGES = 4 };

struct PassParams {
  const RowTable* tab;
  int L;
  const void* const* wpacked;   // device [L][4] tile-major weights: qkv, o, gate/up, down
  const void* const* layer_w;   // device [L][6] original pointers (norm gains: [0] norm1, [3] norm2)
  const float* final_gain;      // gain of the readout's final norm (planes after the last layer)
  int H, Hq, Hkv, F, n_q_heads, n_kv_heads, head_dim, slots;
  float eps, scale;
  float* hid;
  __nv_bfloat16 *xplanes, *aplanes, *splanes;
  float* qbuf;
  float* sumsq;                 // [row][sq_stride]: one partial per cluster
  int sq_stride;
  __nv_bfloat16* kv;            // whole pool
  long long kv_layer_stride, kv_plane_stride, kv_sel_stride;
  const float2* rope;
  float* apart;                 // attention partials
  int* acnt;
  int max_chunks;
  unsigned* bar;                // [0] barrier counter, [1] set once a wait ran out; both zero at launch
  volatile int* err;            // host-visible flag
  unsigned long long* dbg;      // optional: per-stage timestamps of CTA 0 (null in production)
  int n_clusters;
  // per stage: tile groups (pairs of partner tiles or single tiles), k-halves per CTA, k-blocks per row, K
  int n_groups[N_STAGES], paired[N_STAGES], kh[N_STAGES], kpr[N_STAGES], K[N_STAGES];
};

// what one warp does in a stage
struct StageGeo {
  int KH, WG, wg, khalf;  // k-halves per CTA; warps per k-half; this warp's place
  int g_lo, nt;           // first tile group and number of row tiles of this cluster
  int kb_lo, upt;         // k-range of this CTA
  int kb0, nkb;           // this warp's k-blocks: kb0, kb0 + KH, ... (nkb of them)
  int my_nt;              // row tiles of this warp: local tiles wg, wg + WG, ...
  __device__ __forceinline__ void set(const PassParams& p, int st, int cid, int rank, int warp) {
    KH = p.kh[st], WG = 8 / KH, wg = warp % WG, khalf = warp / WG;
    const int ng = p.n_groups[st];
    g_lo = (int)((long long)cid * ng / p.n_clusters);
    const int g_hi = (int)((long long)(cid + 1) * ng / p.n_clusters);
    nt = (g_hi - g_lo) << p.paired[st];
    int kb_hi;
    gemm_krange(p.kpr[st], PASS_CS, rank, kb_lo, kb_hi);
    upt = kb_hi - kb_lo;
    kb0 = kb_lo + khalf;
    nkb = upt > khalf ? (upt - khalf + KH - 1) / KH : 0;
    my_nt = nt > wg ? (nt - wg + WG - 1) / WG : 0;
  }
  // index of this cluster's first tile in the packed weights (partner tiles are adjacent there)
  __device__ __forceinline__ int tile0(const PassParams& p, int st) const { return g_lo << p.paired[st]; }
};

// ---- attention work item on one half of the CTA (128 threads, own named barrier) ----------------------------------
struct AttnSmem {
  float score[4][ATT_CHUNK + MAX_SPEC + 8];
  float red[4][4][128];
  float stat[4][2];
  int last;
};

template <int D, int G>
__device__ __forceinline__ void pass_attention_item(const PassParams& p, const RowTable* tab, int l, int item, AttnSmem& sm,
                                                    int htid, int bar_id) {
  constexpr int NT = 128;
  constexpr int LPP = D / 8, PPW = 32 / LPP, PPR = PPW * (NT / 32);
  constexpr int NPOS = ATT_CHUNK + MAX_SPEC;
  constexpr int ROUNDS = (NPOS + PPR - 1) / PPR;
  constexpr int PSTRIDE = D + 2;
  auto hsync = [&]() { asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(NT) : "memory"); };
  const int warp = htid >> 5, lane = htid & 31, sub = lane / LPP, dl = lane % LPP;
  const int HQ = p.n_q_heads * D;
  const int kvh = item % p.n_kv_heads, rc = item / p.n_kv_heads;
  int row = 0;
  while (row + 1 < tab->n_rows && tab->chunk_start[row + 1] <= rc) ++row;
  const int chunk = rc - tab->chunk_start[row];
  const int n_chunks = tab->chunk_start[row + 1] - tab->chunk_start[row];
  const int p0 = chunk * ATT_CHUNK;
  const int n_can_here = min(ATT_CHUNK, tab->n_canon[row] - p0);
  const int n_spec = (chunk == n_chunks - 1) ? tab->n_spec[row] : 0;
  const int n_here = n_can_here + n_spec;
  const size_t plane = (size_t)l * p.kv_layer_stride + (size_t)(tab->r[row] - 1) * p.kv_plane_stride;
  const size_t headbase = (size_t)(tab->seq[row] * p.n_kv_heads + kvh) * p.slots * D;
  const __nv_bfloat16* Kb = p.kv + plane + headbase;
  const __nv_bfloat16* Vb = p.kv + plane + p.kv_sel_stride + headbase;

  uint4 kreg[ROUNDS], vreg[ROUNDS];
#pragma unroll
  for (int rd = 0; rd < ROUNDS; ++rd) {
    const int jpos = rd * PPR + warp * PPW + sub;
    kreg[rd] = vreg[rd] = make_uint4(0, 0, 0, 0);
    if (jpos < n_here) {
      const int slot = jpos < n_can_here ? p0 + jpos : tab->spec_slot[row][jpos - n_can_here];
      const size_t off = (size_t)slot * D + dl * 8;
      kreg[rd] = __ldcg(reinterpret_cast<const uint4*>(Kb + off));
      vreg[rd] = __ldcg(reinterpret_cast<const uint4*>(Vb + off));
    }
  }
  float q[G][8];
#pragma unroll
  for (int gq = 0; gq < G; ++gq) {
    const float4* qp = reinterpret_cast<const float4*>(p.qbuf + (size_t)row * HQ + (size_t)(kvh * G + gq) * D + dl * 8);
    float4 a = __ldcg(qp), b = __ldcg(qp + 1);
    q[gq][0] = a.x, q[gq][1] = a.y, q[gq][2] = a.z, q[gq][3] = a.w;
    q[gq][4] = b.x, q[gq][5] = b.y, q[gq][6] = b.z, q[gq][7] = b.w;
  }
  hsync();  // the half's shared buffers are free again
#pragma unroll
  for (int rd = 0; rd < ROUNDS; ++rd) {
    const int jpos = rd * PPR + warp * PPW + sub;
    const unsigned w[4] = {kreg[rd].x, kreg[rd].y, kreg[rd].z, kreg[rd].w};
    float kf[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) kf[2 * i] = __uint_as_float(w[i] << 16), kf[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
#pragma unroll
    for (int gq = 0; gq < G; ++gq) {
      float s = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) s = fmaf(q[gq][i], kf[i], s);
#pragma unroll
      for (int o = LPP / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (dl == 0) sm.score[gq][jpos] = (jpos < n_here) ? s * p.scale : -INFINITY;
    }
  }
  hsync();
  for (int gq = warp; gq < G; gq += NT / 32) {
    float m = -INFINITY;
    for (int jj = lane; jj < ROUNDS * PPR; jj += 32) m = fmaxf(m, sm.score[gq][jj]);
    m = warp_max(m);
    float lsum = 0.f;
    for (int jj = lane; jj < ROUNDS * PPR; jj += 32) {
      float e = (jj < n_here) ? expf(sm.score[gq][jj] - m) : 0.f;
      sm.score[gq][jj] = e;
      lsum += e;
    }
    lsum = warp_sum(lsum);
    if (lane == 0) sm.stat[gq][0] = m, sm.stat[gq][1] = lsum;
  }
  hsync();
  float o[G][8];
#pragma unroll
  for (int gq = 0; gq < G; ++gq)
#pragma unroll
    for (int i = 0; i < 8; ++i) o[gq][i] = 0.f;
#pragma unroll
  for (int rd = 0; rd < ROUNDS; ++rd) {
    const int jpos = rd * PPR + warp * PPW + sub;
    const unsigned w[4] = {vreg[rd].x, vreg[rd].y, vreg[rd].z, vreg[rd].w};
    float vf[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) vf[2 * i] = __uint_as_float(w[i] << 16), vf[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
#pragma unroll
    for (int gq = 0; gq < G; ++gq) {
      float pw = sm.score[gq][jpos];
#pragma unroll
      for (int i = 0; i < 8; ++i) o[gq][i] = fmaf(pw, vf[i], o[gq][i]);
    }
  }
#pragma unroll
  for (int gq = 0; gq < G; ++gq)
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float v = o[gq][i];
#pragma unroll
      for (int off = LPP; off < 32; off <<= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
      if (sub == 0) sm.red[warp][gq][dl * 8 + i] = v;
    }
  hsync();
  const int pair = row * p.n_kv_heads + kvh;
  float* mypart = p.apart + ((size_t)pair * p.max_chunks + chunk) * G * PSTRIDE;
  if (n_chunks == 1) {
    for (int idx = htid; idx < G * D; idx += NT) {
      int gq = idx / D, dd = idx % D;
      float v = (sm.red[0][gq][dd] + sm.red[1][gq][dd]) + (sm.red[2][gq][dd] + sm.red[3][gq][dd]);
      store_split(p.aplanes + (size_t)row * 3 * HQ, HQ, (kvh * G + gq) * D + dd, v / sm.stat[gq][1]);
    }
    return;
  }
  for (int idx = htid; idx < G * D; idx += NT) {
    int gq = idx / D, dd = idx % D;
    float v = (sm.red[0][gq][dd] + sm.red[1][gq][dd]) + (sm.red[2][gq][dd] + sm.red[3][gq][dd]);
    __stcg(mypart + gq * PSTRIDE + dd, v);
  }
  if (htid < G) __stcg(mypart + htid * PSTRIDE + D, sm.stat[htid][0]), __stcg(mypart + htid * PSTRIDE + D + 1, sm.stat[htid][1]);
  hsync();
  if (htid == 0) {
    __threadfence();
    int old = atomicAdd(p.acnt + pair, 1);
    sm.last = (old == n_chunks - 1);
    __threadfence();
  }
  hsync();
  if (sm.last) {
    const float* base = p.apart + (size_t)pair * p.max_chunks * G * PSTRIDE;
    for (int idx = htid; idx < G * D; idx += NT) {
      int gq = idx / D, dd = idx % D;
      float m = -INFINITY;
      for (int c0 = 0; c0 < n_chunks; c0 += 8) {
        float mm[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) mm[u] = (c0 + u < n_chunks) ? __ldcg(base + ((size_t)(c0 + u) * G + gq) * PSTRIDE + D) : -INFINITY;
#pragma unroll
        for (int u = 0; u < 8; ++u) m = fmaxf(m, mm[u]);
      }
      float lsum = 0.f, acc = 0.f;
      for (int c0 = 0; c0 < n_chunks; c0 += 8) {
        float mc[8], lc[8], oc[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const bool ok = c0 + u < n_chunks;
          const float* pc = base + ((size_t)(ok ? c0 + u : 0) * G + gq) * PSTRIDE;
          mc[u] = ok ? __ldcg(pc + D) : -INFINITY;
          lc[u] = ok ? __ldcg(pc + D + 1) : 0.f;
          oc[u] = ok ? __ldcg(pc + dd) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          float wgt = expf(mc[u] - m);
          lsum = fmaf(lc[u], wgt, lsum);
          acc = fmaf(oc[u], wgt, acc);
        }
      }
      store_split(p.aplanes + (size_t)row * 3 * HQ, HQ, (kvh * G + gq) * D + dd, acc / lsum);
    }
    if (htid == 0) p.acnt[pair] = 0;
  }
}

__host__ __device__ constexpr int pass_xbuf_uint4() { return 3 * PASS_XCH * 8 * 4; }
__host__ __device__ constexpr int pass_smem_bytes() {
  return PASS_RING * 2 * PASS_THREADS * 16 + pass_xbuf_uint4() * 16 + PASS_RECV_FLOATS * 4 + 16 * 4 + 64;
}

// all clusters arrive: one thread per cluster touches the counter, the cluster barrier fans the release out
template <typename Stamp>
__device__ __forceinline__ void pass_grid_barrier(const PassParams& p, cg::cluster_group& cluster, unsigned& generation, Stamp stamp) {
  __threadfence();  // this thread's global writes of the stage are ordered before the arrival
  stamp();
  cluster.sync();
  stamp();
  ++generation;
  if (cluster.block_rank() == 0 && threadIdx.x == 0) {
    volatile unsigned* bar = p.bar;
    if (bar[1] == 0) {
      const unsigned target = generation * (unsigned)p.n_clusters;
      __threadfence();
      atomicAdd(p.bar, 1u);
      unsigned spins = 0;
      while (bar[0] < target) {
        if (++spins > PASS_SPIN_LIMIT) {  // give up: flag it; every later barrier falls through
          bar[1] = 1;
          *p.err = 4;
          break;
        }
        __nanosleep(40);
      }
      __threadfence();
    }
  }
  stamp();
  cluster.sync();
}

template <int D, int G>
__global__ void __launch_bounds__(PASS_THREADS, 2) pass_kernel(const __grid_constant__ PassParams p) {
  constexpr int XCH = PASS_XCH;
  constexpr int PIECES = 3 * XCH * 8 * 4;
  constexpr int PPT = (PIECES + PASS_THREADS - 1) / PASS_THREADS;

  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4* ring = reinterpret_cast<uint4*>(smem_raw);               // [RING][2][256], slot of thread tid only
  uint4* xbuf = ring + PASS_RING * 2 * PASS_THREADS;                   // [3][XCH][8][4]
  float* recv = reinterpret_cast<float*>(xbuf + pass_xbuf_uint4());  // [8 * KH][nt][16]
  float* s_rstd = recv + PASS_RECV_FLOATS;                        // [8]
  float* s_red = s_rstd + 8;                                      // [8]
  AttnSmem* asm_ = reinterpret_cast<AttnSmem*>(xbuf);             // the activation buffer is idle during attention
  static_assert(2 * sizeof(AttnSmem) <= (size_t)pass_xbuf_uint4() * 16, "attention scratch must fit the activation buffer");

  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int rank = (int)cluster.block_rank(), cid = blockIdx.x / PASS_CS;

  // ---- weight ring, issue side: runs RING-1 units ahead of the consumer, across stages and layers.  Order of a
  // warp's units in a stage: k-blocks outermost, its row tiles innermost (the consumer below walks the same way).
  constexpr unsigned SLOT_BYTES = 2 * PASS_THREADS * 16, RING_MASK = PASS_RING * SLOT_BYTES - 1, HI_OFF = PASS_THREADS * 16;
  const unsigned ring_s = (unsigned)__cvta_generic_to_shared(ring) + tid * 16;
  unsigned i_slot = 0;
  int i_l = 0, i_st = 0, i_s = 0, i_n = 0, i_kleft = 0;
  bool i_done = false;
  const char* i_ptr = nullptr;
  long long i_tile_stride = 0, i_k_rewind = 0;
  auto i_enter = [&]() {  // first stage from (i_l, i_st) in which this warp has units
    for (;;) {
      if (i_l >= p.L) {
        i_done = true;
        return;
      }
      StageGeo ge;
      ge.set(p, i_st, cid, rank, warp);
      if (ge.my_nt > 0 && ge.nkb > 0) {
        const int kpr = p.kpr[i_st];
        const char* W = static_cast<const char*>(p.wpacked[i_l * 4 + i_st]);
        i_ptr = W + ((size_t)(ge.tile0(p, i_st) + ge.wg) * kpr + ge.kb0) * 1024 + lane * 16;
        i_tile_stride = (long long)ge.WG * kpr * 1024;                       // next row tile of this warp
        i_k_rewind = (long long)ge.KH * 1024 - (long long)ge.my_nt * i_tile_stride;  // back to the first tile, next k-block
        i_n = ge.my_nt, i_s = 0, i_kleft = ge.nkb;
        return;
      }
      if (++i_st == N_STAGES) i_st = 0, ++i_l;
    }
  };
  i_enter();
  auto issue_unit = [&]() {
    if (!i_done) {
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ring_s + i_slot), "l"(i_ptr) : "memory");
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ring_s + i_slot + HI_OFF), "l"(i_ptr + 512) : "memory");
      i_slot = (i_slot + SLOT_BYTES) & RING_MASK;
      i_ptr += i_tile_stride;
      if (++i_s == i_n) {
        i_s = 0, i_ptr += i_k_rewind;
        if (--i_kleft == 0) {
          if (++i_st == N_STAGES) i_st = 0, ++i_l;
          i_enter();
        }
      }
    }
    cp_async_commit();
  };
#pragma unroll
  for (int s = 0; s < PASS_RING - 1; ++s) issue_unit();

  pdl_launch_dependents();
  pdl_wait();

  const RowTable* tab = p.tab;
  const int n_cols = min(tab->n_rows, 8);
  if (n_cols <= 0) {  // every CTA takes this exit together: no barrier is ever entered
    cp_async_wait<0>();
    return;
  }
  unsigned generation = 0;
  unsigned c_slot = 0;
  int dbg_n = 0;
  auto stamp = [&]() {
    if (kTune && p.dbg && blockIdx.x == 0 && tid == 0) {
      unsigned long long tns;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(tns));
      p.dbg[dbg_n++] = tns;
    }
  };
  auto lds128 = [](unsigned addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
  };
  const unsigned xs_s = (unsigned)__cvta_generic_to_shared(xbuf) + (g * 4 + t) * 16;
  constexpr unsigned X_KB = 8 * 64, X_PLANE = XCH * 8 * 64;  // bytes per k-block / per plane in xbuf
  const int c_own = rank;  // the token column this CTA finishes
  const bool own = c_own < n_cols;

  for (int l = 0; l < p.L; ++l) {
    for (int st = 0; st < N_STAGES; ++st) {
      stamp();
      StageGeo ge;
      ge.set(p, st, cid, rank, warp);
      const int kpr = p.kpr[st], nt = ge.nt;
      const bool paired = p.paired[st] != 0;
      // ---- activations of this CTA's k-range -> MMA-fragment order (live columns only), 1/rms of the columns
      {
        const __nv_bfloat16* xsrc = st == ST_O ? p.aplanes : (st == ST_DOWN ? p.splanes : p.xplanes);
        const int x_ld = p.K[st];
#pragma unroll
        for (int i = 0; i < PPT; ++i) {
          const int idx = tid + i * PASS_THREADS;
          if (idx < PIECES) {
            const int tt = idx & 3, c = (idx >> 2) & 7, r = idx >> 5, kbl = r % XCH, s = r / XCH;
            const int k = (ge.kb_lo + kbl) * 32 + tt * 8;
            const bool ok = kbl < ge.upt && k < x_ld && c < n_cols;
            cp_async16(xbuf + idx, ok ? xsrc + ((size_t)c * 3 + s) * x_ld + k : xsrc, ok);
          }
        }
        cp_async_commit();
        stamp();
        const bool normed = (st == ST_QKV || st == ST_GU);
        {  // warp c sums the partial sums of squares of column c in a fixed order
          const int c = warp;
          float ss = 0.f;
          if (normed && c < n_cols) {
            const int n_sq = (st == ST_QKV && l == 0) ? 1 : p.n_clusters;
            for (int j = lane; j < n_sq; j += 32) ss += __ldcg(p.sumsq + c * p.sq_stride + j);
          }
          ss = warp_sum(ss);
          if (lane == 0) s_rstd[c] = normed ? 1.0f / sqrtf(ss / (float)p.H + p.eps) : 1.0f;
        }
        stamp();
        cp_async_wait<0>();
        stamp();
        __syncthreads();
        stamp();
      }
      // ---- main loop: this warp's row tiles over its k-blocks
      float acc[3][PASS_TPW][4];
#pragma unroll
      for (int h = 0; h < 3; ++h)
#pragma unroll
        for (int s = 0; s < PASS_TPW; ++s)
#pragma unroll
          for (int i = 0; i < 4; ++i) acc[h][s][i] = 0.f;
      {
        unsigned xk = xs_s + ge.khalf * X_KB;
        for (int kk = 0; kk < ge.nkb; ++kk) {
          const uint4 b0 = lds128(xk), b1 = lds128(xk + X_PLANE), b2 = lds128(xk + 2 * X_PLANE);
#pragma unroll
          for (int s = 0; s < PASS_TPW; ++s) {
            if (s < ge.my_nt) {
              issue_unit();
              cp_async_wait<PASS_RING - 1>();
              const uint4 a_lo = lds128(ring_s + c_slot), a_hi = lds128(ring_s + c_slot + HI_OFF);
              c_slot = (c_slot + SLOT_BYTES) & RING_MASK;
              mma_bf16(acc[0][s], a_lo.x, a_hi.x, a_lo.y, a_hi.y, b0.x, b0.y);
              mma_bf16(acc[0][s], a_lo.z, a_hi.z, a_lo.w, a_hi.w, b0.z, b0.w);
              mma_bf16(acc[1][s], a_lo.x, a_hi.x, a_lo.y, a_hi.y, b1.x, b1.y);
              mma_bf16(acc[1][s], a_lo.z, a_hi.z, a_lo.w, a_hi.w, b1.z, b1.w);
              mma_bf16(acc[2][s], a_lo.x, a_hi.x, a_lo.y, a_hi.y, b2.x, b2.y);
              mma_bf16(acc[2][s], a_lo.z, a_hi.z, a_lo.w, a_hi.w, b2.z, b2.w);
            }
          }
          xk += X_KB * ge.KH;
        }
      }
      stamp();
      // ---- the residual stream and next gain of this CTA's column are requested before the cluster barrier
      const bool resid = (st == ST_O || st == ST_DOWN);
      const float* gain_next = nullptr;
      if (st == ST_O) gain_next = static_cast<const float*>(p.layer_w[l * 6 + 3]);
      else if (st == ST_DOWN) gain_next = l + 1 < p.L ? static_cast<const float*>(p.layer_w[(l + 1) * 6 + 0]) : p.final_gain;
      float pre_h = 0.f, pre_g = 1.f;
      float* h_ptr = nullptr;
      const int n_glob = ge.g_lo * 16 + tid;  // single tiles: output row of thread tid
      const bool live1 = resid && own && tid < nt * 16;
      if (live1) {
        h_ptr = p.hid + (size_t)tab->hid_idx[c_own] * p.H + n_glob;
        pre_h = __ldcg(h_ptr);
        if (gain_next) pre_g = gain_next[n_glob];
      }
      // ---- push the partial tiles to the ranks that finish the columns (hi + (mid + lo), fixed order)
      {
        const int v = rank * ge.KH + ge.khalf;  // contribution index: k-ranges in ascending order
#pragma unroll
        for (int s = 0; s < PASS_TPW; ++s) {
          if (s < ge.my_nt) {
            const int i = ge.wg + s * ge.WG;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const int c = 2 * t + e;
              if (c < n_cols) {
                float* dst = cluster.map_shared_rank(recv, c) + ((size_t)v * nt + i) * 16 + g;
                dst[0] = acc[0][s][e] + (acc[1][s][e] + acc[2][s][e]);
                dst[8] = acc[0][s][2 + e] + (acc[1][s][2 + e] + acc[2][s][2 + e]);
              }
            }
          }
        }
      }
      stamp();
      cluster.sync();
      stamp();
      // ---- finish column c_own: sum the contributions in order, epilogue
      const int n_contrib = PASS_CS * ge.KH;
      if (resid) {
        float xn = 0.f;
        if (live1) {
          const float* src = recv + tid;
          float v = src[0];
          for (int q = 1; q < n_contrib; ++q) v += src[(size_t)q * nt * 16];
          xn = pre_h + v;
          *h_ptr = xn;
          if (gain_next) store_split(p.xplanes + (size_t)c_own * 3 * p.H, p.H, n_glob, xn * pre_g);
        }
        const float ss = warp_sum(xn * xn);
        if (lane == 0) s_red[warp] = ss;
        __syncthreads();
        if (own && tid == 0) {
          float tsum = 0.f;
          for (int w = 0; w < 8; ++w) tsum += s_red[w];
          p.sumsq[c_own * p.sq_stride + cid] = tsum;
        }
      } else if (own && tid < nt * 8) {
        const int gl = tid >> 4, r = tid & 15;
        const float* sa = recv + (2 * gl) * 16 + r;
        float a = sa[0], b = sa[16];
        for (int q = 1; q < n_contrib; ++q) a += sa[(size_t)q * nt * 16], b += sa[(size_t)q * nt * 16 + 16];
        a *= s_rstd[c_own], b *= s_rstd[c_own];
        const int grp = ge.g_lo + gl;
        if (st == ST_GU) {
          store_split(p.splanes + (size_t)c_own * 3 * p.F, p.F, grp * 16 + r, a / (1.0f + expf(-a)) * b);
        } else {  // QKV: group = (head, 16 rotary pairs); a, b are the two halves of the pairs
          constexpr int TH = D / 32, HD2 = D / 2;
          const int hh = grp / TH, i = (grp - hh * TH) * 16 + r;
          const int region = hh < p.n_q_heads ? 0 : (hh < p.n_q_heads + p.n_kv_heads ? 1 : 2);
          float y1 = a, y2 = b;
          if (region < 2) {
            const float2 csn = p.rope[(size_t)tab->pos[c_own] * HD2 + i];
            y1 = a * csn.x - b * csn.y;
            y2 = b * csn.x + a * csn.y;
          }
          if (region == 0) {
            float* q = p.qbuf + (size_t)c_own * p.Hq + hh * D + i;
            q[0] = y1;
            q[HD2] = y2;
          } else {
            const int head = hh - p.n_q_heads - (region == 2 ? p.n_kv_heads : 0);
            __nv_bfloat16* dst = p.kv + (size_t)l * p.kv_layer_stride + (size_t)(tab->r[c_own] - 1) * p.kv_plane_stride +
                                 (size_t)(region - 1) * p.kv_sel_stride +
                                 ((size_t)(tab->seq[c_own] * p.n_kv_heads + head) * p.slots + tab->kv_slot[c_own]) * D + i;
            dst[0] = __float2bfloat16_rn(y1);
            dst[HD2] = __float2bfloat16_rn(y2);
          }
        }
      }
      stamp();
      pass_grid_barrier(p, cluster, generation, stamp);
      // ================= attention (after the QKV stage) =================
      if (st == ST_QKV) {
        stamp();
        const int total_items = tab->attn_items * p.n_kv_heads;
        const int half = tid >> 7, htid = tid & 127;
        for (int item = (int)blockIdx.x * 2 + half; item < total_items; item += 2 * (int)gridDim.x)
          pass_attention_item<D, G>(p, tab, l, item, asm_[half], htid, 1 + half);
        stamp();
        pass_grid_barrier(p, cluster, generation, stamp);
      }
    }
  }
  cp_async_wait<0>();
  cluster.sync();  // nobody leaves while a sibling may still be addressed
}

}  // namespace ls

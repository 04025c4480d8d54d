// One persistent kernel for a whole batched pass through the shared block stack (Sec. 4.2 step 1): for every
// layer QKV -> attention -> O -> gate/up -> down, separated by grid barriers instead of kernel boundaries.
//
// Why: each of the 5 x L stages streams only 1.3-7 us worth of weights, so hand-over latency between stages
// decides the pass time.  Here every CTA walks a fixed, precomputed sequence of weight units (stream-K shares
// of every stage of every layer) and keeps RING units of it in flight in a thread-private cp.async ring that
// never drains at a stage boundary: while a CTA waits at a barrier or gathers activations, the weights of its
// next stage are already arriving.
//
// Every stage is cut into equal contiguous shares of (row block x k-block) units, one per CTA.  A row block
// shared by several CTAs is summed in fixed order by the CTA that finishes it last (a counter per row block),
// which then runs the stage's epilogue.  Data written by other CTAs is read with L2 loads (ld.global.cg).
// The barrier is a monotonic counter; a CTA that waits longer than a bound raises an error flag and leaves.
#pragma once
#include "common.cuh"
#include "gemm.cuh"

namespace ls {

constexpr int PASS_THREADS = 256;
constexpr int PASS_XCH = 24;           // k-blocks of activations staged at a time (NG = 1)
constexpr unsigned PASS_SPIN_LIMIT = 1u << 22;
enum { ST_QKV = 0, ST_O = 1, ST_GU = 2, ST_DOWN = 3, N_STAGES = 4 };

struct PassParams {
  const RowTable* tab;
  int L;
  const void* const* wpacked;   // device [L][4] tile-major weights: qkv, o, gate/up, down
  const void* const* layer_w;   // device [L][6] original pointers (norm gains: [0] norm1, [3] norm2)
  int H, Hq, Hkv, F, n_q_heads, n_kv_heads, head_dim, slots;
  float eps, scale;
  float* hid;
  __nv_bfloat16 *xplanes, *aplanes, *splanes;
  float* qbuf;
  float* sumsq;                 // [row][n_sq]
  int n_sq, sq_stride;
  __nv_bfloat16* kv;            // whole pool
  long long kv_layer_stride, kv_plane_stride, kv_sel_stride;
  const float2* rope;
  float* gpart;                 // split-k partial tiles [rb][max_contrib][8*NG][128]
  int* gcnt;                    // [max n_rb]
  float* apart;                 // attention partials
  int* acnt;
  int max_chunks;
  unsigned* bar;                // grid barrier counter, zero at launch
  volatile int* err;            // host-visible flag
  unsigned long long* dbg;      // optional: per-stage timestamps of CTA 0 (null in production)
  int n_rb[N_STAGES], kpr[N_STAGES], upc[N_STAGES], max_contrib[N_STAGES], N[N_STAGES], K[N_STAGES];
};

__device__ __forceinline__ int pass_row0(const PassParams& p, int st, int rb, int warp) {
  if (st == ST_GU) {
    int j = rb * 64 + (warp & 3) * 16;
    if (j >= p.F) return -1;
    return (warp < 4) ? j : p.F + j;
  }
  int r = rb * RB_ROWS + warp * 16;
  return r < p.N[st] ? r : -1;
}

// position of one CTA in its unit sequence: (layer, stage, unit) and the matching pointer into the packed weights
struct UnitCursor {
  int l, st, u, u_end, rb, kb;
  const __nv_bfloat16* ptr;
  bool ok, done;
  __device__ __forceinline__ void set_block(const PassParams& p, int warp, int lane) {
    rb = u / p.kpr[st];
    kb = u - rb * p.kpr[st];
    int r0 = pass_row0(p, st, rb, warp);
    ok = r0 >= 0;
    const __nv_bfloat16* W = static_cast<const __nv_bfloat16*>(p.wpacked[l * 4 + st]);
    ptr = W + (ok ? ((size_t)(r0 >> 4) * p.kpr[st] + kb) * 512 : 0) + lane * 8;
  }
  __device__ __forceinline__ void enter(const PassParams& p, int warp, int lane) {  // first non-empty stage from (l, st)
    for (;;) {
      if (l >= p.L) { done = true; return; }
      int total = p.n_rb[st] * p.kpr[st];
      u = min((int)blockIdx.x * p.upc[st], total);
      u_end = min(u + p.upc[st], total);
      if (u < u_end) { set_block(p, warp, lane); return; }
      if (++st == N_STAGES) st = 0, ++l;
    }
  }
  __device__ __forceinline__ void init(const PassParams& p, int warp, int lane) {
    l = 0, st = 0, done = false;
    enter(p, warp, lane);
  }
  __device__ __forceinline__ void next(const PassParams& p, int warp, int lane) {
    ++u, ptr += 512;
    if (u == u_end) {
      if (++st == N_STAGES) st = 0, ++l;
      enter(p, warp, lane);
    } else if (++kb == p.kpr[st]) {
      set_block(p, warp, lane);
    }
  }
};

// all CTAs arrive; returns false if the bound ran out (the kernel then leaves)
__device__ __forceinline__ bool grid_barrier(const PassParams& p, unsigned& generation, int* s_ok) {
  __syncthreads();
  if (threadIdx.x == 0) {
    ++generation;
    const unsigned target = generation * gridDim.x;
    __threadfence();
    atomicAdd(p.bar, 1u);
    unsigned spins = 0;
    int ok = 1;
    while (*reinterpret_cast<volatile unsigned*>(p.bar) < target) {
      if (++spins > PASS_SPIN_LIMIT) { ok = 0; *p.err = 4; break; }
      __nanosleep(20);
    }
    __threadfence();
    *s_ok = ok;
  }
  __syncthreads();
  return *s_ok != 0;
}

// ---- epilogue of a finished row block (tile [col][TILE_LD] in shared memory) ----------------------------------
__device__ __forceinline__ void pass_epilogue(const PassParams& p, const RowTable* tab, int l, int st, int rb, int n_cols,
                                              const float* tile, const float* s_rstd) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (st == ST_O || st == ST_DOWN) {
    const float* gain_next = nullptr;
    if (st == ST_O) gain_next = static_cast<const float*>(p.layer_w[l * 6 + 3]);
    else if (l + 1 < p.L) gain_next = static_cast<const float*>(p.layer_w[(l + 1) * 6 + 0]);
    const int n0 = rb * RB_ROWS;
    for (int c = warp; c < n_cols; c += PASS_THREADS / 32) {
      float4* h = reinterpret_cast<float4*>(p.hid + (size_t)tab->hid_idx[c] * p.H + n0) + lane;
      float4 v = __ldcg(h);
      const float* tr = tile + c * TILE_LD + lane * 4;
      v.x += tr[0], v.y += tr[1], v.z += tr[2], v.w += tr[3];
      *h = v;
      float ss = warp_sum(v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w);
      if (lane == 0) p.sumsq[c * p.sq_stride + rb] = ss;
      if (gain_next) {
        float4 gn = *reinterpret_cast<const float4*>(gain_next + n0 + lane * 4);
        float xv[4] = {v.x * gn.x, v.y * gn.y, v.z * gn.z, v.w * gn.w};
        unsigned short hh[4], mm[4], ll[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) split3(xv[i], hh[i], mm[i], ll[i]);
        __nv_bfloat16* dst = p.xplanes + (size_t)c * 3 * p.H + n0 + lane * 4;
        *reinterpret_cast<uint2*>(dst) = make_uint2(hh[0] | ((unsigned)hh[1] << 16), hh[2] | ((unsigned)hh[3] << 16));
        *reinterpret_cast<uint2*>(dst + p.H) = make_uint2(mm[0] | ((unsigned)mm[1] << 16), mm[2] | ((unsigned)mm[3] << 16));
        *reinterpret_cast<uint2*>(dst + 2 * p.H) = make_uint2(ll[0] | ((unsigned)ll[1] << 16), ll[2] | ((unsigned)ll[3] << 16));
      }
    }
  } else if (st == ST_GU) {
    const int j0 = rb * 64;
    for (int idx = tid; idx < n_cols * 64; idx += PASS_THREADS) {
      int c = idx >> 6, jj = idx & 63;
      if (j0 + jj < p.F) {
        float gt = tile[c * TILE_LD + jj] * s_rstd[c], up = tile[c * TILE_LD + 64 + jj] * s_rstd[c];
        store_split(p.splanes + (size_t)c * 3 * p.F, p.F, j0 + jj, gt / (1.0f + expf(-gt)) * up);
      }
    }
  } else {  // ST_QKV
    const int d = p.head_dim, hd2 = d >> 1;
    const int n0 = rb * RB_ROWS;
    const int region = n0 < p.Hq ? 0 : (n0 < p.Hq + p.Hkv ? 1 : 2);
    const int base = region == 0 ? 0 : (region == 1 ? p.Hq : p.Hq + p.Hkv);
    __nv_bfloat16* kvl = p.kv + (size_t)l * p.kv_layer_stride;
    for (int idx = tid; idx < n_cols * 64; idx += PASS_THREADS) {
      int c = idx >> 6, pr = idx & 63;
      int hh = pr / hd2, i = pr - hh * hd2;
      float x1 = tile[c * TILE_LD + hh * d + i] * s_rstd[c], x2 = tile[c * TILE_LD + hh * d + i + hd2] * s_rstd[c];
      float y1 = x1, y2 = x2;
      if (region < 2) {
        float2 cs = p.rope[(size_t)tab->pos[c] * hd2 + i];
        y1 = x1 * cs.x - x2 * cs.y;
        y2 = x2 * cs.x + x1 * cs.y;
      }
      int head = (n0 - base) / d + hh;
      if (region == 0) {
        float* q = p.qbuf + (size_t)c * p.Hq + head * d + i;
        q[0] = y1;
        q[hd2] = y2;
      } else {
        __nv_bfloat16* dst = kvl + (size_t)(tab->r[c] - 1) * p.kv_plane_stride + (size_t)(region - 1) * p.kv_sel_stride +
                             ((size_t)(tab->seq[c] * p.n_kv_heads + head) * p.slots + tab->kv_slot[c]) * d + i;
        dst[0] = __float2bfloat16_rn(y1);
        dst[hd2] = __float2bfloat16_rn(y2);
      }
    }
  }
}

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

__host__ __device__ constexpr int pass_xbuf_uint4(int NG) { return 3 * (PASS_XCH / NG) * 8 * NG * 4; }
__host__ __device__ constexpr int pass_smem_bytes(int NG) {
  return RING * 2 * PASS_THREADS * 16 + pass_xbuf_uint4(NG) * 16 + 8 * NG * TILE_LD * 4 + 8 * NG * 4 + 64;
}

template <int NG, int D, int G>
__global__ void __launch_bounds__(PASS_THREADS, 2) pass_kernel(const __grid_constant__ PassParams p) {
  constexpr int NTOK = 8 * NG;
  constexpr int XCH = PASS_XCH / NG;
  constexpr int PIECES = 3 * XCH * NTOK * 4;
  constexpr int PPT = (PIECES + PASS_THREADS - 1) / PASS_THREADS;

  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4* ring = reinterpret_cast<uint4*>(smem_raw);
  uint4* xbuf = ring + RING * 2 * PASS_THREADS;
  float* tile = reinterpret_cast<float*>(xbuf + pass_xbuf_uint4(NG));
  float* s_rstd = tile + NTOK * TILE_LD;
  AttnSmem* asm_ = reinterpret_cast<AttnSmem*>(xbuf);  // the activation buffer is idle during attention
  static_assert(2 * sizeof(AttnSmem) <= (size_t)pass_xbuf_uint4(NG) * 16, "attention scratch must fit the activation buffer");
  int* s_flag = reinterpret_cast<int*>(s_rstd + NTOK);
  int* s_ok = s_flag + 1;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;

  // ---- weight ring, issue side: runs RING-1 units ahead of the consumer, across stages and layers ----------------
  UnitCursor ic;
  ic.init(p, warp, lane);
  int i_cnt = 0;
  auto issue_unit = [&]() {
    if (!ic.done) {
      uint4* slot = ring + (i_cnt & (RING - 1)) * 2 * PASS_THREADS + tid;
      const __nv_bfloat16* W0 = static_cast<const __nv_bfloat16*>(p.wpacked[0]);
      cp_async16(slot, ic.ok ? ic.ptr : W0, ic.ok);
      cp_async16(slot + PASS_THREADS, ic.ok ? ic.ptr + 256 : W0, ic.ok);
      ++i_cnt;
      ic.next(p, warp, lane);
    }
    cp_async_commit();
  };
#pragma unroll
  for (int s = 0; s < RING - 1; ++s) issue_unit();

  pdl_launch_dependents();
  pdl_wait();

  const RowTable* tab = p.tab;
  int n_cols = min(tab->n_rows, NTOK);
  if (n_cols <= 0) {  // every CTA takes this exit together: no barrier is ever entered
    cp_async_wait<0>();
    return;
  }
  unsigned generation = 0;
  int j = 0;  // units consumed by this CTA so far (ring position)
  int dbg_n = 0;
  auto stamp = [&]() {
    if (p.dbg && blockIdx.x == 0 && tid == 0) {
      unsigned long long tns;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(tns));
      p.dbg[dbg_n++] = tns;
    }
  };

  for (int l = 0; l < p.L; ++l) {
    for (int st = 0; st < N_STAGES; ++st) {
      // ================= weight-streaming stage =================
      const int kpr = p.kpr[st], total = p.n_rb[st] * kpr, upc = p.upc[st];
      int u = min((int)blockIdx.x * upc, total);
      const int u_end = min(u + upc, total);
      stamp();
      if (u < u_end) {
        const __nv_bfloat16* xsrc = st == ST_O ? p.aplanes : (st == ST_DOWN ? p.splanes : p.xplanes);
        const int x_ld = p.K[st];
        const bool normed = (st == ST_QKV || st == ST_GU);
        if (tid < n_cols) {
          float r = 1.0f;
          if (normed) {
            const int n_sq = (st == ST_QKV && l == 0) ? 1 : p.n_sq;
            float ss = 0.f;
            for (int q = 0; q < n_sq; ++q) ss += __ldcg(p.sumsq + tid * p.sq_stride + q);
            r = 1.0f / sqrtf(ss / (float)p.H + p.eps);
          }
          s_rstd[tid] = r;
        }
        while (u < u_end) {
          const int rb = u / kpr, kb0 = u - rb * kpr;
          const int seg_len = min(kpr - kb0, u_end - u);
          const bool warp_valid = pass_row0(p, st, rb, warp) >= 0;
          float acc[3][NG][4];
#pragma unroll
          for (int h = 0; h < 3; ++h)
#pragma unroll
            for (int n = 0; n < NG; ++n)
#pragma unroll
              for (int i = 0; i < 4; ++i) acc[h][n][i] = 0.f;
          for (int ck = 0; ck < seg_len; ck += XCH) {
            const int nkb = min(XCH, seg_len - ck);
            uint4 xr[PPT];
#pragma unroll
            for (int i = 0; i < PPT; ++i) {
              const int idx = tid + i * PASS_THREADS;
              const int tt = idx & 3, c = (idx >> 2) % NTOK, r = idx / (4 * NTOK), kbl = r % XCH, s = r / XCH;
              const int k = (kb0 + ck + kbl) * 32 + tt * 8;
              xr[i] = make_uint4(0, 0, 0, 0);
              if (idx < PIECES && kbl < nkb && c < n_cols && k < x_ld)
                xr[i] = __ldcg(reinterpret_cast<const uint4*>(xsrc + ((size_t)c * 3 + s) * x_ld + k));
            }
            __syncthreads();  // everyone is done with the previous contents of xbuf
#pragma unroll
            for (int i = 0; i < PPT; ++i) {
              const int idx = tid + i * PASS_THREADS;
              if (idx < PIECES) xbuf[idx] = xr[i];
            }
            __syncthreads();
            const uint4* xs = xbuf + g * 4 + t;
            for (int kbl = 0; kbl < nkb; ++kbl, ++j) {
              issue_unit();
              cp_async_wait<RING - 1>();
              if (warp_valid) {
                const uint4* slot = ring + (j & (RING - 1)) * 2 * PASS_THREADS + tid;
                const uint4 a_lo = slot[0], a_hi = slot[PASS_THREADS];
#pragma unroll
                for (int s = 0; s < 3; ++s) {
#pragma unroll
                  for (int n = 0; n < NG; ++n) {
                    const uint4 b = xs[((s * XCH + kbl) * NTOK + n * 8) * 4];
                    mma_bf16(acc[s][n], a_lo.x, a_hi.x, a_lo.y, a_hi.y, b.x, b.y);
                    mma_bf16(acc[s][n], a_lo.z, a_hi.z, a_lo.w, a_hi.w, b.z, b.w);
                  }
                }
              }
            }
          }
          // ---- publish this share of the row block; the last CTA to arrive sums all shares and finishes it --------
          const int c_first = (rb * kpr) / upc, c_last = ((rb + 1) * kpr - 1) / upc;
          const int n_contrib = c_last - c_first + 1;
          const int rl = warp * 16 + g;
          float tot[NG][4];
#pragma unroll
          for (int n = 0; n < NG; ++n)
#pragma unroll
            for (int i = 0; i < 4; ++i) tot[n][i] = acc[0][n][i] + (acc[1][n][i] + acc[2][n][i]);
          bool finish = true;
          if (n_contrib == 1) {
#pragma unroll
            for (int n = 0; n < NG; ++n) {
              const int c0 = n * 8 + 2 * t;
              tile[c0 * TILE_LD + rl] = tot[n][0], tile[(c0 + 1) * TILE_LD + rl] = tot[n][1];
              tile[c0 * TILE_LD + rl + 8] = tot[n][2], tile[(c0 + 1) * TILE_LD + rl + 8] = tot[n][3];
            }
            __syncthreads();
          } else {
            float* dst = p.gpart + ((size_t)rb * p.max_contrib[st] + ((int)blockIdx.x - c_first)) * (NTOK * RB_ROWS);
#pragma unroll
            for (int n = 0; n < NG; ++n) {
              const int c0 = n * 8 + 2 * t;
              if (c0 < n_cols) {
                __stcg(dst + c0 * RB_ROWS + rl, tot[n][0]);
                __stcg(dst + c0 * RB_ROWS + rl + 8, tot[n][2]);
                if (c0 + 1 < n_cols) {
                  __stcg(dst + (c0 + 1) * RB_ROWS + rl, tot[n][1]);
                  __stcg(dst + (c0 + 1) * RB_ROWS + rl + 8, tot[n][3]);
                }
              }
            }
            __syncthreads();
            if (tid == 0) {
              __threadfence();
              int old = atomicAdd(p.gcnt + rb, 1);
              *s_flag = (old == n_contrib - 1);
              __threadfence();
            }
            __syncthreads();
            finish = *s_flag != 0;
            if (finish) {
              const float4* src = reinterpret_cast<const float4*>(p.gpart + (size_t)rb * p.max_contrib[st] * (NTOK * RB_ROWS));
              for (int idx = tid; idx < n_cols * (RB_ROWS / 4); idx += PASS_THREADS) {
                float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int o0 = 0; o0 < n_contrib; o0 += 4) {
                  float4 v4[4];
#pragma unroll
                  for (int q = 0; q < 4; ++q)
                    v4[q] = (o0 + q < n_contrib) ? __ldcg(src + (size_t)(o0 + q) * (NTOK * RB_ROWS / 4) + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                  for (int q = 0; q < 4; ++q) s4.x += v4[q].x, s4.y += v4[q].y, s4.z += v4[q].z, s4.w += v4[q].w;
                }
                const int c = idx / (RB_ROWS / 4), jj = (idx % (RB_ROWS / 4)) * 4;
                float* tr = tile + c * TILE_LD + jj;
                tr[0] = s4.x, tr[1] = s4.y, tr[2] = s4.z, tr[3] = s4.w;
              }
              if (tid == 0) p.gcnt[rb] = 0;
              __syncthreads();
            }
          }
          if (finish) pass_epilogue(p, tab, l, st, rb, n_cols, tile, s_rstd);
          __syncthreads();
          u += seg_len;
        }
      }
      stamp();
      if (!grid_barrier(p, generation, s_ok)) {
        cp_async_wait<0>();
        return;
      }
      stamp();
      // ================= attention (after the QKV stage) =================
      if (st == ST_QKV) {
        const int total_items = tab->attn_items * p.n_kv_heads;
        const int half = tid >> 7, htid = tid & 127;
        for (int item = (int)blockIdx.x * 2 + half; item < total_items; item += 2 * (int)gridDim.x)
          pass_attention_item<D, G>(p, tab, l, item, asm_[half], htid, 1 + half);
        stamp();
        if (!grid_barrier(p, generation, s_ok)) {
          cp_async_wait<0>();
          return;
        }
      }
    }
  }
  cp_async_wait<0>();
}

}  // namespace ls

// Decode attention over the depth-indexed KV cache (App. B "KV Cache Management"): a row advanced to
// recurrence r attends to the keys/values that its prefix produced at the SAME recurrence r -- the
// committed slots [0, n_canon) of plane r plus the speculative slots of its uncommitted ancestors and itself.
//
// Work item = (row, kv head, chunk of ATT_CHUNK key positions).  Chunks are cut at fixed absolute positions
// and combined in ascending order by the CTA that finishes a (row, kv head) last, so a row's result does
// not depend on what else is in the pass.  Softmax statistics are reduced with warp shuffles.
#pragma once
#include "common.cuh"

namespace ls {

constexpr int ATT_THREADS = 256;  // 8 warps per work item; at most 64 registers per thread so that the
                                   // neighbouring GEMM kernels' CTAs can be resident (and prefetching) alongside

struct AttnParams {
  const RowTable* tab;
  const float* qbuf;          // [row][n_q_heads * d], rotary applied, unscaled
  __nv_bfloat16* aplanes;     // out: three bf16 planes per row [row][3][n_q_heads * d]
  const __nv_bfloat16* kv;    // this layer's pool [R][2][S][n_kv][slots][d]
  long long kv_plane_stride, kv_sel_stride;
  int slots, n_kv_heads, n_q_heads;
  float scale;                // 1/sqrt(d)
  float* part;                // [row][n_kv][max_chunks][G][D + 2]
  int max_chunks;
  int* counters;              // [row][n_kv]
  long long* dbg;             // tuning aid: cycle stamps of CTA 0 / thread 0 (null in production)
  unsigned long long* tl;     // tuning aid: kernel timeline (null in production)
  int tl_id;
};

template <int D, int G>
__global__ void __launch_bounds__(ATT_THREADS, 4) attn_kernel(const __grid_constant__ AttnParams p) {
  constexpr int LPP = D / 8;            // lanes per key position (8 bf16 = 16 bytes per lane)
  constexpr int PPW = 32 / LPP;         // positions per warp per load
  constexpr int PPR = PPW * (ATT_THREADS / 32);  // positions per round of the whole CTA
  constexpr int NPOS = ATT_CHUNK + MAX_SPEC;     // the last chunk of a row also carries its speculative slots
  constexpr int ROUNDS = (NPOS + PPR - 1) / PPR;
  constexpr int PSTRIDE = D + 2;

  __shared__ float s_score[G][ROUNDS * PPR];
  __shared__ float s_red[ATT_THREADS / 32][G][D];
  __shared__ float s_stat[G][2];
  __shared__ int s_last;

  int dbg_n = 0;
  auto stamp = [&]() {
    if (kTune && p.dbg && blockIdx.x == 0 && threadIdx.x == 0) p.dbg[dbg_n++] = clock64();
  };
  stamp();
  timeline_mark(p.tl, p.tl_id, false);
  const RowTable* tab = p.tab;   // written before this pass started: safe to read ahead of the predecessor
  const int n_rows = tab->n_rows;
  const int HQ = p.n_q_heads * D;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int sub = lane / LPP, dl = lane % LPP;  // which position of the warp's group, which 8-dim slice
  const int total = tab->attn_items * p.n_kv_heads;
  bool waited = false;

  for (int item = blockIdx.x; item < total; item += gridDim.x) {
    const int kvh = item % p.n_kv_heads;
    const int rc = item / p.n_kv_heads;
    int row = 0;
    while (row + 1 < n_rows && tab->chunk_start[row + 1] <= rc) ++row;
    const int chunk = rc - tab->chunk_start[row];
    const int n_chunks = tab->chunk_start[row + 1] - tab->chunk_start[row];
    const int n_canon = tab->n_canon[row];
    const int p0 = chunk * ATT_CHUNK;
    const int n_can_here = min(ATT_CHUNK, n_canon - p0);
    const int n_spec = (chunk == n_chunks - 1) ? tab->n_spec[row] : 0;
    const int n_here = n_can_here + n_spec;
    // positions below n_safe were cached by earlier passes; the others are written by this pass's QKV kernel
    const int n_safe_can = min(n_can_here, max(0, tab->n_safe[row] - p0));
    const int n_safe = (n_spec > 0) ? n_can_here + n_spec - 1 : n_safe_can;

    const size_t plane = (size_t)(tab->r[row] - 1) * p.kv_plane_stride;
    const size_t headbase = (size_t)(tab->seq[row] * p.n_kv_heads + kvh) * p.slots * D;
    const __nv_bfloat16* Kb = p.kv + plane + headbase;
    const __nv_bfloat16* Vb = p.kv + plane + p.kv_sel_stride + headbase;

    auto slot_of = [&](int jpos) -> int { return jpos < n_can_here ? p0 + jpos : tab->spec_slot[row][jpos - n_can_here]; };
    uint4 kreg[ROUNDS], vreg[ROUNDS];
    auto load_kv = [&](int lo, int hi) {
#pragma unroll
      for (int rd = 0; rd < ROUNDS; ++rd) {
        const int jpos = rd * PPR + warp * PPW + sub;
        if (jpos >= lo && jpos < hi) {
          const size_t off = (size_t)slot_of(jpos) * D + dl * 8;
          kreg[rd] = *reinterpret_cast<const uint4*>(Kb + off);
          vreg[rd] = *reinterpret_cast<const uint4*>(Vb + off);
        }
      }
    };
#pragma unroll
    for (int rd = 0; rd < ROUNDS; ++rd) kreg[rd] = vreg[rd] = make_uint4(0, 0, 0, 0);
    stamp();
    load_kv(0, n_safe);
    stamp();
    if (!waited) {
      pdl_launch_dependents();
      pdl_wait();
      waited = true;
      timeline_mark(p.tl, p.tl_id + 256, false);
    }
    stamp();
    load_kv(n_safe, n_here);

    float q[G][8];
#pragma unroll
    for (int gq = 0; gq < G; ++gq) {
      const float4* qp =
          reinterpret_cast<const float4*>(p.qbuf + (size_t)row * p.n_q_heads * D + (size_t)(kvh * G + gq) * D + dl * 8);
      float4 a = qp[0], b = qp[1];
      q[gq][0] = a.x, q[gq][1] = a.y, q[gq][2] = a.z, q[gq][3] = a.w;
      q[gq][4] = b.x, q[gq][5] = b.y, q[gq][6] = b.z, q[gq][7] = b.w;
    }
    __syncthreads();  // shared buffers of the previous item are free
    stamp();

    // ---- scores ------------------------------------------------------------------------------------
#pragma unroll
    for (int rd = 0; rd < ROUNDS; ++rd) {
      const int jpos = rd * PPR + warp * PPW + sub;
      const unsigned w[4] = {kreg[rd].x, kreg[rd].y, kreg[rd].z, kreg[rd].w};
      float kf[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        kf[2 * i] = __uint_as_float(w[i] << 16);
        kf[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
      }
#pragma unroll
      for (int gq = 0; gq < G; ++gq) {
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) s = fmaf(q[gq][i], kf[i], s);
#pragma unroll
        for (int o = LPP / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (dl == 0) s_score[gq][jpos] = (jpos < n_here) ? s * p.scale : -INFINITY;
      }
    }
    __syncthreads();
    stamp();

    // ---- chunk softmax statistics (one warp per query head, round robin) ----------------------------
    for (int gq = warp; gq < G; gq += ATT_THREADS / 32) {
      float m = -INFINITY;
      for (int jj = lane; jj < ROUNDS * PPR; jj += 32) m = fmaxf(m, s_score[gq][jj]);
      m = warp_max(m);
      float l = 0.f;
      for (int jj = lane; jj < ROUNDS * PPR; jj += 32) {
        float e = (jj < n_here) ? expf(s_score[gq][jj] - m) : 0.f;
        s_score[gq][jj] = e;
        l += e;
      }
      l = warp_sum(l);
      if (lane == 0) s_stat[gq][0] = m, s_stat[gq][1] = l;
    }
    __syncthreads();
    stamp();

    // ---- weighted values ----------------------------------------------------------------------------
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
      for (int i = 0; i < 4; ++i) {
        vf[2 * i] = __uint_as_float(w[i] << 16);
        vf[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
      }
#pragma unroll
      for (int gq = 0; gq < G; ++gq) {
        float pw = s_score[gq][jpos];
#pragma unroll
        for (int i = 0; i < 8; ++i) o[gq][i] = fmaf(pw, vf[i], o[gq][i]);
      }
    }
    // fold the PPW position groups of the warp, then the warps, in fixed order
#pragma unroll
    for (int gq = 0; gq < G; ++gq)
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float v = o[gq][i];
#pragma unroll
        for (int off = LPP; off < 32; off <<= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        if (sub == 0) s_red[warp][gq][dl * 8 + i] = v;
      }
    __syncthreads();
    stamp();

    const int pair = row * p.n_kv_heads + kvh;
    float* mypart = p.part + ((size_t)pair * p.max_chunks + chunk) * G * PSTRIDE;
    if (n_chunks == 1) {
      for (int idx = tid; idx < G * D; idx += ATT_THREADS) {
        int gq = idx / D, dd = idx % D;
        float v = 0.f;
#pragma unroll
        for (int w2 = 0; w2 < ATT_THREADS / 32; ++w2) v += s_red[w2][gq][dd];
        store_split(p.aplanes + (size_t)row * 3 * HQ, HQ, (kvh * G + gq) * D + dd, v / s_stat[gq][1]);
      }
      continue;
    }
    for (int idx = tid; idx < G * D; idx += ATT_THREADS) {
      int gq = idx / D, dd = idx % D;
      float v = 0.f;
#pragma unroll
      for (int w2 = 0; w2 < ATT_THREADS / 32; ++w2) v += s_red[w2][gq][dd];
      __stcg(mypart + gq * PSTRIDE + dd, v);
    }
    if (tid < G) __stcg(mypart + tid * PSTRIDE + D, s_stat[tid][0]), __stcg(mypart + tid * PSTRIDE + D + 1, s_stat[tid][1]);
    __syncthreads();
    if (tid == 0) {
      __threadfence();
      int old = atomicAdd(p.counters + pair, 1);
      s_last = (old == n_chunks - 1);
      __threadfence();
    }
    __syncthreads();
    stamp();
    if (s_last) {  // combine the chunks in ascending order
      const float* base = p.part + (size_t)pair * p.max_chunks * G * PSTRIDE;
      for (int idx = tid; idx < G * D; idx += ATT_THREADS) {
        int gq = idx / D, dd = idx % D;
        float m = -INFINITY;
        for (int c0 = 0; c0 < n_chunks; c0 += 8) {
          float mm[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) mm[u] = (c0 + u < n_chunks) ? __ldcg(base + ((size_t)(c0 + u) * G + gq) * PSTRIDE + D) : -INFINITY;
#pragma unroll
          for (int u = 0; u < 8; ++u) m = fmaxf(m, mm[u]);
        }
        float l = 0.f, acc = 0.f;
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
            l = fmaf(lc[u], wgt, l);
            acc = fmaf(oc[u], wgt, acc);
          }
        }
        store_split(p.aplanes + (size_t)row * 3 * HQ, HQ, (kvh * G + gq) * D + dd, acc / l);
      }
      if (tid == 0) p.counters[pair] = 0;
    }
    stamp();
  }
  if (!waited) {
    pdl_launch_dependents();
    pdl_wait();
  }
  timeline_mark(p.tl, p.tl_id, true);
}

// The same attention for contexts of more than ATT_MAX_RUNS chunks: a work item is a run of consecutive chunks (a
// function of the row's own context only), folded one after the other with the usual softmax rescaling, so that the
// per-item costs (row lookup, partial write, counter) are paid once per run and a (row, kv head) never has more than
// ATT_MAX_RUNS partials.  Kept apart from attn_kernel, whose single-chunk items are the ones the batch-1 decode uses.
template <int D, int G>
__global__ void __launch_bounds__(ATT_THREADS, 4) attn_runs_kernel(const __grid_constant__ AttnParams p) {
  constexpr int LPP = D / 8;            // lanes per key position (8 bf16 = 16 bytes per lane)
  constexpr int PPW = 32 / LPP;         // positions per warp per load
  constexpr int PPR = PPW * (ATT_THREADS / 32);  // positions per round of the whole CTA
  constexpr int NPOS = ATT_CHUNK + MAX_SPEC;     // the last chunk of a row also carries its speculative slots
  constexpr int ROUNDS = (NPOS + PPR - 1) / PPR;
  constexpr int PSTRIDE = D + 2;

  __shared__ float s_score[G][ROUNDS * PPR];
  __shared__ float s_red[ATT_THREADS / 32][G][D];
  __shared__ float s_stat[G][2];
  __shared__ int s_last;

  int dbg_n = 0;
  auto stamp = [&]() {
    if (kTune && p.dbg && blockIdx.x == 0 && threadIdx.x == 0) p.dbg[dbg_n++] = clock64();
  };
  stamp();
  timeline_mark(p.tl, p.tl_id, false);
  const RowTable* tab = p.tab;   // written before this pass started: safe to read ahead of the predecessor
  const int n_rows = tab->n_rows;
  const int HQ = p.n_q_heads * D;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int sub = lane / LPP, dl = lane % LPP;  // which position of the warp's group, which 8-dim slice
  const int total = tab->attn_items * p.n_kv_heads;
  bool waited = false;

  constexpr int EPT = (G * D + ATT_THREADS - 1) / ATT_THREADS;  // output elements (head, dim) a thread folds
  for (int item = blockIdx.x; item < total; item += gridDim.x) {
    const int kvh = item % p.n_kv_heads;
    const int rr = item / p.n_kv_heads;
    int row = 0;
    {  // the row whose items contain rr (binary search over the prefix sums)
      int hi = n_rows - 1;
      while (row < hi) {
        const int mid = (row + hi + 1) >> 1;
        if (tab->chunk_start[mid] <= rr) row = mid;
        else hi = mid - 1;
      }
    }
    const int run = rr - tab->chunk_start[row];
    const int n_runs = tab->chunk_start[row + 1] - tab->chunk_start[row];
    const int n_canon = tab->n_canon[row];
    const int n_chunks = (n_canon + ATT_CHUNK - 1) / ATT_CHUNK;
    const int run_len = att_run_len(n_canon);
    const int chunk_lo = run * run_len, chunk_hi = min(n_chunks, chunk_lo + run_len);
    const int row_spec = tab->n_spec[row], row_safe = tab->n_safe[row];

    const size_t plane = (size_t)(tab->r[row] - 1) * p.kv_plane_stride;
    const size_t headbase = (size_t)(tab->seq[row] * p.n_kv_heads + kvh) * p.slots * D;
    const __nv_bfloat16* Kb = p.kv + plane + headbase;
    const __nv_bfloat16* Vb = p.kv + plane + p.kv_sel_stride + headbase;

    // running softmax state of the run, per output element of this thread: max, mass, weighted values
    float run_m[EPT], run_l[EPT], run_a[EPT];
    for (int chunk = chunk_lo; chunk < chunk_hi; ++chunk) {
      const int p0 = chunk * ATT_CHUNK;
      const int n_can_here = min(ATT_CHUNK, n_canon - p0);
      const int n_spec = (chunk == n_chunks - 1) ? row_spec : 0;
      const int n_here = n_can_here + n_spec;
      // positions below n_safe were cached by earlier passes; the others are written by this pass's QKV kernel
      const int n_safe_can = min(n_can_here, max(0, row_safe - p0));
      const int n_safe = (n_spec > 0) ? n_can_here + n_spec - 1 : n_safe_can;

      auto slot_of = [&](int jpos) -> int { return jpos < n_can_here ? p0 + jpos : tab->spec_slot[row][jpos - n_can_here]; };
      uint4 kreg[ROUNDS], vreg[ROUNDS];
      auto load_kv = [&](int lo, int hi) {
#pragma unroll
        for (int rd = 0; rd < ROUNDS; ++rd) {
          const int jpos = rd * PPR + warp * PPW + sub;
          if (jpos >= lo && jpos < hi) {
            const size_t off = (size_t)slot_of(jpos) * D + dl * 8;
            kreg[rd] = *reinterpret_cast<const uint4*>(Kb + off);
            vreg[rd] = *reinterpret_cast<const uint4*>(Vb + off);
          }
        }
      };
#pragma unroll
      for (int rd = 0; rd < ROUNDS; ++rd) kreg[rd] = vreg[rd] = make_uint4(0, 0, 0, 0);
      stamp();
      load_kv(0, n_safe);
      stamp();
      if (!waited) {
        pdl_launch_dependents();
        pdl_wait();
        waited = true;
        timeline_mark(p.tl, p.tl_id + 256, false);
      }
      stamp();
      load_kv(n_safe, n_here);

      float q[G][8];  // (re-read for every chunk of a run: a cache hit, and it keeps the registers free in between)
#pragma unroll
      for (int gq = 0; gq < G; ++gq) {
        const float4* qp =
            reinterpret_cast<const float4*>(p.qbuf + (size_t)row * p.n_q_heads * D + (size_t)(kvh * G + gq) * D + dl * 8);
        float4 a = qp[0], b = qp[1];
        q[gq][0] = a.x, q[gq][1] = a.y, q[gq][2] = a.z, q[gq][3] = a.w;
        q[gq][4] = b.x, q[gq][5] = b.y, q[gq][6] = b.z, q[gq][7] = b.w;
      }
      __syncthreads();  // shared buffers of the previous chunk are free
      stamp();

      // ---- scores ------------------------------------------------------------------------------------
#pragma unroll
      for (int rd = 0; rd < ROUNDS; ++rd) {
        const int jpos = rd * PPR + warp * PPW + sub;
        const unsigned w[4] = {kreg[rd].x, kreg[rd].y, kreg[rd].z, kreg[rd].w};
        float kf[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          kf[2 * i] = __uint_as_float(w[i] << 16);
          kf[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
#pragma unroll
        for (int gq = 0; gq < G; ++gq) {
          float s = 0.f;
#pragma unroll
          for (int i = 0; i < 8; ++i) s = fmaf(q[gq][i], kf[i], s);
#pragma unroll
          for (int o = LPP / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
          if (dl == 0) s_score[gq][jpos] = (jpos < n_here) ? s * p.scale : -INFINITY;
        }
      }
      __syncthreads();
      stamp();

      // ---- chunk softmax statistics (one warp per query head, round robin) ----------------------------
      for (int gq = warp; gq < G; gq += ATT_THREADS / 32) {
        float m = -INFINITY;
        for (int jj = lane; jj < ROUNDS * PPR; jj += 32) m = fmaxf(m, s_score[gq][jj]);
        m = warp_max(m);
        float l = 0.f;
        for (int jj = lane; jj < ROUNDS * PPR; jj += 32) {
          float e = (jj < n_here) ? expf(s_score[gq][jj] - m) : 0.f;
          s_score[gq][jj] = e;
          l += e;
        }
        l = warp_sum(l);
        if (lane == 0) s_stat[gq][0] = m, s_stat[gq][1] = l;
      }
      __syncthreads();
      stamp();

      // ---- weighted values ----------------------------------------------------------------------------
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
        for (int i = 0; i < 4; ++i) {
          vf[2 * i] = __uint_as_float(w[i] << 16);
          vf[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
#pragma unroll
        for (int gq = 0; gq < G; ++gq) {
          float pw = s_score[gq][jpos];
#pragma unroll
          for (int i = 0; i < 8; ++i) o[gq][i] = fmaf(pw, vf[i], o[gq][i]);
        }
      }
      // fold the PPW position groups of the warp, then the warps, in fixed order
#pragma unroll
      for (int gq = 0; gq < G; ++gq)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          float v = o[gq][i];
#pragma unroll
          for (int off = LPP; off < 32; off <<= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
          if (sub == 0) s_red[warp][gq][dl * 8 + i] = v;
        }
      __syncthreads();
      stamp();

      // ---- fold the chunk into the run: the first chunk is taken as it is, later ones by the usual rescaling ------
#pragma unroll
      for (int e = 0; e < EPT; ++e) {
        const int idx = tid + e * ATT_THREADS;
        if (idx < G * D) {
          const int gq = idx / D, dd = idx % D;
          float v = 0.f;
#pragma unroll
          for (int w2 = 0; w2 < ATT_THREADS / 32; ++w2) v += s_red[w2][gq][dd];
          const float m_c = s_stat[gq][0], l_c = s_stat[gq][1];
          if (chunk == chunk_lo) {
            run_m[e] = m_c, run_l[e] = l_c, run_a[e] = v;
          } else {
            const float mn = fmaxf(run_m[e], m_c), wa = expf(run_m[e] - mn), wb = expf(m_c - mn);
            run_a[e] = fmaf(run_a[e], wa, v * wb), run_l[e] = fmaf(run_l[e], wa, l_c * wb), run_m[e] = mn;
          }
        }
      }
    }

    const int pair = row * p.n_kv_heads + kvh;
    float* mypart = p.part + ((size_t)pair * p.max_chunks + run) * G * PSTRIDE;
    if (n_runs == 1) {
#pragma unroll
      for (int e = 0; e < EPT; ++e) {
        const int idx = tid + e * ATT_THREADS;
        if (idx < G * D) {
          const int gq = idx / D, dd = idx % D;
          store_split(p.aplanes + (size_t)row * 3 * HQ, HQ, (kvh * G + gq) * D + dd, run_a[e] / run_l[e]);
        }
      }
      continue;
    }
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
      const int idx = tid + e * ATT_THREADS;
      if (idx < G * D) {
        const int gq = idx / D, dd = idx % D;
        __stcg(mypart + gq * PSTRIDE + dd, run_a[e]);
        if (dd == 0) __stcg(mypart + gq * PSTRIDE + D, run_m[e]), __stcg(mypart + gq * PSTRIDE + D + 1, run_l[e]);
      }
    }
    __syncthreads();
    if (tid == 0) {
      __threadfence();
      int old = atomicAdd(p.counters + pair, 1);
      s_last = (old == n_runs - 1);
      __threadfence();
    }
    __syncthreads();
    stamp();
    if (s_last) {  // combine the runs in ascending order
      const int n_chunks = n_runs;  // (partials per pair)
      const float* base = p.part + (size_t)pair * p.max_chunks * G * PSTRIDE;
      for (int idx = tid; idx < G * D; idx += ATT_THREADS) {
        int gq = idx / D, dd = idx % D;
        float m = -INFINITY;
        for (int c0 = 0; c0 < n_chunks; c0 += 8) {
          float mm[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) mm[u] = (c0 + u < n_chunks) ? __ldcg(base + ((size_t)(c0 + u) * G + gq) * PSTRIDE + D) : -INFINITY;
#pragma unroll
          for (int u = 0; u < 8; ++u) m = fmaxf(m, mm[u]);
        }
        float l = 0.f, acc = 0.f;
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
            l = fmaf(lc[u], wgt, l);
            acc = fmaf(oc[u], wgt, acc);
          }
        }
        store_split(p.aplanes + (size_t)row * 3 * HQ, HQ, (kvh * G + gq) * D + dd, acc / l);
      }
      if (tid == 0) p.counters[pair] = 0;
    }
    stamp();
  }
  if (!waited) {
    pdl_launch_dependents();
    pdl_wait();
  }
  timeline_mark(p.tl, p.tl_id, true);
}

}  // namespace ls

// Decode attention over the depth-indexed KV cache (App. B "KV Cache Management"): a row advanced to
// recurrence r attends to the keys/values that its prefix produced at the SAME recurrence r -- the
// committed slots [0, n_canon) of plane r plus the speculative slots of its uncommitted ancestors and itself.
//
// Three kernels, by regime:
//   attn_kernel          work item = (row, kv head, chunk of ATT_CHUNK key positions): every chunk in parallel, for the few
//                        rows and short contexts of a single sequence's decode pass (latency matters);
//   attn_runs_kernel     work item = (row, kv head, run of chunks) streamed through a per-thread cp.async ring: long
//                        contexts and contexts of several sequences (bandwidth matters);
//   attn_prefill_mma_kernel  work item = (query head, block of rows, run of chunks) for the consecutive positions of a prefill
//                        pass, which share their keys and values.
// Chunks and runs are cut at fixed absolute positions (or as a function of the row's own context) and folded in
// ascending order, so a row's result does not depend on what else is in the pass.
#pragma once
#include "common.cuh"

namespace ls {

// 16-byte asynchronous copy into shared memory; !valid: the 16 bytes are zero-filled and nothing is read
__device__ __forceinline__ void cp_async16_zfill(void* smem_dst, const void* gsrc, bool valid) {
  const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
  const int n = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(gsrc), "r"(n) : "memory");
}

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

// The same attention for contexts whose rows can have more chunks than single-chunk items are cut for (more than
// ATT_MAX_RUNS chunks; more than ATT_BATCH_SINGLE in contexts of several sequences): a work item is a run of consecutive
// chunks (a function of the row's own context only), so that the per-item costs (row lookup, partial write, counter) are paid
// once per run and a (row, kv head) never has more than ATT_MAX_RUNS partials.  This is the kernel of the KV-bound
// regime, built to stream: every thread owns a ring of (key piece, value piece) slots in shared memory that it fills
// with cp.async and reads back itself, so the K/V of the next rounds are in flight while the current one is used and
// the main loop has no block-wide barrier.  A key position is shared by the D/8 lanes of a group, 8 dims each (groups
// of 4 lanes with D/4 dims each need fewer shuffles and softmax updates per byte but leave too few warps to hide
// their longer dependent chains: 3.6 TB/s against 5.6 TB/s measured on 34 rows x 8192 positions).  Each lane group keeps
// a running softmax (max, mass, weighted values) over the positions it is dealt - position j of a chunk always goes
// to group j mod PPR - the groups of a warp are folded by a fixed butterfly, the warps in ascending order, once per
// run.  Kept apart from attn_kernel, whose single-chunk items are the ones the batch-1 decode uses.
template <int D, int G>
struct AtsCfg {
  static constexpr int NP = 1;                     // 16-byte pieces of a key (and of a value) per lane
  static constexpr int DPL = 8 * NP;               // dims per lane
  static constexpr int LPP = D / DPL;              // lanes per key position
  static constexpr int PPW = 32 / LPP;             // positions per warp per round
  static constexpr int PPR = PPW * (ATT_THREADS / 32);  // positions per round of the whole CTA
  static constexpr int UNIT_BYTES = 2 * NP * ATT_THREADS * 16;  // one round of the CTA: K and V pieces of every thread
  static constexpr int MIN_CTAS = G == 1 ? 4 : 2;  // per SM (grouped-query attention keeps G accumulators per lane)
  static constexpr int UNITS = (G == 1 ? 48 : 96) * 1024 / UNIT_BYTES;  // ring depth: 48 KB in flight per CTA
  static constexpr int COMB_BYTES = (ATT_THREADS / 32) * G * (D + 2) * 4;
  static constexpr int SMEM_BYTES = UNITS * UNIT_BYTES + COMB_BYTES;
};

template <int D, int G>
__global__ void __launch_bounds__(ATT_THREADS, (AtsCfg<D, G>::MIN_CTAS)) attn_runs_kernel(const __grid_constant__ AttnParams p) {
  using C = AtsCfg<D, G>;
  constexpr int NP = C::NP, DPL = C::DPL, LPP = C::LPP, PPW = C::PPW, PPR = C::PPR, UNITS = C::UNITS;
  constexpr int PSTRIDE = D + 2;
  constexpr int EPT = (G * D + ATT_THREADS - 1) / ATT_THREADS;  // output elements (head, dim) a thread folds
  constexpr unsigned PIECE = ATT_THREADS * 16, V_OFF = NP * PIECE, UNIT_BYTES = C::UNIT_BYTES, RING_BYTES = UNITS * UNIT_BYTES;

  extern __shared__ __align__(16) unsigned char ats_smem[];
  float* s_comb = reinterpret_cast<float*>(ats_smem + RING_BYTES);  // [warp][G][PSTRIDE]
  __shared__ int s_last;

  timeline_mark(p.tl, p.tl_id, false);
  const RowTable* tab = p.tab;   // written before this pass started: safe to read ahead of the predecessor
  const int n_rows = tab->n_rows;
  const int HQ = p.n_q_heads * D;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int sub = lane / LPP, dl = lane % LPP;  // which position of the warp's group, which DPL-dim slice
  const int jl = warp * PPW + sub;              // this lane group's position within a round
  const int total = tab->attn_items * p.n_kv_heads;
  const unsigned ring_s = (unsigned)__cvta_generic_to_shared(ats_smem) + tid * 16;
  bool waited = false;

  struct Cursor {  // a round of a chunk of the run, with the chunk's geometry
    int chunk, rd, n_can, n_here, n_safe, rounds;
  };
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
    const int run_len = att_run_len(n_canon, tab->att_mode);
    const int chunk_lo = run * run_len, chunk_hi = min(n_chunks, chunk_lo + run_len);
    const int row_spec = tab->n_spec[row], row_safe = tab->n_safe[row];

    const size_t plane = (size_t)(tab->r[row] - 1) * p.kv_plane_stride;
    const size_t headbase = (size_t)(tab->seq[row] * p.n_kv_heads + kvh) * p.slots * D;
    const __nv_bfloat16* Kb = p.kv + plane + headbase + dl * DPL;
    const __nv_bfloat16* Vb = Kb + p.kv_sel_stride;

    auto setup = [&](Cursor& c, int chunk) {
      const int p0 = chunk * ATT_CHUNK;
      const int n_spec = (chunk == n_chunks - 1) ? row_spec : 0;  // the last chunk of a row also carries its speculative slots
      c.chunk = chunk, c.rd = 0;
      c.n_can = min(ATT_CHUNK, n_canon - p0);
      c.n_here = c.n_can + n_spec;
      // positions below n_safe were cached by earlier passes; the others are written by this pass's QKV kernel
      c.n_safe = (n_spec > 0) ? c.n_can + n_spec - 1 : min(c.n_can, max(0, row_safe - p0));
      c.rounds = (c.n_here + PPR - 1) / PPR;
    };
    auto advance = [&](Cursor& c) {
      if (++c.rd == c.rounds) {
        if (c.chunk + 1 < chunk_hi) setup(c, c.chunk + 1);
        else c.chunk = chunk_hi;
      }
    };
    // ---- ring, issue side: one unit = this thread's pieces of a key and of a value of one round ------------------
    Cursor ic;
    setup(ic, chunk_lo);
    unsigned i_slot = 0, c_slot = 0;
    auto issue = [&]() {
      if (ic.chunk < chunk_hi) {
        const int jpos = ic.rd * PPR + jl;
        if (jpos < ic.n_here) {
          const int slot = jpos < ic.n_can ? ic.chunk * ATT_CHUNK + jpos : tab->spec_slot[row][jpos - ic.n_can];
          const size_t off = (size_t)slot * D;
#pragma unroll
          for (int pc = 0; pc < NP; ++pc) {
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ring_s + i_slot + pc * PIECE), "l"(Kb + off + pc * 8) : "memory");
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ring_s + i_slot + V_OFF + pc * PIECE), "l"(Vb + off + pc * 8)
                         : "memory");
          }
        }
        advance(ic);
      }
      i_slot += UNIT_BYTES;
      if (i_slot == RING_BYTES) i_slot = 0;
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    int issued = 0;
    if (!waited) {
      // rounds whose positions were all cached by earlier passes are requested ahead of the predecessor's completion
      while (issued < UNITS - 1 && ic.chunk < chunk_hi && min((ic.rd + 1) * PPR, ic.n_here) <= ic.n_safe) issue(), ++issued;
      pdl_launch_dependents();
      pdl_wait();
      waited = true;
      timeline_mark(p.tl, p.tl_id + 256, false);
    }
    for (; issued < UNITS - 1; ++issued) issue();

    float q[G][DPL];
#pragma unroll
    for (int gq = 0; gq < G; ++gq) {
      const float4* qp =
          reinterpret_cast<const float4*>(p.qbuf + (size_t)row * p.n_q_heads * D + (size_t)(kvh * G + gq) * D + dl * DPL);
#pragma unroll
      for (int i = 0; i < DPL / 4; ++i) {
        const float4 a = qp[i];
        q[gq][4 * i] = a.x, q[gq][4 * i + 1] = a.y, q[gq][4 * i + 2] = a.z, q[gq][4 * i + 3] = a.w;
      }
    }

    // ---- main loop: running softmax of this lane group over its positions of the run ----------------------------
    float gm[G], gl[G], o[G][DPL];
#pragma unroll
    for (int gq = 0; gq < G; ++gq) {
      gm[gq] = -INFINITY, gl[gq] = 0.f;
#pragma unroll
      for (int i = 0; i < DPL; ++i) o[gq][i] = 0.f;
    }
    auto lds128 = [](unsigned addr) {
      uint4 v;
      asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
      return v;
    };
    Cursor cc;
    setup(cc, chunk_lo);
    while (cc.chunk < chunk_hi) {
      issue();
      asm volatile("cp.async.wait_group %0;" ::"n"(UNITS - 1) : "memory");
      const bool valid = cc.rd * PPR + jl < cc.n_here;
      float sc[G];
#pragma unroll
      for (int gq = 0; gq < G; ++gq) sc[gq] = 0.f;
#pragma unroll
      for (int pc = 0; pc < NP; ++pc) {  // one chain per piece, folded in piece order
        const uint4 kk = valid ? lds128(ring_s + c_slot + pc * PIECE) : make_uint4(0, 0, 0, 0);
        const unsigned kw[4] = {kk.x, kk.y, kk.z, kk.w};
        float sp[G];
#pragma unroll
        for (int gq = 0; gq < G; ++gq) sp[gq] = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float k0 = __uint_as_float(kw[i] << 16), k1 = __uint_as_float(kw[i] & 0xffff0000u);
#pragma unroll
          for (int gq = 0; gq < G; ++gq) sp[gq] = fmaf(q[gq][pc * 8 + 2 * i + 1], k1, fmaf(q[gq][pc * 8 + 2 * i], k0, sp[gq]));
        }
#pragma unroll
        for (int gq = 0; gq < G; ++gq) sc[gq] += sp[gq];
      }
      float wb[G];
#pragma unroll
      for (int gq = 0; gq < G; ++gq) {
#pragma unroll
        for (int off = LPP / 2; off > 0; off >>= 1) sc[gq] += __shfl_xor_sync(0xffffffffu, sc[gq], off);  // (every lane takes part)
        wb[gq] = 0.f;
        if (valid) {
          const float sv = sc[gq] * p.scale;
          if (sv > gm[gq]) {  // a new maximum: rescale what has been gathered (the first position finds -inf: weight 0)
            const float wa = expf(gm[gq] - sv);
            gl[gq] *= wa;
#pragma unroll
            for (int i = 0; i < DPL; ++i) o[gq][i] *= wa;
            gm[gq] = sv;
          }
          wb[gq] = expf(sv - gm[gq]);
          gl[gq] += wb[gq];
        }
      }
      if (valid) {
#pragma unroll
        for (int pc = 0; pc < NP; ++pc) {
          const uint4 vv = lds128(ring_s + c_slot + V_OFF + pc * PIECE);
          const unsigned vw[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float v0 = __uint_as_float(vw[i] << 16), v1 = __uint_as_float(vw[i] & 0xffff0000u);
#pragma unroll
            for (int gq = 0; gq < G; ++gq) {
              o[gq][pc * 8 + 2 * i] = fmaf(wb[gq], v0, o[gq][pc * 8 + 2 * i]);
              o[gq][pc * 8 + 2 * i + 1] = fmaf(wb[gq], v1, o[gq][pc * 8 + 2 * i + 1]);
            }
          }
        }
      }
      c_slot += UNIT_BYTES;
      if (c_slot == RING_BYTES) c_slot = 0;
      advance(cc);
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");  // (only empty groups are left)

    // ---- fold the lane groups of a warp: a butterfly in which the lower lane's state always comes first ---------
#pragma unroll
    for (int off = LPP; off < 32; off <<= 1) {
      const bool upper = (lane & off) != 0;
#pragma unroll
      for (int gq = 0; gq < G; ++gq) {
        const float m2 = __shfl_xor_sync(0xffffffffu, gm[gq], off), l2 = __shfl_xor_sync(0xffffffffu, gl[gq], off);
        const float ma = upper ? m2 : gm[gq], mb = upper ? gm[gq] : m2;  // a: the lower lane's state
        const float la = upper ? l2 : gl[gq], lb = upper ? gl[gq] : l2;
        const float mn = fmaxf(ma, mb);
        const float wa = ma == -INFINITY ? 0.f : expf(ma - mn), wb2 = mb == -INFINITY ? 0.f : expf(mb - mn);
        gl[gq] = fmaf(la, wa, lb * wb2), gm[gq] = mn;
#pragma unroll
        for (int i = 0; i < DPL; ++i) {
          const float o2 = __shfl_xor_sync(0xffffffffu, o[gq][i], off);
          const float oa = upper ? o2 : o[gq][i], ob = upper ? o[gq][i] : o2;
          o[gq][i] = fmaf(oa, wa, ob * wb2);
        }
      }
    }
    // ---- ... and the warps in ascending order -----------------------------------------------------------------
    __syncthreads();  // the previous item's readers are done with s_comb
    if (sub == 0) {
#pragma unroll
      for (int gq = 0; gq < G; ++gq) {
        float* dst = s_comb + ((size_t)warp * G + gq) * PSTRIDE;
#pragma unroll
        for (int i = 0; i < DPL; ++i) dst[dl * DPL + i] = o[gq][i];
        if (dl == 0) dst[D] = gm[gq], dst[D + 1] = gl[gq];
      }
    }
    __syncthreads();
    float run_m[EPT], run_l[EPT], run_a[EPT];
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
      const int idx = tid + e * ATT_THREADS;
      run_m[e] = -INFINITY, run_l[e] = 0.f, run_a[e] = 0.f;
      if (idx < G * D) {
        const int gq = idx / D, dd = idx % D;
        const float* src = s_comb + (size_t)gq * PSTRIDE;
        float m = -INFINITY;
#pragma unroll
        for (int w2 = 0; w2 < ATT_THREADS / 32; ++w2) m = fmaxf(m, src[(size_t)w2 * G * PSTRIDE + D]);
        float l = 0.f, acc = 0.f;
#pragma unroll
        for (int w2 = 0; w2 < ATT_THREADS / 32; ++w2) {
          const float* pc = src + (size_t)w2 * G * PSTRIDE;
          const float wgt = pc[D] == -INFINITY ? 0.f : expf(pc[D] - m);  // a warp that was dealt no position
          l = fmaf(pc[D + 1], wgt, l);
          acc = fmaf(pc[dd], wgt, acc);
        }
        run_m[e] = m, run_l[e] = l, run_a[e] = acc;
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
    if (s_last) {  // combine the runs in ascending order
      const float* base = p.part + (size_t)pair * p.max_chunks * G * PSTRIDE;
      for (int idx = tid; idx < G * D; idx += ATT_THREADS) {
        int gq = idx / D, dd = idx % D;
        float m = -INFINITY;
        for (int c0 = 0; c0 < n_runs; c0 += 8) {
          float mm[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) mm[u] = (c0 + u < n_runs) ? __ldcg(base + ((size_t)(c0 + u) * G + gq) * PSTRIDE + D) : -INFINITY;
#pragma unroll
          for (int u = 0; u < 8; ++u) m = fmaxf(m, mm[u]);
        }
        float l = 0.f, acc = 0.f;
        for (int c0 = 0; c0 < n_runs; c0 += 8) {
          float mc[8], lc[8], oc[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const bool ok = c0 + u < n_runs;
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
  }
  if (!waited) {
    pdl_launch_dependents();
    pdl_wait();
  }
  timeline_mark(p.tl, p.tl_id, true);
}

// ======================= prefill attention: the rows of a pass share every key / value chunk ========================
// A prefill pass carries consecutive prompt positions p0 .. p0 + n - 1 of one sequence at one recurrence, so all its rows
// read the same cached keys and values (row i up to its own position).  A work item is (query head, block of 32 rows, run
// of chunks): a chunk's keys and values are brought into shared memory once for the block, and every row keeps a running
// softmax over the chunks of the run.  Runs are cut at fixed absolute positions - every chunk below position
// ATT_PF_SINGLE * 64 is a run of its own, beyond that runs of ATT_PF_RUN chunks - and a row's runs are folded in ascending
// order by a second kernel (attn_prefill_fold_kernel), so a row's result depends on its own prefix only, not on how the
// prompt was cut into passes.
constexpr int ATT_PF_SINGLE = 8;  // [measured per layer at 2048 / 4096 / 8192 positions, 64 rows: single chunks up to 8 and runs of 4
constexpr int ATT_PF_RUN = 4;     //  beyond: 43 / 68 / 106 us; up to 16: 47 / 66 / 120 us; up to 40: 51 / 78 / 133 us; runs of 8: slower]
__host__ __device__ inline int att_pf_run_of_chunk(int c) { return c < ATT_PF_SINGLE ? c : ATT_PF_SINGLE + (c - ATT_PF_SINGLE) / ATT_PF_RUN; }
__host__ __device__ inline int att_pf_run_first_chunk(int run) {
  return run < ATT_PF_SINGLE ? run : ATT_PF_SINGLE + (run - ATT_PF_SINGLE) * ATT_PF_RUN;
}
constexpr int ATT_PF_ROWS = 64;  // rows of a pass at most (one group of token columns)

// Scores and weighted values of a (32 rows x 64 keys) tile are mma.sync.m16n8k16 contractions (bf16 x bf16 -> fp32).  Keys
// and values are bf16 already; the fp32 queries and the fp32 softmax weights are split exactly into three bf16 planes
// (hi + mid + lo), one accumulator chain per plane, folded hi + (mid + lo) - the arithmetic of the GEMM kernels, so every
// product is exact and a row's result depends on its own operands only (not on its place in the tile, nor on the other
// rows).  (The same tiles as fp32 FMAs in registers took 29 us per layer at 512 positions and 211 us at 8192 against 18 us
// and 134 us here.)
template <int D>
struct AtmCfg {
  static constexpr int IR = 32;                 // rows per item: two 16-row MMA tiles
  static constexpr int QS = D + 8;              // bf16 per row of a query plane (the pad keeps fragment loads off each other's banks)
  static constexpr int KS = D + 8;              // bf16 per key / value row
  static constexpr int PS = ATT_CHUNK + 8;      // bf16 per row of a softmax-weight plane
  static constexpr int SS = ATT_CHUNK + 1;      // floats per score row
  static constexpr int Q_OFF = 0;                                   // [3][IR][QS] bf16
  static constexpr int K_OFF = Q_OFF + 3 * IR * QS * 2;             // [64][KS] bf16
  static constexpr int V_OFF = K_OFF + ATT_CHUNK * KS * 2;          // [64][KS] bf16
  static constexpr int P_OFF = V_OFF + ATT_CHUNK * KS * 2;          // [3][IR][PS] bf16
  static constexpr int S_OFF = P_OFF + 3 * IR * PS * 2;             // [IR][SS] fp32
  static constexpr int ST_OFF = S_OFF + IR * SS * 4;                // [IR][4] fp32
  static constexpr int SMEM_BYTES = ST_OFF + IR * 4 * 4;
};

__device__ __forceinline__ void att_mma(float (&c)[4], const unsigned (&a)[4], unsigned b0, unsigned b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int D>
__global__ void __launch_bounds__(ATT_THREADS, 2) attn_prefill_mma_kernel(const __grid_constant__ AttnParams p) {
  using C = AtmCfg<D>;
  constexpr int IR = C::IR, PSTRIDE = D + 2;
  constexpr int NTO = D / 32;  // 8-dim output tiles per warp (each warp: one 16-row tile x NTO column tiles)
  extern __shared__ __align__(16) unsigned char atm_smem[];
  __nv_bfloat16* s_q = reinterpret_cast<__nv_bfloat16*>(atm_smem + C::Q_OFF);
  __nv_bfloat16* s_k = reinterpret_cast<__nv_bfloat16*>(atm_smem + C::K_OFF);
  __nv_bfloat16* s_v = reinterpret_cast<__nv_bfloat16*>(atm_smem + C::V_OFF);
  __nv_bfloat16* s_p = reinterpret_cast<__nv_bfloat16*>(atm_smem + C::P_OFF);
  float* s_s = reinterpret_cast<float*>(atm_smem + C::S_OFF);
  float* s_st = reinterpret_cast<float*>(atm_smem + C::ST_OFF);  // [row][4]: running max, running mass, rescale of this chunk

  const RowTable* tab = p.tab;  // written before this pass started
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int n_rows = min(tab->n_rows, ATT_PF_ROWS);
  pdl_launch_dependents();
  pdl_wait();  // the queries, and the keys / values of the pass's own positions, come from this pass's QKV kernel
  if (n_rows <= 0) return;
  const int p0 = tab->pos[0], seq = tab->seq[0];
  const int n_ctx = p0 + n_rows;                                   // keys 0 .. n_ctx - 1
  const int n_runs_all = att_pf_run_of_chunk((n_ctx - 1) / ATT_CHUNK) + 1;
  const int n_blocks = (n_rows + IR - 1) / IR;
  const int G = p.n_q_heads / p.n_kv_heads, HQ = p.n_q_heads * D;
  const size_t plane = (size_t)(tab->r[0] - 1) * p.kv_plane_stride;
  const int total = p.n_q_heads * n_blocks * n_runs_all;
  const int mt = warp & 1;   // this warp's 16-row tile
  const int wq = warp >> 1;  // ... and its quarter of the columns (keys of the score tile, dims of the output tile)

  for (int item = blockIdx.x; item < total; item += gridDim.x) {
    const int h = item % p.n_q_heads, rest = item / p.n_q_heads;
    const int blk = rest % n_blocks, run = rest / n_blocks;
    const int row0 = blk * IR, rows_here = min(IR, n_rows - row0);  // this item's rows of the pass
    const int kvh = h / G, gq = h - kvh * G;
    const int c_lo = att_pf_run_first_chunk(run);
    // keys beyond the block's last position are never visible to it: the run ends there
    const int c_hi = min(att_pf_run_first_chunk(run + 1), (p0 + row0 + rows_here - 1) / ATT_CHUNK + 1);
    if (c_lo >= c_hi) continue;  // (uniform over the CTA) none of the block's rows reaches this run
    const __nv_bfloat16* Kb = p.kv + plane + (size_t)(seq * p.n_kv_heads + kvh) * p.slots * D;
    const __nv_bfloat16* Vb = Kb + p.kv_sel_stride;
    __syncthreads();  // the previous item is done with the shared buffers
    // the block's queries for this head, split into three bf16 planes; rows the pass does not have are zeros
    for (int idx = tid; idx < IR * (D / 4); idx += ATT_THREADS) {
      const int lr = idx / (D / 4), d4 = idx - lr * (D / 4);
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (lr < rows_here) v = *reinterpret_cast<const float4*>(p.qbuf + (size_t)(row0 + lr) * HQ + (size_t)h * D + d4 * 4);
      const float x[4] = {v.x, v.y, v.z, v.w};
      unsigned short hh[4], mm[4], ll[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) split3(x[i], hh[i], mm[i], ll[i]);
      __nv_bfloat16* q0 = s_q + lr * C::QS + d4 * 4;
      *reinterpret_cast<uint2*>(q0) = make_uint2(hh[0] | ((unsigned)hh[1] << 16), hh[2] | ((unsigned)hh[3] << 16));
      *reinterpret_cast<uint2*>(q0 + IR * C::QS) = make_uint2(mm[0] | ((unsigned)mm[1] << 16), mm[2] | ((unsigned)mm[3] << 16));
      *reinterpret_cast<uint2*>(q0 + 2 * IR * C::QS) = make_uint2(ll[0] | ((unsigned)ll[1] << 16), ll[2] | ((unsigned)ll[3] << 16));
    }
    if (tid < IR) s_st[tid * 4] = -INFINITY, s_st[tid * 4 + 1] = 0.f, s_st[tid * 4 + 2] = 1.f;
    float o[NTO][4];  // running weighted values: rows 16 mt + g (elements 0, 1) and + 8 (2, 3), dims 8 (wq NTO + j) + 2 t, + 1
#pragma unroll
    for (int j = 0; j < NTO; ++j)
#pragma unroll
      for (int i = 0; i < 4; ++i) o[j][i] = 0.f;

    for (int chunk = c_lo; chunk < c_hi; ++chunk) {
      const int k0 = chunk * ATT_CHUNK;
      const int n_keys = min(ATT_CHUNK, n_ctx - k0);  // keys of this chunk that exist (all of them written)
      if (chunk > c_lo) __syncthreads();               // the previous chunk's readers are done
      // ---- the chunk's keys and values, once for all rows of the block (missing keys: zeros) ----------------------
      for (int idx = tid; idx < ATT_CHUNK * (D / 8); idx += ATT_THREADS) {
        const int key = idx / (D / 8), pc = idx - key * (D / 8);
        const bool ok = key < n_keys;
        const size_t off = (size_t)(k0 + (ok ? key : 0)) * D + pc * 8;
        cp_async16_zfill(s_k + key * C::KS + pc * 8, Kb + off, ok);
        cp_async16_zfill(s_v + key * C::KS + pc * 8, Vb + off, ok);
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      __syncthreads();
      // ---- scores: this warp's 16 rows x 16 keys (two 8-key tiles), three plane chains each --------------------------
      {
        float acc[3][2][4];
#pragma unroll
        for (int pl = 0; pl < 3; ++pl)
#pragma unroll
          for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[pl][j][i] = 0.f;
#pragma unroll 2
        for (int ks = 0; ks < D / 16; ++ks) {
          unsigned a[3][4];
#pragma unroll
          for (int pl = 0; pl < 3; ++pl) {
            const __nv_bfloat16* qa = s_q + (pl * IR + 16 * mt + g) * C::QS + 16 * ks + 2 * t;
            a[pl][0] = *reinterpret_cast<const unsigned*>(qa), a[pl][1] = *reinterpret_cast<const unsigned*>(qa + 8 * C::QS);
            a[pl][2] = *reinterpret_cast<const unsigned*>(qa + 8), a[pl][3] = *reinterpret_cast<const unsigned*>(qa + 8 * C::QS + 8);
          }
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const __nv_bfloat16* kb = s_k + (8 * (2 * wq + j) + g) * C::KS + 16 * ks + 2 * t;
            const unsigned b0 = *reinterpret_cast<const unsigned*>(kb), b1 = *reinterpret_cast<const unsigned*>(kb + 8);
#pragma unroll
            for (int pl = 0; pl < 3; ++pl) att_mma(acc[pl][j], a[pl], b0, b1);
          }
        }
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int lr = 16 * mt + g + (i >> 1) * 8, key = 8 * (2 * wq + j) + 2 * t + (i & 1);
            const float sv = acc[0][j][i] + (acc[1][j][i] + acc[2][j][i]);
            const bool ok = lr < rows_here && key < n_keys && k0 + key <= p0 + row0 + lr;  // causal
            s_s[lr * C::SS + key] = ok ? sv * p.scale : -INFINITY;
          }
      }
      __syncthreads();
      // ---- running softmax of every row: four threads per row, 16 keys each, folded in a fixed order; the weights go
      // to three bf16 planes for the second contraction -------------------------------------------------------------
      if (tid < 4 * IR) {
        const int lr = tid >> 2, part = tid & 3;
        const float* sr = s_s + lr * C::SS + part * 16;
        float m = -INFINITY;
#pragma unroll
        for (int jj = 0; jj < 16; ++jj) m = fmaxf(m, sr[jj]);
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
        const float m_old = s_st[lr * 4], l_old = s_st[lr * 4 + 1];
        const float m_new = fmaxf(m_old, m);
        float l = 0.f;
#pragma unroll
        for (int jj = 0; jj < 16; jj += 2) {
          const float e0 = (sr[jj] == -INFINITY) ? 0.f : expf(sr[jj] - m_new);
          const float e1 = (sr[jj + 1] == -INFINITY) ? 0.f : expf(sr[jj + 1] - m_new);
          l += e0;
          l += e1;
          unsigned short h0, m0, l0, h1, m1, l1;
          split3(e0, h0, m0, l0);
          split3(e1, h1, m1, l1);
          __nv_bfloat16* pp = s_p + lr * C::PS + part * 16 + jj;
          *reinterpret_cast<unsigned*>(pp) = h0 | ((unsigned)h1 << 16);
          *reinterpret_cast<unsigned*>(pp + IR * C::PS) = m0 | ((unsigned)m1 << 16);
          *reinterpret_cast<unsigned*>(pp + 2 * IR * C::PS) = l0 | ((unsigned)l1 << 16);
        }
        const float l1s = __shfl_xor_sync(0xffffffffu, l, 1);
        const float lp = (part & 1) ? l1s + l : l + l1s;       // (part 0 + part 1), (part 2 + part 3)
        const float l2s = __shfl_xor_sync(0xffffffffu, lp, 2);
        const float lc = (part & 2) ? l2s + lp : lp + l2s;     // lower pair first
        __syncwarp();
        if (part == 0) {
          const float wa = (m_old == -INFINITY) ? 0.f : expf(m_old - m_new);  // (a row that has seen no key yet: nothing to rescale)
          s_st[lr * 4] = m_new, s_st[lr * 4 + 1] = fmaf(l_old, wa, lc), s_st[lr * 4 + 2] = (m_new == -INFINITY) ? 1.f : wa;
        }
      }
      __syncthreads();
      // ---- weighted values: this warp's 16 rows x NTO tiles of 8 dims, keys in four steps of 16 ---------------------------
      {
        float acc[3][NTO][4];
#pragma unroll
        for (int pl = 0; pl < 3; ++pl)
#pragma unroll
          for (int j = 0; j < NTO; ++j)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[pl][j][i] = 0.f;
#pragma unroll
        for (int ks = 0; ks < ATT_CHUNK / 16; ++ks) {
          unsigned a[3][4];
#pragma unroll
          for (int pl = 0; pl < 3; ++pl) {
            const __nv_bfloat16* pa = s_p + (pl * IR + 16 * mt + g) * C::PS + 16 * ks + 2 * t;
            a[pl][0] = *reinterpret_cast<const unsigned*>(pa), a[pl][1] = *reinterpret_cast<const unsigned*>(pa + 8 * C::PS);
            a[pl][2] = *reinterpret_cast<const unsigned*>(pa + 8), a[pl][3] = *reinterpret_cast<const unsigned*>(pa + 8 * C::PS + 8);
          }
#pragma unroll
          for (int j = 0; j < NTO; ++j) {
            // B fragment of V[key][dim] (keys = the contraction index): transposing matrix load, lanes 0-15 name the key rows
            const unsigned addr = (unsigned)__cvta_generic_to_shared(s_v + (16 * ks + (lane & 15)) * C::KS + 8 * (wq * NTO + j));
            unsigned b0, b1;
            asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];" : "=r"(b0), "=r"(b1) : "r"(addr));
#pragma unroll
            for (int pl = 0; pl < 3; ++pl) att_mma(acc[pl][j], a[pl], b0, b1);
          }
        }
        const float wa0 = s_st[(16 * mt + g) * 4 + 2], wa1 = s_st[(16 * mt + g + 8) * 4 + 2];
#pragma unroll
        for (int j = 0; j < NTO; ++j)
#pragma unroll
          for (int i = 0; i < 4; ++i)
            o[j][i] = fmaf(o[j][i], (i >> 1) ? wa1 : wa0, acc[0][j][i] + (acc[1][j][i] + acc[2][j][i]));
      }
    }
    __syncthreads();  // every thread has read the final state
    // ---- the run is done: rows with one run only are finished here, the others leave a partial for the fold -----------
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      const int lr = 16 * mt + g + 8 * hf, row = row0 + lr, pos = p0 + row;
      if (lr >= rows_here || c_lo * ATT_CHUNK > pos) continue;   // the row does not reach this run
      const int n_runs_row = att_pf_run_of_chunk(pos / ATT_CHUNK) + 1;
      const float m = s_st[lr * 4], l = s_st[lr * 4 + 1];
      float* mypart = p.part + (((size_t)(row * p.n_kv_heads + kvh) * p.max_chunks + run) * G + gq) * PSTRIDE;
#pragma unroll
      for (int j = 0; j < NTO; ++j)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int dd = 8 * (wq * NTO + j) + 2 * t + e;
          const float v = o[j][2 * hf + e];
          if (n_runs_row == 1) store_split(p.aplanes + (size_t)row * 3 * HQ, HQ, h * D + dd, v / l);
          else __stcg(mypart + dd, v);
        }
      if (n_runs_row > 1 && wq == 0 && t == 0) __stcg(mypart + D, m), __stcg(mypart + D + 1, l);
    }
  }
}

// ... and the fold of a row's runs, in ascending order: one CTA per (row, query head), one lane per four dims.  A
// kernel of its own so that the folds of a pass (up to 64 rows x all heads x up to ATT_PF_SINGLE + max_ctx / 1024 runs)
// spread over the whole device instead of queuing in whichever CTA finished a head last.
template <int D>
__global__ void __launch_bounds__(D / 4) attn_prefill_fold_kernel(const __grid_constant__ AttnParams p) {
  constexpr int PSTRIDE = D + 2;
  const RowTable* tab = p.tab;
  const int row = blockIdx.x, h = blockIdx.y, tid = threadIdx.x;
  pdl_launch_dependents();
  pdl_wait();
  if (row >= min(tab->n_rows, ATT_PF_ROWS)) return;
  const int n_runs = att_pf_run_of_chunk(tab->pos[row] / ATT_CHUNK) + 1;
  if (n_runs == 1) return;  // finished by the attention kernel itself
  const int G = p.n_q_heads / p.n_kv_heads, HQ = p.n_q_heads * D, kvh = h / G, gq = h - kvh * G;
  const float* base = p.part + ((size_t)(row * p.n_kv_heads + kvh) * p.max_chunks * G + gq) * PSTRIDE;
  const size_t rstride = (size_t)G * PSTRIDE;
  float m = -INFINITY;
  for (int c0 = 0; c0 < n_runs; c0 += 8) {
    float mm[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) mm[u] = (c0 + u < n_runs) ? __ldcg(base + (size_t)(c0 + u) * rstride + D) : -INFINITY;
#pragma unroll
    for (int u = 0; u < 8; ++u) m = fmaxf(m, mm[u]);
  }
  float l = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int c0 = 0; c0 < n_runs; c0 += 8) {
    float mc[8], lc[8];
    float2 oa[8], ob[8];  // (a partial's D + 2 floats keep 8-byte alignment only)
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const bool ok = c0 + u < n_runs;
      const float* pc = base + (size_t)(ok ? c0 + u : 0) * rstride;
      mc[u] = ok ? __ldcg(pc + D) : -INFINITY, lc[u] = ok ? __ldcg(pc + D + 1) : 0.f;
      oa[u] = ok ? __ldcg(reinterpret_cast<const float2*>(pc + tid * 4)) : make_float2(0.f, 0.f);
      ob[u] = ok ? __ldcg(reinterpret_cast<const float2*>(pc + tid * 4 + 2)) : make_float2(0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const float wgt = (mc[u] == -INFINITY) ? 0.f : expf(mc[u] - m);
      l = fmaf(lc[u], wgt, l);
      acc[0] = fmaf(oa[u].x, wgt, acc[0]), acc[1] = fmaf(oa[u].y, wgt, acc[1]);
      acc[2] = fmaf(ob[u].x, wgt, acc[2]), acc[3] = fmaf(ob[u].y, wgt, acc[3]);
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) store_split(p.aplanes + (size_t)row * 3 * HQ, HQ, h * D + tid * 4 + i, acc[i] / l);
}

}  // namespace ls

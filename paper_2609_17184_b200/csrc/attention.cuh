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

constexpr int ATT_THREADS = 128;

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
};

template <int D, int G>
__global__ void __launch_bounds__(ATT_THREADS) attn_kernel(const __grid_constant__ AttnParams p) {
  constexpr int LPP = D / 8;            // lanes per key position (8 bf16 = 16 bytes per lane)
  constexpr int PPW = 32 / LPP;         // positions per warp per load
  constexpr int PPR = PPW * (ATT_THREADS / 32);  // positions per round of the whole CTA
  constexpr int ROUNDS = ATT_CHUNK / PPR;
  constexpr int PSTRIDE = D + 2;

  __shared__ float s_score[G][ATT_CHUNK];
  __shared__ float s_red[ATT_THREADS / 32][G][D];
  __shared__ float s_stat[G][2];
  __shared__ int s_slot[ATT_CHUNK];
  __shared__ int s_last;

  pdl_launch_dependents();
  pdl_wait();
  const RowTable* tab = p.tab;
  const int n_rows = tab->n_rows;
  if (n_rows <= 0) return;
  const int HQ = p.n_q_heads * D;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int sub = lane / LPP, dl = lane % LPP;  // which position of the warp's group, which 8-dim slice
  const int total = tab->attn_items * p.n_kv_heads;

  for (int item = blockIdx.x; item < total; item += gridDim.x) {
    const int kvh = item % p.n_kv_heads;
    const int rc = item / p.n_kv_heads;
    int row = 0;
    while (row + 1 < n_rows && tab->chunk_start[row + 1] <= rc) ++row;
    const int chunk = rc - tab->chunk_start[row];
    const int n_chunks = tab->chunk_start[row + 1] - tab->chunk_start[row];
    const int n_canon = tab->n_canon[row], n_spec = tab->n_spec[row];
    const int n_canon_chunks = (n_canon + ATT_CHUNK - 1) / ATT_CHUNK;
    const bool spec_chunk = chunk >= n_canon_chunks;
    const int p0 = chunk * ATT_CHUNK;
    const int n_here = spec_chunk ? n_spec : min(ATT_CHUNK, n_canon - p0);

    __syncthreads();  // shared buffers of the previous item are free
    if (tid < ATT_CHUNK) s_slot[tid] = tid < n_here ? (spec_chunk ? tab->spec_slot[row][tid] : p0 + tid) : 0;

    const size_t plane = (size_t)(tab->r[row] - 1) * p.kv_plane_stride;
    const size_t headbase = (size_t)(tab->seq[row] * p.n_kv_heads + kvh) * p.slots * D;
    const __nv_bfloat16* Kb = p.kv + plane + headbase;
    const __nv_bfloat16* Vb = p.kv + plane + p.kv_sel_stride + headbase;

    float q[G][8];
#pragma unroll
    for (int gq = 0; gq < G; ++gq) {
      const float4* qp =
          reinterpret_cast<const float4*>(p.qbuf + (size_t)row * p.n_q_heads * D + (size_t)(kvh * G + gq) * D + dl * 8);
      float4 a = qp[0], b = qp[1];
      q[gq][0] = a.x, q[gq][1] = a.y, q[gq][2] = a.z, q[gq][3] = a.w;
      q[gq][4] = b.x, q[gq][5] = b.y, q[gq][6] = b.z, q[gq][7] = b.w;
    }
    __syncthreads();

    // ---- scores ------------------------------------------------------------------------------------
    uint4 kreg[ROUNDS];
#pragma unroll
    for (int rd = 0; rd < ROUNDS; ++rd) {
      int j = rd * PPR + warp * PPW + sub;
      kreg[rd] = make_uint4(0, 0, 0, 0);
      if (j < n_here) kreg[rd] = *reinterpret_cast<const uint4*>(Kb + (size_t)s_slot[j] * D + dl * 8);
    }
#pragma unroll
    for (int rd = 0; rd < ROUNDS; ++rd) {
      int j = rd * PPR + warp * PPW + sub;
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
        if (dl == 0) s_score[gq][j] = (j < n_here) ? s * p.scale : -INFINITY;
      }
    }
    __syncthreads();

    // ---- chunk softmax statistics (one warp per query head, round robin) ----------------------------
    for (int gq = warp; gq < G; gq += ATT_THREADS / 32) {
      float m = -INFINITY;
      for (int j = lane; j < ATT_CHUNK; j += 32) m = fmaxf(m, s_score[gq][j]);
      m = warp_max(m);
      float l = 0.f;
      for (int j = lane; j < ATT_CHUNK; j += 32) {
        float e = (j < n_here) ? expf(s_score[gq][j] - m) : 0.f;
        s_score[gq][j] = e;
        l += e;
      }
      l = warp_sum(l);
      if (lane == 0) s_stat[gq][0] = m, s_stat[gq][1] = l;
    }
    __syncthreads();

    // ---- weighted values ----------------------------------------------------------------------------
    float o[G][8];
#pragma unroll
    for (int gq = 0; gq < G; ++gq)
#pragma unroll
      for (int i = 0; i < 8; ++i) o[gq][i] = 0.f;
#pragma unroll
    for (int rd = 0; rd < ROUNDS; ++rd) {
      int j = rd * PPR + warp * PPW + sub;
      kreg[rd] = make_uint4(0, 0, 0, 0);
      if (j < n_here) kreg[rd] = *reinterpret_cast<const uint4*>(Vb + (size_t)s_slot[j] * D + dl * 8);
    }
#pragma unroll
    for (int rd = 0; rd < ROUNDS; ++rd) {
      int j = rd * PPR + warp * PPW + sub;
      const unsigned w[4] = {kreg[rd].x, kreg[rd].y, kreg[rd].z, kreg[rd].w};
      float vf[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        vf[2 * i] = __uint_as_float(w[i] << 16);
        vf[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
      }
#pragma unroll
      for (int gq = 0; gq < G; ++gq) {
        float pw = s_score[gq][j];
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
      mypart[gq * PSTRIDE + dd] = v;
    }
    if (tid < G) mypart[tid * PSTRIDE + D] = s_stat[tid][0], mypart[tid * PSTRIDE + D + 1] = s_stat[tid][1];
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      int old = atomicAdd(p.counters + pair, 1);
      s_last = (old == n_chunks - 1);
    }
    __syncthreads();
    if (s_last) {
      __threadfence();
      const float* base = p.part + (size_t)pair * p.max_chunks * G * PSTRIDE;
      for (int idx = tid; idx < G * D; idx += ATT_THREADS) {
        int gq = idx / D, dd = idx % D;
        float m = -INFINITY;
        for (int c = 0; c < n_chunks; ++c) m = fmaxf(m, __ldcg(base + ((size_t)c * G + gq) * PSTRIDE + D));
        float l = 0.f, acc = 0.f;
        for (int c = 0; c < n_chunks; ++c) {
          const float* pc = base + ((size_t)c * G + gq) * PSTRIDE;
          float wgt = expf(__ldcg(pc + D) - m);
          l = fmaf(__ldcg(pc + D + 1), wgt, l);
          acc = fmaf(__ldcg(pc + dd), wgt, acc);
        }
        store_split(p.aplanes + (size_t)row * 3 * HQ, HQ, (kvh * G + gq) * D + dd, acc / l);
      }
      if (tid == 0) p.counters[pair] = 0;
    }
  }
}

}  // namespace ls

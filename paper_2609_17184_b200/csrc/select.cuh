// Readout decisions of one step: first-proposal draft at d1 (Sec. 4.2 step 2), gate and residual second
// proposal at d2 (Eq. 5-6), cascade verification at R (Sec. 4.3; Algorithm 1 Verify), and the plain draw
// x ~ C(H) used by prefill and vanilla decoding.  One thread-block cluster per reading-out row: every CTA of
// the cluster scans its slice of the vocabulary (a single SM ingests a 196 KB logits row in ~4 us, and the
// sampled paths make several passes over up to three rows), and every reduction over the vocabulary is a
// fixed-order block reduction followed by a fixed-order sum of the CTAs' partials exchanged through
// distributed shared memory - so all CTAs of a cluster hold the same values and take the same branches.
//
// Random draws (the paper only says "x ~ q", "U ~ U(0,1)"): Philox4x32-10 keyed by the seed with counter
// (block, position being decided, sequence, purpose); u = ((word >> 9) + 0.5) * 2^-23; categorical draws
// by the exponential race argmax_v log w_v - log(-log u_v) with ties to the lowest index.
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"

namespace ls {
namespace cg = cooperative_groups;

constexpr int SEL_THREADS = 512;
constexpr int SEL_CS = 8;  // CTAs per reading-out row
constexpr int SEL_NV = 7;  // values reduced together in the nucleus search (3 bits of the cut per pass)
constexpr int SEL_ARG_BLOCK = 128;  // vocabulary rows per argmax partial of the lm_head epilogue
enum { PUR_DRAFT1 = 1, PUR_DRAFT2 = 2, PUR_ACCEPT1 = 3, PUR_ACCEPT2 = 4, PUR_RESAMPLE = 5, PUR_VANILLA = 6 };

struct SelectParams {
  const RowTable* tab;
  const float* logits;  // [logit_idx][V]
  int V, NB;
  NodeTable nodes;
  float temperature;
  int gate, residual_q2;
  int mask_first;       // second-proposal ablation: the first candidate is removed from the second proposal
  unsigned long long seed;
  int kinds_mask;       // bit k set: handle readout kind k
  int* sel_tok;         // per row: drafted / committed token
  int* sel_aux;         // RO_D2: gate open; RO_VERIFY: source 1/2/3
  float* sel_lse;       // RO_D1 / RO_D2: log-sum-exp of z/T
  float* sel_z2;        // RO_D2: normaliser of the residual proposal (0: the proposal is q2~ itself)
  const float2* argpart;  // [readout column][row block]: per-block largest logit and its index, written by the lm_head
  int n_rb;
  // optional filters of C (Sec. 3.1), used when temperature > 0: keep the top_k most probable tokens (0: all), then
  // the shortest prefix of the ranking whose mass reaches top_p (>= 1: all).  The kernel then needs V floats of
  // dynamic shared memory.
  int top_k;
  float top_p;
  int staged;           // 1: dynamic shared memory holds 3 row slices (+1 when filtering) of ceil(V/4/8)*4 floats each
  double* tv_acc;       // [seq][4]: sum and count of TV(p_d1, p_R), sum and count of TV(p_d2, p_R); null: not measured
  float4* sel_flt;      // per row: the nucleus of its readout (max of z/T, kept mass, cut value bits, cut index)
};

// A readout distribution C(H): softmax(z / T), optionally cut to a nucleus.  Ranking: decreasing e = exp(z/T - m)
// (as fp32 bit patterns), ties to the lower index; the nucleus is everything ranked at or before (ecut, vcut).
struct Dist {
  const float* z;   // the logits row in global memory (any index)
  const float* zs;  // the same row for indices of this CTA's vocabulary slice: a shared-memory copy when staged
  float lse;      // unfiltered: log sum_v exp(z_v / T)
  float m, s;     // filtered: max_v z_v / T and the mass of the kept exp(z_v / T - m)
  unsigned ecut;
  int vcut;
  bool filt;
  __device__ __forceinline__ bool kept(unsigned eb, int v) const { return eb > ecut || (eb == ecut && v <= vcut); }
  __device__ __forceinline__ float prob_of(float zv, int v, float T) const {
    if (!filt) return expf(zv / T - lse);
    const float e = expf(zv / T - m);
    return kept(__float_as_uint(e), v) ? e / s : 0.f;
  }
  __device__ __forceinline__ float prob(int v, float T) const { return prob_of(z[v], v, T); }    // any index
  __device__ __forceinline__ float probs(int v, float T) const { return prob_of(zs[v], v, T); }  // index in the slice
  // log of an unnormalised weight for the exponential race (slice indices); -inf outside the support
  __device__ __forceinline__ float logw(int v, float T) const {
    const float zv = zs[v];
    if (!filt) return zv / T;
    return kept(__float_as_uint(expf(zv / T - m)), v) ? zv / T : -INFINITY;
  }
  __device__ __forceinline__ float4 pack() const { return make_float4(m, s, __uint_as_float(ecut), __int_as_float(vcut)); }
  __device__ __forceinline__ void unpack(float4 f) { m = f.x, s = f.y, ecut = __float_as_uint(f.z), vcut = __float_as_int(f.w), filt = true; }
};

__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    unsigned hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    unsigned hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += 0x9E3779B9u;
    k.y += 0xBB67AE85u;
  }
  return c;
}
__device__ __forceinline__ float u01(unsigned w) { return ((float)(w >> 9) + 0.5f) * 1.1920928955078125e-07f; }
__device__ __forceinline__ float gumbel_of(unsigned w) { return -logf(-logf(u01(w))); }

struct ArgMax {
  float v;
  int i;
};
__device__ __forceinline__ ArgMax better(ArgMax a, ArgMax b) { return (b.v > a.v || (b.v == a.v && b.i < a.i)) ? b : a; }

// Reductions over the whole cluster.  Each CTA reduces its own threads (warp shuffles, then the warps' partials in
// order), thread 0 writes the CTA's partial into slot [rank] of every CTA of the cluster, and after one cluster
// barrier every thread combines the slots in rank order.  Two sets of slots alternate, so a CTA that is already in
// the next reduction never overwrites what a slower sibling still reads.
struct ClusterRed {
  cg::cluster_group cluster;
  int n_ranks, rank, phase;
  float* sh_f;    // [SEL_THREADS / 32]
  int* sh_i;      // [SEL_THREADS / 32]
  ArgMax* sh_a;   // [SEL_THREADS / 32]
  float* part_f;  // [2][SEL_CS]
  int* part_i;    // [2][SEL_CS]
  ArgMax* part_a; // [2][SEL_CS]
  float* sh_n;    // [SEL_THREADS / 32][SEL_NV]: several values reduced at once (ints are passed as bit patterns)
  float* part_n;  // [2][SEL_CS][SEL_NV]

  template <typename T>
  __device__ __forceinline__ void publish(T* part, T v) {
    if (threadIdx.x == 0)
      for (int r = 0; r < n_ranks; ++r) *cluster.map_shared_rank(part + phase * SEL_CS + rank, r) = v;
    cluster.sync();
  }
  __device__ __forceinline__ float sum(float v) {
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh_f[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = 0.f;
    for (int w = 0; w < SEL_THREADS / 32; ++w) r += sh_f[w];
    publish(part_f, r);
    r = 0.f;
    for (int q = 0; q < n_ranks; ++q) r += part_f[phase * SEL_CS + q];
    phase ^= 1;
    return r;
  }
  __device__ __forceinline__ float max(float v) {
    v = warp_max(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh_f[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = sh_f[0];
    for (int w = 1; w < SEL_THREADS / 32; ++w) r = fmaxf(r, sh_f[w]);
    publish(part_f, r);
    r = part_f[phase * SEL_CS];
    for (int q = 1; q < n_ranks; ++q) r = fmaxf(r, part_f[phase * SEL_CS + q]);
    phase ^= 1;
    return r;
  }
  __device__ __forceinline__ int sum_int(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh_i[threadIdx.x >> 5] = v;
    __syncthreads();
    int r = 0;
    for (int w = 0; w < SEL_THREADS / 32; ++w) r += sh_i[w];
    publish(part_i, r);
    r = 0;
    for (int q = 0; q < n_ranks; ++q) r += part_i[phase * SEL_CS + q];
    phase ^= 1;
    return r;
  }
  // N <= SEL_NV sums at once, with one exchange: v[i] becomes the cluster-wide sum (floats or, with INT, integers)
  template <int N, bool INT>
  __device__ __forceinline__ void sum_n(float (&v)[N]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int i = 0; i < N; ++i) {
      if (INT) {
        int x = __float_as_int(v[i]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
        v[i] = __int_as_float(x);
      } else {
        v[i] = warp_sum(v[i]);
      }
    }
    __syncthreads();
    if (lane == 0)
#pragma unroll
      for (int i = 0; i < N; ++i) sh_n[warp * SEL_NV + i] = v[i];
    __syncthreads();
    if ((int)threadIdx.x < N) {  // thread i folds value i over the warps (in order) and hands it to every CTA
      const int i = threadIdx.x;
      float r;
      if (INT) {
        int x = 0;
        for (int w = 0; w < SEL_THREADS / 32; ++w) x += __float_as_int(sh_n[w * SEL_NV + i]);
        r = __int_as_float(x);
      } else {
        r = 0.f;
        for (int w = 0; w < SEL_THREADS / 32; ++w) r += sh_n[w * SEL_NV + i];
      }
      for (int q = 0; q < n_ranks; ++q) *cluster.map_shared_rank(part_n + (phase * SEL_CS + rank) * SEL_NV + i, q) = r;
    }
    cluster.sync();
#pragma unroll
    for (int i = 0; i < N; ++i) {
      if (INT) {
        int x = 0;
        for (int q = 0; q < n_ranks; ++q) x += __float_as_int(part_n[(phase * SEL_CS + q) * SEL_NV + i]);
        v[i] = __int_as_float(x);
      } else {
        float r = 0.f;
        for (int q = 0; q < n_ranks; ++q) r += part_n[(phase * SEL_CS + q) * SEL_NV + i];
        v[i] = r;
      }
    }
    phase ^= 1;
  }
  __device__ __forceinline__ ArgMax block_argmax(ArgMax a) {  // this CTA only
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      ArgMax b;
      b.v = __shfl_xor_sync(0xffffffffu, a.v, o);
      b.i = __shfl_xor_sync(0xffffffffu, a.i, o);
      a = better(a, b);
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh_a[threadIdx.x >> 5] = a;
    __syncthreads();
    ArgMax r = sh_a[0];
    for (int w = 1; w < SEL_THREADS / 32; ++w) r = better(r, sh_a[w]);
    return r;
  }
  __device__ __forceinline__ ArgMax argmax(ArgMax a) {
    ArgMax r = block_argmax(a);
    publish(part_a, r);
    r = part_a[phase * SEL_CS];
    for (int q = 1; q < n_ranks; ++q) r = better(r, part_a[phase * SEL_CS + q]);
    phase ^= 1;
    return r;
  }
};

// Nucleus of softmax(z / T) under top-k and top-p.  e_v = exp(z_v/T - m) of this CTA's slice [v_lo, v_hi) is kept in
// shared memory (a thread only ever touches the elements it wrote); the cut is found by searching the bit pattern of
// e from the top bit down (e <= 1, so 30 bits), then the index among equal values; every count / mass is a
// fixed-order reduction, so the result does not depend on timing.  top-k cuts first; top-p then applies to the
// renormalised top-k set.
__device__ __noinline__ void build_nucleus(Dist& d, int V, int v_lo, int v_hi, float T, int top_k, float top_p, float* e_sm,
                                           ClusterRed& R) {
  const int tid = threadIdx.x;
  float m = -INFINITY;
  for (int v = v_lo + tid; v < v_hi; v += SEL_THREADS) m = fmaxf(m, d.zs[v] / T);
  m = R.max(m);
  for (int v = v_lo + tid; v < v_hi; v += SEL_THREADS) e_sm[v - v_lo] = expf(d.zs[v] / T - m);
  d.m = m, d.ecut = 0u, d.vcut = V - 1, d.filt = true;  // everything kept so far
  auto count_if = [&](auto pred) {
    int n = 0;
    for (int v = v_lo + tid; v < v_hi; v += SEL_THREADS) n += pred(__float_as_uint(e_sm[v - v_lo]), v) ? 1 : 0;
    return R.sum_int(n);
  };
  auto mass_if = [&](auto pred) {
    float a = 0.f;
    for (int v = v_lo + tid; v < v_hi; v += SEL_THREADS) a += pred(__float_as_uint(e_sm[v - v_lo]), v) ? e_sm[v - v_lo] : 0.f;
    return R.sum(a);
  };
  // lowest index of an element whose value is c (used when c occurs once: no search over the indices is needed)
  auto first_index_of = [&](unsigned c) {
    int best = V;
    for (int v = v_lo + tid; v < v_hi; v += SEL_THREADS)
      if (__float_as_uint(e_sm[v - v_lo]) == c) best = min(best, v);
    return -R.sum_int(best == V ? 0 : -best);  // exactly one thread of the cluster holds it when the value is unique
  };
  if (top_k > 0 && top_k < V) {
    unsigned c = 0;  // largest c with at least top_k values >= c: the value of the top_k-th ranked token
    for (int shift = 27; shift >= 0; shift -= 3) {  // three bits per pass: the seven candidates c | k << shift at once
      float cnt[SEL_NV];
#pragma unroll
      for (int k = 0; k < SEL_NV; ++k) cnt[k] = __int_as_float(0);
      for (int v = v_lo + tid; v < v_hi; v += SEL_THREADS) {
        const unsigned eb = __float_as_uint(e_sm[v - v_lo]);
#pragma unroll
        for (int k = 0; k < SEL_NV; ++k) cnt[k] = __int_as_float(__float_as_int(cnt[k]) + (eb >= (c | ((unsigned)(k + 1) << shift)) ? 1 : 0));
      }
      R.template sum_n<SEL_NV, true>(cnt);
      unsigned best = 0;
#pragma unroll
      for (int k = 0; k < SEL_NV; ++k)
        if (__float_as_int(cnt[k]) >= top_k) best = k + 1;  // the predicate is monotone in k
      c |= best << shift;
    }
    const int need = top_k - count_if([&](unsigned eb, int) { return eb > c; });  // how many of the equal values stay
    int lo = 0, hi = V - 1;
    if (count_if([&](unsigned eb, int) { return eb == c; }) == 1) lo = hi = first_index_of(c);
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (count_if([&](unsigned eb, int v) { return eb == c && v <= mid; }) >= need) hi = mid;
      else lo = mid + 1;
    }
    d.ecut = c, d.vcut = lo;
  }
  if (top_p < 1.0f) {
    const Dist dk = d;  // the top-k set
    const float target = top_p * mass_if([&](unsigned eb, int v) { return dk.kept(eb, v); });
    unsigned c = 0;     // largest c such that the kept values >= c carry at least the target mass
    for (int shift = 27; shift >= 0; shift -= 3) {
      float mass[SEL_NV];
#pragma unroll
      for (int k = 0; k < SEL_NV; ++k) mass[k] = 0.f;
      for (int v = v_lo + tid; v < v_hi; v += SEL_THREADS) {
        const float e = e_sm[v - v_lo];
        const unsigned eb = __float_as_uint(e);
        const bool in_k = dk.kept(eb, v);
#pragma unroll
        for (int k = 0; k < SEL_NV; ++k) mass[k] += (in_k && eb >= (c | ((unsigned)(k + 1) << shift))) ? e : 0.f;
      }
      R.template sum_n<SEL_NV, false>(mass);
      unsigned best = 0;
#pragma unroll
      for (int k = 0; k < SEL_NV; ++k)
        if (mass[k] >= target) best = k + 1;
      c |= best << shift;
    }
    if (c < dk.ecut) c = dk.ecut;
    const float m_gt = mass_if([&](unsigned eb, int v) { return dk.kept(eb, v) && eb > c; });
    const float e_c = __uint_as_float(c);
    int lo = 0, hi = (c == dk.ecut) ? dk.vcut : V - 1;
    if (count_if([&](unsigned eb, int) { return eb == c; }) == 1) lo = hi = first_index_of(c);
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      const int n = count_if([&](unsigned eb, int v) { return eb == c && v <= mid; });
      if (m_gt + (float)n * e_c >= target) hi = mid;
      else lo = mid + 1;
    }
    d.ecut = c, d.vcut = lo;
  }
  const Dist df = d;
  d.s = mass_if([&](unsigned eb, int v) { return df.kept(eb, v); });
}

// argmax of the logits row of readout column `col` from the per-block maxima the lm_head epilogue left (ties to the
// lowest index)
__device__ __forceinline__ int greedy_argmax(const float2* argpart, int n_rb, int col, ClusterRed& R) {
  ArgMax a = {-INFINITY, 0x7fffffff};
  for (int b = threadIdx.x; b < n_rb; b += SEL_THREADS) {
    const float2 v = __ldcg(argpart + (size_t)col * n_rb + b);
    a = better(a, ArgMax{v.x, __float_as_int(v.y)});
  }
  return R.block_argmax(a).i;  // every CTA of the cluster reads all partials: no exchange needed
}

__global__ void __launch_bounds__(SEL_THREADS) select_kernel(const __grid_constant__ SelectParams p) {
  __shared__ ArgMax sh_am[SEL_THREADS / 32];
  __shared__ float sh_f[SEL_THREADS / 32];
  __shared__ int sh_i[SEL_THREADS / 32];
  __shared__ float part_f[2 * SEL_CS];
  __shared__ int part_i[2 * SEL_CS];
  __shared__ ArgMax part_a[2 * SEL_CS];
  __shared__ float sh_n[(SEL_THREADS / 32) * SEL_NV];
  __shared__ float part_n[2 * SEL_CS * SEL_NV];
  cg::cluster_group this_cl = cg::this_cluster();
  ClusterRed R{this_cl, (int)this_cl.num_blocks(), (int)this_cl.block_rank(), 0, sh_f, sh_i, sh_am, part_f, part_i, part_a, sh_n, part_n};
  const int col = (int)blockIdx.x / R.n_ranks;  // readout column = this cluster
  tune_mark(602, false);
  pdl_launch_dependents();
  // the row table was written before this pass started: everything but the logits can be read ahead of the lm_head
  const RowTable* tab = p.tab;
  if (col >= tab->n_readout) {  // every CTA waits: a kernel that ends early would release its dependents early
    pdl_wait();
    return;
  }
  struct EndMark { __device__ ~EndMark() { tune_mark(602, true); } } end_mark;
  const int row = tab->ro_rows[col];
  const int kind = tab->readout[row];
  if (!((p.kinds_mask >> kind) & 1)) {
    pdl_wait();
    return;
  }
  const int V = p.V, tid = threadIdx.x;
  const bool writer = R.rank == 0 && tid == 0;  // all CTAs of the cluster hold the same results; one thread stores them
  // this CTA's slice of the vocabulary: whole Philox blocks of 4 indices
  const int per = ((V / 4 + R.n_ranks - 1) / R.n_ranks) * 4;
  const int v_lo = min(V, R.rank * per), v_hi = min(V, v_lo + per);
  const float T = p.temperature;
  const float* z = p.logits + (size_t)tab->logit_idx[row] * V;
  const int gn = tab->node[row];
  const float* z1 = p.logits + (size_t)(gn < 0 ? 0 : gn) * 2 * V;  // stored first-proposal readout
  const float* z2 = z1 + V;                                        // stored second-proposal readout
  const unsigned position = (unsigned)(tab->pos[row] + 1);         // the position being decided
  const unsigned seq = (unsigned)tab->seq[row];
  const uint2 key = make_uint2((unsigned)(p.seed & 0xffffffffull), (unsigned)(p.seed >> 32));

  const bool filt = T > 0.f && ((p.top_k > 0 && p.top_k < V) || p.top_p < 1.0f);
  // dynamic shared memory: [staged ? 3 : 0] row slices, then the slice of exp(z/T - max) when filters are on
  extern __shared__ __align__(16) float dyn_sm[];
  float* e_sm = dyn_sm + (p.staged ? 3 * per : 0);
  // Copy this CTA's slice of a logits row into shared memory with every load in flight at once (the sampled paths
  // pass over up to three rows several times; from global memory each pass is a chain of L2 round trips).  Returns a
  // pointer indexed by the vocabulary index.
  auto stage = [&](const float* zz, int slot) -> const float* {
    if (!p.staged) return zz;
    float* dst = dyn_sm + slot * per;
    const float4* src = reinterpret_cast<const float4*>(zz + v_lo);
    for (int i = tid; i < (v_hi - v_lo) / 4; i += SEL_THREADS) reinterpret_cast<float4*>(dst)[i] = __ldcg(src + i);
    __syncthreads();
    return dst - v_lo;
  };
  // the distribution C(H) of a freshly computed logits row
  auto fresh = [&](const float* zz, int slot) -> Dist {
    Dist d;
    d.z = zz, d.zs = stage(zz, slot), d.filt = false, d.lse = 0.f, d.m = 0.f, d.s = 1.f, d.ecut = 0u, d.vcut = V - 1;
    if (filt) {
      build_nucleus(d, V, v_lo, v_hi, T, p.top_k, p.top_p, e_sm, R);
    } else {  // log sum_v exp(zz_v / T)
      float m = -INFINITY;
      for (int v = v_lo + tid; v < v_hi; v += SEL_THREADS) m = fmaxf(m, d.zs[v] / T);
      m = R.max(m);
      float s = 0.f;
      for (int v = v_lo + tid; v < v_hi; v += SEL_THREADS) s += expf(d.zs[v] / T - m);
      s = R.sum(s);
      d.lse = m + logf(s);
    }
    return d;
  };
  // a distribution stored with a proposal record: its logits row, log-normaliser and (if filtered) nucleus
  auto stored = [&](const float* zz, int slot, float lse, const float4* flt) -> Dist {
    Dist d;
    d.z = zz, d.zs = stage(zz, slot), d.filt = false, d.lse = lse, d.m = 0.f, d.s = 1.f, d.ecut = 0u, d.vcut = V - 1;
    if (filt) d.unpack(*flt);
    return d;
  };
  // greedy readouts are always taken from the row the lm_head just produced
  auto greedy = [&](const float*) -> int { return greedy_argmax(p.argpart, p.n_rb, col, R); };
  // exponential race over weights given through logw(v) (-inf = zero weight)
  auto race = [&](auto logw, int purpose) -> int {
    ArgMax a = {-INFINITY, 0x7fffffff};
    for (int b = v_lo / 4 + tid; b < v_hi / 4; b += SEL_THREADS) {
      uint4 w = philox4x32_10(make_uint4((unsigned)b, position, seq, (unsigned)purpose), key);
      const unsigned ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        int v = 4 * b + e;
        float lw = logw(v);
        if (lw > -INFINITY) a = better(a, ArgMax{lw + gumbel_of(ww[e]), v});
      }
    }
    return R.argmax(a).i;
  };
  auto uniform = [&](int purpose) -> float {
    return u01(philox4x32_10(make_uint4(0u, position, seq, (unsigned)purpose), key).x);
  };

  pdl_wait();
  if (kind == RO_TARGET) {
    int tok;
    if (T == 0.f) {
      tok = greedy(z);
    } else {
      const Dist dz = fresh(z, 0);
      tok = race([&](int v) { return dz.logw(v, T); }, PUR_VANILLA);
    }
    if (writer) p.sel_tok[row] = tok;
    return;
  }
  if (kind == RO_D1) {
    if (T == 0.f) {
      int tok = greedy(z);
      if (writer) p.sel_tok[row] = tok, p.sel_lse[row] = 0.f;
    } else {
      const Dist dz = fresh(z, 0);
      int tok = race([&](int v) { return dz.logw(v, T); }, PUR_DRAFT1);
      if (writer) {
        p.sel_tok[row] = tok, p.sel_lse[row] = dz.lse;
        if (filt) p.sel_flt[row] = dz.pack();
      }
    }
    return;
  }
  if (kind == RO_D2) {
    const int x1 = p.nodes.tok1[gn];
    if (T == 0.f) {
      int top = greedy(z);
      const bool open = (top != x1) || !p.gate;
      if (open && top == x1 && p.mask_first) {
        // the best token other than the first candidate: the per-block maxima of the other blocks, and the logits of
        // the candidate's own block one by one
        ArgMax a = {-INFINITY, 0x7fffffff};
        const int xb = x1 / SEL_ARG_BLOCK;
        for (int b = tid; b < p.n_rb; b += SEL_THREADS)
          if (b != xb) {
            const float2 v = __ldcg(p.argpart + (size_t)col * p.n_rb + b);
            a = better(a, ArgMax{v.x, __float_as_int(v.y)});
          }
        if (tid < SEL_ARG_BLOCK) {
          const int v = xb * SEL_ARG_BLOCK + tid;
          if (v < V && v != x1) a = better(a, ArgMax{__ldcg(z + v), v});
        }
        top = R.block_argmax(a).i;
      }
      if (writer) p.sel_tok[row] = top, p.sel_aux[row] = open, p.sel_lse[row] = 0.f, p.sel_z2[row] = 0.f;
      return;
    }
    const Dist d1 = stored(z1, 1, p.nodes.lse1[gn], p.nodes.flt1 + gn);
    const Dist d2 = fresh(z, 0);
    // Eq. 6; without filters the comparison is made on log-probabilities, as before
    const bool lower = filt ? (d2.prob(x1, T) < d1.prob(x1, T)) : (z[x1] / T - d2.lse < z1[x1] / T - d1.lse);
    bool open = lower || !p.gate;
    const bool mask = p.mask_first != 0;
    int tok = 0;
    // how the record's proposal is normalised: > 0: [q2~ - q1]_+ over this mass; < 0: q2~ over minus this mass
    // (first candidate masked out); 0: q2~ as it is
    float Z2 = 0.f;
    if (open) {
      if (p.residual_q2) {
        float s = 0.f;
        for (int v = v_lo + tid; v < v_hi; v += SEL_THREADS)
          if (!(mask && v == x1)) s += fmaxf(d2.probs(v, T) - d1.probs(v, T), 0.f);
        Z2 = R.sum(s);
      }
      if (Z2 > 0.f) {
        tok = race([&](int v) {
          float w = (mask && v == x1) ? 0.f : d2.probs(v, T) - d1.probs(v, T);
          return w > 0.f ? logf(w) : -INFINITY; }, PUR_DRAFT2);
      } else if (!mask) {
        tok = race([&](int v) { return d2.logw(v, T); }, PUR_DRAFT2);
      } else {  // q2~ without the first candidate
        float s = 0.f;
        for (int v = v_lo + tid; v < v_hi; v += SEL_THREADS)
          if (v != x1) s += d2.probs(v, T);
        const float rest = R.sum(s);
        if (rest > 0.f) {
          Z2 = -rest;
          tok = race([&](int v) { return v == x1 ? -INFINITY : d2.logw(v, T); }, PUR_DRAFT2);
        } else {
          open = false;  // all of q2~ sits on the first candidate: no second proposal
        }
      }
    }
    if (writer) {
      p.sel_tok[row] = tok, p.sel_aux[row] = open, p.sel_lse[row] = d2.lse, p.sel_z2[row] = Z2;
      if (filt) p.sel_flt[row] = d2.pack();
    }
    return;
  }
  // ---- RO_VERIFY: z is the target readout p_R of the root branch ------------------------------------
  const int x1 = p.nodes.tok1[gn], has2 = p.nodes.has2[gn], x2 = p.nodes.tok2[gn];
  if (T == 0.f) {
    int top = greedy(z);
    int src = (top == x1) ? 1 : ((has2 && top == x2) ? 2 : 3);
    if (writer) p.sel_tok[row] = top, p.sel_aux[row] = src;
    return;
  }
  const float Z2 = p.nodes.z2[gn];
  const Dist d1 = stored(z1, 1, p.nodes.lse1[gn], p.nodes.flt1 + gn);
  const Dist d2 = has2 ? stored(z2, 2, p.nodes.lse2[gn], p.nodes.flt2 + gn) : d1;
  const Dist dp = fresh(z, 0);
  // p_R, the first proposal and the deeper readout: (v) for indices of this CTA's slice, (v, true) for any index
  auto pp = [&](int v, bool any = false) { return any ? dp.prob(v, T) : dp.probs(v, T); };
  auto q1 = [&](int v, bool any = false) { return any ? d1.prob(v, T) : d1.probs(v, T); };
  auto q2t = [&](int v, bool any = false) { return any ? d2.prob(v, T) : d2.probs(v, T); };
  // sum_v [p - q1]_+ : the normaliser of rho1 = p (-) q1 (Eq. 2) and, both being normalised, TV(q1, p)
  auto mass_above_q1 = [&]() {
    float a = 0.f;
    for (int v = v_lo + tid; v < v_hi; v += SEL_THREADS) a += fmaxf(pp(v) - q1(v), 0.f);
    return R.sum(a);
  };
  float Z1 = 0.f;
  if (p.tv_acc) {  // the empirical TV profile of Sec. 4.1, recorded at every verification
    Z1 = mass_above_q1();
    float tv2 = 0.f;
    if (has2) {
      float a = 0.f;
      for (int v = v_lo + tid; v < v_hi; v += SEL_THREADS) a += fmaxf(pp(v) - q2t(v), 0.f);
      tv2 = R.sum(a);
    }
    if (writer) {  // one verification per sequence and pass: no other writer
      double* acc = p.tv_acc + 4 * seq;
      acc[0] += (double)Z1, acc[1] += 1.0;
      if (has2) acc[2] += (double)tv2, acc[3] += 1.0;
    }
  }
  // first proposal: accept with probability min{1, p(x1)/q1(x1)} (Eq. 3)
  const float U1 = uniform(PUR_ACCEPT1);
  if (U1 < fminf(1.0f, pp(x1, true) / q1(x1, true))) {
    if (writer) p.sel_tok[row] = x1, p.sel_aux[row] = 1;
    return;
  }
  // rho1 = p (-) q1 (Eq. 2); if the positive part has no mass rho1 = p
  if (!p.tv_acc) Z1 = mass_above_q1();
  float s = 0.f;
  auto rho1 = [&](int v, bool any = false) { return Z1 > 0.f ? fmaxf(pp(v, any) - q1(v, any), 0.f) / Z1 : pp(v, any); };
  if (!has2) {
    int tok = race([&](int v) { float w = rho1(v); return w > 0.f ? logf(w) : -INFINITY; }, PUR_RESAMPLE);
    if (writer) p.sel_tok[row] = tok, p.sel_aux[row] = 3;
    return;
  }
  const bool mask = p.mask_first != 0;
  auto q2 = [&](int v, bool any = false) {  // the second proposal as it was drafted (see the record's normaliser)
    if (mask && v == x1) return 0.f;
    if (Z2 > 0.f) return fmaxf(q2t(v, any) - q1(v, any), 0.f) / Z2;
    return Z2 < 0.f ? q2t(v, any) / -Z2 : q2t(v, any);
  };
  const float U2 = uniform(PUR_ACCEPT2);
  if (U2 < fminf(1.0f, rho1(x2, true) / q2(x2, true))) {
    if (writer) p.sel_tok[row] = x2, p.sel_aux[row] = 2;
    return;
  }
  s = 0.f;
  for (int v = v_lo + tid; v < v_hi; v += SEL_THREADS) s += fmaxf(rho1(v) - q2(v), 0.f);
  const float S2 = R.sum(s);
  int tok = race([&](int v) {
    float w = S2 > 0.f ? fmaxf(rho1(v) - q2(v), 0.f) : rho1(v);
    return w > 0.f ? logf(w) : -INFINITY; }, PUR_RESAMPLE);
  if (writer) p.sel_tok[row] = tok, p.sel_aux[row] = 3;
}

}  // namespace ls

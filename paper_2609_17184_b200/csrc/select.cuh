// Readout decisions of one step: first-proposal draft at d1 (Sec. 4.2 step 2), gate and residual second
// proposal at d2 (Eq. 5-6), cascade verification at R (Sec. 4.3; Algorithm 1 Verify), and the plain draw
// x ~ C(H) used by prefill and vanilla decoding.  One CTA per reading-out row; every reduction over the
// vocabulary is a fixed-order block reduction.
//
// Random draws (the paper only says "x ~ q", "U ~ U(0,1)"): Philox4x32-10 keyed by the seed with counter
// (block, position being decided, sequence, purpose); u = ((word >> 9) + 0.5) * 2^-23; categorical draws
// by the exponential race argmax_v log w_v - log(-log u_v) with ties to the lowest index.
#pragma once
#include "common.cuh"

namespace ls {

constexpr int SEL_THREADS = 1024;
enum { PUR_DRAFT1 = 1, PUR_DRAFT2 = 2, PUR_ACCEPT1 = 3, PUR_ACCEPT2 = 4, PUR_RESAMPLE = 5, PUR_VANILLA = 6 };

struct SelectParams {
  const RowTable* tab;
  const float* logits;  // [logit_idx][V]
  int V, NB;
  NodeTable nodes;
  float temperature;
  int gate, residual_q2;
  unsigned long long seed;
  int kinds_mask;       // bit k set: handle readout kind k
  int* sel_tok;         // per row: drafted / committed token
  int* sel_aux;         // RO_D2: gate open; RO_VERIFY: source 1/2/3
  float* sel_lse;       // RO_D1 / RO_D2: log-sum-exp of z/T
  float* sel_z2;        // RO_D2: normaliser of the residual proposal (0: the proposal is q2~ itself)
  const float2* argpart;  // [readout column][row block]: per-block largest logit and its index, written by the lm_head
  int n_rb;
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

__device__ __forceinline__ ArgMax block_argmax(ArgMax a, ArgMax* sh) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ArgMax b;
    b.v = __shfl_xor_sync(0xffffffffu, a.v, o);
    b.i = __shfl_xor_sync(0xffffffffu, a.i, o);
    a = better(a, b);
  }
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = a;
  __syncthreads();
  ArgMax r = sh[0];
  for (int w = 1; w < SEL_THREADS / 32; ++w) r = better(r, sh[w]);
  return r;
}
__device__ __forceinline__ float block_sum(float v, float* sh) {
  v = warp_sum(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = 0.f;
  for (int w = 0; w < SEL_THREADS / 32; ++w) r += sh[w];
  return r;
}
__device__ __forceinline__ float block_max(float v, float* sh) {
  v = warp_max(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = sh[0];
  for (int w = 1; w < SEL_THREADS / 32; ++w) r = fmaxf(r, sh[w]);
  return r;
}

// argmax of the logits row of readout column `col` from the per-block maxima the lm_head epilogue left (ties to the
// lowest index)
__device__ __forceinline__ int greedy_argmax(const float2* argpart, int n_rb, int col, ArgMax* sh_am) {
  ArgMax a = {-INFINITY, 0x7fffffff};
  for (int b = threadIdx.x; b < n_rb; b += SEL_THREADS) {
    const float2 v = __ldcg(argpart + (size_t)col * n_rb + b);
    a = better(a, ArgMax{v.x, __float_as_int(v.y)});
  }
  return block_argmax(a, sh_am).i;
}

__global__ void __launch_bounds__(SEL_THREADS) select_kernel(const __grid_constant__ SelectParams p) {
  __shared__ ArgMax sh_am[SEL_THREADS / 32];
  __shared__ float sh_f[SEL_THREADS / 32];
  tune_mark(602, false);
  pdl_launch_dependents();
  // the row table was written before this pass started: everything but the logits can be read ahead of the lm_head
  const RowTable* tab = p.tab;
  if ((int)blockIdx.x >= tab->n_readout) {  // every CTA waits: a kernel that ends early would release its dependents early
    pdl_wait();
    return;
  }
  struct EndMark { __device__ ~EndMark() { tune_mark(602, true); } } end_mark;
  const int row = tab->ro_rows[blockIdx.x];
  const int kind = tab->readout[row];
  if (!((p.kinds_mask >> kind) & 1)) {
    pdl_wait();
    return;
  }
  const int V = p.V, tid = threadIdx.x;
  const float T = p.temperature;
  const float* z = p.logits + (size_t)tab->logit_idx[row] * V;
  const int gn = tab->node[row];
  const float* z1 = p.logits + (size_t)(gn < 0 ? 0 : gn) * 2 * V;  // stored first-proposal readout
  const float* z2 = z1 + V;                                        // stored second-proposal readout
  const unsigned position = (unsigned)(tab->pos[row] + 1);         // the position being decided
  const unsigned seq = (unsigned)tab->seq[row];
  const uint2 key = make_uint2((unsigned)(p.seed & 0xffffffffull), (unsigned)(p.seed >> 32));

  auto lse_of = [&](const float* zz) -> float {  // log sum_v exp(zz_v / T)
    float m = -INFINITY;
    for (int v = tid; v < V; v += SEL_THREADS) m = fmaxf(m, zz[v] / T);
    m = block_max(m, sh_f);
    float s = 0.f;
    for (int v = tid; v < V; v += SEL_THREADS) s += expf(zz[v] / T - m);
    s = block_sum(s, sh_f);
    return m + logf(s);
  };
  // greedy readouts are always taken from the row the lm_head just produced
  auto greedy = [&](const float*) -> int { return greedy_argmax(p.argpart, p.n_rb, (int)blockIdx.x, sh_am); };
  // exponential race over weights given through logw(v) (-inf = zero weight)
  auto race = [&](auto logw, int purpose) -> int {
    ArgMax a = {-INFINITY, 0x7fffffff};
    for (int b = tid; b < V / 4; b += SEL_THREADS) {
      uint4 w = philox4x32_10(make_uint4((unsigned)b, position, seq, (unsigned)purpose), key);
      const unsigned ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        int v = 4 * b + e;
        float lw = logw(v);
        if (lw > -INFINITY) a = better(a, ArgMax{lw + gumbel_of(ww[e]), v});
      }
    }
    return block_argmax(a, sh_am).i;
  };
  auto uniform = [&](int purpose) -> float {
    return u01(philox4x32_10(make_uint4(0u, position, seq, (unsigned)purpose), key).x);
  };

  pdl_wait();
  if (kind == RO_TARGET) {
    int tok = (T == 0.f) ? greedy(z) : race([&](int v) { return z[v] / T; }, PUR_VANILLA);
    if (tid == 0) p.sel_tok[row] = tok;
    return;
  }
  if (kind == RO_D1) {
    if (T == 0.f) {
      int tok = greedy(z);
      if (tid == 0) p.sel_tok[row] = tok, p.sel_lse[row] = 0.f;
    } else {
      float lse = lse_of(z);
      int tok = race([&](int v) { return z[v] / T; }, PUR_DRAFT1);
      if (tid == 0) p.sel_tok[row] = tok, p.sel_lse[row] = lse;
    }
    return;
  }
  if (kind == RO_D2) {
    const int x1 = p.nodes.tok1[gn];
    if (T == 0.f) {
      int top = greedy(z);
      if (tid == 0) p.sel_tok[row] = top, p.sel_aux[row] = (top != x1) || !p.gate, p.sel_lse[row] = 0.f, p.sel_z2[row] = 0.f;
      return;
    }
    const float lse1 = p.nodes.lse1[gn];
    const float lse2 = lse_of(z);
    const bool open = (z[x1] / T - lse2 < z1[x1] / T - lse1) || !p.gate;
    int tok = 0;
    float Z2 = 0.f;
    if (open) {
      if (p.residual_q2) {
        float s = 0.f;
        for (int v = tid; v < V; v += SEL_THREADS) s += fmaxf(expf(z[v] / T - lse2) - expf(z1[v] / T - lse1), 0.f);
        Z2 = block_sum(s, sh_f);
      }
      if (Z2 > 0.f)
        tok = race([&](int v) {
          float w = expf(z[v] / T - lse2) - expf(z1[v] / T - lse1);
          return w > 0.f ? logf(w) : -INFINITY; }, PUR_DRAFT2);
      else
        tok = race([&](int v) { return z[v] / T; }, PUR_DRAFT2);
    }
    if (tid == 0) p.sel_tok[row] = tok, p.sel_aux[row] = open, p.sel_lse[row] = lse2, p.sel_z2[row] = Z2;
    return;
  }
  // ---- RO_VERIFY: z is the target readout p_R of the root branch ------------------------------------
  const int x1 = p.nodes.tok1[gn], has2 = p.nodes.has2[gn], x2 = p.nodes.tok2[gn];
  if (T == 0.f) {
    int top = greedy(z);
    int src = (top == x1) ? 1 : ((has2 && top == x2) ? 2 : 3);
    if (tid == 0) p.sel_tok[row] = top, p.sel_aux[row] = src;
    return;
  }
  const float lse1 = p.nodes.lse1[gn], lse2 = p.nodes.lse2[gn], Z2 = p.nodes.z2[gn];
  const float lsep = lse_of(z);
  auto pp = [&](int v) { return expf(z[v] / T - lsep); };     // p_R
  auto q1 = [&](int v) { return expf(z1[v] / T - lse1); };    // first proposal
  auto q2t = [&](int v) { return expf(z2[v] / T - lse2); };   // deeper readout
  // first proposal: accept with probability min{1, p(x1)/q1(x1)} (Eq. 3)
  const float U1 = uniform(PUR_ACCEPT1);
  if (U1 < fminf(1.0f, pp(x1) / q1(x1))) {
    if (tid == 0) p.sel_tok[row] = x1, p.sel_aux[row] = 1;
    return;
  }
  // rho1 = p (-) q1 (Eq. 2); if the positive part has no mass rho1 = p
  float s = 0.f;
  for (int v = tid; v < V; v += SEL_THREADS) s += fmaxf(pp(v) - q1(v), 0.f);
  const float Z1 = block_sum(s, sh_f);
  auto rho1 = [&](int v) { return Z1 > 0.f ? fmaxf(pp(v) - q1(v), 0.f) / Z1 : pp(v); };
  if (!has2) {
    int tok = race([&](int v) { float w = rho1(v); return w > 0.f ? logf(w) : -INFINITY; }, PUR_RESAMPLE);
    if (tid == 0) p.sel_tok[row] = tok, p.sel_aux[row] = 3;
    return;
  }
  auto q2 = [&](int v) { return Z2 > 0.f ? fmaxf(q2t(v) - q1(v), 0.f) / Z2 : q2t(v); };
  const float U2 = uniform(PUR_ACCEPT2);
  if (U2 < fminf(1.0f, rho1(x2) / q2(x2))) {
    if (tid == 0) p.sel_tok[row] = x2, p.sel_aux[row] = 2;
    return;
  }
  s = 0.f;
  for (int v = tid; v < V; v += SEL_THREADS) s += fmaxf(rho1(v) - q2(v), 0.f);
  const float S2 = block_sum(s, sh_f);
  int tok = race([&](int v) {
    float w = S2 > 0.f ? fmaxf(rho1(v) - q2(v), 0.f) : rho1(v);
    return w > 0.f ? logf(w) : -INFINITY; }, PUR_RESAMPLE);
  if (tid == 0) p.sel_tok[row] = tok, p.sel_aux[row] = 3;
}

}  // namespace ls

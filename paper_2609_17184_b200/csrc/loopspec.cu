// C ABI of the LoopSpec decode path (see include/loopspec.h): context, workspace layout, the launch
// sequence of one batched pass, CUDA-graph capture of the decode step and the host side of the scheduler.
#include "../../include/loopspec.h"

#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstddef>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#if __has_include(<nvtx3/nvToolsExt.h>)
#include <nvtx3/nvToolsExt.h>  // header-only: ranges show up when a profiler injects the NVTX library, cost nothing otherwise
#define LOOPSPEC_NVTX 1
#endif

#include "attention.cuh"
#include "common.cuh"
#include "control.cuh"
#include "gemm.cuh"
#include "select.cuh"
#include "linear_tc.cuh"
#include "gemm_dec.cuh"

using namespace ls;

namespace {

#ifndef LS_CTAS
#define LS_CTAS 2
#endif
constexpr int kCtasPerSm = LS_CTAS;  // GEMM CTAs that fit one SM (shared memory and registers)

struct GemmPlan {
  int n_rb, kpr, cs, n_clusters, grid;
};

// Cluster size = how many CTAs split K for one block of 128 output rows.  Enough CTAs to fill the resident
// slots (two per SM), a k-range short enough that a decode pass keeps its activations staged once, and whole
// rounds of row blocks per cluster so that every CTA streams the same number of bytes.
GemmPlan plan_gemm(int n_rb, int K, int slots, bool pow2_only, int kh = 1, int cs_cap = 8) {
  GemmPlan g;
  g.n_rb = n_rb;
  g.kpr = (K + 31) / 32;
  int cs_min = (g.kpr + MAX_XCH_BLOCKS - 1) / MAX_XCH_BLOCKS;
  int cs = std::max(1, slots / std::max(n_rb, 1));
  // a warp should keep at least 8 k-blocks: below that the fixed cost of a CTA (staging, reduction, epilogue)
  // outweighs what more CTAs stream in parallel, and a smaller grid leaves room for the next kernel's CTAs to
  // become resident (and prefetch) early  [measured: O projection, 8 -> 4 CTAs per cluster]
  cs = std::min(cs, std::max(1, g.kpr / (8 * kh)));
  cs = std::max(cs, cs_min);
  cs = std::min(std::min(cs, cs_cap), g.kpr);
  auto pow2_at_least = [&](int v) {
    int q = 1;
    while (q < v) q <<= 1;
    q = std::min(std::min(q, 8), g.kpr);
    while (q & (q - 1)) --q;
    return q;
  };
  if (pow2_only || n_rb * cs_min > slots) {
    cs = pow2_at_least(cs);  // several rounds of row blocks per cluster: measured best with power-of-two clusters
  } else {
    // the largest cluster size up to `cs` whose grid leaves a tenth of the resident slots free: a grid that fills them
    // all keeps the next kernel's CTAs from becoming resident (and requesting their weights) while this one runs
    // [measured on the QKV shape of Ouro-1.4B, 48 row blocks on 296 slots: clusters of 3 / 4 / 5 / 6 give passes of
    // 1.141 / 1.121 / 1.108 / 1.209 ms; k-ranges that differ by one k-block cost less than the idle slots]
    for (int v = cs; v >= std::max(cs_min, 1); --v)
      if (n_rb * v * 10 <= slots * 9 || v == std::max(cs_min, 1)) {
        cs = v;
        break;
      }
  }
  g.cs = cs;
  int max_clusters = std::max(1, slots / cs);
  int rounds = (n_rb + max_clusters - 1) / max_clusters;
  g.n_clusters = (n_rb + rounds - 1) / rounds;
  g.grid = g.n_clusters * cs;
  return g;
}

size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

// ---- plan of a decode-pass GEMM on the tcgen05 kernel (dgemm_kernel) ----
// One CTA per SM and kernel.  Among the cluster sizes the device can co-schedule, the one that gives the busiest CTA
// the fewest (row block, k-block) units; ties go to the smaller cluster (fewer contributions to sum per column).
struct DgPlan {
  int n_rb, cs, n_clusters, stages, acc_bufs, recv_bufs;
  size_t smem;
};
constexpr int kDgSmem = 200 * 1024;  // one CTA per SM: the ring takes (nearly) all of its shared memory
int dg_mp_for_rows(int rows) { return rows <= 8 ? 8 : (rows + 15) / 16 * 16; }
DgPlan plan_dg(int n_rb, int K, int MP, const int* max_clusters /* [9], by cluster size */) {
  const int kb = (K + TC_BK - 1) / TC_BK;
  DgPlan best{};
  long long best_cost = -1;
  for (int cs = 1; cs <= std::min(8, kb); ++cs) {
    const int n_cl_max = max_clusters[cs];
    if (n_cl_max < 1) continue;
    const int n_cl = std::min(n_rb, n_cl_max);
    const int tasks = (n_rb + n_cl - 1) / n_cl, kbm = (kb + cs - 1) / cs;
    const long long cost = (long long)tasks * kbm;
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      best.n_rb = n_rb, best.cs = cs, best.n_clusters = (n_rb + tasks - 1) / tasks;
      best.recv_bufs = tasks > 1 ? 2 : 1;
    }
  }
  if (best_cost < 0) return best;
  best.acc_bufs = 2 * DG_CHAINS * dg_mma_n(MP) <= 512 ? 2 : 1;
  const int budget = kDgSmem;
  const int fixed = 1024 + best.recv_bufs * dg_recv_floats(MP, best.cs) * 4;
  best.stages = std::max(2, std::min(DG_MAX_STAGES, (budget - fixed) / dg_stage_bytes(MP)));
  best.smem = (size_t)dg_smem_bytes(MP, best.cs, best.stages, best.recv_bufs);
  return best;
}
int ng_for_rows(int rows) { return rows <= 8 ? 1 : rows <= 16 ? 2 : rows <= 32 ? 4 : 8; }

static_assert(SEL_ARG_BLOCK == RB_ROWS, "the selection reads one argmax partial per lm_head row block");

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}
// bf16 matrix [rows][K], K contiguous; box = 64 k x box_rows rows, 128-byte swizzle, zeros beyond the edges
bool make_map_bf16(CUtensorMap* map, const void* ptr, int rows, int K, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// the activation planes of a pass, [column][3][x_ld] bf16, as a (k, plane, column) tensor; box = 64 k x 1 plane x cols
bool make_map_planes3d(CUtensorMap* map, const void* ptr, int K, int x_ld, int n_cols, int box_cols) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)K, 3, (cuuint64_t)n_cols};
  cuuint64_t strides[2] = {(cuuint64_t)x_ld * 2, (cuuint64_t)x_ld * 6};
  cuuint32_t box[3] = {(cuuint32_t)TC_BK, 1, (cuuint32_t)box_cols};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// the same buffer with all three planes of `box_rows` rows in one box: the tile's 128-byte rows are (row, plane) pairs
bool make_map_planes_all(CUtensorMap* map, const void* ptr, int K, int x_ld, int n_rows, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)K, 3, (cuuint64_t)n_rows};
  cuuint64_t strides[2] = {(cuuint64_t)x_ld * 2, (cuuint64_t)x_ld * 6};
  cuuint32_t box[3] = {(cuuint32_t)TC_BK, 3, (cuuint32_t)box_rows};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// k-split of a prefill GEMM on the tcgen05 kernel: a function of the matrix alone, so that a prompt position's sums
// do not depend on how many positions share the pass
struct TcPfPlan {
  int n_tiles, n_split, kb_per_split;
};
TcPfPlan tc_pf_plan(int N, int K) {
  TcPfPlan t;
  t.n_tiles = (N + TC_BM - 1) / TC_BM;
  const int total_kb = K / TC_BK;
#ifndef LS_TC_SLOTS
#define LS_TC_SLOTS 296
#endif
  const int want = std::max(1, std::min(LS_TC_SLOTS / t.n_tiles, total_kb / 4));
  t.kb_per_split = (total_kb + want - 1) / want;
  t.n_split = (total_kb + t.kb_per_split - 1) / t.kb_per_split;
  return t;
}
// the prefill passes can run their four layer GEMMs on the tcgen05 kernel: bf16 weights, every K a multiple of 64
bool tc_prefill_shapes_ok(const loopspec_model* m) {
  return m->weight_dtype == 1 && m->hidden % TC_BK == 0 && (m->n_q_heads * m->head_dim) % TC_BK == 0 && m->ffn % TC_BK == 0;
}
int tc_pf_cols(int max_rows_pf) { return (max_rows_pf + 15) / 16 * 16; }

struct Layout {  // byte offsets into the workspace
  size_t wpack, rope, kv, hid, qbuf, xplanes, aplanes, splanes, sumsq, logits, argpart, tcpart, flt, sel_flt, tv, tune, tune_bytes, apart, acnt, nodes, seqs, ctr, tab_dec, tab_pf,
      estore, cplanes, tab_pre, tab_coda, tab_pfc, tab_vanc, tab_van, sel_tok, sel_aux, sel_lse, sel_z2, kvcopy, out_ids, commits, trace, trace_n, prompt, total;
};

struct Derived {
  int att_mode;   // attention work items: 0 one sequence per context, 1 several (see att_run_len)
  int att_runs;   // the context's rows can have items of several chunks: the streaming attention kernel runs
  int S, NB, B, max_rows_dec, max_rows_pf, max_rows, slots, ids_cap, n_hid, n_logit_vecs, p_logit_base, n_sq, sq_stride, max_chunks,
      trace_cap, Hq, Hkv, d1, d2;
  // Raven-style layout (P and C hold transformer blocks): all layers in one list - prelude, recurrent, coda
  int raven, n_pre, n_coda, NL, n_classes, class_depth[3], hid_coda_base;
};

int max_branches(int R, int d1, int d2) {
  int n = R / d1;
  if (d2 == 0) return n;
  int lag = d2 / d1;
  std::vector<long long> s(n);
  long long tot = 0;
  for (int k = 0; k < n; ++k) {
    s[k] = k < lag ? 1 : s[k - 1] + s[k - lag];
    tot += s[k];
  }
  return (int)std::min<long long>(tot, 1 << 20);
}

// Theorem 2 / Eq. 8
void closed_form(double a, double b, double R, double* d1, double* d2) {
  double D = a * a + a + 1.0, ab = a * b, tar = 2.0 * a * R;
  *d1 = std::pow(ab, (a + 1.0) / D) * std::pow(tar, 1.0 / D);
  *d2 = std::pow(ab, a / D) * std::pow(tar, (a + 1.0) / D);
}
double steps_bound(double d1, double d2, double a, double b, double R) {
  return d1 + b * std::pow(d1, -a) * d2 + 2.0 * b * std::pow(d2, -a) * R;
}
bool snap_depths(double a, double b, int R, int* o1, int* o2) {
  double best = 0;
  bool found = false;
  for (int x = 1; x < R; ++x)
    for (int y = x + 1; y < R; ++y) {
      if (y % x || R % x) continue;
      double f = steps_bound(x, y, a, b, R);
      if (!found || f < best) best = f, *o1 = x, *o2 = y, found = true;
    }
  return found;
}

bool validate_model(const loopspec_model* m, int* why) {
  *why = LOOPSPEC_EINVAL;
  if (!m) return false;
  if (m->vocab <= 0 || m->hidden <= 0 || m->n_q_heads <= 0 || m->n_kv_heads <= 0 || m->ffn <= 0 || m->R < 2 ||
      m->n_recurrent <= 0 || (m->weight_dtype != 0 && m->weight_dtype != 1) || !(m->rms_eps > 0) || !(m->rope_theta > 0))
    return false;
  if (m->n_q_heads % m->n_kv_heads) return false;
  if (m->n_prelude < 0 || m->n_coda < 0) return false;
  *why = LOOPSPEC_EUNSUPPORTED;
  if (m->head_dim != 64 && m->head_dim != 128) return false;
  int g = m->n_q_heads / m->n_kv_heads;
  if (g != 1 && g != 4) return false;
  if (m->hidden % 128 || (m->n_q_heads * m->head_dim) % 128 || (m->n_kv_heads * m->head_dim) % 128) return false;
  if (m->ffn % 16 || m->vocab % 16) return false;
  return true;
}

bool resolve_sched(const loopspec_model* m, const loopspec_sched* s, Derived* d, int* why) {
  *why = LOOPSPEC_EINVAL;
  if (!s || s->max_seqs <= 0 || s->max_ctx < 4 || s->temperature < 0 || s->max_prefill_rows < 0) return false;
  if (s->top_k < 0 || s->top_p < 0.f || s->top_p != s->top_p) return false;
  int d1 = s->d1, d2 = s->d2;
  if (d1 == 0 && d2 == 0) {
    if (!(s->alpha > 0) || !(s->beta > 0)) return false;
    if (!snap_depths(s->alpha, s->beta, m->R, &d1, &d2)) {  // R too small for two proposals
      d1 = 1, d2 = 0;
    }
  }
  if (d1 < 1 || d1 >= m->R || m->R % d1) return false;
  if (d2 != 0 && (d2 <= d1 || d2 >= m->R || d2 % d1)) return false;
  d->d1 = d1, d->d2 = d2;
  *why = LOOPSPEC_ECAPACITY;
  d->S = s->max_seqs;
  d->B = max_branches(m->R, d1, d2);
  d->NB = 2 * d->B + 1;
  if (m->R / d1 > MAX_SPEC) return false;
  if (d->S > MAX_SEQS || d->S * d->NB > MAX_NODES || d->S * d->B > MAX_ROWS) return false;
  d->max_rows_dec = d->S * d->B;
  d->max_rows_pf = s->max_prefill_rows ? s->max_prefill_rows : 32;
  if (d->max_rows_pf > GROUP_ROWS) return false;
  {  // rows of the pass buffers: one group of 8 / 16 / 32 / 64 token columns, or whole groups of 64
    const int need = std::max(d->max_rows_dec, d->max_rows_pf);
    d->max_rows = need <= GROUP_ROWS ? 8 * ng_for_rows(need) : (need + GROUP_ROWS - 1) / GROUP_ROWS * GROUP_ROWS;
  }
  d->slots = s->max_ctx + d->NB;
  d->ids_cap = s->max_ctx;
  d->n_pre = m->n_prelude, d->n_coda = m->n_coda, d->raven = (m->n_prelude || m->n_coda) ? 1 : 0;
  d->NL = m->n_prelude + m->n_recurrent + m->n_coda;
  d->n_classes = d->raven ? (d2 ? 3 : 2) : 0;  // coda caches: depth d1, depth d2 (if any), depth R
  d->class_depth[0] = d1, d->class_depth[1] = d2 ? d2 : m->R, d->class_depth[2] = m->R;
  if (d->raven && d->n_classes > m->R) return false;  // the pool gives every layer R planes
  d->hid_coda_base = d->S * d->NB + GROUP_ROWS;
  d->n_hid = d->S * d->NB + GROUP_ROWS + (d->raven ? MAX_ROWS : 0);  // branches, prefill rows, copies for the coda pass
  d->p_logit_base = d->S * d->NB * 2;
  d->n_logit_vecs = d->p_logit_base + d->S;
  d->n_sq = m->hidden / 128;  // row blocks of the residual GEMMs = partial sums of squares per row
  d->sq_stride = std::max(d->n_sq, 64);  // room for one partial per cluster of the persistent pass kernel
  d->max_chunks = (s->max_ctx + ATT_CHUNK - 1) / ATT_CHUNK;
  d->att_mode = d->S >= 2 ? 1 : 0;
  d->att_runs = d->max_chunks > (d->att_mode ? ATT_BATCH_SINGLE : ATT_MAX_RUNS) ? 1 : 0;
  d->trace_cap = m->R * s->max_ctx + 64;  // a token can take R passes (restart)
  d->Hq = m->n_q_heads * m->head_dim;
  d->Hkv = m->n_kv_heads * m->head_dim;
  return true;
}

// bytes of one matrix in the tile-major streaming layout (bf16 weights only; fp32 weights are used in place)
size_t packed_bytes(int N, int K) { return align_up((size_t)(N / 16) * ((K + 31) / 32) * 1024); }
size_t packed_total_bytes(const loopspec_model* m, const Derived& d) {
  if (m->weight_dtype != 1) return 0;
  size_t per_layer = packed_bytes(d.Hq + 2 * d.Hkv, m->hidden) + packed_bytes(m->hidden, d.Hq) +
                     packed_bytes(2 * m->ffn, m->hidden) + packed_bytes(m->hidden, m->ffn);
  return per_layer * d.NL + packed_bytes(m->vocab, m->hidden) + (d.raven ? packed_bytes(m->hidden, 2 * m->hidden) : 0);
}

Layout make_layout(const loopspec_model* m, const loopspec_sched* s, const Derived& d) {
  Layout L;
  size_t o = 0;
  auto take = [&](size_t bytes) {
    size_t at = o;
    o = align_up(o + bytes);
    return at;
  };
  const size_t MR = d.max_rows;
  L.wpack = take(packed_total_bytes(m, d));
  L.rope = take((size_t)s->max_ctx * (m->head_dim / 2) * sizeof(float2));
  L.kv = take((size_t)d.NL * m->R * 2 * d.S * m->n_kv_heads * d.slots * m->head_dim * 2);
  L.hid = take((size_t)d.n_hid * m->hidden * 4);
  L.estore = take(d.raven ? (size_t)d.n_hid * m->hidden * 4 : 0);
  L.cplanes = take(d.raven ? MR * 3 * 2 * m->hidden * 2 : 0);
  L.qbuf = take(MR * d.Hq * 4);
  L.xplanes = take(MR * 3 * m->hidden * 2);
  L.aplanes = take(MR * 3 * d.Hq * 2);
  L.splanes = take(MR * 3 * m->ffn * 2);
  L.sumsq = take(MR * d.sq_stride * 4);
  L.logits = take((size_t)d.n_logit_vecs * m->vocab * 4);
  L.argpart = take(MR * ((m->vocab + 127) / 128) * sizeof(float2));
  {  // k-split partial sums of the GEMMs that run on the tcgen05 kernel (the largest of them, prefill or decode columns)
    size_t need = 0;
    if (tc_prefill_shapes_ok(m)) {
      const int Ns[5] = {d.Hq + 2 * d.Hkv, m->hidden, 2 * m->ffn, m->hidden, m->hidden};
      const int Ks[5] = {m->hidden, d.Hq, m->hidden, m->ffn, 2 * m->hidden};
      const int groups = (d.max_rows_dec + GROUP_ROWS - 1) / GROUP_ROWS;  // decode passes: one slice per group of 64 columns
      const size_t cols = std::max((size_t)tc_pf_cols(d.max_rows_pf), (size_t)groups * tc_pf_cols(std::min(d.max_rows_dec, (int)GROUP_ROWS)));
      for (int i = 0; i < (d.raven ? 5 : 4); ++i) need = std::max(need, (size_t)tc_pf_plan(Ns[i], Ks[i]).n_split * cols * Ns[i] * 4);
    }
    L.tcpart = take(need);
  }
  L.tune_bytes = kTune ? (size_t)1 << 20 : 0;  // kernel timeline of tuning builds
  L.tune = take(L.tune_bytes);
  int G = m->n_q_heads / m->n_kv_heads;
  L.apart = take(MR * m->n_kv_heads * d.max_chunks * G * (m->head_dim + 2) * 4);
  L.acnt = take(MR * m->n_q_heads * 4);  // arrival counters per (row, kv head) of the decode kernels, (row, query head) of the prefill kernel
  L.nodes = take((size_t)13 * MAX_NODES * 4);
  L.flt = take((size_t)2 * MAX_NODES * sizeof(float4));
  L.sel_flt = take((size_t)MAX_ROWS * sizeof(float4));
  L.seqs = take((size_t)5 * MAX_SEQS * 4);
  L.ctr = take(sizeof(Counters));
  L.tv = take((size_t)MAX_SEQS * 4 * sizeof(double));
  L.tab_dec = take(sizeof(RowTable));
  L.tab_pf = take(sizeof(RowTable));
  L.tab_pre = take(sizeof(RowTable));
  L.tab_coda = take(sizeof(RowTable));
  L.tab_pfc = take(sizeof(RowTable));
  L.tab_vanc = take(sizeof(RowTable));
  L.tab_van = take(sizeof(RowTable) * m->R);
  L.sel_tok = take(MAX_ROWS * 4);
  L.sel_aux = take(MAX_ROWS * 4);
  L.sel_lse = take(MAX_ROWS * 4);
  L.sel_z2 = take(MAX_ROWS * 4);
  L.kvcopy = take(MAX_SEQS * sizeof(KvCopyCmd));
  L.out_ids = take((size_t)d.S * d.ids_cap * 4);
  L.commits = take((size_t)d.S * d.ids_cap * 8 * 4);
  L.trace = take((size_t)d.trace_cap * 4);
  L.trace_n = take(4);
  L.prompt = take((size_t)s->max_ctx * 4);
  L.total = o;
  return L;
}

}  // namespace

struct loopspec_ctx {
  loopspec_model m;
  loopspec_sched s;
  Derived d;
  Layout L;
  cudaStream_t stream = nullptr;
  unsigned char* ws = nullptr;
  const void* embed = nullptr;
  const void* lm_head = nullptr;
  const float* final_norm = nullptr;
  std::vector<const void*> layers;  // 6 per layer: prelude blocks, recurrent blocks, coda blocks
  std::vector<const void*> packed;  // 4 per layer (qkv, o, gate/up, down), then lm_head, then the adapter; empty for fp32 weights
  const void* adapter = nullptr;    // Raven-style layout: [H][2H]
  int n_sm = 148;
  int ng_dec = 1, ng_pf = 1;
  GemmPlan plan[6];      // mma.sync kernels of the decode passes
  GemmPlan plan_pf[6];   // ... of prefill passes that run on them (clusters of up to 8: the receive buffer of a wide pass
                         // holds several columns per rank)
  const GemmPlan* cur_plan = plan;  // the set the launch helpers read (loopspec_prefill switches it for its duration)
  // prefill on the tcgen05 kernel: tensor maps of the row-major weights (4 per layer) and of the three plane buffers
  // ... and the decode passes of contexts whose passes carry 9 to 64 rows (batches, deep recurrences), where the
  // mma.sync kernels are bound by their three-plane arithmetic rather than by the weight stream
  struct TcCfg {
    bool on = false;
    int cols = 0, stages = 0;   // token columns of a launch (multiple of 16), ring stages
    size_t smem = 0;
    CUtensorMap xmaps[4];       // planes read by QKV and gate/up, by O, by down, by the adapter
  };
  TcCfg tc[2];                  // 0: prefill passes, 1: decode passes
  std::vector<CUtensorMap> tc_wmaps;  // 4 per block, then the adapter
  TcPfPlan tc_plan[5];          // qkv, o, gate/up, down, adapter
  // readout GEMM of the decode passes on the tcgen05 kernel (bf16 weights): plan, tensor maps of the row-major lm_head
  // (one box per 128-row tile) and of the hidden-state planes (all three planes of dg_mp rows in one box)
  bool dg = false;
  int dg_mp = 8;
  DgPlan dgp;
  CUtensorMap dg_wmap, dg_xmap;
  long long dg_wait_cycles = TC_WAIT_CYCLES;
  int dg_drop_unit = -1;  // test hook: see loopspec_debug_fail_next_step
  volatile int* host_flags = nullptr;  // pinned + mapped
  int* host_flags_dev = nullptr;
  int* pin_ids = nullptr;              // pinned staging for prompt / ids
  size_t pin_ids_cap = 0;
  cudaGraphExec_t g_step = nullptr, g_vanilla = nullptr;
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  std::vector<char> prefilled;
  bool pending_verify = false, sticky = false, vanilla_mode = false, use_pdl = true;
  bool pf_attn = false;  // prefill passes run the attention kernel that shares K/V chunks among the rows
  bool filters = false;  // C applies top-k / top-p (sampling only)
  int sel_staged = 0;    // the selection kernel keeps its row slices in shared memory
  size_t sel_smem = 0;
  int launches_per_step = 0;
  std::string err;

  template <typename T>
  T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
  NodeTable nodes() const {
    int* b = at<int>(L.nodes);
    NodeTable n;
    n.state = b, n.depth = b + MAX_NODES, n.pos = b + 2 * MAX_NODES, n.token = b + 3 * MAX_NODES;
    n.parent = b + 4 * MAX_NODES, n.child1 = b + 5 * MAX_NODES, n.child2 = b + 6 * MAX_NODES, n.tok1 = b + 7 * MAX_NODES;
    n.tok2 = b + 8 * MAX_NODES, n.has2 = b + 9 * MAX_NODES;
    n.lse1 = reinterpret_cast<float*>(b + 10 * MAX_NODES), n.lse2 = reinterpret_cast<float*>(b + 11 * MAX_NODES);
    n.z2 = reinterpret_cast<float*>(b + 12 * MAX_NODES);
    n.flt1 = at<float4>(L.flt), n.flt2 = n.flt1 + MAX_NODES;
    return n;
  }
  SeqState seqs() const {
    int* b = at<int>(L.seqs);
    SeqState q;
    q.root = b, q.n_ids = b + MAX_SEQS, q.n_dec = b + 2 * MAX_SEQS, q.n_target = b + 3 * MAX_SEQS, q.need_verify = b + 4 * MAX_SEQS;
    return q;
  }
  long long kv_sel_stride() const { return (long long)d.S * m.n_kv_heads * d.slots * m.head_dim; }
  long long kv_plane_stride() const { return 2 * kv_sel_stride(); }
  long long kv_layer_stride() const { return (long long)m.R * kv_plane_stride(); }
};

namespace {

// a named range around a C-ABI call (prefill, step, verify, decode), visible on a profiler's timeline
struct Range {
#ifdef LOOPSPEC_NVTX
  explicit Range(const char* name) { nvtxRangePushA(name); }
  ~Range() { nvtxRangePop(); }
#else
  explicit Range(const char*) {}
#endif
};

int fail(loopspec_ctx* c, int code, const char* fmt, ...) {
  if (c) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    c->err = buf;
    if (code == LOOPSPEC_ECUDA) c->sticky = true;
  }
  return code;
}

#define CU(c, call)                                                                                       \
  do {                                                                                                    \
    cudaError_t e_ = (call);                                                                              \
    if (e_ != cudaSuccess) return fail(c, LOOPSPEC_ECUDA, "%s failed: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

// ---- kernel dispatch ---------------------------------------------------------------------------------
using GemmFn = void (*)(const GemmParams);

template <int NG>
GemmFn gemm_fn_epi(int wdt, int epi) {
  if (wdt == 1) {
    switch (epi) {
      case EPI_PLAIN: return gemm_bf16_kernel<NG, EPI_PLAIN>;
      case EPI_QKV: return gemm_bf16_kernel<NG, EPI_QKV>;
      case EPI_RESID: return gemm_bf16_kernel<NG, EPI_RESID>;
      case EPI_SWIGLU: return gemm_bf16_kernel<NG, EPI_SWIGLU>;
      default: return gemm_bf16_kernel<NG, EPI_LOGITS>;
    }
  }
  switch (epi) {
    case EPI_PLAIN: return gemm_f32_kernel<NG, EPI_PLAIN>;
    case EPI_QKV: return gemm_f32_kernel<NG, EPI_QKV>;
    case EPI_RESID: return gemm_f32_kernel<NG, EPI_RESID>;
    case EPI_SWIGLU: return gemm_f32_kernel<NG, EPI_SWIGLU>;
    default: return gemm_f32_kernel<NG, EPI_LOGITS>;
  }
}
GemmFn gemm_fn(int wdt, int ng, int epi) {
  switch (ng) {
    case 1: return gemm_fn_epi<1>(wdt, epi);
    case 2: return gemm_fn_epi<2>(wdt, epi);
    case 4: return gemm_fn_epi<4>(wdt, epi);
    default: return gemm_fn_epi<8>(wdt, epi);
  }
}
int gemm_smem(int wdt, int ng) { return wdt == 1 ? gemm_smem_bytes(ng) : gemm_f32_smem_bytes(ng); }

// Launch with programmatic stream serialization: the kernel may start while its predecessor in the stream is
// still running; it orders itself with griddepcontrol.wait before touching anything the predecessor writes.
template <typename P>
cudaError_t launch_k(void (*fn)(const P), dim3 grid, dim3 block, size_t smem, cudaStream_t st, const P& params, bool pdl,
                     int cluster = 1) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = grid, cfg.blockDim = block, cfg.dynamicSmemBytes = smem, cfg.stream = st;
  cudaLaunchAttribute at[2];
  int n = 0;
  if (pdl) {
    at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster > 1) {
    at[n].id = cudaLaunchAttributeClusterDimension;
    at[n].val.clusterDim.x = cluster, at[n].val.clusterDim.y = 1, at[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = at, cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, fn, params);
}

cudaError_t launch_gemm(int wdt, int ng, int epi, const GemmParams& p, cudaStream_t st, bool pdl = true) {
  return launch_k(gemm_fn(wdt, ng, epi), dim3(p.n_clusters * p.cluster_size), dim3(GEMM_THREADS), (size_t)gemm_smem(wdt, ng), st, p,
                  pdl, p.cluster_size);
}

using AttnFn = void (*)(const AttnParams);
AttnFn attn_fn(int d, int G, bool runs) {  // runs: rows of this context can have work items of several chunks
  if (runs) {
    if (d == 128) return G == 1 ? attn_runs_kernel<128, 1> : attn_runs_kernel<128, 4>;
    return G == 1 ? attn_runs_kernel<64, 1> : attn_runs_kernel<64, 4>;
  }
  if (d == 128) return G == 1 ? attn_kernel<128, 1> : attn_kernel<128, 4>;
  return G == 1 ? attn_kernel<64, 1> : attn_kernel<64, 4>;
}

// dynamic shared memory and grid of the attention launch (the streaming kernel of long contexts: its rings, and one
// CTA per slot the SMs offer)
size_t attn_smem(int d, int G, bool runs) {
  if (!runs) return 0;
  if (d == 128) return G == 1 ? AtsCfg<128, 1>::SMEM_BYTES : AtsCfg<128, 4>::SMEM_BYTES;
  return G == 1 ? AtsCfg<64, 1>::SMEM_BYTES : AtsCfg<64, 4>::SMEM_BYTES;
}
int attn_grid(int n_sm, int G, bool runs) { return runs ? n_sm * (G == 1 ? AtsCfg<128, 1>::MIN_CTAS : AtsCfg<128, 4>::MIN_CTAS) : n_sm * 8; }

// tuning builds (-DLOOPSPEC_TUNE) with LOOPSPEC_DBG set record a kernel timeline in a workspace region of their own
unsigned long long* tune_timeline(loopspec_ctx* c) {
  return (kTune && c->L.tune_bytes && getenv("LOOPSPEC_DBG")) ? reinterpret_cast<unsigned long long*>(c->ws + c->L.tune) : nullptr;
}

// ---- one batched pass through the shared block stack (all layers) on the rows of `tab` ------------------
enum { G_QKV = 0, G_O = 1, G_GU = 2, G_DOWN = 3, G_LM = 4, G_ADAPT = 5 };
const int kEpiOf[6] = {EPI_QKV, EPI_RESID, EPI_SWIGLU, EPI_RESID, EPI_LOGITS, EPI_RESID};
// `layer` is the index in the list prelude blocks | recurrent blocks | coda blocks
bool first_of_stack(const Derived& d, int n_rec, int layer) { return layer == 0 || layer == d.n_pre || layer == d.n_pre + n_rec; }
bool last_of_stack(const Derived& d, int n_rec, int layer) {
  return layer == d.n_pre - 1 || layer == d.n_pre + n_rec - 1 || layer == d.NL - 1;
}

GemmParams gemm_params(loopspec_ctx* c, int which, int layer, const RowTable* tab, int col0 = 0) {
  const loopspec_model& m = c->m;
  const Derived& d = c->d;
  GemmParams p;
  memset(&p, 0, sizeof p);
  const GemmPlan& g = c->cur_plan[which];
  p.n_rb = g.n_rb, p.kb_per_rb = g.kpr, p.cluster_size = g.cs, p.n_clusters = g.n_clusters;
  p.hid = c->at<float>(c->L.hid), p.H = m.hidden, p.eps = m.rms_eps, p.tab = tab;
  p.err = c->host_flags_dev + HF_ERROR;
  const void* const* lp = (which == G_LM || which == G_ADAPT) ? nullptr : &c->layers[6 * layer];
  __nv_bfloat16* xpl = c->at<__nv_bfloat16>(c->L.xplanes);
  switch (which) {
    case G_QKV:
      p.W = c->packed.empty() ? lp[1] : c->packed[4 * layer + 0], p.N = d.Hq + 2 * d.Hkv, p.K = m.hidden;
      p.xplanes = xpl, p.x_ld = m.hidden;
      // the first block of a stack reads the full sums its preparation kernel wrote (the recurrent blocks of a
      // Raven-style model follow the adapter, which leaves partials like every other residual GEMM); later blocks
      // read the down projection's partials
      p.sumsq = c->at<float>(c->L.sumsq), p.sq_stride = d.sq_stride;
      p.n_sq = (first_of_stack(d, m.n_recurrent, layer) && !(d.raven && layer == d.n_pre)) ? 1 : d.n_sq;
      if (!c->packed.empty() ) p.perm = 2, p.perm_a = m.head_dim / 32, p.perm_d = m.head_dim;
      p.qbuf = c->at<float>(c->L.qbuf);
      p.kv = c->at<__nv_bfloat16>(c->L.kv) + (size_t)layer * c->kv_layer_stride();
      p.kv_plane_stride = c->kv_plane_stride(), p.kv_sel_stride = c->kv_sel_stride();
      p.slots = d.slots, p.n_kv_heads = m.n_kv_heads, p.n_q_heads = m.n_q_heads, p.head_dim = m.head_dim;
      p.rope = c->at<float2>(c->L.rope);
      break;
    case G_O:
      p.W = c->packed.empty() ? lp[2] : c->packed[4 * layer + 1], p.N = m.hidden, p.K = d.Hq;
      p.xplanes = c->at<__nv_bfloat16>(c->L.aplanes), p.x_ld = d.Hq;
      p.sumsq_out = c->at<float>(c->L.sumsq), p.n_sq_out = d.sq_stride;
      p.out_planes = xpl, p.planes_ld = m.hidden, p.gain_next = static_cast<const float*>(lp[3]);
      break;
    case G_GU:
      p.W = c->packed.empty() ? lp[4] : c->packed[4 * layer + 2], p.N = 2 * m.ffn, p.K = m.hidden, p.F = m.ffn;
      if (!c->packed.empty() ) p.perm = 1, p.perm_a = m.ffn;
      p.xplanes = xpl, p.x_ld = m.hidden;
      p.sumsq = c->at<float>(c->L.sumsq), p.n_sq = d.n_sq, p.sq_stride = d.sq_stride;
      p.out_planes = c->at<__nv_bfloat16>(c->L.splanes), p.planes_ld = m.ffn;
      break;
    case G_DOWN:
      p.W = c->packed.empty() ? lp[5] : c->packed[4 * layer + 3], p.N = m.hidden, p.K = m.ffn;
      p.xplanes = c->at<__nv_bfloat16>(c->L.splanes), p.x_ld = m.ffn;
      p.sumsq_out = c->at<float>(c->L.sumsq), p.n_sq_out = d.sq_stride;
      // planes for the next consumer of the residual stream: the next layer's first norm, or - after the last
      // layer - the final norm of the readout (the lm_head picks the reading-out rows out of them)
      p.out_planes = xpl, p.planes_ld = m.hidden;
      p.gain_next = last_of_stack(d, m.n_recurrent, layer) ? c->final_norm : static_cast<const float*>(c->layers[6 * (layer + 1)]);
      break;
    case G_ADAPT:  // H <- W_a [H; e]: replaces the stream; leaves planes and sums of squares for the first recurrent block
      p.W = c->packed.empty() ? c->adapter : c->packed[4 * d.NL + 1], p.N = m.hidden, p.K = 2 * m.hidden;
      p.xplanes = c->at<__nv_bfloat16>(c->L.cplanes), p.x_ld = 2 * m.hidden, p.no_resid = 1;
      p.sumsq_out = c->at<float>(c->L.sumsq), p.n_sq_out = d.sq_stride;
      p.out_planes = xpl, p.planes_ld = m.hidden, p.gain_next = static_cast<const float*>(c->layers[6 * d.n_pre]);
      break;
    default:
      p.W = c->packed.empty() ? c->lm_head : c->packed[4 * d.NL], p.N = m.vocab, p.K = m.hidden;
      p.xplanes = xpl, p.x_ld = m.hidden, p.cols_from_readout = 1;
      // 1/rms from the partial sums of squares the last down projection left for the row
      p.sumsq = c->at<float>(c->L.sumsq), p.n_sq = d.n_sq, p.sq_stride = d.sq_stride;
      p.logits = c->at<float>(c->L.logits), p.argpart = c->at<float2>(c->L.argpart);
      break;
  }
  if (col0 > 0) {  // a later group of token columns: its slices of the per-column buffers
    p.col0 = col0;
    if (which == G_LM) {
      p.argpart += (size_t)col0 * p.n_rb;  // the planes and sums of squares are addressed by pass row, not by column
    } else {
      p.xplanes += (size_t)col0 * 3 * p.x_ld;
      if (p.out_planes) p.out_planes += (size_t)col0 * 3 * p.planes_ld;
      if (p.sumsq) p.sumsq += (size_t)col0 * p.sq_stride;
      if (p.sumsq_out) p.sumsq_out += (size_t)col0 * p.n_sq_out;
      if (p.qbuf) p.qbuf += (size_t)col0 * d.Hq;
    }
  }
  return p;
}

// planes and sums of squares for the first block of a stack (`first_layer`); use_src: on copies of the rows' states
cudaError_t launch_prep(loopspec_ctx* c, const RowTable* tab, int first_layer = 0, bool use_src = false) {
  PrepParams q;
  memset(&q, 0, sizeof q);
  q.tab = tab, q.hid = c->at<float>(c->L.hid), q.K = c->m.hidden, q.planes = c->at<__nv_bfloat16>(c->L.xplanes);
  q.gain = static_cast<const float*>(c->layers[6 * first_layer]), q.sumsq = c->at<float>(c->L.sumsq), q.sq_stride = c->d.sq_stride;
  q.use_src = use_src ? 1 : 0;
  return launch_k(prep_planes_kernel, dim3(c->d.max_rows), dim3(256), 0, c->stream, q, c->use_pdl);
}


int col_groups(loopspec_ctx* c, const RowTable* tab);
// one layer GEMM of a prefill pass on the tcgen05 kernel: raw k-split sums, then the fused epilogue
template <int EPI>
cudaError_t launch_tc_epi(const TcEpiParams& q, int groups, cudaStream_t st, bool pdl) {
  if (groups > 1) return launch_k(tc_epilogue_kernel<EPI, true>, dim3(q.g.n_rb, TCE_GROUPS, groups), dim3(GEMM_THREADS), 0, st, q, pdl);
  return launch_k(tc_epilogue_kernel<EPI, false>, dim3(q.g.n_rb, TCE_GROUPS), dim3(GEMM_THREADS), 0, st, q, pdl);
}
cudaError_t launch_tc_gemm(loopspec_ctx* c, int which, int layer, const RowTable* tab, int cfg_i) {
  const loopspec_ctx::TcCfg& tc = c->tc[cfg_i];
  const int pi = which == G_ADAPT ? 4 : which;
  const TcPfPlan& t = c->tc_plan[pi];
  TcEpiParams q;
  // one grid plane per group of 64 token columns (a plane whose group holds no row returns at once)
  const int groups = cfg_i == 1 ? col_groups(c, tab) : 1;
  q.g = gemm_params(c, which, layer, tab);
  q.g.cluster_size = TCE_GROUPS, q.g.recv_ranks = 1, q.Hq = c->d.Hq;
  q.part = c->at<float>(c->L.tcpart), q.n_split = t.n_split, q.cols_ld = tc.cols;
  LinearTcParams p;
  memset(&p, 0, sizeof p);
  p.out = c->at<float>(c->L.tcpart);
  p.M = tc.cols, p.MP = tc.cols, p.N = q.g.N, p.K = q.g.K, p.kb_per_split = t.kb_per_split, p.stages = tc.stages;
  p.err = const_cast<int*>(c->host_flags_dev + HF_ERROR), p.err_code = 5, p.x3d = 1;
  p.row0 = 0, p.group_cols = GROUP_ROWS, p.group_stride = (long long)t.n_split * tc.cols * q.g.N;
  // (only a pass of several groups can have an empty one worth skipping)
  p.n_live = groups > 1 ? reinterpret_cast<const int*>(reinterpret_cast<const char*>(tab) + offsetof(RowTable, n_rows)) : nullptr;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3(t.n_tiles, t.n_split, groups), cfg.blockDim = dim3(TC_THREADS), cfg.dynamicSmemBytes = tc.smem, cfg.stream = c->stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at, cfg.numAttrs = c->use_pdl ? 1 : 0;
  const int xi = which == G_O ? 1 : which == G_DOWN ? 2 : which == G_ADAPT ? 3 : 0;
  const CUtensorMap& wm = which == G_ADAPT ? c->tc_wmaps[4 * c->d.NL] : c->tc_wmaps[4 * layer + which];
  cudaError_t e = cudaLaunchKernelEx(&cfg, linear_tc_kernel, wm, tc.xmaps[xi], p);
  if (e != cudaSuccess) return e;
  switch (which) {
    case G_QKV: return launch_tc_epi<EPI_QKV>(q, groups, c->stream, c->use_pdl);
    case G_GU: return launch_tc_epi<EPI_SWIGLU>(q, groups, c->stream, c->use_pdl);
    default: return launch_tc_epi<EPI_RESID>(q, groups, c->stream, c->use_pdl);
  }
}

using DgFn = void (*)(const CUtensorMap, const CUtensorMap, const DgParams);
DgFn dg_fn(int epi) { return epi == EPI_LOGITS ? dgemm_kernel<EPI_LOGITS> : dgemm_kernel<EPI_PLAIN>; }
cudaError_t launch_dg_raw(int epi, const DgPlan& g, const CUtensorMap& mw, const CUtensorMap& mx, const DgParams& q, cudaStream_t st,
                          bool pdl) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3(g.n_clusters * g.cs), cfg.blockDim = dim3(DG_THREADS), cfg.dynamicSmemBytes = g.smem, cfg.stream = st;
  cudaLaunchAttribute at[2];
  int n = 0;
  if (pdl) {
    at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (g.cs > 1) {
    at[n].id = cudaLaunchAttributeClusterDimension;
    at[n].val.clusterDim.x = g.cs, at[n].val.clusterDim.y = 1, at[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = at, cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, dg_fn(epi), mw, mx, q);
}
// the readout GEMM of a decode pass on the tcgen05 kernel
cudaError_t launch_dg_lm(loopspec_ctx* c, const RowTable* tab) {
  const DgPlan& g = c->dgp;
  DgParams q;
  memset(&q, 0, sizeof q);
  q.g = gemm_params(c, G_LM, 0, tab);
  q.g.cluster_size = g.cs, q.g.n_clusters = g.n_clusters, q.g.n_rb = g.n_rb;
  q.g.err = c->host_flags_dev + HF_ERROR, q.g.tl_id = 120;
  q.MP = c->dg_mp, q.stages = g.stages, q.acc_bufs = g.acc_bufs, q.recv_bufs = g.recv_bufs, q.err_code = ERR_WAIT;
  q.wait_cycles = c->dg_wait_cycles;
  q.drop_unit = c->dg_drop_unit;
  return launch_dg_raw(EPI_LOGITS, g, c->dg_wmap, c->dg_xmap, q, c->stream, c->use_pdl);
}

// launches a GEMM of a pass over `tab` takes: decode passes that can carry more than 64 rows run every GEMM once per group of
// 64 token columns (a launch whose group holds no row returns at once); prefill passes carry at most 64 rows
int col_groups(loopspec_ctx* c, const RowTable* tab) {
  if (tab == c->at<RowTable>(c->L.tab_pf) || tab == c->at<RowTable>(c->L.tab_pfc)) return 1;
  return (c->d.max_rows_dec + GROUP_ROWS - 1) / GROUP_ROWS;
}

// decode attention of block `l` on the rows of `tab`
cudaError_t launch_attention(loopspec_ctx* c, const RowTable* tab, int l, unsigned long long* tl, int tl_id, bool prefill_rows = false) {
  const loopspec_model& m = c->m;
  const Derived& d = c->d;
  const int G = m.n_q_heads / m.n_kv_heads;
  AttnParams a;
  memset(&a, 0, sizeof a);
  a.tab = tab, a.qbuf = c->at<float>(c->L.qbuf), a.aplanes = c->at<__nv_bfloat16>(c->L.aplanes);
  a.kv = c->at<__nv_bfloat16>(c->L.kv) + (size_t)l * c->kv_layer_stride();
  a.kv_plane_stride = c->kv_plane_stride(), a.kv_sel_stride = c->kv_sel_stride();
  a.slots = d.slots, a.n_kv_heads = m.n_kv_heads, a.n_q_heads = m.n_q_heads;
  a.scale = 1.0f / sqrtf((float)m.head_dim);
  a.part = c->at<float>(c->L.apart), a.max_chunks = d.max_chunks, a.counters = c->at<int>(c->L.acnt);
  a.tl = tl, a.tl_id = tl_id;
  if (prefill_rows && c->pf_attn) {  // consecutive prompt positions of one sequence: the rows share every K/V chunk
    const dim3 fold_grid(d.max_rows_pf, m.n_q_heads);
    cudaError_t e;
    if (m.head_dim == 128) {
      if ((e = launch_k(attn_prefill_mma_kernel<128>, dim3(c->n_sm * 2), dim3(ATT_THREADS), (size_t)AtmCfg<128>::SMEM_BYTES, c->stream, a, c->use_pdl)))
        return e;
      return launch_k(attn_prefill_fold_kernel<128>, fold_grid, dim3(32), 0, c->stream, a, c->use_pdl);
    }
    if ((e = launch_k(attn_prefill_mma_kernel<64>, dim3(c->n_sm * 2), dim3(ATT_THREADS), (size_t)AtmCfg<64>::SMEM_BYTES, c->stream, a, c->use_pdl)))
      return e;
    return launch_k(attn_prefill_fold_kernel<64>, fold_grid, dim3(16), 0, c->stream, a, c->use_pdl);
  }
  const bool runs = d.att_runs != 0;
  return launch_k(attn_fn(m.head_dim, G, runs), dim3(attn_grid(c->n_sm, G, runs)), dim3(ATT_THREADS), attn_smem(m.head_dim, G, runs), c->stream, a,
                  c->use_pdl);
}

// the blocks [l0, l0 + count) of the layer list on the rows of `tab`
cudaError_t launch_stack(loopspec_ctx* c, const RowTable* tab, int ng, int l0, int count, int* n_launch, int tc) {
  const loopspec_model& m = c->m;
  const Derived& d = c->d;
  const int G = m.n_q_heads / m.n_kv_heads;
  const bool pdl = c->use_pdl;
  cudaError_t e;
  const int groups = col_groups(c, tab);
  // a GEMM of the pass: one launch per group of token columns (one group unless a decode pass can carry more than 64 rows)
  auto gemm = [&](int which, int l, int tl_id) -> cudaError_t {
    if (tc >= 0) return launch_tc_gemm(c, which, l, tab, tc);  // (all groups of token columns in one pair of launches)
    for (int g = 0; g < groups; ++g) {
      GemmParams gp = gemm_params(c, which, l, tab, g * GROUP_ROWS);
      gp.tl = tune_timeline(c), gp.tl_id = tl_id;
      cudaError_t e2 = launch_gemm(m.weight_dtype, ng, kEpiOf[which], gp, c->stream, pdl);
      if (e2) return e2;
    }
    return cudaSuccess;
  };
  for (int l = l0; l < l0 + count; ++l) {
    unsigned long long* tl = tune_timeline(c);
    if ((e = gemm(G_QKV, l, l * 5 + 0))) return e;
    if ((e = launch_attention(c, tab, l, tl, l * 5 + 1, tab == c->at<RowTable>(c->L.tab_pf) || tab == c->at<RowTable>(c->L.tab_pfc)))) return e;
    if ((e = gemm(G_O, l, l * 5 + 2))) return e;
    if ((e = gemm(G_GU, l, l * 5 + 3))) return e;
    if ((e = gemm(G_DOWN, l, l * 5 + 4))) return e;
    if (n_launch) *n_launch += 1 + 4 * (tc >= 0 ? 2 : groups);
  }
  return cudaSuccess;
}

// One batched pass of B over the rows of `tab` (Sec. 4.2 step 1).  Ouro layout: preparation + the shared blocks.
// Raven-style layout: the rows entering their first recurrence (`tab_pre`, may be null) go through the prelude blocks,
// then every row through the adapter on [H; e] and the recurrent blocks.
cudaError_t launch_layers(loopspec_ctx* c, const RowTable* tab, int ng, int* n_launch, int tc = -1, const RowTable* tab_pre = nullptr) {
  const loopspec_model& m = c->m;
  const Derived& d = c->d;
  cudaError_t e;
  if (!d.raven) {
    if ((e = launch_prep(c, tab))) return e;
    if (n_launch) *n_launch += 1;
    return launch_stack(c, tab, ng, 0, m.n_recurrent, n_launch, tc);
  }
  if (tab_pre && d.n_pre > 0) {
    if ((e = launch_prep(c, tab_pre, 0))) return e;
    if ((e = launch_stack(c, tab_pre, ng, 0, d.n_pre, n_launch, tc))) return e;
    if (n_launch) *n_launch += 1;
  }
  ConcatParams cp;
  cp.tab = tab, cp.hid = c->at<float>(c->L.hid), cp.e_store = c->at<float>(c->L.estore), cp.H = m.hidden;
  cp.planes = c->at<__nv_bfloat16>(c->L.cplanes);
  if ((e = launch_k(raven_concat_kernel, dim3(d.max_rows), dim3(256), 0, c->stream, cp, c->use_pdl))) return e;
  const int groups = col_groups(c, tab);
  if (tc >= 0) {
    if ((e = launch_tc_gemm(c, G_ADAPT, 0, tab, tc))) return e;
  } else {
    for (int g = 0; g < groups; ++g)
      if ((e = launch_gemm(m.weight_dtype, ng, EPI_RESID, gemm_params(c, G_ADAPT, 0, tab, g * GROUP_ROWS), c->stream, c->use_pdl))) return e;
  }
  if (n_launch) *n_launch += 1 + (tc >= 0 ? 2 : groups);
  return launch_stack(c, tab, ng, d.n_pre, m.n_recurrent, n_launch, tc);
}

// Raven-style layout: the post-layers' blocks on copies of the reading-out rows' states (`tab_coda`), writing the coda
// cache of each row's readout depth; leaves the planes the lm_head reads
cudaError_t launch_coda(loopspec_ctx* c, const RowTable* tab_coda, int ng, int* n_launch, int tc = -1) {
  const Derived& d = c->d;
  cudaError_t e;
  if ((e = launch_prep(c, tab_coda, d.n_pre + c->m.n_recurrent, true))) return e;
  if (n_launch) *n_launch += 1;
  return launch_stack(c, tab_coda, ng, d.n_pre + c->m.n_recurrent, d.n_coda, n_launch, tc);
}

cudaError_t launch_lm_head(loopspec_ctx* c, const RowTable* tab, int ng) {
  if (c->dg && tab != c->at<RowTable>(c->L.tab_pf) && tab != c->at<RowTable>(c->L.tab_pfc)) return launch_dg_lm(c, tab);
  const int groups = col_groups(c, tab);
  for (int g = 0; g < groups; ++g) {
    GemmParams gl = gemm_params(c, G_LM, 0, tab, g * GROUP_ROWS);
    gl.tl = tune_timeline(c), gl.tl_id = 120;
    cudaError_t e = launch_gemm(c->m.weight_dtype, ng, EPI_LOGITS, gl, c->stream, c->use_pdl);
    if (e) return e;
  }
  return cudaSuccess;
}

cudaError_t launch_select(loopspec_ctx* c, const RowTable* tab, int kinds_mask) {
  SelectParams sp;
  sp.tab = tab, sp.logits = c->at<float>(c->L.logits), sp.V = c->m.vocab, sp.NB = c->d.NB, sp.nodes = c->nodes();
  sp.temperature = c->s.temperature, sp.gate = c->s.gate, sp.residual_q2 = c->s.residual_q2, sp.seed = c->s.seed;
  sp.mask_first = c->s.mask_first;
  sp.kinds_mask = kinds_mask;
  sp.sel_tok = c->at<int>(c->L.sel_tok), sp.sel_aux = c->at<int>(c->L.sel_aux);
  sp.sel_lse = c->at<float>(c->L.sel_lse), sp.sel_z2 = c->at<float>(c->L.sel_z2);
  sp.argpart = c->at<float2>(c->L.argpart), sp.n_rb = c->plan[G_LM].n_rb;
  sp.top_k = c->filters ? c->s.top_k : 0, sp.top_p = c->filters ? c->s.top_p : 1.0f, sp.sel_flt = c->at<float4>(c->L.sel_flt);
  sp.staged = c->sel_staged;
  sp.tv_acc = (c->s.measure_tv && c->s.temperature > 0.f) ? c->at<double>(c->L.tv) : nullptr;
  return launch_k(select_kernel, dim3(c->d.max_rows * SEL_CS), dim3(SEL_THREADS), c->sel_smem, c->stream, sp, c->use_pdl, SEL_CS);
}

ControlParams control_params(loopspec_ctx* c, int phases) {
  ControlParams p;
  memset(&p, 0, sizeof p);
  p.att_mode = c->d.att_mode;
  p.tab = c->at<RowTable>(c->L.tab_dec), p.nodes = c->nodes(), p.seqs = c->seqs(), p.ctr = c->at<Counters>(c->L.ctr);
  p.S = c->d.S, p.NB = c->d.NB, p.R = c->m.R, p.d1 = c->d.d1, p.d2 = c->d.d2, p.ctx_cap = c->s.max_ctx;
  p.sel_tok = c->at<int>(c->L.sel_tok), p.sel_aux = c->at<int>(c->L.sel_aux);
  p.sel_lse = c->at<float>(c->L.sel_lse), p.sel_z2 = c->at<float>(c->L.sel_z2);
  p.sel_flt = c->filters ? c->at<float4>(c->L.sel_flt) : nullptr;
  p.phases = phases;
  p.out_ids = c->at<int>(c->L.out_ids), p.ids_cap = c->d.ids_cap, p.commits = c->at<int>(c->L.commits);
  p.row_trace = c->at<int>(c->L.trace), p.trace_n = c->at<int>(c->L.trace_n), p.trace_cap = c->d.trace_cap;
  p.kvcopy = c->at<KvCopyCmd>(c->L.kvcopy);
  p.hid = c->at<float>(c->L.hid), p.H = c->m.hidden, p.embed = c->embed, p.weight_dtype = c->m.weight_dtype;
  p.p_logit_base = c->d.p_logit_base, p.host_flags = c->host_flags_dev;
  if (c->d.raven) p.tab_pre = c->at<RowTable>(c->L.tab_pre), p.tab_coda = c->at<RowTable>(c->L.tab_coda), p.hid_coda_base = c->d.hid_coda_base;
  return p;
}

cudaError_t launch_control(loopspec_ctx* c, int phases) {
  return launch_k(control_kernel, dim3(1), dim3(CTRL_THREADS), sizeof(ControlSmem), c->stream, control_params(c, phases), c->use_pdl);
}

cudaError_t launch_kv_commit(loopspec_ctx* c) {
  KvCommitParams k;
  k.cmds = c->at<KvCopyCmd>(c->L.kvcopy), k.kv = c->at<__nv_bfloat16>(c->L.kv);
  k.layer_stride = c->kv_layer_stride(), k.plane_stride = c->kv_plane_stride(), k.sel_stride = c->kv_sel_stride();
  k.S = c->d.S, k.L = c->d.NL, k.n_kv_heads = c->m.n_kv_heads, k.slots = c->d.slots, k.d = c->m.head_dim;
  k.n_prelude = c->d.n_pre, k.n_rec = c->m.n_recurrent, k.n_classes = c->d.n_classes;
  for (int i = 0; i < 3; ++i) k.class_depth[i] = c->d.class_depth[i];
  dim3 grid(c->d.NL, c->m.R, 2 * c->d.S);
  return launch_k(kv_commit_kernel, grid, dim3(128), 0, c->stream, k, c->use_pdl);
}

// the whole decode step: pass, readouts, decisions, bookkeeping, KV commit
cudaError_t launch_step(loopspec_ctx* c, int kinds_mask, int phases, bool kv_commit, int* n_launch) {
  const RowTable* tab = c->at<RowTable>(c->L.tab_dec);
  cudaError_t e;
  const int tc = c->tc[1].on ? 1 : -1;  // decode passes of 9 to 64 rows: the layers' GEMMs on the tcgen05 kernel
  if ((e = launch_layers(c, tab, c->ng_dec, n_launch, tc, c->d.raven ? c->at<RowTable>(c->L.tab_pre) : nullptr))) return e;
  const RowTable* tab_ro = tab;  // the rows the lm_head reads
  if (c->d.raven && c->d.n_coda > 0) {
    tab_ro = c->at<RowTable>(c->L.tab_coda);
    if ((e = launch_coda(c, tab_ro, c->ng_dec, n_launch, tc))) return e;
  }
  if ((e = launch_lm_head(c, tab_ro, c->ng_dec))) return e;
  if ((e = launch_select(c, tab, kinds_mask))) return e;
  if ((e = launch_control(c, phases))) return e;
  if (n_launch) *n_launch += 3;
  if (kv_commit) {
    if ((e = launch_kv_commit(c))) return e;
    if (n_launch) *n_launch += 1;
  }
  return cudaSuccess;
}

VanillaParams vanilla_params(loopspec_ctx* c, int commit) {
  VanillaParams v;
  memset(&v, 0, sizeof v);
  v.att_mode = c->d.att_mode;
  v.tabs = c->at<RowTable>(c->L.tab_van), v.nodes = c->nodes(), v.seqs = c->seqs();
  v.S = c->d.S, v.NB = c->d.NB, v.R = c->m.R, v.sel_tok = c->at<int>(c->L.sel_tok), v.commit = commit;
  v.out_ids = c->at<int>(c->L.out_ids), v.ids_cap = c->d.ids_cap;
  v.hid = c->at<float>(c->L.hid), v.H = c->m.hidden, v.embed = c->embed, v.weight_dtype = c->m.weight_dtype;
  v.p_logit_base = c->d.p_logit_base, v.ctx_cap = c->s.max_ctx, v.host_flags = c->host_flags_dev;
  if (c->d.raven && c->d.n_coda > 0) v.tab_coda = c->at<RowTable>(c->L.tab_vanc), v.hid_coda_base = c->d.hid_coda_base, v.n_classes = c->d.n_classes;
  return v;
}

cudaError_t launch_vanilla_token(loopspec_ctx* c) {
  cudaError_t e;
  RowTable* tabs = c->at<RowTable>(c->L.tab_van);
  for (int r = 0; r < c->m.R; ++r)  // every row enters recurrence 1 in the first pass: the prelude pass is that table itself
    if ((e = launch_layers(c, tabs + r, c->ng_dec, nullptr, c->tc[1].on ? 1 : -1, (c->d.raven && r == 0) ? tabs : nullptr))) return e;
  const RowTable* tab_ro = tabs + c->m.R - 1;
  if (c->d.raven && c->d.n_coda > 0) {
    tab_ro = c->at<RowTable>(c->L.tab_vanc);
    if ((e = launch_coda(c, tab_ro, c->ng_dec, nullptr, c->tc[1].on ? 1 : -1))) return e;
  }
  if ((e = launch_lm_head(c, tab_ro, c->ng_dec))) return e;
  if ((e = launch_select(c, tabs + c->m.R - 1, 1 << RO_TARGET))) return e;
  return launch_k(vanilla_control_kernel, dim3(1), dim3(CTRL_THREADS), 0, c->stream, vanilla_params(c, 1), c->use_pdl);
}

int check_device_error(loopspec_ctx* c) {
  int e = c->host_flags[HF_ERROR];
  if (!e) return LOOPSPEC_OK;
  c->host_flags[HF_ERROR] = 0;
  if (e == ERR_WAIT || e == ERR_WAIT_PF)  // a bounded wait inside a kernel ran out: the pass's results are void, the context is not
    return fail(c, LOOPSPEC_ETIMEOUT, "a bounded device-side wait ran out (%s)", e == ERR_WAIT ? "decode-pass GEMM" : "prefill GEMM or grid barrier");
  return fail(c, LOOPSPEC_ECAPACITY, "device scheduler reported %s",
              e == ERR_NODES ? "node/row table overflow" : e == ERR_CTX ? "max_ctx exceeded" : "speculative chain too deep");
}

int capture(loopspec_ctx* c, cudaGraphExec_t* out, bool vanilla) {
  cudaGraph_t g = nullptr;
  CU(c, cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal));
  cudaError_t e;
  if (vanilla) e = launch_vanilla_token(c);
  else {
    int n = 0;
    e = launch_step(c, 0x1e, PH_ADVANCE | PH_VERIFY | PH_BUILD, true, &n);
    c->launches_per_step = n;
  }
  cudaError_t e2 = cudaStreamEndCapture(c->stream, &g);
  if (e != cudaSuccess || e2 != cudaSuccess) {
    if (g) cudaGraphDestroy(g);
    return fail(c, LOOPSPEC_ECUDA, "graph capture failed: %s", cudaGetErrorString(e != cudaSuccess ? e : e2));
  }
  e = cudaGraphInstantiate(out, g, 0);
  cudaGraphDestroy(g);
  if (e != cudaSuccess) return fail(c, LOOPSPEC_ECUDA, "cudaGraphInstantiate failed: %s", cudaGetErrorString(e));
  return LOOPSPEC_OK;
}

bool any_prefilled(loopspec_ctx* c) {
  for (char p : c->prefilled)
    if (p) return true;
  return false;
}

}  // namespace

// =============================================== C ABI =================================================
extern "C" {

size_t loopspec_workspace_bytes(const loopspec_model* m, const loopspec_sched* s) {
  int why;
  Derived d;
  if (!validate_model(m, &why) || !resolve_sched(m, s, &d, &why)) return 0;
  return make_layout(m, s, d).total;
}

int loopspec_pick_depths(float alpha, float beta, int32_t R, double* d1_star, double* d2_star, int32_t* d1, int32_t* d2) {
  if (!(alpha > 0) || !(beta > 0) || R < 2) return LOOPSPEC_EINVAL;
  double a, b;
  closed_form(alpha, beta, R, &a, &b);
  if (d1_star) *d1_star = a;
  if (d2_star) *d2_star = b;
  int x = 1, y = 0;
  if (!snap_depths(alpha, beta, R, &x, &y)) x = 1, y = 0;
  if (d1) *d1 = x;
  if (d2) *d2 = y;
  return LOOPSPEC_OK;
}

int loopspec_fit_envelope(const double* tv, int32_t n, double* alpha, double* beta) {
  if (!tv || n < 2 || !alpha || !beta) return LOOPSPEC_EINVAL;
  for (int i = 0; i < n; ++i)
    if (!(tv[i] > 0)) return LOOPSPEC_EINVAL;
  // With u_r(a) = log tv_r + a log r the constraint is log beta >= max_r u_r(a) and, at the tightest beta, the worst
  // log-ratio is max_r u_r(a) - min_r u_r(a): convex and piecewise linear in a, so its minimum over a > 0 is at a slope
  // where two of the lines u_i, u_j cross.  Every such slope is tried.
  double best_gap = 0, best_a = 0, best_logb = 0;
  bool have = false;
  for (int i = 0; i < n; ++i)
    for (int j = i + 1; j < n; ++j) {
      const double a = -(std::log(tv[j]) - std::log(tv[i])) / (std::log((double)(j + 1)) - std::log((double)(i + 1)));
      if (!(a > 0)) continue;
      double hi = -1e300, lo = 1e300;
      for (int r = 0; r < n; ++r) {
        const double u = std::log(tv[r]) + a * std::log((double)(r + 1));
        hi = std::max(hi, u), lo = std::min(lo, u);
      }
      if (!have || hi - lo < best_gap - 1e-15 || (std::fabs(hi - lo - best_gap) <= 1e-15 && a < best_a)) {
        best_gap = hi - lo, best_a = a, best_logb = hi, have = true;
      }
    }
  if (!have) return LOOPSPEC_EINVAL;  // the profile never decreases: no positive exponent fits
  *alpha = best_a, *beta = std::exp(best_logb);
  return LOOPSPEC_OK;
}

int32_t loopspec_max_branches(int32_t R, int32_t d1, int32_t d2) {
  if (d1 < 1 || R < 2 || d1 >= R || R % d1 || (d2 && (d2 <= d1 || d2 >= R || d2 % d1))) return 0;
  return max_branches(R, d1, d2);
}

int loopspec_init(const loopspec_model* m, const loopspec_sched* s, const loopspec_weights* w, void* workspace,
                  size_t workspace_bytes, void* cuda_stream, loopspec_ctx** out) {
  if (!out) return LOOPSPEC_EINVAL;
  *out = nullptr;
  int why;
  Derived d;
  if (!validate_model(m, &why)) return why;
  if (!resolve_sched(m, s, &d, &why)) return why;
  if (!w || !w->embed || !w->final_norm || !w->layer_ptrs || (!m->tied_lm_head && !w->lm_head)) return LOOPSPEC_EINVAL;
  if ((d.raven != 0) != (w->adapter != nullptr)) return LOOPSPEC_EINVAL;  // the adapter belongs to the Raven-style layout
  if (w->adapter && (reinterpret_cast<uintptr_t>(w->adapter) & 15)) return LOOPSPEC_EINVAL;
  for (int i = 0; i < 6 * d.NL; ++i)
    if (!w->layer_ptrs[i]) return LOOPSPEC_EINVAL;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255)) return LOOPSPEC_EINVAL;
  // every tensor is read with 16-byte loads
  if ((reinterpret_cast<uintptr_t>(w->embed) & 15) || (w->lm_head && (reinterpret_cast<uintptr_t>(w->lm_head) & 15)) ||
      (reinterpret_cast<uintptr_t>(w->final_norm) & 15))
    return LOOPSPEC_EINVAL;
  for (int i = 0; i < 6 * d.NL; ++i)
    if (reinterpret_cast<uintptr_t>(w->layer_ptrs[i]) & 15) return LOOPSPEC_EINVAL;
  if (!cuda_stream) return LOOPSPEC_EINVAL;  // the legacy default stream cannot be captured into a graph
  int dev = 0, n_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return LOOPSPEC_ECUDA;
  Layout L = make_layout(m, s, d);
  if (workspace_bytes < L.total) return LOOPSPEC_ECAPACITY;

  loopspec_ctx* c = new loopspec_ctx();
  c->m = *m, c->s = *s, c->d = d, c->L = L, c->n_sm = n_sm;
  c->s.d1 = d.d1, c->s.d2 = d.d2;
  if (c->s.top_p <= 0.f || c->s.top_p > 1.f) c->s.top_p = 1.f;  // 0 and anything above 1: no nucleus cut
  c->filters = c->s.temperature > 0.f && ((c->s.top_k > 0 && c->s.top_k < m->vocab) || c->s.top_p < 1.f);
  {  // selection kernel, sampling: every CTA stages its slice of up to three logits rows in shared memory, plus the
     // slice of exp(z/T - max) when C filters; rows too long for that are read from global memory in every pass
    const size_t slice = (size_t)((m->vocab / 4 + SEL_CS - 1) / SEL_CS) * 4 * sizeof(float);
    c->sel_staged = c->s.temperature > 0.f && (3 + (c->filters ? 1 : 0)) * slice <= 200 * 1024;
    c->sel_smem = (c->sel_staged ? 3 * slice : 0) + (c->filters ? slice : 0);
    if (c->sel_smem > 200 * 1024 ||
        (c->sel_smem > 48 * 1024 &&
         cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->sel_smem) != cudaSuccess)) {
      (void)cudaGetLastError();
      delete c;
      return LOOPSPEC_EUNSUPPORTED;
    }
  }
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  c->ws = static_cast<unsigned char*>(workspace);
  c->embed = w->embed, c->lm_head = m->tied_lm_head ? w->embed : w->lm_head;
  c->final_norm = static_cast<const float*>(w->final_norm);
  c->layers.assign(w->layer_ptrs, w->layer_ptrs + 6 * d.NL);
  c->adapter = w->adapter;
  c->ng_dec = ng_for_rows(d.max_rows_dec), c->ng_pf = ng_for_rows(d.max_rows_pf);
  c->prefilled.assign(d.S, 0);
  const int resid_rows = 128;
  const int n_rbs[6] = {(d.Hq + 2 * d.Hkv) / 128, m->hidden / resid_rows, (m->ffn + 63) / 64, m->hidden / resid_rows, (m->vocab + 127) / 128,
                        m->hidden / resid_rows};
  const int Ks[6] = {m->hidden, d.Hq, m->hidden, m->ffn, m->hidden, 2 * m->hidden};
  int slots = n_sm * kCtasPerSm;
  // Passes of up to 8 rows may split K over up to 11 CTAs (clusters beyond 8 are opt-in; a rank's slot of the receive
  // buffer holds one column then): the down projection's 176 k-blocks over 11 ranks instead of 8 [measured: pass 1.122 ->
  // 1.099 ms; 12 ranks 1.110 ms, 16 ranks 1.21 ms - they no longer fit at once]
  const int cs_cap = c->ng_dec == 1 ? 11 : 8;
  for (int i = 0; i < 6; ++i) c->plan[i] = plan_gemm(n_rbs[i], Ks[i], slots, false, 1, cs_cap);
  for (int i = 0; i < 6; ++i) c->plan_pf[i] = plan_gemm(n_rbs[i], Ks[i], slots, false);
  if (kTune) {  // tuning aid: cluster size of GEMM i from LOOPSPEC_CS_i
    for (int i = 0; i < 6; ++i) {
      char name[32];
      snprintf(name, sizeof name, "LOOPSPEC_CS_%d", i);
      if (const char* v = getenv(name)) {
        GemmPlan& g = c->plan[i];
        g.cs = std::max(1, std::min(16, atoi(v)));
        const int max_clusters = std::max(1, slots / g.cs), rounds = (g.n_rb + max_clusters - 1) / max_clusters;
        g.n_clusters = (g.n_rb + rounds - 1) / rounds, g.grid = g.n_clusters * g.cs;
      }
    }
  }
  // Every kernel of the chain asks for the same (largest) shared-memory carve-out: the GEMM CTAs need it, and an SM
  // whose partition was set by a small-shared-memory kernel would have to drain before it can host one.
  {
    const void* small_fns[] = {(const void*)attn_fn(m->head_dim, m->n_q_heads / m->n_kv_heads, d.att_runs != 0), (const void*)prep_planes_kernel,
                               (const void*)select_kernel, (const void*)control_kernel, (const void*)vanilla_control_kernel,
                               (const void*)kv_commit_kernel};
    for (const void* f : small_fns)
      if (cudaFuncSetAttribute(f, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess)
        (void)cudaGetLastError();
  }
  {
    const int G = m->n_q_heads / m->n_kv_heads;
    const bool runs = d.att_runs != 0;
    if (runs && cudaFuncSetAttribute((const void*)attn_fn(m->head_dim, G, runs), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)attn_smem(m->head_dim, G, runs)) != cudaSuccess) {
      delete c;
      return LOOPSPEC_ECUDA;
    }
  }
  if (!s->prefill_skinny) {  // (prefill_skinny keeps the decode kernels for the prefill passes, attention included)
    bool ok = true;
    if (m->head_dim == 128)
      ok = cudaFuncSetAttribute(attn_prefill_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, AtmCfg<128>::SMEM_BYTES) == cudaSuccess;
    else
      ok = cudaFuncSetAttribute(attn_prefill_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, AtmCfg<64>::SMEM_BYTES) == cudaSuccess;
    if (!ok) (void)cudaGetLastError();
    c->pf_attn = ok;
  }
  if (cudaFuncSetAttribute(control_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ControlSmem)) != cudaSuccess) {
    delete c;
    return LOOPSPEC_ECUDA;
  }
  for (int epi = 0; epi < 5; ++epi)  // clusters of more than 8 CTAs (the O and down projections' k-split) are opt-in
    if (cudaFuncSetAttribute(gemm_fn(m->weight_dtype, c->ng_dec, epi), cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)
      (void)cudaGetLastError();
  for (int ng : {c->ng_dec, c->ng_pf})
    if (gemm_smem(m->weight_dtype, ng) > 48 * 1024)
      for (int epi = 0; epi < 5; ++epi)
        if (cudaFuncSetAttribute(gemm_fn(m->weight_dtype, ng, epi), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 gemm_smem(m->weight_dtype, ng)) != cudaSuccess) {
          delete c;
          return LOOPSPEC_ECUDA;
        }
#ifdef LOOPSPEC_TUNE
  if (unsigned long long* tl = tune_timeline(c)) cudaMemcpyToSymbol(g_tune_tl, &tl, sizeof tl);
#endif
  // cluster sizes that are not powers of two are used only if the device can co-schedule them
  for (int i = 0; i < 12; ++i) {
    const bool pf = i >= 6;
    GemmPlan& g = pf ? c->plan_pf[i - 6] : c->plan[i];
    if ((g.cs & (g.cs - 1)) == 0 && g.cs <= 8) continue;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    const int ng = pf ? c->ng_pf : c->ng_dec;
    cfg.gridDim = dim3(g.grid), cfg.blockDim = dim3(GEMM_THREADS), cfg.dynamicSmemBytes = gemm_smem(m->weight_dtype, ng);
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = g.cs, at[0].val.clusterDim.y = 1, at[0].val.clusterDim.z = 1;
    cfg.attrs = at, cfg.numAttrs = 1;
    int n_active = 0;
    cudaError_t e = cudaOccupancyMaxActiveClusters(&n_active, gemm_fn(m->weight_dtype, ng, kEpiOf[i % 6]), &cfg);
    if (e != cudaSuccess || n_active < 1 || (g.cs > 8 && n_active < g.n_clusters)) {
      (void)cudaGetLastError();
      g = g.cs > 8 ? plan_gemm(n_rbs[i % 6], Ks[i % 6], slots, false) : plan_gemm(n_rbs[i % 6], Ks[i % 6], slots, true);
    }
  }
  // prefill passes on the tcgen05 kernel (shapes it does not take, and fp32 weights: the kernels of the decode passes);
  // decode passes too when they carry 9 to 64 rows
  if (tc_prefill_shapes_ok(m) && encode_tiled_fn()) {
    const Derived& dd = c->d;
    const int Ns[5] = {dd.Hq + 2 * dd.Hkv, m->hidden, 2 * m->ffn, m->hidden, m->hidden};
    const int Ks[5] = {m->hidden, dd.Hq, m->hidden, m->ffn, 2 * m->hidden};
    const int w_idx[4] = {1, 2, 4, 5};  // qkv, o, gate/up, down among a layer's six pointers
    bool ok = true;
    c->tc_wmaps.resize((size_t)4 * dd.NL + 1);
    for (int l = 0; l < dd.NL && ok; ++l)
      for (int i = 0; i < 4 && ok; ++i) ok = make_map_bf16(&c->tc_wmaps[4 * l + i], c->layers[6 * l + w_idx[i]], Ns[i], Ks[i], TC_BM);
    if (dd.raven) ok = ok && make_map_bf16(&c->tc_wmaps[4 * dd.NL], c->adapter, Ns[4], Ks[4], TC_BM);
    for (int i = 0; i < 5; ++i) c->tc_plan[i] = tc_pf_plan(Ns[i], Ks[i]);
    const size_t x_off[4] = {c->L.xplanes, c->L.aplanes, c->L.splanes, c->L.cplanes};
    const int x_k[4] = {m->hidden, dd.Hq, m->ffn, 2 * m->hidden};
    const bool want[2] = {!s->prefill_skinny, c->ng_dec > 1};
    const int rows[2] = {dd.max_rows_pf, std::min(dd.max_rows_dec, (int)GROUP_ROWS)};  // (wider decode passes: groups of 64 columns)
    size_t smem_max = 0;
    for (int k = 0; k < 2 && ok; ++k) {
      if (!want[k]) continue;
      loopspec_ctx::TcCfg& tc = c->tc[k];
      tc.cols = tc_pf_cols(rows[k]);
      const int sb = tc_stage_bytes(tc.cols);
      tc.stages = std::max(2, std::min(TC_MAX_STAGES, (100 * 1024) / sb));
      tc.smem = (size_t)tc.stages * sb + 1024;
      smem_max = std::max(smem_max, tc.smem);
      for (int i = 0; i < (dd.raven ? 4 : 3) && ok; ++i)
        ok = make_map_planes3d(&tc.xmaps[i], c->ws + x_off[i], x_k[i], x_k[i], dd.max_rows, tc.cols);
    }
    if (smem_max) ok = ok && cudaFuncSetAttribute(linear_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max) == cudaSuccess;
    if (!ok) (void)cudaGetLastError();
    for (int k = 0; k < 2; ++k) c->tc[k].on = ok && want[k];
  }
  // readout GEMM of the decode passes on the tcgen05 kernel: bf16 weights whose rows are 16-byte multiples (TMA strides)
  if (m->weight_dtype == 1 && encode_tiled_fn() && m->hidden % 8 == 0) {
    const Derived& dd = c->d;
    c->dg_mp = dg_mp_for_rows(dd.max_rows_dec);
    bool ok = c->dg_mp <= DG_MAX_COLS;
    const int budget = kDgSmem;
    for (int epi : {EPI_LOGITS, EPI_PLAIN})
      ok = ok && cudaFuncSetAttribute(dg_fn(epi), cudaFuncAttributeMaxDynamicSharedMemorySize, budget) == cudaSuccess;
    int max_cl[9] = {0};
    for (int cs = 1; cs <= 8 && ok; ++cs) {  // clusters of this size the device runs at once (one CTA per SM at most)
      cudaLaunchConfig_t cfg;
      memset(&cfg, 0, sizeof cfg);
      cfg.gridDim = dim3(cs * n_sm), cfg.blockDim = dim3(DG_THREADS), cfg.dynamicSmemBytes = budget;
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = cs, at[0].val.clusterDim.y = 1, at[0].val.clusterDim.z = 1;
      cfg.attrs = at, cfg.numAttrs = 1;
      int n_active = 0;
      if (cudaOccupancyMaxActiveClusters(&n_active, dg_fn(EPI_LOGITS), &cfg) != cudaSuccess) (void)cudaGetLastError(), n_active = 0;
      // Inside the chain a kernel's clusters are placed while its predecessor's CTAs still leave: measured on the gate/up
      // shape, three of the 45 clusters of three that the query (and a probe on the idle device) promised found no place
      // and ran as a second wave, doubling the kernel's time; a tenth of the promise is left unused.
      max_cl[cs] = std::min(n_active, n_sm / cs);
      if (cs > 1) max_cl[cs] = max_cl[cs] * 9 / 10;
    }
    if (ok) c->dgp = plan_dg((m->vocab + 127) / 128, m->hidden, c->dg_mp, max_cl);
    ok = ok && c->dgp.cs >= 1;
    ok = ok && make_map_bf16(&c->dg_wmap, c->lm_head, m->vocab, m->hidden, TC_BM);
    ok = ok && make_map_planes_all(&c->dg_xmap, c->ws + c->L.xplanes, m->hidden, m->hidden, dd.max_rows, c->dg_mp);
    if (!ok) (void)cudaGetLastError();
    c->dg = ok;
  }
  if (kTune && getenv("LOOPSPEC_DBG")) fprintf(stderr, "LOOPSPEC_TUNE region at workspace offset %zu\n", c->L.tune);
  auto bail = [&](int code, const char* what) {
    loopspec_destroy(c);
    (void)what;
    return code;
  };
  int* hf = nullptr;
  if (cudaHostAlloc(reinterpret_cast<void**>(&hf), HF_COUNT * sizeof(int), cudaHostAllocMapped) != cudaSuccess)
    return bail(LOOPSPEC_ECUDA, "cudaHostAlloc");
  memset(hf, 0, HF_COUNT * sizeof(int));
  c->host_flags = hf;
  if (cudaHostGetDevicePointer(reinterpret_cast<void**>(&c->host_flags_dev), hf, 0) != cudaSuccess)
    return bail(LOOPSPEC_ECUDA, "cudaHostGetDevicePointer");
  c->pin_ids_cap = (size_t)std::max(s->max_ctx, d.S * d.ids_cap) * 8 + 64;
  if (cudaHostAlloc(reinterpret_cast<void**>(&c->pin_ids), c->pin_ids_cap * sizeof(int), cudaHostAllocDefault) != cudaSuccess)
    return bail(LOOPSPEC_ECUDA, "cudaHostAlloc");
  if (cudaEventCreate(&c->ev0) != cudaSuccess || cudaEventCreate(&c->ev1) != cudaSuccess) return bail(LOOPSPEC_ECUDA, "event");

  // rotary table in double precision on the host: cos/sin(pos * theta^(-2i/d))
  {
    const int hd2 = m->head_dim / 2;
    std::vector<float2> tab((size_t)s->max_ctx * hd2);
    for (int i = 0; i < hd2; ++i) {
      double inv = std::pow((double)m->rope_theta, -2.0 * i / m->head_dim);
      for (int p = 0; p < s->max_ctx; ++p) {
        double a = p * inv;
        tab[(size_t)p * hd2 + i] = make_float2((float)std::cos(a), (float)std::sin(a));
      }
    }
    if (cudaMemcpyAsync(c->ws + L.rope, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice, c->stream) != cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess)
      return bail(LOOPSPEC_ECUDA, "rope upload");
  }
  // bf16 weights: repack every matrix once into the tile-major streaming layout held in the workspace
  if (m->weight_dtype == 1) {
    unsigned char* dst = c->ws + L.wpack;
    auto pack = [&](const void* src, int N, int K, int perm = 0, int perm_a = 0) -> bool {
      PackParams pp;
      pp.src = static_cast<const __nv_bfloat16*>(src), pp.dst = reinterpret_cast<__nv_bfloat16*>(dst), pp.N = N, pp.K = K;
      pp.kpr = (K + 31) / 32, pp.perm = perm, pp.perm_a = perm_a, pp.perm_d = m->head_dim;
      pack_weights_kernel<<<n_sm * 8, 256, 0, c->stream>>>(pp);
      c->packed.push_back(dst);
      dst += packed_bytes(N, K);
      return cudaGetLastError() == cudaSuccess;
    };
    bool ok = true;
    for (int l = 0; l < d.NL && ok; ++l) {
      const void* const* lp = &c->layers[6 * l];
      // rotary partners (QKV) and gate/up partners are stored as adjacent row tiles
      ok = pack(lp[1], d.Hq + 2 * d.Hkv, m->hidden, 2, m->head_dim / 32) && pack(lp[2], m->hidden, d.Hq) &&
           pack(lp[4], 2 * m->ffn, m->hidden, 1, m->ffn) && pack(lp[5], m->hidden, m->ffn);
    }
    ok = ok && pack(c->lm_head, m->vocab, m->hidden);
    if (d.raven) ok = ok && pack(c->adapter, m->hidden, 2 * m->hidden);
    if (!ok || cudaStreamSynchronize(c->stream) != cudaSuccess) return bail(LOOPSPEC_ECUDA, "weight repack");
  }
  // clear everything after the KV pool's predecessor tables: scratch counters must start at zero, tables idle
  if (cudaMemsetAsync(c->ws + L.acnt, 0, L.total - L.acnt, c->stream) != cudaSuccess ||
      cudaMemsetAsync(c->ws + L.seqs, 0xff, (size_t)MAX_SEQS * 4, c->stream) != cudaSuccess ||  // root = -1
      cudaStreamSynchronize(c->stream) != cudaSuccess)
    return bail(LOOPSPEC_ECUDA, "workspace clear");
  *out = c;
  return LOOPSPEC_OK;
}

int loopspec_destroy(loopspec_ctx* c) {
  if (!c) return LOOPSPEC_OK;
  if (c->g_step) cudaGraphExecDestroy(c->g_step);
  if (c->g_vanilla) cudaGraphExecDestroy(c->g_vanilla);
  if (c->ev0) cudaEventDestroy(c->ev0);
  if (c->ev1) cudaEventDestroy(c->ev1);
  if (c->host_flags) cudaFreeHost(const_cast<int*>(c->host_flags));
  if (c->pin_ids) cudaFreeHost(c->pin_ids);
  delete c;
  return LOOPSPEC_OK;
}

const char* loopspec_last_error(loopspec_ctx* c) { return c ? c->err.c_str() : "null context"; }

int loopspec_prefill(loopspec_ctx* c, int32_t seq, const int32_t* prompt_ids, int32_t n, int32_t* first_token) {
  Range nvtx_range("loopspec_prefill");
  struct PlanGuard {  // prefill passes on the mma.sync kernels use their own cluster plans
    loopspec_ctx* c;
    explicit PlanGuard(loopspec_ctx* c_) : c(c_) {
      if (c) c->cur_plan = c->plan_pf;
    }
    ~PlanGuard() {
      if (c) c->cur_plan = c->plan;
    }
  } plan_guard(c);
  if (!c) return LOOPSPEC_EINVAL;
  if (c->sticky) return LOOPSPEC_ECUDA;
  if (seq < 0 || seq >= c->d.S || !prompt_ids || n < 1) return fail(c, LOOPSPEC_EINVAL, "bad prefill arguments");
  if (n + 3 >= c->s.max_ctx) return fail(c, LOOPSPEC_ECAPACITY, "prompt of %d tokens does not fit max_ctx %d", n, c->s.max_ctx);
  for (int i = 0; i < n; ++i)
    if (prompt_ids[i] < 0 || prompt_ids[i] >= c->m.vocab) return fail(c, LOOPSPEC_EINVAL, "prompt id out of range");
  if (c->pending_verify) return fail(c, LOOPSPEC_ESTATE, "verification pending");
  memcpy(c->pin_ids, prompt_ids, (size_t)n * 4);
  CU(c, cudaMemcpyAsync(c->ws + c->L.prompt, c->pin_ids, (size_t)n * 4, cudaMemcpyHostToDevice, c->stream));
  RowTable* tab = c->at<RowTable>(c->L.tab_pf);
  const int chunk = c->d.max_rows_pf;
  for (int p0 = 0; p0 < n; p0 += chunk) {
    int cnt = std::min(chunk, n - p0);
    for (int r = 1; r <= c->m.R; ++r) {
      PrefillParams pp;
      pp.att_mode = c->d.att_mode;
      pp.tab = tab, pp.prompt = c->at<int>(c->L.prompt), pp.seq = seq, pp.p0 = p0, pp.count = cnt, pp.r = r, pp.R = c->m.R;
      pp.n_prompt = n, pp.hid_base = c->d.S * c->d.NB, pp.p_logit_base = c->d.p_logit_base;
      pp.hid = c->at<float>(c->L.hid), pp.H = c->m.hidden, pp.embed = c->embed, pp.weight_dtype = c->m.weight_dtype;
      pp.tab_coda = nullptr, pp.coda_class = 0, pp.hid_coda_base = c->d.hid_coda_base;
      if (c->d.raven && c->d.n_coda > 0) {  // the prompt fills the coda cache of every readout depth (App. B)
        pp.tab_coda = c->at<RowTable>(c->L.tab_pfc);
        for (int k = 0; k < c->d.n_classes; ++k)
          if (c->d.class_depth[k] == r && pp.coda_class == 0) pp.coda_class = k + 1;
        if (r == c->m.R) pp.coda_class = c->d.n_classes;
      }
      prefill_setup_kernel<<<1, CTRL_THREADS, 0, c->stream>>>(pp);
      CU(c, cudaGetLastError());
      CU(c, launch_layers(c, tab, c->ng_pf, nullptr, c->tc[0].on ? 0 : -1, (c->d.raven && r == 1) ? tab : nullptr));
      if (pp.coda_class > 0) CU(c, launch_coda(c, pp.tab_coda, c->ng_pf, nullptr, c->tc[0].on ? 0 : -1));
    }
  }
  if (c->d.raven && c->d.n_coda > 0) tab = c->at<RowTable>(c->L.tab_pfc);  // its last state: last chunk, depth R
  CU(c, launch_lm_head(c, tab, c->ng_pf));
  CU(c, launch_select(c, tab, 1 << RO_TARGET));
  PrefillFinishParams fp;
  fp.tab = c->at<RowTable>(c->L.tab_pf), fp.nodes = c->nodes(), fp.seqs = c->seqs(), fp.seq = seq, fp.NB = c->d.NB, fp.n_prompt = n, fp.n_target = 0;
  fp.sel_tok = c->at<int>(c->L.sel_tok), fp.hid = c->at<float>(c->L.hid), fp.H = c->m.hidden, fp.embed = c->embed;
  fp.weight_dtype = c->m.weight_dtype, fp.host_flags = c->host_flags_dev;
  prefill_finish_kernel<<<1, CTRL_THREADS, 0, c->stream>>>(fp);
  CU(c, cudaGetLastError());
  // statistics and traces restart with the sequence set
  CU(c, cudaMemsetAsync(c->ws + c->L.ctr, 0, sizeof(Counters), c->stream));
  CU(c, cudaMemsetAsync(c->ws + c->L.tv, 0, (size_t)MAX_SEQS * 4 * sizeof(double), c->stream));
  CU(c, cudaMemsetAsync(c->ws + c->L.trace_n, 0, 4, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  c->prefilled[seq] = 1;
  c->vanilla_mode = false;
  if (first_token) *first_token = c->host_flags[HF_FIRST_TOKEN];
  return check_device_error(c);
}

// set every prefilled sequence's target to n more tokens and (re)build the decode rows
static int arm_decode(loopspec_ctx* c, int n_tokens, bool unlimited = false) {
  std::vector<int> ndec(MAX_SEQS), nids(MAX_SEQS), tgt(MAX_SEQS, 0);
  CU(c, cudaMemcpyAsync(ndec.data(), c->seqs().n_dec, MAX_SEQS * 4, cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaMemcpyAsync(nids.data(), c->seqs().n_ids, MAX_SEQS * 4, cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  // Positions a sequence can reach: its committed ids, the tokens asked for (a manual step commits at most one) and
  // the deepest chain of uncommitted drafts, R/d1; the scheduler wants two more below max_ctx.  Checked here, before
  // anything is launched, so that no pass ever carries a row whose position lies outside the KV pool.
  const int spec_depth = c->m.R / c->d.d1;
  for (int s = 0; s < c->d.S; ++s) {
    if (!c->prefilled[s]) continue;
    const long long want = unlimited ? 1 : n_tokens;
    if ((long long)nids[s] + want + spec_depth + 2 > c->s.max_ctx || (long long)ndec[s] + want > c->d.ids_cap)
      return fail(c, LOOPSPEC_ECAPACITY, "sequence %d: %d committed ids + %lld more + %d speculative + 2 exceed max_ctx %d", s, nids[s],
                  want, spec_depth, c->s.max_ctx);
    tgt[s] = unlimited ? c->d.ids_cap : ndec[s] + n_tokens;
  }
  memcpy(c->pin_ids, tgt.data(), MAX_SEQS * 4);
  CU(c, cudaMemcpyAsync(c->seqs().n_target, c->pin_ids, MAX_SEQS * 4, cudaMemcpyHostToDevice, c->stream));
  if (c->vanilla_mode) {  // drop back from vanilla decoding: the root restarts at depth 0
    vanilla_control_kernel<<<1, CTRL_THREADS, 0, c->stream>>>(vanilla_params(c, 0));
    CU(c, cudaGetLastError());
    c->vanilla_mode = false;
  }
  CU(c, launch_control(c, PH_BUILD));
  CU(c, cudaStreamSynchronize(c->stream));
  return check_device_error(c);
}

int loopspec_step(loopspec_ctx* c, int32_t* n_rows_out, int32_t* n_need_verify_out) {
  Range nvtx_range("loopspec_step");
  if (!c) return LOOPSPEC_EINVAL;
  if (c->sticky) return LOOPSPEC_ECUDA;
  if (!any_prefilled(c)) return fail(c, LOOPSPEC_ESTATE, "step before prefill");
  if (c->pending_verify) return fail(c, LOOPSPEC_ESTATE, "verification pending: call loopspec_verify first");
  // a manual step never stops on a token target; (re)building the rows is idempotent
  int rc = arm_decode(c, 0, true);
  if (rc) return rc;
  int rows = c->host_flags[HF_N_ROWS];
  CU(c, launch_step(c, (1 << RO_D1) | (1 << RO_D2), PH_ADVANCE | PH_BUILD, false, nullptr));
  CU(c, cudaStreamSynchronize(c->stream));
  int need = c->host_flags[HF_NEED_VERIFY];
  c->pending_verify = need > 0;
  if (n_rows_out) *n_rows_out = rows;
  if (n_need_verify_out) *n_need_verify_out = need;
  return check_device_error(c);
}

int loopspec_verify(loopspec_ctx* c, loopspec_commit* out, int32_t max_out, int32_t* n_out) {
  Range nvtx_range("loopspec_verify");
  if (!c) return LOOPSPEC_EINVAL;
  if (c->sticky) return LOOPSPEC_ECUDA;
  if (!c->pending_verify) return fail(c, LOOPSPEC_ESTATE, "no branch is at depth R");
  if (max_out < 0 || (max_out > 0 && !out)) return fail(c, LOOPSPEC_EINVAL, "bad output array");
  std::vector<int> before(MAX_SEQS), after(MAX_SEQS);
  CU(c, cudaMemcpyAsync(before.data(), c->seqs().n_dec, MAX_SEQS * 4, cudaMemcpyDeviceToHost, c->stream));
  CU(c, launch_select(c, c->at<RowTable>(c->L.tab_dec), 1 << RO_VERIFY));
  CU(c, launch_control(c, PH_VERIFY | PH_BUILD));
  CU(c, launch_kv_commit(c));
  CU(c, cudaMemcpyAsync(after.data(), c->seqs().n_dec, MAX_SEQS * 4, cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  c->pending_verify = false;
  int n = 0;
  for (int s = 0; s < c->d.S; ++s) {
    if (after[s] == before[s]) continue;
    if (n < max_out) {
      int rec[8];
      CU(c, cudaMemcpy(rec, c->at<int>(c->L.commits) + ((size_t)s * c->d.ids_cap + before[s]) * 8, sizeof rec, cudaMemcpyDeviceToHost));
      out[n] = loopspec_commit{rec[0], rec[1], rec[2], rec[3], rec[4], rec[5], rec[6], rec[7]};
    }
    ++n;
  }
  if (n_out) *n_out = n;
  return check_device_error(c);
}

static int copy_ids_out(loopspec_ctx* c, const std::vector<int>& start, int n_tokens, int32_t* ids_out) {
  if (!ids_out) return LOOPSPEC_OK;
  for (int s = 0; s < c->d.S; ++s) {
    if (!c->prefilled[s]) continue;
    CU(c, cudaMemcpyAsync(c->pin_ids + (size_t)s * n_tokens, c->at<int>(c->L.out_ids) + (size_t)s * c->d.ids_cap + start[s],
                          (size_t)n_tokens * 4, cudaMemcpyDeviceToHost, c->stream));
  }
  CU(c, cudaStreamSynchronize(c->stream));
  for (int s = 0; s < c->d.S; ++s)
    if (c->prefilled[s]) memcpy(ids_out + (size_t)s * n_tokens, c->pin_ids + (size_t)s * n_tokens, (size_t)n_tokens * 4);
  return LOOPSPEC_OK;
}

int loopspec_decode(loopspec_ctx* c, int32_t n_tokens, int32_t* ids_out) {
  Range nvtx_range("loopspec_decode");
  if (!c) return LOOPSPEC_EINVAL;
  if (c->sticky) return LOOPSPEC_ECUDA;
  if (n_tokens < 1) return fail(c, LOOPSPEC_EINVAL, "n_tokens must be positive");
  if (!any_prefilled(c)) return fail(c, LOOPSPEC_ESTATE, "decode before prefill");
  if (c->pending_verify) return fail(c, LOOPSPEC_ESTATE, "verification pending");
  std::vector<int> start(MAX_SEQS);
  CU(c, cudaMemcpyAsync(start.data(), c->seqs().n_dec, MAX_SEQS * 4, cudaMemcpyDeviceToHost, c->stream));
  int rc = arm_decode(c, n_tokens);
  if (rc) return rc;
  if (!c->g_step && (rc = capture(c, &c->g_step, false))) return rc;
  // every commit needs at least d1 more passes, so `remaining * d1` replays can never overshoot
  std::vector<int> ndec(MAX_SEQS);
  for (;;) {
    CU(c, cudaMemcpyAsync(ndec.data(), c->seqs().n_dec, MAX_SEQS * 4, cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
    if ((rc = check_device_error(c))) return rc;
    int remaining = 0;
    for (int s = 0; s < c->d.S; ++s)
      if (c->prefilled[s]) remaining = std::max(remaining, start[s] + n_tokens - ndec[s]);
    if (remaining <= 0) break;
    if (kTune && getenv("LOOPSPEC_DBG_REPLAYS")) {  // tuning aid: a fixed number of replays, whatever they commit
      for (int i = 0; i < atoi(getenv("LOOPSPEC_DBG_REPLAYS")); ++i) CU(c, cudaGraphLaunch(c->g_step, c->stream));
      CU(c, cudaStreamSynchronize(c->stream));
      return LOOPSPEC_OK;
    }
    for (int i = 0; i < remaining * c->d.d1; ++i) CU(c, cudaGraphLaunch(c->g_step, c->stream));
  }
  return copy_ids_out(c, start, n_tokens, ids_out);
}

int loopspec_vanilla_decode(loopspec_ctx* c, int32_t n_tokens, int32_t* ids_out) {
  Range nvtx_range("loopspec_vanilla_decode");
  if (!c) return LOOPSPEC_EINVAL;
  if (c->sticky) return LOOPSPEC_ECUDA;
  if (n_tokens < 1) return fail(c, LOOPSPEC_EINVAL, "n_tokens must be positive");
  if (!any_prefilled(c)) return fail(c, LOOPSPEC_ESTATE, "decode before prefill");
  if (c->pending_verify) return fail(c, LOOPSPEC_ESTATE, "verification pending");
  std::vector<int> start(MAX_SEQS), nids(MAX_SEQS);
  CU(c, cudaMemcpyAsync(start.data(), c->seqs().n_dec, MAX_SEQS * 4, cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaMemcpyAsync(nids.data(), c->seqs().n_ids, MAX_SEQS * 4, cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  for (int s = 0; s < c->d.S; ++s)  // no drafts here: the last position is committed ids + n_tokens - 1, two more must fit
    if (c->prefilled[s] && ((long long)nids[s] + n_tokens + 2 > c->s.max_ctx || (long long)start[s] + n_tokens > c->d.ids_cap))
      return fail(c, LOOPSPEC_ECAPACITY, "sequence %d: %d committed ids + %d more + 2 exceed max_ctx %d", s, nids[s], n_tokens, c->s.max_ctx);
  vanilla_control_kernel<<<1, CTRL_THREADS, 0, c->stream>>>(vanilla_params(c, 0));
  CU(c, cudaGetLastError());
  c->vanilla_mode = true;
  int rc;
  if (!c->g_vanilla && (rc = capture(c, &c->g_vanilla, true))) return rc;
  for (int i = 0; i < n_tokens; ++i) CU(c, cudaGraphLaunch(c->g_vanilla, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  if ((rc = check_device_error(c))) return rc;
  return copy_ids_out(c, start, n_tokens, ids_out);
}

int loopspec_get_stats(loopspec_ctx* c, loopspec_stats* out) {
  if (!c || !out) return LOOPSPEC_EINVAL;
  Counters k;
  CU(c, cudaMemcpyAsync(&k, c->ws + c->L.ctr, sizeof k, cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  out->steps = k.steps, out->n_decode = k.n_decode, out->n_accept1 = k.n_accept1, out->n_accept2 = k.n_accept2;
  out->n_restart = k.n_restart, out->gate_evals = k.gate_evals, out->gate_opens = k.gate_opens;
  out->rows_total = k.rows_total, out->rows_max = k.rows_max, out->readout_rows_total = k.readout_rows_total;
  double den = (double)k.n_accept1 * c->d.d1 + (double)k.n_accept2 * c->d.d2 + (double)k.n_restart * c->m.R;
  out->gamma = den > 0 ? (double)k.n_decode * c->m.R / den : 0.0;  // Sec. 6 "Implementation and Metrics", definition of gamma
  double tv[MAX_SEQS * 4];
  CU(c, cudaMemcpy(tv, c->ws + c->L.tv, sizeof tv, cudaMemcpyDeviceToHost));
  double s1 = 0, n1 = 0, s2 = 0, n2 = 0;
  for (int s = 0; s < c->d.S; ++s) s1 += tv[4 * s], n1 += tv[4 * s + 1], s2 += tv[4 * s + 2], n2 += tv[4 * s + 3];
  out->tv_d1 = n1 > 0 ? s1 / n1 : 0.0, out->tv_d2 = n2 > 0 ? s2 / n2 : 0.0;
  out->tv_n1 = (int64_t)n1, out->tv_n2 = (int64_t)n2;
  return LOOPSPEC_OK;
}

int loopspec_get_commits(loopspec_ctx* c, int32_t seq, loopspec_commit* out, int32_t max_out, int32_t* n_out) {
  if (!c || seq < 0 || seq >= c->d.S || max_out < 0 || (max_out && !out)) return LOOPSPEC_EINVAL;
  int n = 0;
  CU(c, cudaMemcpyAsync(&n, c->seqs().n_dec + seq, 4, cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  int k = std::min(n, (int)max_out);
  if (k > 0) {
    std::vector<int> rec((size_t)k * 8);
    CU(c, cudaMemcpy(rec.data(), c->at<int>(c->L.commits) + (size_t)seq * c->d.ids_cap * 8, rec.size() * 4, cudaMemcpyDeviceToHost));
    for (int i = 0; i < k; ++i) {
      const int* r = &rec[(size_t)i * 8];
      out[i] = loopspec_commit{r[0], r[1], r[2], r[3], r[4], r[5], r[6], r[7]};
    }
  }
  if (n_out) *n_out = n;
  return LOOPSPEC_OK;
}

int loopspec_get_row_trace(loopspec_ctx* c, int32_t* out, int32_t max_out, int32_t* n_out) {
  if (!c || max_out < 0 || (max_out && !out)) return LOOPSPEC_EINVAL;
  int n = 0;
  CU(c, cudaMemcpyAsync(&n, c->ws + c->L.trace_n, 4, cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  int k = std::min(std::min(n, c->d.trace_cap), (int)max_out);
  if (k > 0) CU(c, cudaMemcpy(out, c->ws + c->L.trace, (size_t)k * 4, cudaMemcpyDeviceToHost));
  if (n_out) *n_out = n;
  return LOOPSPEC_OK;
}

int loopspec_debug_logits(loopspec_ctx* c, int32_t seq, int32_t which, float* out_V) {
  if (!c || !out_V || seq < 0 || seq >= c->d.S || which < 0 || which > 2) return LOOPSPEC_EINVAL;
  size_t idx;
  if (which == 0) idx = c->d.p_logit_base + seq;
  else {
    int root = -1;
    CU(c, cudaMemcpy(&root, c->seqs().root + seq, 4, cudaMemcpyDeviceToHost));
    if (root < 0) return fail(c, LOOPSPEC_ESTATE, "sequence has no root branch");
    idx = (size_t)(seq * c->d.NB + root) * 2 + (which - 1);
  }
  CU(c, cudaStreamSynchronize(c->stream));
  CU(c, cudaMemcpy(out_V, c->at<float>(c->L.logits) + idx * c->m.vocab, (size_t)c->m.vocab * 4, cudaMemcpyDeviceToHost));
  return LOOPSPEC_OK;
}

int loopspec_debug_drop_tile(loopspec_ctx* c, int32_t unit, int32_t wait_us) {
  if (!c || unit < -1 || wait_us < 0) return LOOPSPEC_EINVAL;
  if (!c->dg) return fail(c, LOOPSPEC_EUNSUPPORTED, "no tcgen05 readout kernel in this context (fp32 weights)");
  c->dg_drop_unit = unit;
  c->dg_wait_cycles = (unit >= 0 && wait_us > 0) ? (long long)wait_us * 2000 : TC_WAIT_CYCLES;
  if (c->g_step) cudaGraphExecDestroy(c->g_step), c->g_step = nullptr;  // captured launches carry the old setting
  if (c->g_vanilla) cudaGraphExecDestroy(c->g_vanilla), c->g_vanilla = nullptr;
  return LOOPSPEC_OK;
}

int loopspec_launches_per_step(loopspec_ctx* c, int32_t* out) {
  if (!c || !out) return LOOPSPEC_EINVAL;
  const Derived& d = c->d;
  // launches per GEMM: one per group of 64 token columns, or the tcgen05 kernel and its epilogue
  const int groups = (d.max_rows_dec + GROUP_ROWS - 1) / GROUP_ROWS;
  const int g = c->tc[1].on ? 2 : groups;
  const int per_block = 1 + 4 * g, lm = c->dg ? 1 : groups;  // attention + four GEMMs
  int n = 1 + c->m.n_recurrent * per_block + lm + 3;               // preparation, blocks, lm_head, selection, control, KV commit
  if (d.raven)  // prelude pass (preparation + blocks), concatenation + adapter instead of the preparation, coda pass
    n = (d.n_pre ? 1 + per_block * d.n_pre : 0) + 1 + g + per_block * c->m.n_recurrent + (d.n_coda ? 1 + per_block * d.n_coda : 0) + lm + 3;
  *out = n;
  return LOOPSPEC_OK;
}

int loopspec_decode_paths(loopspec_ctx* c, int32_t* gemm_path, int32_t* attention_path) {
  if (!c) return LOOPSPEC_EINVAL;
  if (gemm_path) *gemm_path = c->tc[1].on ? 1 : 0;
  if (attention_path) *attention_path = c->d.att_runs != 0 ? 1 : 0;
  return LOOPSPEC_OK;
}

int loopspec_time_kernel(loopspec_ctx* c, int32_t which, int32_t rows, int32_t iters, float* ms_out, double* bytes_out) {
  if (!c || which < 0 || which > 6 || rows < 1 || rows > (which == 6 ? c->d.max_rows_pf : 8 * c->ng_dec) || iters < 1 || !ms_out)
    return LOOPSPEC_EINVAL;
  if (c->sticky) return LOOPSPEC_ECUDA;
  if (c->pending_verify) return fail(c, LOOPSPEC_ESTATE, "verification pending");
  // a scratch row table with `rows` plain rows on sequence 0 (hidden states of the prefill area; outputs go to
  // the pass buffers and to KV slot 0 of plane 1, which the next prefill overwrites)
  RowTable t;
  memset(&t, 0, sizeof t);
  t.n_rows = rows, t.n_readout = rows, t.att_mode = c->d.att_mode;
  for (int i = 0; i < rows; ++i) {
    t.r[i] = 1, t.hid_idx[i] = c->d.S * c->d.NB + i, t.ro_rows[i] = i, t.readout[i] = RO_TARGET, t.n_canon[i] = 1, t.n_safe[i] = 0;
    t.logit_idx[i] = c->d.p_logit_base, t.node[i] = -1, t.chunk_start[i] = i;
  }
  t.chunk_start[rows] = rows, t.attn_items = rows;
  if (which == 5) {
    // attention: row i reads the whole cached context (the capacity minus one chunk) of sequence i mod S at recurrence
    // 1 + (i / S) mod R, so that no two rows share keys or values (as rows at different depths do not)
    const int ctx = std::max(1, c->d.ids_cap - ATT_CHUNK);
    int items = 0;
    for (int i = 0; i < rows; ++i) {
      t.seq[i] = i % c->d.S, t.r[i] = 1 + (i / c->d.S) % c->m.R;
      t.n_canon[i] = ctx, t.n_safe[i] = ctx, t.n_spec[i] = 0, t.chunk_start[i] = items;
      items += att_items(ctx, c->d.att_mode);
    }
    t.chunk_start[rows] = items, t.attn_items = items;
  }
  if (which == 6) {
    // prefill attention: `rows` consecutive prompt positions of sequence 0 at recurrence 1, the last one at the end of
    // the cached context (the capacity minus one chunk)
    const int ctx = std::max(rows, c->d.ids_cap - ATT_CHUNK);
    int items = 0;
    for (int i = 0; i < rows; ++i) {
      const int pos = ctx - rows + i;
      t.seq[i] = 0, t.r[i] = 1, t.pos[i] = pos, t.kv_slot[i] = pos, t.n_canon[i] = pos + 1, t.n_safe[i] = ctx - rows, t.n_spec[i] = 0;
      t.chunk_start[i] = items;
      items += att_items(pos + 1, c->d.att_mode);
    }
    t.chunk_start[rows] = items, t.attn_items = items;
  }
  CU(c, cudaMemcpyAsync(c->ws + c->L.tab_pf, &t, sizeof t, cudaMemcpyHostToDevice, c->stream));
  CU(c, cudaMemsetAsync(c->ws + c->L.hid + (size_t)c->d.S * c->d.NB * c->m.hidden * 4, 0, (size_t)rows * c->m.hidden * 4, c->stream));
  const RowTable* tab = c->at<RowTable>(c->L.tab_pf);
  int L = c->m.n_recurrent;
  if (kTune && getenv("LOOPSPEC_TK_LAYERS")) L = std::max(1, std::min(L, atoi(getenv("LOOPSPEC_TK_LAYERS"))));  // L2-resident weights
  auto run = [&](int n) -> cudaError_t {
    for (int i = 0; i < n; ++i) {
      if (which >= 5) {
        cudaError_t e = launch_attention(c, tab, i % L, nullptr, 0, which == 6);
        if (e) return e;
        continue;
      }
      GemmParams p = gemm_params(c, which, i % L, tab);
      if (kTune && tune_timeline(c)) p.dbg = reinterpret_cast<long long*>(tune_timeline(c));  // phase stamps of CTA 0 (tuning builds)
      cudaError_t e = (c->dg && which == G_LM)         ? launch_dg_lm(c, tab)
                      : (c->tc[1].on && which != G_LM) ? launch_tc_gemm(c, which, i % L, tab, 1)
                                                       : launch_gemm(c->m.weight_dtype, c->ng_dec, kEpiOf[which], p, c->stream, c->use_pdl);
      if (e) return e;
    }
    return cudaSuccess;
  };
  CU(c, run(std::min(iters, 8)));
  CU(c, cudaEventRecord(c->ev0, c->stream));
  CU(c, run(iters));
  CU(c, cudaEventRecord(c->ev1, c->stream));
  CU(c, cudaEventSynchronize(c->ev1));
  float ms = 0;
  CU(c, cudaEventElapsedTime(&ms, c->ev0, c->ev1));
  *ms_out = ms / iters;
  const size_t wb = c->m.weight_dtype ? 2 : 4;
  const Derived& d = c->d;
  double nk[5] = {(double)(d.Hq + 2 * d.Hkv) * c->m.hidden, (double)c->m.hidden * d.Hq, 2.0 * c->m.ffn * c->m.hidden,
                  (double)c->m.hidden * c->m.ffn, (double)c->m.vocab * c->m.hidden};
  if (bytes_out) {
    const double kv_ctx = 2.0 * c->m.n_kv_heads * (double)std::max(1, d.ids_cap - ATT_CHUNK) * c->m.head_dim * 2;  // K and V of a context, bf16
    *bytes_out = which < 5 ? nk[which] * wb : which == 5 ? rows * kv_ctx : kv_ctx;  // (the rows of a prefill pass share one context)
  }
  // the timed launches touched sequence state only through scratch; mark sequences as needing a new prefill
  std::fill(c->prefilled.begin(), c->prefilled.end(), 0);
  return LOOPSPEC_OK;
}

size_t loopspec_linear_scratch_bytes(int32_t M, int32_t N, int32_t K) {
  if (M < 1 || M > 64 || N < 16 || K < 8 || N % 16 || K % 8) return 0;
  return align_up((size_t)M * 3 * K * 2) + packed_bytes(N, K);
}

int loopspec_op_linear(const void* W, int32_t weight_dtype, const float* x, float* y, int32_t M, int32_t N, int32_t K,
                       void* scratch, size_t scratch_bytes, void* cuda_stream) {
  if (!W || !x || !y || (weight_dtype != 0 && weight_dtype != 1)) return LOOPSPEC_EINVAL;
  size_t need = loopspec_linear_scratch_bytes(M, N, K);
  if (!need) return LOOPSPEC_EINVAL;
  if (!scratch || scratch_bytes < need || (reinterpret_cast<uintptr_t>(scratch) & 15)) return LOOPSPEC_ECAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int ng = ng_for_rows(M);
  GemmPlan g = plan_gemm((N + 127) / 128, K, 148 * kCtasPerSm, true);
  PrepParams q;
  memset(&q, 0, sizeof q);
  q.m_fixed = M, q.x = x, q.K = K, q.planes = static_cast<__nv_bfloat16*>(scratch);
  if (launch_k(prep_planes_kernel, dim3(M), dim3(256), 0, st, q, false) != cudaSuccess) return LOOPSPEC_ECUDA;
  if (weight_dtype == 1) {  // stream from a tile-major copy, as the decode path does
    PackParams pp;
    memset(&pp, 0, sizeof pp);
    pp.src = static_cast<const __nv_bfloat16*>(W), pp.N = N, pp.K = K, pp.kpr = (K + 31) / 32;
    pp.dst = reinterpret_cast<__nv_bfloat16*>(static_cast<unsigned char*>(scratch) + align_up((size_t)M * 3 * K * 2));
    pack_weights_kernel<<<296, 256, 0, st>>>(pp);
    if (cudaGetLastError() != cudaSuccess) return LOOPSPEC_ECUDA;
    W = pp.dst;
  }
  GemmParams p;
  memset(&p, 0, sizeof p);
  p.W = W, p.N = N, p.K = K, p.n_rb = g.n_rb, p.kb_per_rb = g.kpr, p.cluster_size = g.cs, p.n_clusters = g.n_clusters;
  p.xplanes = q.planes, p.x_ld = K, p.m_fixed = M;
  p.out = y, p.out_ld = N;
  GemmFn fn = gemm_fn(weight_dtype, ng, EPI_PLAIN);
  if (gemm_smem(weight_dtype, ng) > 48 * 1024 &&
      cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, gemm_smem(weight_dtype, ng)) != cudaSuccess)
    return LOOPSPEC_ECUDA;
  cudaError_t e = launch_gemm(weight_dtype, ng, EPI_PLAIN, p, st, false);
  return e == cudaSuccess ? LOOPSPEC_OK : LOOPSPEC_ECUDA;
}

// ---- linear map without any caller- or library-side allocation ---------------------------------------------
// Scratch for loopspec_op_linear_static: one fixed array in the library's device image.  Host code may only use
// the symbol through cudaGetSymbolAddress; the address is looked up once per device and cached.
#define LOOPSPEC_STATIC_SCRATCH_BYTES (16u << 20)
static __device__ __align__(256) unsigned char g_static_scratch[LOOPSPEC_STATIC_SCRATCH_BYTES];

int loopspec_op_linear_static(const void* W, int32_t weight_dtype, const float* x, float* y, int32_t M, int32_t N, int32_t K,
                              void* cuda_stream) {
  // one slot per device; the address of a device symbol never changes, so two threads racing on a first call store
  // the same value and the atomic only makes the publication well defined
  static std::atomic<void*> scratch_of_device[64];
  size_t need = loopspec_linear_scratch_bytes(M, N, K);
  if (!need) return LOOPSPEC_EINVAL;
  if (need > LOOPSPEC_STATIC_SCRATCH_BYTES) return LOOPSPEC_ECAPACITY;  // beyond the built-in scratch: use loopspec_op_linear
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LOOPSPEC_ECUDA;
  void* ptr = scratch_of_device[dev].load(std::memory_order_acquire);
  if (!ptr) {  // first call on this device (it is the current one): resolve the array's device address; this is
               // also the moment the library's device image, the 16 MiB array included, becomes resident there
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
      (void)cudaGetLastError();
      return LOOPSPEC_ECUDA;
    }
    scratch_of_device[dev].store(ptr, std::memory_order_release);
  }
  return loopspec_op_linear(W, weight_dtype, x, y, M, N, K, ptr, LOOPSPEC_STATIC_SCRATCH_BYTES, cuda_stream);
}

}  // extern "C"

// ---- the same linear map on tcgen05 / TMA (stand-alone operator) ---------------------------------------------
namespace {
struct TcPlan {
  int MP, stages, n_rb, n_split, kb_per_split;
  size_t smem, planes_off, part_off, total;
};
bool plan_tc(int M, int N, int K, TcPlan* t) {
  if (M < 1 || M > 64 || N < 8 || N % 8 || K < TC_BK || K % TC_BK) return false;
  t->MP = (M + 15) / 16 * 16;
  const int sb = tc_stage_bytes(t->MP);
  // measured on the Ouro-1.4B shapes: up to 16 columns stream best from many small CTAs (two stages, four CTAs per
  // SM); wider tiles from two CTAs per SM with deeper rings
  const int kb_budget = t->MP <= 16 ? 56 : 100;
  const int slots = t->MP <= 16 ? 592 : 296;
  t->stages = std::max(2, std::min(TC_MAX_STAGES, (kb_budget * 1024) / sb));
  t->smem = (size_t)t->stages * sb + 1024;
  t->n_rb = (N + TC_BM - 1) / TC_BM;
  const int total_kb = K / TC_BK;
  int want = std::max(1, std::min(slots / t->n_rb, total_kb / 4));
  t->kb_per_split = (total_kb + want - 1) / want;
  t->n_split = (total_kb + t->kb_per_split - 1) / t->kb_per_split;
  t->planes_off = 256;
  t->part_off = t->planes_off + align_up((size_t)3 * t->MP * K * 2);
  t->total = t->part_off + align_up((size_t)t->n_split * M * N * 4);
  return true;
}
}  // namespace

extern "C" {

size_t loopspec_linear_tc_scratch_bytes(int32_t M, int32_t N, int32_t K) {
  TcPlan t;
  return plan_tc(M, N, K, &t) ? t.total : 0;
}

int loopspec_op_linear_tc(const void* W, const float* x, float* y, int32_t M, int32_t N, int32_t K, void* scratch,
                          size_t scratch_bytes, void* cuda_stream) {
  TcPlan t;
  if (!W || !x || !y || !plan_tc(M, N, K, &t) || (reinterpret_cast<uintptr_t>(W) & 15)) return LOOPSPEC_EINVAL;
  if (!scratch || scratch_bytes < t.total || (reinterpret_cast<uintptr_t>(scratch) & 255)) return LOOPSPEC_ECAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* sc = static_cast<unsigned char*>(scratch);
  __nv_bfloat16* planes = reinterpret_cast<__nv_bfloat16*>(sc + t.planes_off);
  CUtensorMap map_w, map_x;
  if (!make_map_bf16(&map_w, W, N, K, TC_BM) || !make_map_bf16(&map_x, planes, 3 * t.MP, K, 3 * t.MP)) return LOOPSPEC_ECUDA;
  if (cudaMemsetAsync(sc, 0, 256, st) != cudaSuccess) return LOOPSPEC_ECUDA;
  tc_split_kernel<<<t.MP, 256, 0, st>>>(x, planes, M, t.MP, K);
  LinearTcParams p;
  memset(&p, 0, sizeof p);
  p.out = t.n_split > 1 ? reinterpret_cast<float*>(sc + t.part_off) : y;
  p.M = M, p.MP = t.MP, p.N = N, p.K = K, p.kb_per_split = t.kb_per_split, p.stages = t.stages;
  p.err = reinterpret_cast<int*>(sc), p.err_code = 1;
  if (cudaFuncSetAttribute(linear_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)t.smem) != cudaSuccess)
    return LOOPSPEC_ECUDA;
  linear_tc_kernel<<<dim3(t.n_rb, t.n_split), TC_THREADS, t.smem, st>>>(map_w, map_x, p);
  if (t.n_split > 1) tc_sum_splits_kernel<<<296, 256, 0, st>>>(p.out, y, (size_t)M * N, t.n_split);
  return cudaGetLastError() == cudaSuccess ? LOOPSPEC_OK : LOOPSPEC_ECUDA;
}

int loopspec_time_linear_tc(const void* const* Ws, int32_t n_w, const float* x, int32_t M, int32_t N, int32_t K,
                            void* scratch, size_t scratch_bytes, int32_t iters, float* us_out, void* cuda_stream) {
  TcPlan t;
  if (!Ws || n_w < 1 || n_w > 64 || !x || !us_out || iters < 1 || !plan_tc(M, N, K, &t)) return LOOPSPEC_EINVAL;
  const size_t part_bytes = align_up((size_t)t.n_split * M * N * 4);
  if (!scratch || scratch_bytes < t.part_off + part_bytes || (reinterpret_cast<uintptr_t>(scratch) & 255)) return LOOPSPEC_ECAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* sc = static_cast<unsigned char*>(scratch);
  __nv_bfloat16* planes = reinterpret_cast<__nv_bfloat16*>(sc + t.planes_off);
  std::vector<CUtensorMap> maps(n_w);
  CUtensorMap map_x;
  for (int i = 0; i < n_w; ++i)
    if (!Ws[i] || (reinterpret_cast<uintptr_t>(Ws[i]) & 15) || !make_map_bf16(&maps[i], Ws[i], N, K, TC_BM)) return LOOPSPEC_EINVAL;
  if (!make_map_bf16(&map_x, planes, 3 * t.MP, K, 3 * t.MP)) return LOOPSPEC_ECUDA;
  if (cudaMemsetAsync(sc, 0, 256, st) != cudaSuccess) return LOOPSPEC_ECUDA;
  tc_split_kernel<<<t.MP, 256, 0, st>>>(x, planes, M, t.MP, K);
  LinearTcParams p;
  memset(&p, 0, sizeof p);
  p.out = reinterpret_cast<float*>(sc + t.part_off);
  p.M = M, p.MP = t.MP, p.N = N, p.K = K, p.kb_per_split = t.kb_per_split, p.stages = t.stages;
  p.err = reinterpret_cast<int*>(sc), p.err_code = 1;
  if (cudaFuncSetAttribute(linear_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)t.smem) != cudaSuccess)
    return LOOPSPEC_ECUDA;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3(t.n_rb, t.n_split), cfg.blockDim = dim3(TC_THREADS), cfg.dynamicSmemBytes = t.smem, cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at, cfg.numAttrs = 1;
  cudaEvent_t e0, e1;
  if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return LOOPSPEC_ECUDA;
  cudaError_t e = cudaSuccess;
  for (int rep = 0; rep < iters + 1 && e == cudaSuccess; ++rep) {  // the first round warms up
    if (rep == 1) e = cudaEventRecord(e0, st);
    for (int i = 0; i < n_w && e == cudaSuccess; ++i) e = cudaLaunchKernelEx(&cfg, linear_tc_kernel, maps[i], map_x, p);
  }
  if (e == cudaSuccess) e = cudaEventRecord(e1, st);
  if (e == cudaSuccess) e = cudaEventSynchronize(e1);
  float ms = 0.f;
  if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
  cudaEventDestroy(e0), cudaEventDestroy(e1);
  if (e != cudaSuccess) return LOOPSPEC_ECUDA;
  *us_out = ms * 1e3f / ((float)iters * n_w);
  return LOOPSPEC_OK;
}

}  // extern "C"

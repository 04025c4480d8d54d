// Device-resident scheduler: the branch bookkeeping of Algorithm 1 (Spawn, the readout branches at d1/d2,
// Verify's outcome, Reroot) and the construction of the next pass's row table, so that a decode step is a
// CUDA-graph replay with no host round trip.  All kernels here run as ONE CTA: the tables are a few KB,
// are pulled into shared memory, updated there (one thread per sequence) and written back.
#pragma once
#include "common.cuh"

namespace ls {

constexpr int CTRL_THREADS = 256;
constexpr int MAX_NODES = 512;   // max_seqs * nodes-per-sequence
enum { PH_ADVANCE = 1, PH_VERIFY = 2, PH_BUILD = 4 };
enum { HF_ERROR = 0, HF_MIN_DEC = 1, HF_N_ROWS = 2, HF_NEED_VERIFY = 3, HF_FIRST_TOKEN = 4, HF_COUNT = 8 };
enum { ERR_NODES = 1, ERR_CTX = 2, ERR_SPEC = 3, ERR_WAIT = 4 /* bounded wait, decode GEMM */, ERR_WAIT_PF = 5 /* prefill GEMM, grid barrier */ };

struct ControlParams {
  int att_mode;     // how attention work items are cut (att_run_len)
  RowTable* tab;
  NodeTable nodes;
  SeqState seqs;
  Counters* ctr;
  int S, NB, R, d1, d2, ctx_cap;
  const int* sel_tok;
  const int* sel_aux;
  const float* sel_lse;
  const float* sel_z2;
  const float4* sel_flt;  // nucleus of a drafted row's readout (null unless C filters)
  int phases;
  int* out_ids;      // [S][ids_cap] decoded tokens since prefill
  int ids_cap;
  int* commits;      // [S][ids_cap][8]
  int* row_trace;    // [trace_cap], trace_n[0] entries used
  int* trace_n;
  int trace_cap;
  KvCopyCmd* kvcopy; // [S]
  float* hid;        // [hid_idx][H]
  int H;
  const void* embed; // [V][H]
  int weight_dtype;
  int p_logit_base;  // logits index of sequence 0's target readout
  volatile int* host_flags;  // pinned, host-mapped
  // Raven-style layout (P and C hold transformer blocks, Sec. 3.1): the rows entering their first recurrence go through
  // the prelude blocks first (tab_pre), the reading-out rows through the coda blocks on a copy of their state (tab_coda)
  RowTable* tab_pre;   // null for the Ouro layout
  RowTable* tab_coda;
  int hid_coda_base;   // first hidden-state index of the coda pass's copies
};

// Sub-pass tables of the Raven-style layout, derived from the pass's rows (thread 0, straight to global memory).
// class_of_readout: RO_D1 -> coda cache 1, RO_D2 -> 2, RO_VERIFY / RO_TARGET -> the last one (its plane index + 1 is `r`).
__device__ void derive_raven_tables(const RowTable& t, RowTable* pre, RowTable* coda, int hid_coda_base, int n_classes) {
  auto copy_row = [&](RowTable* dst, int j, int i) {
    dst->seq[j] = t.seq[i], dst->pos[j] = t.pos[i], dst->kv_slot[j] = t.kv_slot[i], dst->n_canon[j] = t.n_canon[i];
    dst->n_spec[j] = t.n_spec[i], dst->n_safe[j] = t.n_safe[i], dst->node[j] = t.node[i], dst->logit_idx[j] = t.logit_idx[i];
    for (int k = 0; k < MAX_SPEC; ++k) dst->spec_slot[j][k] = t.spec_slot[i][k];
  };
  int items = 0;
  if (pre) {
    int np = 0;
    for (int i = 0; i < t.n_rows; ++i) {
      if (t.r[i] != 1) continue;  // P runs once per branch, before its first recurrence
      copy_row(pre, np, i);
      pre->r[np] = 1, pre->hid_idx[np] = t.hid_idx[i], pre->src_hid[np] = -1, pre->readout[np] = RO_NONE;
      pre->chunk_start[np] = items;
      items += att_items(t.n_canon[i], t.att_mode);
      ++np;
    }
    pre->chunk_start[np] = items;
    pre->n_rows = np, pre->n_readout = 0, pre->attn_items = items, pre->att_mode = t.att_mode;
  }
  int nc = 0;
  items = 0;
  for (int j = 0; j < t.n_readout; ++j) {
    const int i = t.ro_rows[j];
    copy_row(coda, nc, i);
    const int ro = t.readout[i];
    coda->r[nc] = ro == RO_D1 ? 1 : (ro == RO_D2 ? 2 : n_classes);
    coda->hid_idx[nc] = hid_coda_base + nc, coda->src_hid[nc] = t.hid_idx[i];
    coda->readout[nc] = ro, coda->ro_rows[nc] = nc;
    coda->chunk_start[nc] = items;
    items += att_items(t.n_canon[i], t.att_mode);
    ++nc;
  }
  coda->chunk_start[nc] = items;
  coda->n_rows = nc, coda->n_readout = nc, coda->attn_items = items, coda->att_mode = t.att_mode;
}

struct NodeSmem {
  int state[MAX_NODES], depth[MAX_NODES], pos[MAX_NODES], token[MAX_NODES], parent[MAX_NODES], child1[MAX_NODES],
      child2[MAX_NODES], tok1[MAX_NODES], tok2[MAX_NODES], has2[MAX_NODES];
  float lse1[MAX_NODES], lse2[MAX_NODES], z2[MAX_NODES];
};

__device__ __forceinline__ void nodes_load(NodeSmem& s, const NodeTable& g, int n) {
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    s.state[i] = g.state[i], s.depth[i] = g.depth[i], s.pos[i] = g.pos[i], s.token[i] = g.token[i];
    s.parent[i] = g.parent[i], s.child1[i] = g.child1[i], s.child2[i] = g.child2[i], s.tok1[i] = g.tok1[i];
    s.tok2[i] = g.tok2[i], s.has2[i] = g.has2[i], s.lse1[i] = g.lse1[i], s.lse2[i] = g.lse2[i], s.z2[i] = g.z2[i];
  }
}
__device__ __forceinline__ void nodes_store(const NodeSmem& s, const NodeTable& g, int n) {
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    g.state[i] = s.state[i], g.depth[i] = s.depth[i], g.pos[i] = s.pos[i], g.token[i] = s.token[i];
    g.parent[i] = s.parent[i], g.child1[i] = s.child1[i], g.child2[i] = s.child2[i], g.tok1[i] = s.tok1[i];
    g.tok2[i] = s.tok2[i], g.has2[i] = s.has2[i], g.lse1[i] = s.lse1[i], g.lse2[i] = s.lse2[i], g.z2[i] = s.z2[i];
  }
}

// P of Eq. 1 for the Ouro layout: hidden state at depth 0 = embedding row of the prefix's last token.  All rows are
// copied in one flat loop so that every load is in flight before the first store (H is a multiple of 128).  A node slot
// freed and handed out again within one step appears twice in the list: the later entry is the live one.
__device__ __forceinline__ void embed_rows(const int (*list)[2], int n, float* hid, int H, const void* embed, int wdt) {
  const int per_row = H / 8;  // 8 elements per thread and step
  for (int idx = threadIdx.x; idx < n * per_row; idx += blockDim.x) {
    const int e = idx / per_row, i = (idx - e * per_row) * 8;
    bool superseded = false;
    for (int e2 = e + 1; e2 < n; ++e2) superseded |= list[e2][0] == list[e][0];
    if (superseded) continue;
    float4* dst = reinterpret_cast<float4*>(hid + (size_t)list[e][0] * H + i);
    if (wdt == 1) {
      const uint4 w = *reinterpret_cast<const uint4*>(static_cast<const unsigned short*>(embed) + (size_t)list[e][1] * H + i);
      dst[0] = make_float4(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xffff0000u), __uint_as_float(w.y << 16),
                           __uint_as_float(w.y & 0xffff0000u));
      dst[1] = make_float4(__uint_as_float(w.z << 16), __uint_as_float(w.z & 0xffff0000u), __uint_as_float(w.w << 16),
                           __uint_as_float(w.w & 0xffff0000u));
    } else {
      const float4* src = reinterpret_cast<const float4*>(static_cast<const float*>(embed) + (size_t)list[e][1] * H + i);
      dst[0] = src[0], dst[1] = src[1];
    }
  }
}

__device__ __forceinline__ int alloc_node(int* state, int NB) {
  for (int i = 0; i < NB; ++i)
    if (!state[i]) return i;
  return -1;
}

// Fill the row table from the active branches (thread 0; tables live in shared memory).
__device__ void build_rows(RowTable& t, const NodeSmem& nd, const int* root, const int* n_dec, const int* n_target,
                           const ControlParams& p, int* err) {
  int n_rows = 0, n_ro = 0, items = 0;
  for (int s = 0; s < p.S; ++s) {
    if (root[s] < 0 || n_dec[s] >= n_target[s]) continue;
    const int o = s * p.NB;
    const int rt = root[s];
    for (int n = 0; n < p.NB; ++n) {
      if (!nd.state[o + n]) continue;
      if (n_rows >= MAX_ROWS) { *err = ERR_NODES; break; }
      // a position outside the KV pool is never scheduled (the host refuses such a decode before it starts; this is
      // the second line of defence): the branch stays where it is and the flag tells the host
      if (nd.pos[o + n] + 2 >= p.ctx_cap) { *err = ERR_CTX; continue; }
      const int i = n_rows++;
      const int r = nd.depth[o + n] + 1;
      const bool is_root = nd.parent[o + n] < 0;
      t.seq[i] = s, t.r[i] = r, t.pos[i] = nd.pos[o + n], t.node[i] = o + n, t.hid_idx[i] = o + n;
      t.kv_slot[i] = is_root ? nd.pos[o + n] : p.ctx_cap + n;
      t.src_hid[i] = -1;
      t.n_canon[i] = nd.pos[o + rt] + 1;
      t.n_safe[i] = is_root ? nd.pos[o + n] : t.n_canon[i];
      int chain[MAX_SPEC], len = 0;
      for (int a = n; a >= 0 && nd.parent[o + a] >= 0; a = nd.parent[o + a]) {
        if (len >= MAX_SPEC) { *err = ERR_SPEC; break; }
        chain[len++] = a;
      }
      t.n_spec[i] = len;
      for (int j = 0; j < len; ++j) t.spec_slot[i][j] = p.ctx_cap + chain[len - 1 - j];
      int ro = RO_NONE, li = 0;
      if (r == p.d1) ro = RO_D1, li = (o + n) * 2;
      else if (p.d2 > 0 && r == p.d2) ro = RO_D2, li = (o + n) * 2 + 1;
      else if (r == p.R) ro = RO_VERIFY, li = p.p_logit_base + s;
      t.readout[i] = ro, t.logit_idx[i] = li;
      if (ro) t.ro_rows[n_ro++] = i;
      t.chunk_start[i] = items;
      items += att_items(t.n_canon[i], p.att_mode);
    }
  }
  t.chunk_start[n_rows] = items;
  t.n_rows = n_rows, t.n_readout = n_ro, t.attn_items = items, t.att_mode = p.att_mode;
}

// dynamic shared memory of control_kernel: the branch table, the row table and the per-row selection results
struct ControlSmem {
  NodeSmem nd;
  RowTable t;
  int emb[2 * MAX_ROWS][2];
  int sel_tok[MAX_ROWS], sel_aux[MAX_ROWS];
  float sel_lse[MAX_ROWS], sel_z2[MAX_ROWS];
};

__global__ void __launch_bounds__(CTRL_THREADS) control_kernel(const __grid_constant__ ControlParams p) {
  extern __shared__ __align__(16) unsigned char ctrl_smem_raw[];
  ControlSmem& sm = *reinterpret_cast<ControlSmem*>(ctrl_smem_raw);
  NodeSmem& nd = sm.nd;
  RowTable& t = sm.t;
  int (*s_emb)[2] = sm.emb;
  int *s_sel_tok = sm.sel_tok, *s_sel_aux = sm.sel_aux;
  float *s_sel_lse = sm.sel_lse, *s_sel_z2 = sm.sel_z2;
  __shared__ int s_root[MAX_SEQS], s_nids[MAX_SEQS], s_ndec[MAX_SEQS], s_ntarget[MAX_SEQS], s_needv[MAX_SEQS];
  __shared__ int s_nemb, s_err;
  __shared__ unsigned long long s_steps;
  __shared__ int s_trace_n;
  const int tid = threadIdx.x;
  const int n_nodes = p.S * p.NB;
  tune_mark(603, false);
  pdl_launch_dependents();
  // Everything the serial bookkeeping reads is pulled into shared memory with one round of parallel loads.  The branch
  // table, the row table and the sequence state were last written by the previous step, so they are read while this
  // step's readout kernels are still running; only the selection results have to wait for them.
  if (tid == CTRL_THREADS - 1) s_steps = p.ctr->steps;
  if (tid == CTRL_THREADS - 2) s_trace_n = *p.trace_n;
  nodes_load(nd, p.nodes, n_nodes);
  {
    const int* src = reinterpret_cast<const int*>(p.tab);
    int* dst = reinterpret_cast<int*>(&t);
    for (int i = tid; i < (int)(sizeof(RowTable) / 4); i += CTRL_THREADS) dst[i] = src[i];
  }
  if (tid < p.S) {
    s_root[tid] = p.seqs.root[tid], s_nids[tid] = p.seqs.n_ids[tid], s_ndec[tid] = p.seqs.n_dec[tid];
    s_ntarget[tid] = p.seqs.n_target[tid], s_needv[tid] = p.seqs.need_verify[tid];
  }
  pdl_wait();
  for (int i = tid; i < MAX_ROWS; i += CTRL_THREADS) {
    s_sel_tok[i] = p.sel_tok[i], s_sel_aux[i] = p.sel_aux[i];
    s_sel_lse[i] = p.sel_lse[i], s_sel_z2[i] = p.sel_z2[i];
  }
  if (tid == 0) s_nemb = 0, s_err = 0;
  __syncthreads();

  if (tid < p.S) {
    const int s = tid, o = s * p.NB;
    int* st = nd.state + o;
    // ---- advance, first proposal at d1, gated second proposal at d2 (Algorithm 1 main loop body) ----
    if (p.phases & PH_ADVANCE) {
      for (int i = 0; i < t.n_rows; ++i)
        if (t.seq[i] == s) nd.depth[t.node[i]] = t.r[i];
      for (int i = 0; i < t.n_rows; ++i) {
        if (t.seq[i] != s) continue;
        const int gn = t.node[i], ro = t.readout[i];
        if (ro == RO_D1 || (ro == RO_D2 && s_sel_aux[i])) {
          int c = alloc_node(st, p.NB);
          if (c < 0) { s_err = ERR_NODES; continue; }
          st[c] = 1, nd.depth[o + c] = 0, nd.pos[o + c] = nd.pos[gn] + 1, nd.token[o + c] = s_sel_tok[i];
          nd.parent[o + c] = gn - o, nd.child1[o + c] = nd.child2[o + c] = -1, nd.has2[o + c] = 0;
          if (ro == RO_D1) {
            nd.tok1[gn] = s_sel_tok[i], nd.child1[gn] = c, nd.lse1[gn] = s_sel_lse[i], nd.has2[gn] = 0, nd.child2[gn] = -1;
            if (p.sel_flt) p.nodes.flt1[gn] = p.sel_flt[i];
          } else {
            nd.tok2[gn] = s_sel_tok[i], nd.child2[gn] = c, nd.lse2[gn] = s_sel_lse[i], nd.z2[gn] = s_sel_z2[i], nd.has2[gn] = 1;
            if (p.sel_flt) p.nodes.flt2[gn] = p.sel_flt[i];
            atomicAdd(&p.ctr->gate_opens, 1ull);
          }
          int e = atomicAdd(&s_nemb, 1);
          s_emb[e][0] = o + c, s_emb[e][1] = s_sel_tok[i];
        }
        if (ro == RO_D2) atomicAdd(&p.ctr->gate_evals, 1ull);
        if (ro == RO_VERIFY) s_needv[s] = 1;
      }
    }
    // ---- the deepest branch reached R: commit and Reroot ---------------------------------------------
    p.kvcopy[s].n_planes = 0;
    if ((p.phases & PH_VERIFY) && s_needv[s]) {
      int vrow = -1;
      for (int i = 0; i < t.n_rows; ++i)
        if (t.seq[i] == s && t.readout[i] == RO_VERIFY) vrow = i;
      const int rt = s_root[s];
      const int tok = s_sel_tok[vrow], src = s_sel_aux[vrow];
      const int k = s_ndec[s];
      if (k < p.ids_cap) {
        p.out_ids[(size_t)s * p.ids_cap + k] = tok;
        int* cm = p.commits + ((size_t)s * p.ids_cap + k) * 8;
        cm[0] = s, cm[1] = 1, cm[2] = tok, cm[3] = src, cm[4] = (src == 1), cm[5] = (src == 2), cm[6] = nd.has2[o + rt];
        cm[7] = (int)s_steps + ((p.phases & PH_ADVANCE) ? 1 : 0);
      }
      s_ndec[s] = k + 1, s_nids[s] += 1;
      atomicAdd(&p.ctr->n_decode, 1ull);
      atomicAdd(src == 1 ? &p.ctr->n_accept1 : (src == 2 ? &p.ctr->n_accept2 : &p.ctr->n_restart), 1ull);
      const int keep = src == 1 ? nd.child1[o + rt] : (src == 2 ? nd.child2[o + rt] : -1);
      const int new_pos = nd.pos[o + rt] + 1;
      for (int n = 0; n < p.NB; ++n) {
        if (!st[n]) continue;
        bool in = false;
        for (int a = n; a >= 0; a = nd.parent[o + a])
          if (a == keep) { in = true; break; }
        if (!in) st[n] = 0;
      }
      if (keep < 0) {  // restart: fresh branch on the verified prefix
        const int c = alloc_node(st, p.NB);
        st[c] = 1, nd.depth[o + c] = 0, nd.pos[o + c] = new_pos, nd.token[o + c] = tok, nd.parent[o + c] = -1;
        nd.child1[o + c] = nd.child2[o + c] = -1, nd.has2[o + c] = 0;
        s_root[s] = c;
        int e = atomicAdd(&s_nemb, 1);
        s_emb[e][0] = o + c, s_emb[e][1] = tok;
      } else {         // keep the chosen child and its descendants; its KV joins the committed prefix
        nd.parent[o + keep] = -1;
        s_root[s] = keep;
        p.kvcopy[s].src_slot = p.ctx_cap + keep, p.kvcopy[s].dst_slot = nd.pos[o + keep];
        p.kvcopy[s].n_planes = nd.depth[o + keep];
      }
      s_needv[s] = 0;
    }
  }
  __syncthreads();
  if (tid == 0) {
    if (p.phases & PH_ADVANCE) {  // counters: no value is read back, so nothing here waits for memory
      atomicAdd(&p.ctr->steps, 1ull), atomicAdd(&p.ctr->rows_total, (unsigned long long)t.n_rows);
      atomicAdd(&p.ctr->readout_rows_total, (unsigned long long)t.n_readout);
      atomicMax(&p.ctr->rows_max, (unsigned long long)t.n_rows);
      const int k = s_trace_n;
      if (k < p.trace_cap) p.row_trace[k] = t.n_rows;
      *p.trace_n = k + 1;
    }
    int need = 0, min_dec = 0x7fffffff;
    for (int s = 0; s < p.S; ++s) {
      need += s_needv[s];
      if (s_root[s] >= 0) min_dec = min(min_dec, s_ndec[s]);
    }
    int err = s_err;
    // rows are rebuilt only when no verification is pending (the verify phase needs the current rows)
    if ((p.phases & PH_BUILD) && need == 0) {
      build_rows(t, nd, s_root, s_ndec, s_ntarget, p, &err);
      if (p.tab_pre) derive_raven_tables(t, p.tab_pre, p.tab_coda, p.hid_coda_base, p.d2 > 0 ? 3 : 2);
    }
    p.host_flags[HF_MIN_DEC] = min_dec, p.host_flags[HF_N_ROWS] = t.n_rows, p.host_flags[HF_NEED_VERIFY] = need;
    if (err) p.host_flags[HF_ERROR] = err;
  }
  __syncthreads();
  nodes_store(nd, p.nodes, n_nodes);
  {
    int* dst = reinterpret_cast<int*>(p.tab);
    const int* src = reinterpret_cast<const int*>(&t);
    for (int i = tid; i < (int)(sizeof(RowTable) / 4); i += CTRL_THREADS) dst[i] = src[i];
  }
  if (tid < p.S) {
    p.seqs.root[tid] = s_root[tid], p.seqs.n_ids[tid] = s_nids[tid], p.seqs.n_dec[tid] = s_ndec[tid];
    p.seqs.need_verify[tid] = s_needv[tid];
  }
  embed_rows(s_emb, s_nemb, p.hid, p.H, p.embed, p.weight_dtype);
  tune_mark(603, true);
}

// ---- vanilla decoding (Fig. 1a): one row per sequence, R passes per token ---------------------------
struct VanillaParams {
  int att_mode;     // how attention work items are cut (att_run_len)
  RowTable* tabs;   // [R] one table per recurrence
  NodeTable nodes;
  SeqState seqs;
  int S, NB, R;
  const int* sel_tok;
  int commit;       // 0: set up from the current committed prefix; 1: commit sel_tok of each sequence first
  int* out_ids;
  int ids_cap;
  float* hid;
  int H;
  const void* embed;
  int weight_dtype, p_logit_base, ctx_cap;
  volatile int* host_flags;
  RowTable* tab_coda;  // Raven-style layout: the readout rows of the last recurrence on copies of their states (else null)
  int hid_coda_base, n_classes;
};

__global__ void __launch_bounds__(CTRL_THREADS) vanilla_control_kernel(const __grid_constant__ VanillaParams p) {
  __shared__ int s_emb[MAX_SEQS][2];
  __shared__ int s_rowof[MAX_SEQS];
  __shared__ int s_n;
  const int tid = threadIdx.x;
  pdl_launch_dependents();
  pdl_wait();
  if (tid == 0) {
    int n = 0;
    const RowTable& cur = p.tabs[p.R - 1];
    for (int s = 0; s < p.S; ++s) {
      int rt = p.seqs.root[s];
      if (rt < 0) continue;
      const int o = s * p.NB;
      if (p.commit) {
        int row = -1;
        for (int i = 0; i < cur.n_rows; ++i)
          if (cur.seq[i] == s) row = i;
        if (row < 0) continue;  // the sequence had no row in the last pass (dropped at the capacity limit)
        int tok = p.sel_tok[row];
        int k = p.seqs.n_dec[s];
        if (k < p.ids_cap) p.out_ids[(size_t)s * p.ids_cap + k] = tok;
        p.seqs.n_dec[s] = k + 1, p.seqs.n_ids[s] += 1;
        p.nodes.token[o + rt] = tok, p.nodes.pos[o + rt] += 1;
      } else {
        for (int i = 0; i < p.NB; ++i)
          if (i != rt) p.nodes.state[o + i] = 0;
      }
      p.nodes.depth[o + rt] = 0, p.nodes.child1[o + rt] = p.nodes.child2[o + rt] = -1, p.nodes.has2[o + rt] = 0;
      p.seqs.need_verify[s] = 0;
      if (p.nodes.pos[o + rt] + 2 >= p.ctx_cap) {  // never schedule a position outside the KV pool
        p.host_flags[HF_ERROR] = ERR_CTX;
        continue;
      }
      s_emb[n][0] = o + rt, s_emb[n][1] = p.nodes.token[o + rt];
      s_rowof[n] = s;
      ++n;
    }
    s_n = n;
    for (int r = 1; r <= p.R; ++r) {
      RowTable& t = p.tabs[r - 1];
      int items = 0;
      for (int i = 0; i < n; ++i) {
        int s = s_rowof[i], gn = s_emb[i][0], pos = p.nodes.pos[gn];
        t.seq[i] = s, t.r[i] = r, t.pos[i] = pos, t.kv_slot[i] = pos, t.n_canon[i] = pos + 1, t.n_spec[i] = 0;
        t.n_safe[i] = pos;
        t.hid_idx[i] = gn, t.node[i] = gn, t.readout[i] = (r == p.R) ? RO_TARGET : RO_NONE, t.src_hid[i] = -1;
        t.logit_idx[i] = p.p_logit_base + s, t.ro_rows[i] = i, t.chunk_start[i] = items;
        items += att_items(pos + 1, p.att_mode);
      }
      t.chunk_start[n] = items;
      t.n_rows = n, t.n_readout = (r == p.R) ? n : 0, t.attn_items = items, t.att_mode = p.att_mode;
    }
    if (p.tab_coda) {  // the prelude pass of a vanilla token is the first table itself (every row enters recurrence 1)
      derive_raven_tables(p.tabs[p.R - 1], nullptr, p.tab_coda, p.hid_coda_base, p.n_classes);
    }
  }
  __syncthreads();
  embed_rows(s_emb, s_n, p.hid, p.H, p.embed, p.weight_dtype);
}

// ---- prefill (Algorithm 1, lines before the main loop): rows = consecutive prompt positions ---------
struct PrefillParams {
  int att_mode;       // how attention work items are cut (att_run_len)
  RowTable* tab;
  const int* prompt;  // device ids of the sequence
  int seq, p0, count, r, R, n_prompt;
  int hid_base;       // first hidden-state index of the prefill rows
  int p_logit_base;
  float* hid;
  int H;
  const void* embed;
  int weight_dtype;
  RowTable* tab_coda;  // Raven-style layout: every prompt row goes through the coda blocks at the readout depths, on copies
  int coda_class;      // cache of this recurrence's readout depth (1-based; 0: this recurrence is no readout depth)
  int hid_coda_base;
};

__global__ void __launch_bounds__(CTRL_THREADS) prefill_setup_kernel(const PrefillParams p) {
  __shared__ int s_emb[MAX_ROWS][2];
  const int tid = threadIdx.x;
  // one thread per row (rows are independent: consecutive positions of one sequence); the reading-out row, if the
  // pass has one, is the prompt's last position at the last recurrence
  RowTable& t = *p.tab;
  RowTable* c = (p.tab_coda && p.coda_class > 0) ? p.tab_coda : nullptr;  // the same rows, on copies of their states,
                                                                          // writing this depth's coda cache
  const int ro_row = (p.r == p.R && p.n_prompt - 1 >= p.p0 && p.n_prompt - 1 < p.p0 + p.count) ? p.n_prompt - 1 - p.p0 : -1;
  for (int i = tid; i <= p.count; i += CTRL_THREADS) {
    int items = 0;  // work items of the rows before this one
    for (int k = 0; k < i; ++k) items += att_items(p.p0 + k + 1, p.att_mode);
    t.chunk_start[i] = items;
    if (c) c->chunk_start[i] = items;
    if (i == p.count) {
      t.n_rows = p.count, t.n_readout = ro_row >= 0 ? 1 : 0, t.attn_items = items, t.att_mode = p.att_mode;
      if (ro_row >= 0) t.ro_rows[0] = ro_row;
      if (c) {
        c->n_rows = p.count, c->n_readout = ro_row >= 0 ? 1 : 0, c->attn_items = items, c->att_mode = p.att_mode;
        if (ro_row >= 0) c->ro_rows[0] = ro_row;
      }
      break;
    }
    const int pos = p.p0 + i, ro = i == ro_row ? RO_TARGET : RO_NONE;
    t.seq[i] = p.seq, t.r[i] = p.r, t.pos[i] = pos, t.kv_slot[i] = pos, t.n_canon[i] = pos + 1, t.n_spec[i] = 0;
    t.n_safe[i] = p.p0;
    t.hid_idx[i] = p.hid_base + i, t.node[i] = -1, t.src_hid[i] = -1;
    t.readout[i] = ro, t.logit_idx[i] = p.p_logit_base + p.seq;
    s_emb[i][0] = p.hid_base + i, s_emb[i][1] = p.prompt[pos];
    if (c) {
      c->seq[i] = p.seq, c->r[i] = p.coda_class, c->pos[i] = pos, c->kv_slot[i] = pos, c->n_canon[i] = pos + 1;
      c->n_spec[i] = 0, c->n_safe[i] = p.p0, c->hid_idx[i] = p.hid_coda_base + i, c->src_hid[i] = p.hid_base + i, c->node[i] = -1;
      c->readout[i] = ro, c->logit_idx[i] = p.p_logit_base + p.seq;
    }
  }
  __syncthreads();
  if (p.r == 1) embed_rows(s_emb, p.count, p.hid, p.H, p.embed, p.weight_dtype);
}

struct PrefillFinishParams {
  const RowTable* tab;
  NodeTable nodes;
  SeqState seqs;
  int seq, NB, n_prompt, n_target;
  const int* sel_tok;
  float* hid;
  int H;
  const void* embed;
  int weight_dtype;
  volatile int* host_flags;
};

// commit the first token and Spawn(prompt || token) as the root branch at depth 0
__global__ void __launch_bounds__(CTRL_THREADS) prefill_finish_kernel(const PrefillFinishParams p) {
  __shared__ int s_emb[1][2];
  if (threadIdx.x == 0) {
    const int o = p.seq * p.NB;
    const int tok = p.sel_tok[p.tab->ro_rows[0]];
    for (int i = 0; i < p.NB; ++i) p.nodes.state[o + i] = 0;
    p.nodes.state[o] = 1, p.nodes.depth[o] = 0, p.nodes.pos[o] = p.n_prompt, p.nodes.token[o] = tok, p.nodes.parent[o] = -1;
    p.nodes.child1[o] = p.nodes.child2[o] = -1, p.nodes.has2[o] = 0;
    p.seqs.root[p.seq] = 0, p.seqs.n_ids[p.seq] = p.n_prompt + 1, p.seqs.n_dec[p.seq] = 0;
    p.seqs.n_target[p.seq] = p.n_target, p.seqs.need_verify[p.seq] = 0;
    p.host_flags[HF_FIRST_TOKEN] = tok;
    s_emb[0][0] = o, s_emb[0][1] = tok;
  }
  __syncthreads();
  embed_rows(s_emb, 1, p.hid, p.H, p.embed, p.weight_dtype);
}

// ---- KV rollback / commit: the kept branch's keys and values become the committed ones of its position ---
struct KvCommitParams {
  const KvCopyCmd* cmds;  // [S]
  __nv_bfloat16* kv;      // whole pool [L][R][2][S][n_kv][slots][d]
  long long layer_stride, plane_stride, sel_stride;
  int S, L, n_kv_heads, slots, d;
  // Raven-style layout: the pool's layers are prelude blocks (one plane), recurrent blocks (a plane per recurrence) and coda
  // blocks (a plane per readout depth); n_prelude = 0 and n_classes = 0 for the Ouro layout
  int n_prelude, n_rec, n_classes;
  int class_depth[3];
};

__global__ void kv_commit_kernel(const __grid_constant__ KvCommitParams p) {
  // grid: (L, R, 2 * S); one CTA copies n_kv_heads rows of d bf16
  tune_mark(604, false);
  pdl_launch_dependents();
  pdl_wait();
  struct EndMark { __device__ ~EndMark() { tune_mark(604, true); } } end_mark;
  const int l = blockIdx.x, plane = blockIdx.y, sel = blockIdx.z & 1, s = blockIdx.z >> 1;
  const KvCopyCmd c = p.cmds[s];
  if (c.n_planes <= 0) return;                 // nothing kept for this sequence (n_planes = recurrent depth of the kept child)
  if (l < p.n_prelude) {
    if (plane != 0) return;                    // its prelude keys / values
  } else if (l < p.n_prelude + p.n_rec) {
    if (plane >= c.n_planes) return;           // the recurrences it has been through
  } else {
    if (plane >= p.n_classes || p.class_depth[plane] > c.n_planes) return;  // the readout depths it has reached
  }
  __nv_bfloat16* base = p.kv + (size_t)l * p.layer_stride + (size_t)plane * p.plane_stride + (size_t)sel * p.sel_stride;
  const int per_head = p.d / 8;  // uint4 per head row
  for (int i = threadIdx.x; i < p.n_kv_heads * per_head; i += blockDim.x) {
    int h = i / per_head, j = i % per_head;
    size_t hb = (size_t)(s * p.n_kv_heads + h) * p.slots;
    const uint4* src = reinterpret_cast<const uint4*>(base + (hb + c.src_slot) * p.d) + j;
    uint4* dst = reinterpret_cast<uint4*>(base + (hb + c.dst_slot) * p.d) + j;
    *dst = *src;
  }
}

}  // namespace ls

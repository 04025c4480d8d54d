// Shared device-side declarations of the LoopSpec decode path: the row table every kernel of a batched
// pass reads, the branch (node) table of Algorithm 1, and small numeric helpers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ls {

// tuning aids (cycle stamps, kernel timeline) are compiled in only with -DLOOPSPEC_TUNE:
// the decode kernels run for a few microseconds each and every kilobyte of code they carry costs fetch time
#ifdef LOOPSPEC_TUNE
constexpr bool kTune = true;
#else
constexpr bool kTune = false;
#endif

constexpr int MAX_ROWS = 256; // rows (branches) one batched pass can carry (Sec. 4.3: the branch bound for R = 32 with
                              // (d1, d2) = (2, 8) is 249); the GEMMs take them in groups of up to 64 token columns
constexpr int GROUP_ROWS = 64;  // token columns one GEMM launch carries
constexpr int MAX_SEQS = 64;  // sequences a context can hold
constexpr int MAX_SPEC = 16;  // speculative ancestors (incl. the row itself) a row can attend to: R/d1 levels
constexpr int ATT_CHUNK = 64; // key positions per attention chunk (cut at fixed absolute positions)
constexpr int ATT_MAX_RUNS = 40;  // attention work items per (row, kv head) at most (contexts up to 2560: one chunk each)
constexpr int ATT_LONG_RUNS = 8;  // ... and for longer contexts
constexpr int ATT_BATCH_SINGLE = 8;  // contexts that hold several sequences: single-chunk items only up to 8 chunks
// A work item covers a run of consecutive chunks.  mode 0 (a context of one sequence: few rows per pass, every chunk in
// parallel matters): one chunk for contexts up to ATT_MAX_RUNS chunks, beyond that as many as leave ATT_LONG_RUNS items.
// mode 1 (contexts of several sequences: many rows per pass, the stream matters): one chunk up to ATT_BATCH_SINGLE
// chunks, beyond that as many as leave ATT_LONG_RUNS items.  Either way a function of the row's own context only, so a
// row's arithmetic does not depend on what shares the pass.
__host__ __device__ inline int att_run_len(int n_canon, int mode) {
  const int nc = (n_canon + ATT_CHUNK - 1) / ATT_CHUNK;
  return nc <= (mode ? ATT_BATCH_SINGLE : ATT_MAX_RUNS) ? 1 : (nc + ATT_LONG_RUNS - 1) / ATT_LONG_RUNS;
}
__host__ __device__ inline int att_items(int n_canon, int mode) {
  const int nc = (n_canon + ATT_CHUNK - 1) / ATT_CHUNK, rl = att_run_len(n_canon, mode);
  return (nc + rl - 1) / rl;
}

// readout kinds of a row after its advance (Algorithm 1: r_b = d1, r_b = d2, r_b = R)
enum { RO_NONE = 0, RO_D1 = 1, RO_D2 = 2, RO_VERIFY = 3, RO_TARGET = 4 /* x ~ C(H): prefill, vanilla */ };

// One batched pass = the rows below.  A row is one branch: one token position at one recurrent depth.
struct RowTable {
  int n_rows;
  int n_readout;             // rows whose new depth is d1, d2 or R
  int attn_items;            // sum over rows of attention work items (runs of chunks)
  int att_mode;              // how attention work items are cut (see att_run_len)
  int seq[MAX_ROWS];         // sequence of the row
  int r[MAX_ROWS];           // recurrence the row is advanced TO (1..R): KV plane it writes and reads
  int pos[MAX_ROWS];         // position of the row's token (rotary index)
  int kv_slot[MAX_ROWS];     // slot its K,V are written to
  int n_canon[MAX_ROWS];     // committed slots [0, n_canon) it attends to
  int n_spec[MAX_ROWS];      // speculative slots it attends to (its uncommitted ancestors and itself)
  int n_safe[MAX_ROWS];      // committed slots [0, n_safe) were cached by earlier passes (not written in this one)
  int spec_slot[MAX_ROWS][MAX_SPEC];
  int hid_idx[MAX_ROWS];     // where its hidden state lives (updated in place)
  int readout[MAX_ROWS];     // RO_*
  int logit_idx[MAX_ROWS];   // which logits vector its readout fills
  int node[MAX_ROWS];        // global node index (seq * NB + node), -1 for prefill rows
  int ro_rows[MAX_ROWS];     // compact list of rows with readout != 0
  int src_hid[MAX_ROWS];     // >= 0: the pass works on a copy of this hidden state, made into hid_idx by its preparation
                             // (the post-layers C of a Raven-style model must not disturb the branch's recurrent state)
  int chunk_start[MAX_ROWS + 1];  // exclusive prefix sum of attention work items per row
};

// Branch table of Algorithm 1 (a branch: prefix, hidden state, depth, proposal records), per sequence NB nodes.
struct NodeTable {
  int* state;    // 0 free, 1 active
  int* depth;    // r_b
  int* pos;      // position of the last token of the prefix
  int* token;    // that token
  int* parent;   // node index within the sequence, -1 for the root (whole prefix committed)
  int* child1;   // record 1: child spawned for the first proposal
  int* child2;   // record 2
  int* tok1;
  int* tok2;
  int* has2;     // the gate opened and record 2 exists
  float* lse1;   // log-sum-exp of z/T of the first readout
  float* lse2;
  float* z2;     // sum of [q2~ - q1]_+ (normaliser of the residual proposal), 0 if it had no mass
  float4* flt1;  // nucleus of the first readout when C filters (top-k / top-p): max z/T, kept mass, cut value, cut index
  float4* flt2;
};

struct SeqState {
  int* root;         // node index of the root branch, -1 if the sequence is idle
  int* n_ids;        // committed tokens (prompt + decoded)
  int* n_dec;        // decoded tokens since prefill (excluding the prefill token)
  int* n_target;     // decode stops committing for the sequence at this many
  int* need_verify;  // set by the step phase when the root reached R
};

struct Counters {  // App. D / App. E statistics
  unsigned long long steps, n_decode, n_accept1, n_accept2, n_restart, gate_evals, gate_opens, rows_total, rows_max,
      readout_rows_total;
};

struct KvCopyCmd {
  int src_slot, dst_slot, n_planes, pad;
};

__device__ __forceinline__ float bf16_bits_to_float(unsigned short b) { return __uint_as_float(((unsigned)b) << 16); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// x = hi + mid + lo with hi, mid, lo bf16 (round-to-nearest at each stage; the remainders are exact in fp32)
__device__ __forceinline__ void split3(float x, unsigned short& hi, unsigned short& mid, unsigned short& lo) {
  __nv_bfloat16 h = __float2bfloat16_rn(x);
  float r1 = x - __bfloat162float(h);
  __nv_bfloat16 m = __float2bfloat16_rn(r1);
  float r2 = r1 - __bfloat162float(m);
  __nv_bfloat16 l = __float2bfloat16_rn(r2);
  hi = __bfloat16_as_ushort(h);
  mid = __bfloat16_as_ushort(m);
  lo = __bfloat16_as_ushort(l);
}
// write one value into the three planes of a row: planes + plane * ld
__device__ __forceinline__ void store_split(__nv_bfloat16* row_planes, int ld, int k, float v) {
  unsigned short h, m, l;
  split3(v, h, m, l);
  row_planes[k] = __ushort_as_bfloat16(h);
  row_planes[ld + k] = __ushort_as_bfloat16(m);
  row_planes[2 * ld + k] = __ushort_as_bfloat16(l);
}

// tuning aid: earliest CTA start / latest CTA end of kernel `id` on the global nanosecond timer
__device__ __forceinline__ void timeline_mark(unsigned long long* tl, int id, bool end) {
  if (!kTune || tl == nullptr || threadIdx.x != 0) return;
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  if (end) atomicMax(tl + 2 * id + 1, t);
  else {
    atomicMin(tl + 2 * id, t);
    if (id < 256) atomicMax(tl + 2 * (id + 512) + 1, t);  // the latest CTA start
  }
}

// tuning aid for kernels without a timeline pointer of their own: a pointer set once by the host
#ifdef LOOPSPEC_TUNE
__device__ unsigned long long* g_tune_tl = nullptr;
__device__ __forceinline__ void tune_mark(int id, bool end) { timeline_mark(g_tune_tl, id, end); }
#else
__device__ __forceinline__ void tune_mark(int, bool) {}
#endif

// programmatic dependent launch: wait for the kernels this launch depends on / let dependents start launching
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

}  // namespace ls

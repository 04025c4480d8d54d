/*
 * loopspec.h -- C ABI of the LoopSpec pipelined decode path for looped transformers on B200 (sm_100a).
 *
 * The library runs the decode loop of Algorithm 1 (App. H) of "LoopSpec: Pipelined Self-Speculative
 * Decoding for Looped Transformers": in every step all active branches -- the token being verified at
 * recurrent depth R, first-proposal drafts spawned at depth d1 and, when the gate of Eq. 6 opens,
 * residual second proposals spawned at depth d2 (Eq. 5) -- go through the shared block stack in ONE
 * batched pass (Sec. 4.2 step 1), so the shared weights are read from HBM once per step.
 *
 * Conventions (all entry points):
 *   - Every call returns a loopspec_status; nothing throws or aborts across this boundary.
 *   - "device" pointers are CUDA device memory of the current device, "host" pointers are ordinary host memory.
 *   - Weights and the workspace are allocated by the caller, borrowed for the life of the context and never
 *     freed by the library; weights are never written.  The library itself allocates only host memory, CUDA
 *     graphs/events and two small pinned host buffers; it never allocates device memory.
 *   - Linear weights are row-major [out_features][in_features]; bf16 weights are raw 16-bit bfloat16,
 *     fp32 weights IEEE binary32.  Norm gains are always fp32.
 *   - Argument errors are detected on the host before any launch and leave the context usable.
 *     LOOPSPEC_ECUDA is sticky (the context must be destroyed).
 *   - A context is not thread safe; all work is issued on the stream given at init.
 */
#ifndef LOOPSPEC_H
#define LOOPSPEC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct loopspec_ctx loopspec_ctx; /* opaque, owned by the library */

typedef enum {
  LOOPSPEC_OK = 0,
  LOOPSPEC_EINVAL = -1,       /* bad argument */
  LOOPSPEC_ESTATE = -2,       /* call out of order (step before prefill, verify with nothing at depth R, ...) */
  LOOPSPEC_ECAPACITY = -3,    /* max_ctx, max_seqs, node table or workspace too small */
  LOOPSPEC_ECUDA = -4,        /* a CUDA call failed; see loopspec_last_error */
  LOOPSPEC_ETIMEOUT = -5,     /* a bounded device-side wait (mbarrier, grid barrier) ran out; the pass's results are void */
  LOOPSPEC_EUNSUPPORTED = -6  /* shape outside what the kernels support */
} loopspec_status;

/* Looped transformer of Sec. 3.1 (Eq. 1).  Ouro layout: n_prelude = n_coda = 0, P = embedding, C = final
 * RMSNorm + lm_head.  Raven-style layout (n_prelude or n_coda > 0; Sec. 3.1: P and C hold transformer blocks too):
 * P = embedding + n_prelude blocks giving e, H0 = e, one recurrence is H <- RecurrentBlocks(W_a [H; e]) with the adapter
 * W_a [hidden][2 hidden], C = n_coda blocks + final RMSNorm + lm_head.  The prelude blocks have an ordinary KV cache, the
 * coda blocks one cache per readout depth (d1, d2, R: App. B "KV Cache Management"); the prompt fills all of them.
 * Blocks are pre-RMSNorm, rotary attention (rotate-half pairing), SwiGLU, no biases. */
typedef struct {
  int32_t vocab, hidden, n_q_heads, n_kv_heads, head_dim, ffn;
  int32_t n_prelude, n_recurrent, n_coda; /* transformer blocks in P, B, C */
  int32_t R;                              /* recurrences of B */
  int32_t weight_dtype;                   /* 0 = fp32, 1 = bf16 (all matrices incl. embedding) */
  int32_t tied_lm_head;                   /* 1: lm_head pointer ignored, the embedding is used */
  float rms_eps, rope_theta;
} loopspec_model;

/* Scheduler settings (Sec. 4.2-4.3, App. B "Depth Configuration").
 * d1 < d2 < R with d1 | d2 and d1 | R; d2 == 0 selects the single-proposal pipeline of Sec. 4.2;
 * d1 == d2 == 0 picks the pair from the closed form of Theorem 2 using (alpha, beta).
 * gate = 1 applies Eq. 6, gate = 0 always creates the second proposal; residual_q2 = 1 drafts it from
 * p_{d2} (-) p_{d1} (Eq. 5), 0 from p_{d2} itself.  temperature 0 = greedy.  max_prefill_rows (0 = default)
 * bounds how many prompt positions one prefill pass carries.
 * Capacity: max_ctx counts positions per sequence, the speculative ones included: a sequence needs
 * max_ctx >= prompt + decoded tokens + R/d1 + 2 (the deepest chain of uncommitted positions); R/d1 may not exceed 16,
 * max_seqs 64, and max_seqs times the branch bound of Sec. 4.3 256 rows per pass (LOOPSPEC_ECAPACITY otherwise; the bound
 * for R = 32 with (d1, d2) = (2, 8) is 249).  Passes that can carry more than 64 rows run every GEMM once per group of 64
 * rows, i.e. stream the weights once per group.
 * top_k, top_p: the optional filters of the post-layers C (Sec. 3.1), applied at EVERY readout depth when
 * temperature > 0: tokens are ranked by decreasing probability (ties: lower index first); top_k > 0 keeps the first
 * top_k and renormalises; 0 < top_p < 1 then keeps the shortest prefix of the ranking whose mass reaches top_p and
 * renormalises.  top_k = 0 and top_p = 0 (or >= 1) switch the filters off.
 * measure_tv = 1 (sampling only): every verification also records TV(p_d1, p_R) and, where a second-proposal record
 * exists, TV(p_d2, p_R) of the readouts involved (Sec. 4.1's empirical profile; see loopspec_stats and
 * loopspec_fit_envelope).  With the gate on, the depth-d2 readout exists only where the gate opened.
 * mask_first = 1: the variant of the paper's second-proposal ablation (Sec. 6): the first candidate is removed from the
 * second proposal's distribution (the residual one if it has mass elsewhere, else p_{d2}) and the rest renormalised, so
 * the two candidates always differ; a branch whose p_{d2} has all its mass on the first candidate gets no second
 * proposal.  Under greedy decoding the second candidate is then the best token other than the first. */
typedef struct {
  int32_t d1, d2;
  float alpha, beta;
  int32_t gate, residual_q2;
  float temperature;
  uint64_t seed;
  int32_t max_seqs, max_ctx;
  int32_t max_prefill_rows;
  int32_t top_k;
  float top_p;
  int32_t measure_tv;
  int32_t mask_first;
  int32_t prefill_skinny; /* 1: the prefill passes run the kernels of the decode passes - layer GEMMs on mma.sync instead of
                             the wide tcgen05 kernel, attention row by row instead of the kernel that shares K/V among the
                             rows of a pass (slower; for comparing the two paths) */
} loopspec_sched;

/* Device pointers to the weights.  layer_ptrs is a HOST array of 6 * (n_prelude + n_recurrent + n_coda) device pointers -
 * the prelude blocks, then the recurrent blocks, then the coda blocks - per block:
 * norm1 [H], wqkv [(nq + 2 nkv) * d][H] (q rows, then k rows, then v rows), wo [H][nq * d], norm2 [H],
 * wgateup [2F][H] (gate rows, then up rows), wdown [H][F].  adapter: [H][2H] (columns: state, then prelude output) for
 * the Raven-style layout, NULL for the Ouro layout. */
typedef struct {
  const void* embed;      /* [V][H] */
  const void* lm_head;    /* [V][H], ignored when tied */
  const void* final_norm; /* fp32 [H] */
  const void* adapter;
  const void* const* layer_ptrs;
} loopspec_weights;

/* One committed token (Algorithm 1, main loop, the commit after Verify). source: 1 = accepted first
 * proposal, 2 = accepted second proposal, 3 = resampled at depth R (restart). step = index (from 1) of the
 * batched pass after which it was committed. */
typedef struct {
  int32_t seq, n_committed, token, source, accepted1, accepted2, gate_open, step;
} loopspec_commit;

/* Counters of Sec. 6 (gamma), App. D (gate openings, effective batch size) and App. E (commit sources).
 * tv_d1 / tv_d2: mean total-variation distance between the depth-d1 / depth-d2 readout and the target over the
 * tv_n1 / tv_n2 verifications that had one (0 unless the scheduler was created with measure_tv). */
typedef struct {
  int64_t steps, n_decode, n_accept1, n_accept2, n_restart, gate_evals, gate_opens, rows_total, rows_max,
      readout_rows_total;
  double gamma;
  double tv_d1, tv_d2;
  int64_t tv_n1, tv_n2;
} loopspec_stats;

/* Bytes of device workspace loopspec_init needs for this model and scheduler (0 on invalid input).  For bf16
 * weights this includes a second, tile-major copy of every matrix that the kernels stream from. */
size_t loopspec_workspace_bytes(const loopspec_model*, const loopspec_sched*);

/* Create a context.  workspace: device memory, 256-byte aligned, at least loopspec_workspace_bytes large.
 * cuda_stream: a cudaStream_t created by the caller; NULL (the legacy default stream) is rejected with EINVAL
 * because the decode step is captured into a CUDA graph on it.
 * Host structs are copied.  Synchronous; uploads the rotary table and clears the workspace tables. */
int loopspec_init(const loopspec_model*, const loopspec_sched*, const loopspec_weights*, void* workspace,
                  size_t workspace_bytes, void* cuda_stream, loopspec_ctx** out);

/* Algorithm 1, lines before the main loop: run all R recurrences over the prompt of sequence `seq`
 * (host array of n ids), fill every (layer, recurrence) KV plane, commit the first token drawn from C(H^R)
 * and spawn the initial branch on prompt||token.  first_token (host, may be NULL) receives that token.
 * Synchronous.  Calling it again for the same seq restarts that sequence. */
int loopspec_prefill(loopspec_ctx*, int32_t seq, const int32_t* prompt_ids, int32_t n, int32_t* first_token);

/* One iteration of the body of Algorithm 1's main loop up to, not including, verification: advance every
 * active branch by one recurrent depth in one batched pass, read out branches reaching d1 / d2 / R, draw
 * first proposals, evaluate the gate, draw second proposals, spawn their children.  n_rows_out: branches
 * advanced; n_need_verify_out: sequences whose deepest branch reached R (call loopspec_verify before the
 * next step if > 0).  Synchronous. */
int loopspec_step(loopspec_ctx*, int32_t* n_rows_out, int32_t* n_need_verify_out);

/* Cascade verification (Sec. 4.3; Algorithm 1 Verify + Reroot) for every sequence whose deepest branch is
 * at depth R: accept the first candidate w.p. min{1, p/q1}, else the second against p (-) q1, else
 * resample; commit, keep the chosen child's subtree, release the rest, make the kept branch's KV part of
 * the committed prefix.  out: host array of max_out entries.  ESTATE if nothing is at depth R. */
int loopspec_verify(loopspec_ctx*, loopspec_commit* out, int32_t max_out, int32_t* n_out);

/* Run step+verify until every prefilled sequence has committed n_tokens more tokens, as CUDA-graph
 * replays with the branch table on the device.  ids_out: host [max_seqs][n_tokens] (rows of sequences
 * that were not prefilled are left untouched).  Produces exactly the tokens of alternating step/verify. */
int loopspec_decode(loopspec_ctx*, int32_t n_tokens, int32_t* ids_out);

/* Baseline of Fig. 1(a): all R recurrences of a token before the next, from the same kernels. */
int loopspec_vanilla_decode(loopspec_ctx*, int32_t n_tokens, int32_t* ids_out);

/* Power-law envelope phi(r) = beta r^-alpha over a measured total-variation profile tv[r-1] = TV(p_r, p_R),
 * r = 1..n (Sec. 4.1, the min-max-ratio fit of the envelope), read as:
 * minimise max_r phi(r) / tv[r-1] subject to phi(r) >= tv[r-1] for every r, alpha > 0.  The pair feeds
 * loopspec_pick_depths.  Host only.  tv: host array of n >= 2 positive values that decreases somewhere;
 * EINVAL otherwise. */
int loopspec_fit_envelope(const double* tv, int32_t n, double* alpha, double* beta);

/* Theorem 2 / Eq. 8: real-valued optimum and the admissible integer pair (d1 | d2, d1 | R, d1 < d2 < R)
 * minimising the bound d1 + beta d1^-alpha d2 + 2 beta d2^-alpha R.  Host only; any output may be NULL. */
int loopspec_pick_depths(float alpha, float beta, int32_t R, double* d1_star, double* d2_star, int32_t* d1,
                         int32_t* d2);

/* Maximum number of simultaneously active branches (Sec. 4.3 recurrence); d2 = 0: single proposal. */
int32_t loopspec_max_branches(int32_t R, int32_t d1, int32_t d2);

int loopspec_get_stats(loopspec_ctx*, loopspec_stats*);
/* Commit records of the last decode/verify calls of sequence seq since its prefill (host array). */
int loopspec_get_commits(loopspec_ctx*, int32_t seq, loopspec_commit* out, int32_t max_out, int32_t* n_out);
/* Rows advanced by each step since the last prefill of any sequence (host array of int32). */
int loopspec_get_row_trace(loopspec_ctx*, int32_t* out, int32_t max_out, int32_t* n_out);

/* Copy fp32 logits (before temperature) to host out_V[vocab]: which = 0 the last verified target p_R
 * (or the prefill / vanilla readout), 1 / 2 the root branch's stored first / second proposal readout. */
int loopspec_debug_logits(loopspec_ctx*, int32_t seq, int32_t which, float* out_V);

/* Failure injection on the host side of the bounded device waits (App. B describes no failure handling; this serves the
 * library's own tests).  Every wait inside the tcgen05 kernels (an mbarrier a TMA copy completes, a stage the tensor
 * core releases, a cluster partner's partial sums) is bounded by the clock; when one runs out the kernel raises a flag,
 * carries on with whatever data it has so that every barrier still receives its arrivals, and ends; the call that
 * launched it returns LOOPSPEC_ETIMEOUT, the results of that pass are void, the context stays usable (prefill the
 * sequence again).  This call makes such a wait run out: from now on CTA 0 of the readout GEMM never requests ring unit
 * `unit` (unit >= 0), so the wait for it gives up after about wait_us microseconds.  unit = -1 restores normal operation
 * (and the normal bound of ~0.2 s).  Nothing faults or hangs: the skipped copy is simply never issued. */
int loopspec_debug_drop_tile(loopspec_ctx*, int32_t unit, int32_t wait_us);

/* Number of kernels one decode step (one graph replay of loopspec_decode) launches. */
int loopspec_launches_per_step(loopspec_ctx*, int32_t* out);

/* Which kernels a decode pass of this context runs (fixed at loopspec_init by the row capacity of a pass and the
 * context capacity): *gemm_path = 0 the mma.sync cluster kernels (passes of up to 8 rows, fp32 weights), 1 the
 * tcgen05 / TMA kernel + epilogue kernel (bf16 weights, passes of 9 or more rows, one pair of launches per group of 64
 * token columns);
 * *attention_path = 0 one work item per 64-position chunk (context capacity up to 2560 positions; up to 512 when the
 * context holds several sequences), 1 the streaming kernel over runs of chunks.  Either pointer may be null. */
int loopspec_decode_paths(loopspec_ctx*, int32_t* gemm_path, int32_t* attention_path);

/* Time `iters` back-to-back launches of one kernel of the pass in the decode launch configuration, cycling
 * over the layers' weights (so successive launches read different memory): which = 0 qkv, 1 o-proj,
 * 2 gate/up, 3 down, 4 lm_head, 5 the attention kernel with every row reading a cached context of (max_ctx - 64)
 * positions of its own (row i: sequence i mod max_seqs, recurrence 1 + (i / max_seqs) mod R), 6 the attention of a
 * prefill pass: `rows` (<= max_prefill_rows) consecutive positions of sequence 0 ending at position max_ctx - 65, which
 * share the cached keys and values (bytes_out: those of one context).  rows = token rows
 * carried.  ms_out: mean milliseconds per launch measured with CUDA events on the context's stream; bytes_out: weight
 * (which = 5: key and value) bytes one launch streams.  Sequences need a new prefill afterwards. */
int loopspec_time_kernel(loopspec_ctx*, int32_t which, int32_t rows, int32_t iters, float* ms_out,
                         double* bytes_out);

/* Stand-alone linear map y[M][N] = x[M][K] * W[N][K]^T through the same weight-streaming kernel (token
 * activations split into three bf16 terms, fp32 accumulation; fp32 weights use the CUDA-core path).
 * All pointers device; x, y fp32; scratch: device, 16-byte aligned, loopspec_linear_scratch_bytes(M, N, K)
 * bytes (it receives the bf16 planes of x and, for bf16 weights, a tile-major copy of W; contents on entry are
 * irrelevant).  M <= 64, N % 16 == 0, K % 8 == 0. */
size_t loopspec_linear_scratch_bytes(int32_t M, int32_t N, int32_t K);
int loopspec_op_linear(const void* W, int32_t weight_dtype, const float* x, float* y, int32_t M, int32_t N,
                       int32_t K, void* scratch, size_t scratch_bytes, void* cuda_stream);

/* The same linear map for bf16 weights on the tensor-memory path of sm_100a: weight tiles and activation planes arrive
 * by TMA into a shared-memory ring, one thread issues tcgen05.mma (128 weight rows x up to 64 token columns per
 * instruction, three exact bf16 planes of x per k-step, fp32 accumulator in tensor memory), K is split over CTAs and
 * the partial sums are added in split order.  W is read in place (row-major, 16-byte aligned; no packed copy).
 * All pointers device; x, y fp32; scratch: device, 256-byte aligned, loopspec_linear_tc_scratch_bytes(M, N, K) bytes
 * (0 = unsupported shape).  1 <= M <= 64, N % 8 == 0, K % 64 == 0, else LOOPSPEC_EINVAL.  Stream-ordered; every wait
 * inside the kernel is bounded: after the stream has been synchronised the first int32 of scratch is non-zero if one ran
 * out (y is then undefined).  The prefill passes of a context run their layer GEMMs on the same kernel; the decode passes
 * do not. */
size_t loopspec_linear_tc_scratch_bytes(int32_t M, int32_t N, int32_t K);
int loopspec_op_linear_tc(const void* W, const float* x, float* y, int32_t M, int32_t N, int32_t K, void* scratch,
                          size_t scratch_bytes, void* cuda_stream);
/* Measurement aid for the operator above: the tcgen05 kernel alone, launched back to back with programmatic dependent
 * launch (each launch requests its first weight tiles while the previous one still runs, as a kernel of the decode
 * pass does), cycling over n_w (<= 64) weight matrices Ws[i] (HOST array of device pointers, each [N][K] bf16) so that
 * consecutive launches stream different memory.  x is split once; the k-split partial sums stay in scratch (same size
 * rule as above).  One untimed round over the matrices, then iters timed rounds; us_out (host) = mean microseconds per
 * launch from CUDA events on cuda_stream.  Blocks until done. */
int loopspec_time_linear_tc(const void* const* Ws, int32_t n_w, const float* x, int32_t M, int32_t N, int32_t K,
                            void* scratch, size_t scratch_bytes, int32_t iters, float* us_out, void* cuda_stream);

/* The same linear map for callers that cannot allocate device memory at all.  (The paper has no counterpart;
 * this is a packaging convenience.)  Two kinds of caller are meant: a serving process whose allocator has reserved
 * the whole device up front, so that a later cudaMalloc -- theirs or ours -- fails or fragments the pool; and a
 * latency-critical thread for which cudaMalloc/cudaFree are off limits because they synchronise the device and stall
 * every other stream.  Such callers pass only inputs and the output; the scratch that loopspec_op_linear wants lives
 * in a fixed 16 MiB array inside the library's device image (every GPU that loads the library carries it until the
 * process exits).  The call allocates nothing and frees nothing.
 *   - Sizes: loopspec_linear_scratch_bytes(M, N, K) must not exceed 16 MiB (roughly N*K <= 8M bf16 weights);
 *     larger requests return LOOPSPEC_ECAPACITY and do nothing.  Bad shapes return LOOPSPEC_EINVAL.
 *   - The first call on each device looks up the array's device address (with that device current); make that
 *     first call outside any stream capture.  Later calls only launch kernels on cuda_stream.  With lazy module
 *     loading that first call is also when the library's device image -- the 16 MiB array with it -- becomes
 *     resident on the device: make it BEFORE the process's pool reserves the device's memory (a warm-up call on a
 *     small shape is enough); made afterwards it can return LOOPSPEC_ECUDA for lack of memory.
 *   - The array is the CURRENT device's (cudaGetDevice at the time of the call): cuda_stream, W, x and y must
 *     belong to that device.  Nothing checks this; a stream or pointer of another device gives a CUDA error or
 *     wrong results.  The first-call look-up is safe to race from several host threads.
 *   - All calls on a device share the one array, which keeps whatever the previous call left there.  Nothing in
 *     it has to start at zero: every call overwrites the part it reads.  Two calls that overlap on the GPU (different
 *     streams, or threads racing on one stream's ordering) overwrite each other's scratch and give wrong results:
 *     serialise them. */
int loopspec_op_linear_static(const void* W, int32_t weight_dtype, const float* x, float* y, int32_t M, int32_t N,
                              int32_t K, void* cuda_stream);

const char* loopspec_last_error(loopspec_ctx*);
int loopspec_destroy(loopspec_ctx*);

#ifdef __cplusplus
}
#endif
#endif /* LOOPSPEC_H */

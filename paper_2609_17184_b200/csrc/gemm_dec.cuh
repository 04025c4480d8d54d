// The readout GEMM of a decode pass - final RMSNorm's 1/rms, lm_head, fp32 logits and the per-block arg max that the
// greedy selection reads (Sec. 3.1: p_r = C(H^r) at the proposal depths d1, d2 and at R) - on the Blackwell path:
// TMA ring -> tcgen05.mma with the accumulator in tensor memory -> tcgen05.ld -> split-K sum over distributed shared
// memory -> epilogue.  It is the one GEMM of a pass that streams long enough (201 MB at the Ouro-1.4B shape) for the
// stream to dominate its fixed cost: alone it runs at 0.85 of the measured copy bandwidth, against 0.69 for the
// mma.sync kernel it replaces here.  The layers' four GEMMs stream 8-46 MB each; for them the same kernel was measured
// slower than the mma.sync kernels (fixed cost per launch ~5 us against ~4 us, fewer CTAs because a cluster must own
// whole 128-row blocks), so they stay there.  `EPI_PLAIN` serves tests of the kernel as a plain linear map.
//
// Shape of the problem: y[c][n] = sum_k x[c][k] W[n][k] with at most a few token rows c per pass (the branches of
// Algorithm 1 at their staggered depths) and W streaming from HBM.  The weights are the 128-row A operand of the MMA,
// the token rows are its N columns.  Activations arrive as three bf16 planes (an exact split of the fp32 value); the
// planes sit side by side as accumulator columns (row r, plane pl -> column 3 r + pl), so one MMA per 16-wide k-step
// feeds three separate accumulation chains, folded hi + (mid + lo) when the accumulator is read; the even and the odd
// k-steps go to two accumulators of their own, issued by two threads (an MMA of so few columns costs its issuing thread
// ~150 cycles) and added in fixed order.  A token's arithmetic therefore does not depend on which other tokens share
// the pass, nor on the pass width.
//
// Work split.  A cluster of `cs` CTAs owns row blocks rb = cluster, cluster + n_clusters, ... (128 output rows each);
// its CTAs split K into contiguous ranges of 64-wide k-blocks.  One CTA per SM with (nearly) the whole shared memory as
// its ring: what decides the streaming rate is the number of bytes in flight per SM.
//
// Roles inside a CTA (256 threads): the lanes of warp 4 keep the ring's weight tiles coming and those of warp 6 the
// activation tiles of the same k-blocks - lane s owns ring stage s (so it is never more than one use ahead of the
// stage's barrier, which a parity wait requires), and every tile is ONE TMA request (a 128-row box of the weights, one
// box with all three planes of the pass's rows): requesting a tile costs a thread a few hundred cycles, and a single
// thread issuing five requests per stage was measured to cap the stream at ~3 TB/s.  The first ring-full of weights is
// requested ahead of griddepcontrol.wait.  Warps 5 and 7 (lane 0) issue the MMAs and release stages with
// tcgen05.commit, warps 0-3 read finished accumulators (lane = weight row), push every live column into the receive
// buffer of the rank that finishes it, wait on that rank's mbarrier for all ranks' contributions and run the epilogue.
// Producers and MMA issuers run ahead across row blocks (two accumulator buffers in tensor memory, two receive
// buffers), so the reduction and epilogue of block t overlap the stream of t + 1.  Every wait is bounded by the clock:
// a wait that runs out raises the error flag and carries on, so all barriers still receive their arrivals and the
// kernel ends (the host then reports LOOPSPEC_ETIMEOUT).
#pragma once
#include <cooperative_groups.h>

#include "gemm.cuh"
#include "linear_tc.cuh"

namespace ls {

constexpr int DG_THREADS = 256;
constexpr int DG_CHAINS = 2;  // accumulation chains per accumulator, one MMA-issuing thread each
constexpr int DG_W_BYTES = TC_BM * TC_BK * 2;  // weight tile of a stage: 128 rows x 64 k, 128-byte swizzle
constexpr int DG_MAX_STAGES = 12;
constexpr int DG_MAX_COLS = 64;                // token columns one MMA carries (three planes: 192 accumulator columns)

struct DgParams {
  GemmParams g;     // shapes, row table, epilogue operands; cluster_size / n_clusters / n_rb as planned by the host
  int MP;           // MMA columns per plane: 8 (passes of up to 8 rows) or a multiple of 16 up to 64
  int stages;       // ring depth
  int acc_bufs;     // accumulator buffers in tensor memory (2 unless the tile is too wide)
  int recv_bufs;    // receive buffers (2 when a cluster finishes more than one row block)
  int err_code;     // written to g.err when a bounded wait ran out
  long long wait_cycles;
  int drop_unit;    // test hook: the producer skips this unit of CTA 0 (-1: none), so that the wait for it runs out
};

__host__ __device__ constexpr int dg_x_bytes(int MP) { return 3 * MP * TC_BK * 2; }
__host__ __device__ constexpr int dg_stage_bytes(int MP) { return dg_x_bytes(MP) + DG_W_BYTES; }
__host__ __device__ constexpr int dg_mma_n(int MP) { return (3 * MP + 15) / 16 * 16; }
__host__ __device__ constexpr int dg_recv_floats(int MP, int cs) { return ((MP + cs - 1) / cs) * cs * RB_ROWS; }
__host__ __device__ constexpr int dg_smem_bytes(int MP, int cs, int stages, int recv_bufs) {
  return 1024 + stages * dg_stage_bytes(MP) + recv_bufs * dg_recv_floats(MP, cs) * 4;
}

__device__ __forceinline__ bool dg_wait(unsigned bar, unsigned parity, long long limit) {
  const long long t0 = clock64();
  for (;;) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
    if (clock64() - t0 > limit) return false;
  }
}
// the same with cluster-scope acquire: the arrivals come from other CTAs of the cluster, after their pushes
__device__ __forceinline__ bool dg_wait_cluster(unsigned bar, unsigned parity, long long limit) {
  const long long t0 = clock64();
  for (;;) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
    if (clock64() - t0 > limit) return false;
  }
}
__device__ __forceinline__ unsigned dg_mapa(unsigned addr, unsigned rank) {
  unsigned r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void dg_st_cluster(unsigned addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void dg_arrive_cluster(unsigned addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(addr) : "memory");
}
__device__ __forceinline__ void dg_arrive(unsigned bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void dg_team_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }  // warps 0-3

// ---- the epilogue team (threads 0..127, thread j = row j of the block) finishes this rank's columns -------------
// recv holds, for every rank rk and owned slot, the 128 partial sums that rank pushed: [rk][slot][128].
template <int EPI>
__device__ __forceinline__ void dg_epilogue(const GemmParams& p, const int* ct, int rb, int n_cols, const float* recv, int own_max,
                                            const float* s_rstd, float* s_red, int rank, int cs) {
  static_assert(EPI == EPI_PLAIN || EPI == EPI_LOGITS, "the tcgen05 decode kernel finishes plain outputs and logits");
  const int j = threadIdx.x, lane = j & 31, hw = j >> 5;
  constexpr int NT = DG_MAX_COLS;  // column stride of the table
  int it = 0;
  for (int c = rank; c < n_cols; c += cs, ++it) {
    const float* src = recv + (size_t)(c / cs) * RB_ROWS + j;
    float v = src[0];
    for (int rk = 1; rk < cs; ++rk) v += src[(size_t)rk * own_max * RB_ROWS];  // rank order, the same in every launch
    v *= s_rstd[c];
    const int n = rb * RB_ROWS + j;
    if (n < p.N) {
      if (EPI == EPI_PLAIN) p.out[(size_t)c * p.out_ld + n] = v;
      else p.logits[(size_t)ct[CT_LOGIT * NT + c] * p.N + n] = v;
    }
    if (EPI == EPI_LOGITS) {  // the block's largest logit (ties: lowest index) for the greedy selection
      float bv = n < p.N ? v : -INFINITY;
      int bi = n;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) bv = ov, bi = oi;
      }
      float* av = s_red + (it & 1) * 8;
      if (lane == 0) av[hw] = bv, av[4 + hw] = __int_as_float(bi);
      dg_team_sync();
      if (j == 0) {
        for (int w = 1; w < 4; ++w) {
          const float ov = av[w];
          const int oi = __float_as_int(av[4 + w]);
          if (ov > bv || (ov == bv && oi < bi)) bv = ov, bi = oi;
        }
        p.argpart[(size_t)c * p.n_rb + rb] = make_float2(bv, __int_as_float(bi));
      }
    }
  }
}

template <int EPI>
__global__ void __launch_bounds__(DG_THREADS) dgemm_kernel(const __grid_constant__ CUtensorMap map_w,  // row-major weights [N][K], box 64 k x 128 rows
                                                           const __grid_constant__ CUtensorMap map_x,  // (k, plane, row), box 64 x 3 x MP
                                                           const __grid_constant__ DgParams q) {
  namespace cg = cooperative_groups;
  extern __shared__ unsigned char dg_smem_raw[];
  __shared__ __align__(8) unsigned long long s_full[DG_MAX_STAGES], s_empty[DG_MAX_STAGES], s_accf[2], s_acce[2], s_recvf[2];
  __shared__ unsigned s_tmem;
  __shared__ int s_fail;
  __shared__ float s_rstd[DG_MAX_COLS];
  __shared__ int s_ct[CT_FIELDS * DG_MAX_COLS];
  __shared__ int s_colof[DG_MAX_COLS];   // pass row (= MMA column) -> output column, -1: not finished by this GEMM
  __shared__ float s_red[16];

  const GemmParams& p = q.g;
  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cs = p.cluster_size, rank = cs > 1 ? (int)cluster.block_rank() : 0, cid = blockIdx.x / cs;
  const int MP = q.MP, S = q.stages;
  const int own_max = (MP + cs - 1) / cs;
  const unsigned base = (tc_smem_u32(dg_smem_raw) + 1023u) & ~1023u;
  const int stage_bytes = dg_stage_bytes(MP), x_bytes = dg_x_bytes(MP);
  float* recv0 = reinterpret_cast<float*>(dg_smem_raw + (base - tc_smem_u32(dg_smem_raw)) + S * stage_bytes);
  const int recv_floats = dg_recv_floats(MP, cs);
  const long long limit = q.wait_cycles;

  pdl_launch_dependents();
  tune_mark(p.tl_id, false);
  // the row table of a pass is final before the pass starts: read ahead of the predecessor
  const RowTable* tab = p.tab;
  int n_rows = tab ? tab->n_rows : p.m_fixed;          // rows of the pass = live MMA columns
  int n_cols = tab ? (p.cols_from_readout ? tab->n_readout : n_rows) : p.m_fixed;  // columns this GEMM finishes
  if (n_rows > MP) n_rows = MP;
  if (n_cols > MP) n_cols = MP;
  if (n_cols <= 0) {  // uniform over the grid: nothing reads out in this pass - nothing is requested, nothing allocated
    pdl_wait();     // (a kernel that ended before its predecessor would release its own dependents too early)
    return;
  }

  int kb_lo, kb_hi;
  gemm_krange((p.K + TC_BK - 1) / TC_BK, cs, rank, kb_lo, kb_hi);
  const int n_kb = kb_hi - kb_lo;
  const int n_tasks = (p.n_rb - cid + p.n_clusters - 1) / p.n_clusters;
  const int total_units = n_tasks * n_kb;
  const int pre = min(S, total_units);

  auto load_w = [&](int u, int s) {  // the weight tile of unit u (row block of its task, k-block of this rank) into stage s
    const int task = u / n_kb, kb = kb_lo + u - task * n_kb, rb = cid + task * p.n_clusters;
    const unsigned a = base + s * stage_bytes + x_bytes, bar = tc_smem_u32(&s_full[s]);
    tc_tma_load_2d(a, &map_w, bar, kb * TC_BK, rb * RB_ROWS);
  };
  auto load_x = [&](int u, int s) {  // all three planes of the pass's rows for the same k-block: tile rows = (row, plane)
    const int kb = kb_lo + u % n_kb;
    tc_tma_load_3d(base + s * stage_bytes, &map_x, tc_smem_u32(&s_full[s]), kb * TC_BK, 0, 0);
  };
  const bool dropper = q.drop_unit >= 0 && blockIdx.x == 0;

  if (tid == 128) {  // producer: its own barriers first, then the first ring-full of weights - constants, so nothing
                     // here waits for the predecessor
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<unsigned long long>(&map_w)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<unsigned long long>(&map_x)) : "memory");
    for (int s = 0; s < S; ++s) tc_mbar_init(tc_smem_u32(&s_full[s]), 1), tc_mbar_init(tc_smem_u32(&s_empty[s]), DG_CHAINS);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    for (int u = 0; u < pre; ++u) {
      if (dropper && u == q.drop_unit) continue;
      tc_mbar_expect_tx(tc_smem_u32(&s_full[u]), (unsigned)stage_bytes);
      load_w(u, u);
    }
  }
  if (tid == 0) {
    for (int b = 0; b < 2; ++b) {
      tc_mbar_init(tc_smem_u32(&s_accf[b]), DG_CHAINS);
      tc_mbar_init(tc_smem_u32(&s_acce[b]), 4);
      tc_mbar_init(tc_smem_u32(&s_recvf[b]), 4 * cs);
    }
    s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  const unsigned mma_n = (unsigned)dg_mma_n(MP);
  const unsigned acc_stride = DG_CHAINS * mma_n;  // chain ch of a buffer at columns ch * mma_n
  const unsigned acc_cols = acc_stride * q.acc_bufs;
  const unsigned tmem_cols = acc_cols <= 32 ? 32u : acc_cols <= 64 ? 64u : acc_cols <= 128 ? 128u : acc_cols <= 256 ? 256u : 512u;
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem_u32(&s_tmem)), "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp < 4) {
    if (tid < DG_MAX_COLS) s_colof[tid] = (!p.cols_from_readout && tid < n_cols) ? tid : -1;
    gemm_load_cols(p, n_cols, DG_MAX_COLS, s_ct);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  if (p.cols_from_readout && tid < n_cols) s_colof[s_ct[CT_XROW * DG_MAX_COLS + tid]] = tid;
  const unsigned tmem = s_tmem;
  if (cs > 1) cluster.sync();  // every rank's barriers exist before anybody arrives on them remotely
  else __syncthreads();

  if (warp == 4) {
    if (lane < S) {
      // ---- weight producers: lane s owns stage s and requests the tiles of units s + S, s + 2 S, ... in order (the first
      // ring-full went out in the prologue); a stage is free once the MMAs of its previous unit have read it ----
      bool ok = true;
      unsigned par = 0;
      for (int u = lane + S; u < total_units; u += S, par ^= 1u) {
        if (!dg_wait(tc_smem_u32(&s_empty[lane]), par, limit)) ok = false;
        if (dropper && u == q.drop_unit) continue;
        tc_mbar_expect_tx(tc_smem_u32(&s_full[lane]), (unsigned)stage_bytes);
        load_w(u, lane);
      }
      if (!ok) s_fail = 1, *p.err = q.err_code;
    }
  } else if (warp == 6) {
    if (lane < S) {
      // ---- activation producers (lane s owns stage s): the planes are the predecessor's output ----
      pdl_wait();
      bool ok = true;
      unsigned par = 1;
      for (int u = lane; u < total_units; u += S, par ^= 1u) {
        if (u >= S && !dg_wait(tc_smem_u32(&s_empty[lane]), par, limit)) ok = false;
        if (dropper && u == q.drop_unit) continue;
        load_x(u, lane);
      }
      if (!ok) s_fail = 1, *p.err = q.err_code;
    }
  } else if (warp == 5 || warp == 7) {
    if (lane == 0) {
      // ---- MMA issuers: issuing an MMA of so few columns costs its thread ~150 cycles, so two threads share a k-block:
      // thread ch issues the 16-wide k-steps ch, ch + 2 into its own accumulation chain (the chains are added in fixed
      // order when the accumulator is read); a stage is free when both have committed ----
      const int ch = warp == 5 ? 0 : 1;
      const unsigned idesc = tc_idesc(TC_BM, (int)mma_n);
      const unsigned long long desc0 = tc_smem_desc(0);  // the fixed bits of a shared-memory descriptor
      bool ok = true;
      int s = 0;
      unsigned par = 0;
      for (int task = 0; task < n_tasks; ++task) {
        const int buf = q.acc_bufs > 1 ? (task & 1) : 0;
        const int uses = q.acc_bufs > 1 ? (task >> 1) : task;  // earlier uses of this accumulator buffer
        if (uses > 0 && !dg_wait(tc_smem_u32(&s_acce[buf]), (uses - 1) & 1, limit)) ok = false;  // its readers are done
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const unsigned d_tmem = tmem + (unsigned)buf * acc_stride + (unsigned)ch * mma_n;
        for (int kbl = 0; kbl < n_kb; ++kbl) {
          if (!dg_wait(tc_smem_u32(&s_full[s]), par, limit)) ok = false;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const unsigned b = base + s * stage_bytes;
          const unsigned long long bdesc = desc0 | (unsigned long long)((b >> 4) & 0x3FFF);
          const unsigned long long adesc = desc0 | (unsigned long long)(((b + x_bytes) >> 4) & 0x3FFF);
#pragma unroll
          for (int ks = ch; ks < TC_BK / 16; ks += DG_CHAINS) tc_mma(d_tmem, adesc + 2 * ks, bdesc + 2 * ks, idesc, (kbl | (ks / DG_CHAINS)) != 0);
          tc_commit(tc_smem_u32(&s_empty[s]));
          if (++s == S) s = 0, par ^= 1u;
        }
        tc_commit(tc_smem_u32(&s_accf[buf]));
      }
      if (!ok) s_fail = 1, *p.err = q.err_code;
    }
  } else {
    // ---- accumulator readers / epilogue team: thread j = row j of the block ----
    pdl_wait();
    tune_mark(p.tl_id + 256, false);
    // 1/rms of every column this GEMM finishes (one partial per lane, butterfly sum: the same order in every launch)
    for (int c = warp; c < n_cols; c += 4) {
      const int xr = p.cols_from_readout ? s_ct[CT_XROW * DG_MAX_COLS + c] : c;
      float ss = 0.f;
      if (p.sumsq)
        for (int i = lane; i < p.n_sq; i += 32) ss += p.sumsq[xr * p.sq_stride + i];
      ss = warp_sum(ss);
      if (lane == 0) s_rstd[c] = p.sumsq ? 1.0f / sqrtf(ss / (float)p.H + p.eps) : 1.0f;
    }
    dg_team_sync();
    bool ok = true;
    for (int task = 0; task < n_tasks; ++task) {
      const int rb = cid + task * p.n_clusters;
      const int buf = q.acc_bufs > 1 ? (task & 1) : 0, uses = q.acc_bufs > 1 ? (task >> 1) : task;
      const int rbuf = q.recv_bufs > 1 ? (task & 1) : 0, ruses = q.recv_bufs > 1 ? (task >> 1) : task;
      float* recv = recv0 + (size_t)rbuf * recv_floats;
      if (!dg_wait(tc_smem_u32(&s_accf[buf]), uses & 1, limit)) ok = false;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const unsigned recv_s = tc_smem_u32(recv);
      for (int c0 = 0; c0 < n_rows; c0 += 8) {
        float v8[8];  // rows c0 .. c0 + 7: accumulator column of (row r, plane pl) = 3 r + pl, per chain
#pragma unroll
        for (int ch = 0; ch < DG_CHAINS; ++ch) {
          unsigned w[24];
#pragma unroll
          for (int g = 0; g < 3; ++g) {
            const unsigned taddr = tmem + ((unsigned)(warp * 32) << 16) + (unsigned)(buf * acc_stride + ch * mma_n + 3 * c0 + 8 * g);
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(w[8 * g]), "=r"(w[8 * g + 1]), "=r"(w[8 * g + 2]), "=r"(w[8 * g + 3]), "=r"(w[8 * g + 4]), "=r"(w[8 * g + 5]),
                           "=r"(w[8 * g + 6]), "=r"(w[8 * g + 7])
                         : "r"(taddr)
                         : "memory");
          }
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
          for (int jj = 0; jj < 8; ++jj) {
            const float x = __uint_as_float(w[3 * jj]) + (__uint_as_float(w[3 * jj + 1]) + __uint_as_float(w[3 * jj + 2]));
            v8[jj] = ch == 0 ? x : v8[jj] + x;
          }
        }
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
          const int c = c0 + jj < MP ? s_colof[c0 + jj] : -1;
          if (c >= 0) {
            const float v = v8[jj];
            const int owner = c % cs, slot = c / cs;
            const unsigned off = (unsigned)(((rank * own_max + slot) * RB_ROWS + tid) * 4);
            if (cs > 1) dg_st_cluster(dg_mapa(recv_s + off, owner), v);
            else recv[(rank * own_max + slot) * RB_ROWS + tid] = v;
          }
        }
      }
      // this warp has read its quarter of the accumulator: the buffer may be overwritten once all four have
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) dg_arrive(tc_smem_u32(&s_acce[buf]));
      if (cs > 1) {
        asm volatile("fence.acq_rel.cluster;" ::: "memory");
        __syncwarp();
        if (lane < cs) dg_arrive_cluster(dg_mapa(tc_smem_u32(&s_recvf[rbuf]), lane));  // one arrival per warp and rank
        if (!dg_wait_cluster(tc_smem_u32(&s_recvf[rbuf]), ruses & 1, limit)) ok = false;
      } else {
        dg_team_sync();
      }
      dg_epilogue<EPI>(p, s_ct, rb, n_cols, recv, own_max, s_rstd, s_red, rank, cs);
      if (cs == 1 && q.recv_bufs == 1) dg_team_sync();  // the one receive buffer is free again
    }
    if (!ok && lane == 0) s_fail = 1, *p.err = q.err_code;
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 5) {
    if (s_fail) {  // a wait gave up: copies may still be in flight; give them a bounded time before the memory goes
      const long long t0 = clock64();
      while (clock64() - t0 < 2000000LL) {
      }
    }
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
  }
  tune_mark(p.tl_id, true);
}

}  // namespace ls

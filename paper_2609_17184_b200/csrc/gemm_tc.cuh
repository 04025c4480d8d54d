// A layer GEMM of a prefill pass in one kernel on the Blackwell path: TMA ring + tcgen05.mma with the accumulator in
// tensor memory (as linear_tc_kernel), then the cluster split-K reduction and the fused epilogues of the mma.sync
// kernels (gemm_reduce_epilogue), fed from tcgen05.ld instead of MMA fragments.
//
// A cluster owns one block of 128 output rows (for gate/up: 64 gate rows and the 64 matching up rows, two weight boxes);
// its CTAs split K into equal ranges of 64-wide k-blocks.  After its last MMA a CTA reads its accumulator (lane = row,
// column = token) and pushes every column into the receive buffer of the rank that owns it (distributed shared memory);
// one cluster barrier; the owner sums the ranks' contributions in rank order and finishes the column.
#pragma once
#include <cooperative_groups.h>

#include "gemm.cuh"
#include "linear_tc.cuh"

namespace ls {

constexpr int GTC_COLS = 64;  // token columns of a prefill pass at most

struct GemmTcParams {
  GemmParams g;   // cluster_size = CTAs per row block; n_rb row blocks; the epilogue's operands
  int MP;         // columns of the MMA (multiple of 16, <= GTC_COLS)
  int stages;
  int err_code;
};

__host__ __device__ constexpr int gtc_stage_bytes(int MP) { return TC_BM * TC_BK * 2 + 3 * MP * TC_BK * 2; }
__host__ __device__ constexpr int gtc_recv_floats(int MP) { return (MP + 7) * RB_ROWS; }
__host__ __device__ constexpr int gtc_tail_bytes(int MP) {
  return gtc_recv_floats(MP) * 4 + 2 * RB_ROWS * 4 + GTC_COLS * 4 + CT_FIELDS * GTC_COLS * 4;
}

template <int EPI>
__global__ void __launch_bounds__(GEMM_THREADS) gemm_tc_kernel(const __grid_constant__ CUtensorMap map_w,  // box 64 k x 64 rows
                                                               const __grid_constant__ CUtensorMap map_x,  // (k, plane, column)
                                                               const __grid_constant__ GemmTcParams q) {
  namespace cg = cooperative_groups;
  extern __shared__ unsigned char gtc_smem_raw[];
  __shared__ __align__(8) unsigned long long s_full[TC_MAX_STAGES], s_empty[TC_MAX_STAGES], s_done;
  __shared__ unsigned s_tmem;

  const GemmParams& p = q.g;
  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cs = p.cluster_size, rank = (int)cluster.block_rank(), rb = blockIdx.x / cs;
  const int own_max = (q.MP + cs - 1) / cs;
  const unsigned base = (tc_smem_u32(gtc_smem_raw) + 1023u) & ~1023u;
  const int stage_bytes = gtc_stage_bytes(q.MP);
  unsigned char* tail = gtc_smem_raw + (base - tc_smem_u32(gtc_smem_raw)) + q.stages * stage_bytes;
  float* recv = reinterpret_cast<float*>(tail);                // [cs][own_max][128]
  float* colbuf = recv + gtc_recv_floats(q.MP);                    // [2][128]
  float* s_rstd = colbuf + 2 * RB_ROWS;
  int* s_ct = reinterpret_cast<int*>(s_rstd + GTC_COLS);       // [CT_FIELDS][GTC_COLS]

  const RowTable* tab = p.tab;  // final before the pass starts
  int n_cols = tab->n_rows;
  if (n_cols > q.MP) n_cols = q.MP;
  pdl_launch_dependents();
  if (n_cols <= 0) {  // uniform over the grid
    pdl_wait();
    return;
  }
  int kb_lo, kb_hi;
  gemm_krange(p.K / TC_BK, cs, rank, kb_lo, kb_hi);
  const int n_kb = kb_hi - kb_lo;
  // weight rows of the two 64-row halves of this block
  int row_a, row_b;
  if (EPI == EPI_SWIGLU) row_a = rb * 64, row_b = p.F + rb * 64;
  else row_a = rb * RB_ROWS, row_b = row_a + 64;
  // the three planes of the activations are three groups of MP accumulator columns: one MMA of N = 3 MP per k-step,
  // three separate chains as in the mma.sync kernels, folded hi + (mid + lo) when the accumulator is read
  const unsigned tmem_cols = 3 * q.MP <= 64 ? 64u : (3 * q.MP <= 128 ? 128u : 256u);

  if (tid == 32) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<unsigned long long>(&map_w)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<unsigned long long>(&map_x)) : "memory");
  }
  if (tid == 0) {
    for (int s = 0; s < q.stages; ++s) tc_mbar_init(tc_smem_u32(&s_full[s]), 1), tc_mbar_init(tc_smem_u32(&s_empty[s]), 1);
    tc_mbar_init(tc_smem_u32(&s_done), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  gemm_load_cols(p, n_cols, GTC_COLS, s_ct);
  __syncthreads();
  auto load_w = [&](unsigned a, unsigned bar, int k) {
    tc_tma_load_2d(a, &map_w, bar, k, row_a);
    tc_tma_load_2d(a + 64 * TC_BK * 2, &map_w, bar, k, row_b);
  };
  const int pre = min(q.stages, n_kb);
  if (tid == 32) {  // weights are constants: requested ahead of the predecessor's completion
    for (int kb = 0; kb < pre; ++kb) {
      const unsigned bar = tc_smem_u32(&s_full[kb]);
      tc_mbar_expect_tx(bar, (unsigned)stage_bytes);
      load_w(base + kb * stage_bytes, bar, (kb_lo + kb) * TC_BK);
    }
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem_u32(&s_tmem)), "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const unsigned tmem = s_tmem;

  pdl_wait();
  bool failed = false;
  if (tid == 32) {
    // ---- producer ----
    for (int kb = 0; kb < pre; ++kb) {
      const unsigned b = base + kb * stage_bytes + TC_BM * TC_BK * 2, bar = tc_smem_u32(&s_full[kb]);
#pragma unroll
      for (int pl = 0; pl < 3; ++pl) tc_tma_load_3d(b + pl * q.MP * TC_BK * 2, &map_x, bar, (kb_lo + kb) * TC_BK, pl, 0);
    }
    bool ok = true;
    for (int kb = pre; kb < n_kb && ok; ++kb) {
      const int s = kb % q.stages;
      ok = tc_mbar_wait(tc_smem_u32(&s_empty[s]), ((kb / q.stages) - 1) & 1);
      if (!ok) break;
      const unsigned bar = tc_smem_u32(&s_full[s]);
      const unsigned a = base + s * stage_bytes, b = a + TC_BM * TC_BK * 2;
      tc_mbar_expect_tx(bar, (unsigned)stage_bytes);
      load_w(a, bar, (kb_lo + kb) * TC_BK);
#pragma unroll
      for (int pl = 0; pl < 3; ++pl) tc_tma_load_3d(b + pl * q.MP * TC_BK * 2, &map_x, bar, (kb_lo + kb) * TC_BK, pl, 0);
    }
    if (!ok) *p.err = q.err_code;
  } else if (tid == 0) {
    // ---- MMA issuer ----
    const unsigned idesc = tc_idesc(TC_BM, 3 * q.MP);
    bool ok = true;
    for (int kb = 0; kb < n_kb && ok; ++kb) {
      const int s = kb % q.stages;
      ok = tc_mbar_wait(tc_smem_u32(&s_full[s]), (kb / q.stages) & 1);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const unsigned a = base + s * stage_bytes, b = a + TC_BM * TC_BK * 2;
      const unsigned long long adesc = tc_smem_desc(a);
      const unsigned long long bdesc = tc_smem_desc(b);  // rows pl * MP + column: the planes stacked
#pragma unroll
      for (int ks = 0; ks < TC_BK / 16; ++ks) tc_mma(tmem, adesc + 2 * ks, bdesc + 2 * ks, idesc, (kb | ks) != 0);
      tc_commit(tc_smem_u32(&s_empty[s]));
    }
    if (ok) tc_commit(tc_smem_u32(&s_done));
    else *p.err = q.err_code;
  }
  // operands of this CTA's first output column, requested ahead of the accumulator (as the mma.sync kernels do)
  float pre_h = 0.f, pre_g = 1.f;
  float2 pre_rope = make_float2(1.f, 0.f);
  {
    const int c = rank + cs * (tid >> 7), jr = tid & 127;
    if (EPI == EPI_RESID && c < n_cols) {
      pre_h = p.hid[(size_t)s_ct[CT_HID * GTC_COLS + c] * p.H + rb * RB_ROWS + jr];
      if (p.out_planes) pre_g = p.gain_next[rb * RB_ROWS + jr];
    }
    if (EPI == EPI_QKV && c < n_cols && jr < 64) {
      const int hd2 = p.head_dim >> 1;
      pre_rope = p.rope[(size_t)s_ct[CT_POS * GTC_COLS + c] * hd2 + jr % hd2];
    }
  }
  // 1/rms of the columns this rank finishes (gemm_rstd's arithmetic), by the warps that do not read the accumulator
  if (warp >= 4) {
    for (int c = rank + cs * (warp - 4); c < n_cols; c += cs * 4) {
      float ss = 0.f;
      if (p.sumsq)
        for (int i = lane; i < p.n_sq; i += 32) ss += p.sumsq[c * p.sq_stride + i];
      ss = warp_sum(ss);
      if (lane == 0) s_rstd[c] = p.sumsq ? 1.0f / sqrtf(ss / (float)p.H + p.eps) : 1.0f;
    }
  }
  // ---- accumulator -> the owners' receive buffers ----
  if (warp < 4) {
    bool have = n_kb > 0;
    if (have) have = tc_mbar_wait(tc_smem_u32(&s_done), 0);
    failed = n_kb > 0 && !have;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const int row = warp * 32 + lane;
    for (int c0 = 0; c0 < q.MP; c0 += 16) {
      unsigned v[16];
      if (have) {
        unsigned w[3][16];
#pragma unroll
        for (int pl = 0; pl < 3; ++pl) {
          const unsigned taddr = tmem + ((unsigned)(warp * 32) << 16) + (unsigned)(pl * q.MP + c0);
          asm volatile(
              "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
              : "=r"(w[pl][0]), "=r"(w[pl][1]), "=r"(w[pl][2]), "=r"(w[pl][3]), "=r"(w[pl][4]), "=r"(w[pl][5]), "=r"(w[pl][6]),
                "=r"(w[pl][7]), "=r"(w[pl][8]), "=r"(w[pl][9]), "=r"(w[pl][10]), "=r"(w[pl][11]), "=r"(w[pl][12]),
                "=r"(w[pl][13]), "=r"(w[pl][14]), "=r"(w[pl][15])
              : "r"(taddr)
              : "memory");
        }
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int j = 0; j < 16; ++j)
          v[j] = __float_as_uint(__uint_as_float(w[0][j]) + (__uint_as_float(w[1][j]) + __uint_as_float(w[2][j])));
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = 0u;  // a rank without k-blocks contributes zeros
      }
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const int c = c0 + j;
        if (c < n_cols) {
          const int owner = c % cs, slot = c / cs;
          float* dst = (cs > 1 ? cluster.map_shared_rank(recv, owner) : recv) + ((size_t)rank * own_max + slot) * RB_ROWS + row;
          *dst = __uint_as_float(v[j]);
        }
      }
    }
    if (failed && lane == 0) *p.err = q.err_code;
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  cluster.sync();
  gemm_reduce_epilogue<EPI>(p, s_ct, GTC_COLS, rb, n_cols, recv, own_max, colbuf, s_rstd, rank, pre_h, pre_g, pre_rope,
                            EPI == EPI_RESID || EPI == EPI_QKV);
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
}

}  // namespace ls

// Weight-streaming linear map on the fifth-generation tensor cores: y[m][n] = sum_k x[m][k] W[n][k].
//
// The same contraction as the skinny GEMMs of the decode pass (Sec. 4.2 step 1: the token-at-depth rows are the
// narrow side, the shared weights the wide side that streams from HBM), built from the Blackwell pieces: tiles of
// the row-major weights and of the activation planes arrive by TMA (cp.async.bulk.tensor, 128-byte swizzle) in a
// ring of shared-memory stages guarded by mbarriers; one thread issues tcgen05.mma (128 weight rows x up to 64 token
// columns, K = 16 per instruction) with the accumulator in tensor memory; four warps read it back with tcgen05.ld.
// Activations are fp32 split exactly into three bf16 planes; the planes are stacked as 3 MP columns of one MMA per
// k-step (three accumulator chains, as in the mma.sync kernels) and folded hi + (mid + lo) when the accumulator is read.
// K may be split over blockIdx.y; the partial sums are added in split order by a second kernel (no atomics).  Passes of
// more than 64 token columns put one group of 64 columns in each blockIdx.z plane.
//
// Used by the stand-alone operator loopspec_op_linear_tc, by the prefill passes and by the decode passes that carry 9 or
// more rows (tc_epilogue_kernel then applies the fused epilogue of the GEMM); decode passes of up to 8 rows run
// gemm_bf16_kernel, whose launch is cheaper than this pair's.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace ls {

constexpr int TC_THREADS = 128;
constexpr int TC_BM = 128;         // weight rows per CTA = rows of one MMA
constexpr int TC_BK = 64;          // k per stage: 64 bf16 = one 128-byte swizzled row
constexpr int TC_MAX_STAGES = 8;
constexpr long long TC_WAIT_CYCLES = 400000000LL;  // ~0.2 s: a wait that runs this long gives up and raises the flag

struct LinearTcParams {
  float* out;          // [n_split][M][N] partial sums (n_split == 1: y itself)
  int M, MP, N, K;     // MP = M rounded up to 16: columns of the MMA
  int kb_per_split;    // 64-wide k-blocks per blockIdx.y
  int stages;
  int* err;            // flag the host reads: set to err_code when a bounded wait ran out
  int err_code;
  int x3d;             // 0: x planes stacked [3][MP][K], one box; 1: the decode pass's layout [column][3][x_ld], a
                       // three-dimensional map (k, plane, column) and one box per plane
  int row0;            // x3d: first column of the map this launch carries; blockIdx.z adds group_cols to it and
  int group_cols;      //      group_stride floats to `out` (passes wider than one MMA's columns: one grid plane per
  long long group_stride;  //  group of columns)
  const int* n_live;   // x3d: number of live columns of the pass (may be null); a group beyond it has nothing to do
};

__device__ __forceinline__ unsigned tc_smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void tc_mbar_init(unsigned bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void tc_mbar_expect_tx(unsigned bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// bounded wait on a phase parity: false when it gave up
__device__ __forceinline__ bool tc_mbar_wait(unsigned bar, unsigned parity) {
  const long long t0 = clock64();
  for (;;) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
    if (clock64() - t0 > TC_WAIT_CYCLES) return false;
  }
}
__device__ __forceinline__ void tc_tma_load_2d(unsigned dst, const CUtensorMap* map, unsigned bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(reinterpret_cast<unsigned long long>(map)), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tc_tma_load_3d(unsigned dst, const CUtensorMap* map, unsigned bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
      "l"(reinterpret_cast<unsigned long long>(map)), "r"(bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}
// shared-memory matrix descriptor: K-major tile of 128-byte rows, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ unsigned long long tc_smem_desc(unsigned addr) {
  unsigned long long d = 0;
  d |= (unsigned long long)((addr >> 4) & 0x3FFF);
  d |= (unsigned long long)(1024 >> 4) << 32;  // stride between 8-row groups
  d |= 1ull << 46;                             // descriptor version of this architecture
  d |= 2ull << 61;                             // 128-byte swizzle
  return d;
}
// instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N
__host__ __device__ constexpr unsigned tc_idesc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((unsigned)(N >> 3) << 17) | ((unsigned)(M >> 4) << 24);
}
__device__ __forceinline__ void tc_mma(unsigned d_tmem, unsigned long long adesc, unsigned long long bdesc, unsigned idesc,
                                       unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_commit(unsigned bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__host__ __device__ constexpr int tc_stage_bytes(int MP) { return TC_BM * TC_BK * 2 + 3 * MP * TC_BK * 2; }

__global__ void __launch_bounds__(TC_THREADS) linear_tc_kernel(const __grid_constant__ CUtensorMap map_w,
                                                               const __grid_constant__ CUtensorMap map_x,
                                                               const __grid_constant__ LinearTcParams p) {
  extern __shared__ unsigned char tc_smem_raw[];
  __shared__ __align__(8) unsigned long long s_full[TC_MAX_STAGES], s_empty[TC_MAX_STAGES], s_done;
  __shared__ unsigned s_tmem;
  __shared__ int s_fail;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const unsigned base = (tc_smem_u32(tc_smem_raw) + 1023u) & ~1023u;  // swizzled tiles sit on 1024-byte boundaries
  const int stage_bytes = tc_stage_bytes(p.MP);
  const int n0 = blockIdx.x * TC_BM;
  const int kb0 = blockIdx.y * p.kb_per_split;
  const int n_kb = min(p.kb_per_split, p.K / TC_BK - kb0);
  // the three planes of the activations are three groups of MP accumulator columns: one MMA of N = 3 MP per k-step
  // (three separate chains, as in the mma.sync kernels), folded hi + (mid + lo) when the accumulator is read
  const unsigned tmem_cols = 3 * p.MP <= 64 ? 64u : (3 * p.MP <= 128 ? 128u : 256u);

  if (tid == 32) {  // the producer fetches the two tensor maps while the barriers are set up
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<unsigned long long>(&map_w)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<unsigned long long>(&map_x)) : "memory");
  }
  if (tid == 0) {
    for (int s = 0; s < p.stages; ++s) tc_mbar_init(tc_smem_u32(&s_full[s]), 1), tc_mbar_init(tc_smem_u32(&s_empty[s]), 1);
    tc_mbar_init(tc_smem_u32(&s_done), 1);
    s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  pdl_launch_dependents();
  const int row0 = p.row0 + (int)blockIdx.z * p.group_cols;
  if (p.n_live && *p.n_live <= row0) {  // (final before the pass starts; uniform over the CTA) this group of columns is empty
    pdl_wait();  // a kernel that ended before its predecessor would release its own dependents too early
    return;
  }
  // The weights are constants, so the first ring-full of weight tiles is requested ahead of the predecessor's
  // completion - and while warp 0 still allocates the tensor memory; the activation tiles (which the predecessor may
  // still be writing) follow after the dependency wait, on the same barriers.
  const int pre = min(p.stages, n_kb);
  if (tid == 32) {
    for (int kb = 0; kb < pre; ++kb) {
      const unsigned bar = tc_smem_u32(&s_full[kb]);
      tc_mbar_expect_tx(bar, (unsigned)stage_bytes);
      tc_tma_load_2d(base + kb * stage_bytes, &map_w, bar, (kb0 + kb) * TC_BK, n0);
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
  auto load_x = [&](unsigned b, unsigned bar, int k) {  // the three planes of the activations, plane pl at b + pl * MP * 128
    if (p.x3d) {
#pragma unroll
      for (int pl = 0; pl < 3; ++pl) tc_tma_load_3d(b + pl * p.MP * TC_BK * 2, &map_x, bar, k, pl, row0);
    } else {
      tc_tma_load_2d(b, &map_x, bar, k, 0);
    }
  };
  if (tid == 32 && n_kb > 0) {
    // ---- producer: one thread keeps the ring of stages filled by TMA ----
    for (int kb = 0; kb < pre; ++kb)
      load_x(base + kb * stage_bytes + TC_BM * TC_BK * 2, tc_smem_u32(&s_full[kb]), (kb0 + kb) * TC_BK);
    bool ok = true;
    for (int kb = pre; kb < n_kb && ok; ++kb) {
      const int s = kb % p.stages;
      ok = tc_mbar_wait(tc_smem_u32(&s_empty[s]), ((kb / p.stages) - 1) & 1);  // the stage's MMAs are done
      if (!ok) break;
      const unsigned bar = tc_smem_u32(&s_full[s]);
      const unsigned a = base + s * stage_bytes, b = a + TC_BM * TC_BK * 2;
      tc_mbar_expect_tx(bar, (unsigned)stage_bytes);
      tc_tma_load_2d(a, &map_w, bar, (kb0 + kb) * TC_BK, n0);
      load_x(b, bar, (kb0 + kb) * TC_BK);
    }
    if (!ok) s_fail = 1, *p.err = p.err_code;
  }
  if (tid == 0 && n_kb > 0) {
    // ---- MMA issuer: one thread, the accumulator lives in tensor memory ----
    const unsigned idesc = tc_idesc(TC_BM, 3 * p.MP);
    bool ok = true;
    for (int kb = 0; kb < n_kb && ok; ++kb) {
      const int s = kb % p.stages;
      ok = tc_mbar_wait(tc_smem_u32(&s_full[s]), (kb / p.stages) & 1);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const unsigned a = base + s * stage_bytes, b = a + TC_BM * TC_BK * 2;
      const unsigned long long adesc = tc_smem_desc(a);
      const unsigned long long bdesc = tc_smem_desc(b);  // rows pl * MP + column: the hi, mid, lo planes stacked
#pragma unroll
      for (int ks = 0; ks < TC_BK / 16; ++ks) tc_mma(tmem, adesc + 2 * ks, bdesc + 2 * ks, idesc, (kb | ks) != 0);
      tc_commit(tc_smem_u32(&s_empty[s]));  // arrives when the MMAs issued so far have read their operands
    }
    if (ok) tc_commit(tc_smem_u32(&s_done));
    else s_fail = 1, *p.err = p.err_code;
  }
  // everyone: the accumulator is complete when the last commit arrives
  bool have = n_kb > 0;
  if (have) have = tc_mbar_wait(tc_smem_u32(&s_done), 0);
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const int n = n0 + warp * 32 + lane;  // this thread's weight row = its TMEM lane
  float* out = p.out + (size_t)blockIdx.z * p.group_stride + (size_t)blockIdx.y * p.M * p.N;
  if (n_kb <= 0) {
    for (int m = 0; m < p.M; ++m)
      if (n < p.N) out[(size_t)m * p.N + n] = 0.f;
  } else if (have) {
    for (int c0 = 0; c0 < p.MP; c0 += 16) {
      unsigned w[3][16];
#pragma unroll
      for (int pl = 0; pl < 3; ++pl) {
        const unsigned taddr = tmem + ((unsigned)(warp * 32) << 16) + (unsigned)(pl * p.MP + c0);
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
            : "=r"(w[pl][0]), "=r"(w[pl][1]), "=r"(w[pl][2]), "=r"(w[pl][3]), "=r"(w[pl][4]), "=r"(w[pl][5]), "=r"(w[pl][6]),
              "=r"(w[pl][7]), "=r"(w[pl][8]), "=r"(w[pl][9]), "=r"(w[pl][10]), "=r"(w[pl][11]), "=r"(w[pl][12]),
              "=r"(w[pl][13]), "=r"(w[pl][14]), "=r"(w[pl][15])
            : "r"(taddr)
            : "memory");
      }
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      unsigned v[16];
#pragma unroll
      for (int j = 0; j < 16; ++j)
        v[j] = __float_as_uint(__uint_as_float(w[0][j]) + (__uint_as_float(w[1][j]) + __uint_as_float(w[2][j])));
#pragma unroll
      for (int j = 0; j < 16; ++j)
        if (c0 + j < p.M && n < p.N) out[(size_t)(c0 + j) * p.N + n] = __uint_as_float(v[j]);
    }
  } else if (tid == 0) {
    *p.err = p.err_code;
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    // a wait that gave up may have left copies in flight: give them a bounded time to land before the memory is freed
    if (s_fail) {
      const long long t0 = clock64();
      while (clock64() - t0 < 2000000LL) {
      }
    }
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
  }
}

// x fp32 [M][K] -> planes bf16 [3][MP][K] (rows M..MP-1 zero)
__global__ void tc_split_kernel(const float* __restrict__ x, __nv_bfloat16* __restrict__ planes, int M, int MP, int K) {
  const int m = blockIdx.x;
  for (int k = threadIdx.x; k < K; k += blockDim.x) {
    unsigned short h = 0, mi = 0, l = 0;
    if (m < M) split3(x[(size_t)m * K + k], h, mi, l);
    planes[((size_t)0 * MP + m) * K + k] = __ushort_as_bfloat16(h);
    planes[((size_t)1 * MP + m) * K + k] = __ushort_as_bfloat16(mi);
    planes[((size_t)2 * MP + m) * K + k] = __ushort_as_bfloat16(l);
  }
}

// y = sum over the k-splits, in split order
__global__ void tc_sum_splits_kernel(const float* __restrict__ part, float* __restrict__ y, size_t MN, int n_split) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < MN; i += (size_t)gridDim.x * blockDim.x) {
    float v = part[i];
    for (int s = 1; s < n_split; ++s) v += part[(size_t)s * MN + i];
    y[i] = v;
  }
}

}  // namespace ls

// Stand-alone microbenchmark (not part of the library): cycles per tcgen05.mma for several tile widths, operand
// layouts and CTA groupings, with the operands resident in shared memory and no loads in flight.  It bounds what
// the GEMM kernels' tensor pipe can reach for a given tile shape.  Build and run on a B200:
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -I include -I paper_1910_05124_b200/csrc \
//        -o mma_issue_bench paper_1910_05124_b200/csrc/mma_issue_bench.cu && ./mma_issue_bench
// Every wait is bounded; the operands are constant bit patterns (their values do not matter).
#include <cstdio>
#include <cuda_runtime.h>
#include "pm_ptx.cuh"
using namespace pm;

template <int PAIR>
__global__ void __launch_bounds__(128, 1) bench(int N, int a_mn, int b_mn, int iters, int n_acc, long long* out, int* status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;
  const uint32_t bar = tiles + 4 * 49152;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_raw + (bar + 64 - raw));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = PAIR ? (int)cluster_ctarank() : 0;
  // zero shared memory operands
  for (uint32_t i = threadIdx.x; i < 4 * 49152 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem_raw + (tiles - raw))[i] = 0x3c003c00u;
  if (threadIdx.x == 0) { mbar_init(bar, 1); *abort_flag = 0; asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
  fence_async_smem();
  if (warp == 1) { __syncwarp(); if (PAIR) { tmem_alloc_pair(smem_u32(tmem_slot), 512); tmem_relinquish_pair(); } else { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); } }
  tc_fence_before();
  if (PAIR) cluster_sync_all(); else __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (warp == 0 && lane == 0 && rank == 0) {
    const int M = PAIR ? 256 : 128;
    const uint32_t idesc = make_idesc_mn(M, N, a_mn, b_mn);
    const int nb_cta = PAIR ? N / 2 : N;                 // B columns held by this CTA
    const uint64_t dba = a_mn ? desc_base(8192, 1024) : desc_base(16, 1024);
    const uint64_t dbb = b_mn ? desc_base(8192, 1024) : desc_base(16, 1024);
    const uint32_t ka = a_mn ? 2048 : 32, kb = b_mn ? 2048 : 32;
    (void)nb_cta;
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
      const uint32_t sa = tiles + (it & 3) * 49152, sb = sa + 16384;
      const uint32_t acc = tmem_base + (uint32_t)((it % n_acc) * N);
#pragma unroll
      for (int k16 = 0; k16 < 4; ++k16) {
        if (PAIR) tc_mma_bf16_pair(acc, desc_at(dba, sa + k16 * ka), desc_at(dbb, sb + k16 * kb), idesc, 1u);
        else tc_mma_bf16(acc, desc_at(dba, sa + k16 * ka), desc_at(dbb, sb + k16 * kb), idesc, 1u);
      }
    }
    const long long t1 = clock64();
    if (PAIR) tc_commit_pair(bar, 1); else tc_commit(bar);
    mbar_wait(bar, 0, abort_flag, status, 1);
    const long long t2 = clock64();
    if (blockIdx.x == 0) { out[0] = t1 - t0; out[1] = t2 - t0; }
  }
  tc_fence_before();
  if (PAIR) cluster_sync_all(); else __syncthreads();
  if (warp == 1) { __syncwarp(); tc_fence_after(); if (PAIR) tmem_dealloc_pair(tmem_base, 512); else tmem_dealloc(tmem_base, 512); }
}

template <int PAIR> void run(int grid, int N, int a_mn, int b_mn, int n_acc) {
  long long* out; int* status; cudaMalloc(&out, 16); cudaMalloc(&status, 4); cudaMemset(status, 0, 4);
  const int smem = 4 * 49152 + 2048;
  cudaFuncSetAttribute((const void*)bench<PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  const int iters = 2000;
  cudaLaunchConfig_t cfg = {}; cfg.gridDim = dim3(grid); cfg.blockDim = dim3(128); cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute at[1]; at[0].id = cudaLaunchAttributeClusterDimension; at[0].val.clusterDim.x = PAIR ? 2 : 1; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  for (int rep = 0; rep < 2; ++rep) cudaLaunchKernelEx(&cfg, bench<PAIR>, N, a_mn, b_mn, iters, n_acc, out, status);
  cudaError_t e = cudaDeviceSynchronize();
  long long h[2]; int hs; cudaMemcpy(h, out, 16, cudaMemcpyDeviceToHost); cudaMemcpy(&hs, status, 4, cudaMemcpyDeviceToHost);
  const double clk_per_mma = (double)h[1] / (iters * 4.0);
  const double macs = (PAIR ? 128.0 : 128.0) * N * 16;   // per SM per MMA
  printf("pair=%d grid=%3d N=%3d a_mn=%d b_mn=%d n_acc=%d : %.1f clk/MMA (issue %.1f)  %.0f MAC/clk/SM  err=%s status=%d\n", PAIR, grid, N, a_mn, b_mn, n_acc,
         clk_per_mma, (double)h[0] / (iters * 4.0), macs / clk_per_mma, cudaGetErrorString(e), hs);
  cudaFree(out); cudaFree(status);
}

int main() {
  for (int grid : {2, 148}) {
    for (int N : {64, 128, 256}) {
      run<0>(grid, N, 0, 0, 1); run<0>(grid, N, 0, 1, 1); run<0>(grid, N, 1, 1, 1);
      if (N <= 128) run<0>(grid, N, 0, 1, 2);
    }
    for (int N : {128, 256}) {
      run<1>(grid, N, 0, 0, 1); run<1>(grid, N, 0, 1, 1); run<1>(grid, N, 1, 1, 1);
      if (N <= 128) run<1>(grid, N, 0, 1, 2);
    }
  }
  return 0;
}

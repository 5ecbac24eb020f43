// Element-wise tick kernels (ingest, loss, activation backward) and the fp32 SIMT grouped GEMMs.
//
// Every kernel is "grouped": blockIdx.z (or .y) selects the stage, the per-tick table says
// whether that stage is active and which ring slots it touches.  Within a tick the stages
// only read what earlier ticks left in their rings and mailboxes, so one launch covers all.
#include "pm_tick.cuh"

namespace pm {

template <typename AT> __device__ __forceinline__ AT* ring_ptr(const TickArgs& t, uint64_t off, int slot, uint64_t slot_elems) {
  return ring_at<AT>(t, off, slot, slot_elems);
}
template <typename AT> __device__ __forceinline__ AT* ws_ptr(const TickArgs& t, uint64_t off) { return ws_at<AT>(t, off); }

// ---- ingest -----------------------------------------------------------------------------------
// MLP: inputs [T, n_in] (activation type) -> stage 1's input ring slot; targets [T, n_out] float -> target ring.
// Encoder: token ids [T] int32 -> stage 1's id ring slot; target ids [T] int32 -> target ring.
template <typename AT>
__global__ void ingest_kernel(TickArgs t, const void* __restrict__ inputs, const void* __restrict__ targets, int64_t mb) {
  const StageDev& s0 = t.st[0];
  const uint64_t gid = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (uint64_t)gridDim.x * blockDim.x;
  if (s0.pre == PRE_EMBED) {
    int32_t* idst = ring_ptr<int32_t>(t, s0.ids_ring, (int)(mb % s0.ids_depth), (uint64_t)t.T);
    for (uint64_t i = gid; i < (uint64_t)t.T; i += stride) idst[i] = reinterpret_cast<const int32_t*>(inputs)[i];
    if (t.n_streams > 1) {                                    // second token stream -> the stage that embeds it
      const StageDev& s1 = t.st[t.second_embed_stage];
      int32_t* d1 = ring_ptr<int32_t>(t, s1.ids_ring, (int)(mb % s1.ids_depth), (uint64_t)t.T);
      for (uint64_t i = gid; i < (uint64_t)t.T; i += stride) d1[i] = reinterpret_cast<const int32_t*>(inputs)[(uint64_t)t.T + i];
    }
  } else {
    const uint64_t n_x = (uint64_t)t.T * t.n_in_first;
    AT* xdst = ring_ptr<AT>(t, s0.x_ring, (int)(mb % s0.xdepth), n_x);
    for (uint64_t i = gid; i < n_x; i += stride) xdst[i] = reinterpret_cast<const AT*>(inputs)[i];
  }
  if (t.loss_kind == PM_LOSS_CE) {
    int32_t* tdst = ws_ptr<int32_t>(t, t.tgt_off) + (uint64_t)(mb % (t.P + 1)) * t.T;
    for (uint64_t i = gid; i < (uint64_t)t.T; i += stride) tdst[i] = reinterpret_cast<const int32_t*>(targets)[i];
  } else {
    const uint64_t n_t = (uint64_t)t.T * t.n_out_last;
    float* tdst = ws_ptr<float>(t, t.tgt_off) + (uint64_t)(mb % (t.P + 1)) * n_t;
    for (uint64_t i = gid; i < n_t; i += stride) tdst[i] = reinterpret_cast<const float*>(targets)[i];
  }
}

cudaError_t launch_ingest(const TickArgs& t, int dtype, const void* inputs, const float* targets, int64_t mb, cudaStream_t stream) {
  uint64_t n = (uint64_t)t.T * (t.n_in_first > t.n_out_last ? t.n_in_first : t.n_out_last);
  int blocks = (int)((n + 255) / 256);
  if (blocks > 1184) blocks = 1184;
  if (dtype == PM_F32) ingest_kernel<float><<<blocks, 256, 0, stream>>>(t, inputs, targets, mb);
  else ingest_kernel<__nv_bfloat16><<<blocks, 256, 0, stream>>>(t, inputs, targets, mb);
  return cudaGetLastError();
}

// ---- MSE loss at the last stage ------------------------------------------------------------------
// loss = mean over T*out of (y - y*)^2 ;  dy = 2 (y - y*) / (T*out), stored in the activation type.
// Fixed summation order: each block sums a contiguous chunk (strided per-thread partials, fixed tree),
// the last block to finish adds the per-block partials in block order.
constexpr int kLossBlocks = 64, kLossThreads = 256;

template <typename AT>
__global__ void __launch_bounds__(kLossThreads) mse_loss_kernel(TickArgs t) {
  const StageDyn& d = t.dyn[t.P - 1];
  if (d.b_mb < 0) return;
  const StageDev& sl = t.st[t.P - 1];
  const uint64_t n = (uint64_t)t.T * t.n_out_last;
  const int par = (int)((d.tick + 1) & 1);            // written during the previous tick
  const AT* y = ws_ptr<AT>(t, t.yout_off) + (uint64_t)par * n;
  const float* tg = ws_ptr<float>(t, t.tgt_off) + (uint64_t)(d.b_mb % (t.P + 1)) * n;
  AT* dy = gin_read<AT>(t, sl, d);
  float* partial = ws_ptr<float>(t, t.lossred_off);
  unsigned int* counter = reinterpret_cast<unsigned int*>(partial + kLossBlocks);
  const float scale = (float)(2.0 / (double)n * (double)t.loss_scale);
  const uint64_t chunk = (n + gridDim.x - 1) / gridDim.x;
  const uint64_t lo = (uint64_t)blockIdx.x * chunk, hi = lo + chunk < n ? lo + chunk : n;
  float part = 0.f;
  for (uint64_t i = lo + threadIdx.x; i < hi; i += blockDim.x) {
    float r = __fsub_rn(to_f<AT>(y[i]), tg[i]);
    part = __fadd_rn(part, __fmul_rn(r, r));
    dy[i] = from_f<AT>(__fmul_rn(scale, r));
  }
  __shared__ float red[kLossThreads];
  __shared__ bool last;
  red[threadIdx.x] = part;
  __syncthreads();
  for (int off = kLossThreads / 2; off > 0; off >>= 1) {
    if ((int)threadIdx.x < off) red[threadIdx.x] = __fadd_rn(red[threadIdx.x], red[threadIdx.x + off]);
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    partial[blockIdx.x] = red[0];
    __threadfence();
    last = atomicAdd(counter, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (last && threadIdx.x == 0) {
    __threadfence();
    float sum = 0.f;
    for (int b = 0; b < (int)gridDim.x; ++b) sum = __fadd_rn(sum, reinterpret_cast<volatile float*>(partial)[b]);
    ws_ptr<float>(t, t.loss_off)[d.b_mb % t.loss_cap] = sum / (float)n;
    *counter = 0;                                     // ready for the next tick
  }
}

cudaError_t launch_ce_loss(const TickArgs& t, int dtype, cudaStream_t stream);   // pm_xfmr.cu

cudaError_t launch_loss(const TickArgs& t, int dtype, cudaStream_t stream) {
  if (t.loss_kind == PM_LOSS_CE) return launch_ce_loss(t, dtype, stream);
  if (dtype == PM_F32) mse_loss_kernel<float><<<kLossBlocks, kLossThreads, 0, stream>>>(t);
  else mse_loss_kernel<__nv_bfloat16><<<kLossBlocks, kLossThreads, 0, stream>>>(t);
  return cudaGetLastError();
}

// ---- activation backward + bias gradient ---------------------------------------------------------
// dz = dy * act'(z) (stored in the activation type); db[c] = sum over rows of the stored dz.
// A block owns 64 columns; warp w takes rows w, w+8, ... (ascending), two columns per thread; the eight
// per-warp partial sums of a column are added in warp order.
constexpr int kActCols = 64, kActWarps = 8;

template <typename AT> struct Pair;
template <> struct Pair<float> {
  static __device__ __forceinline__ float2 ld(const float* p) { return *reinterpret_cast<const float2*>(p); }
  static __device__ __forceinline__ void st(float* p, float2 v) { *reinterpret_cast<float2*>(p) = v; }
};
template <> struct Pair<__nv_bfloat16> {
  static __device__ __forceinline__ float2 ld(const __nv_bfloat16* p) { return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(p)); }
  static __device__ __forceinline__ void st(__nv_bfloat16* p, float2 v) { *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(v.x, v.y); }
};

constexpr int kActColsV = 256;                        // columns per block: 8 per lane
constexpr int kColsumGroup = 8;                       // row chunks per block in a launch that only sums columns
constexpr int kStageGroup = 4;                        // ... and in a launch of one stage
// Row chunks one block of the activation-backward launch covers; its sum is partial row (first chunk / group) of the stage.
__host__ __device__ inline int act_chunk_group(const TickArgs& t) {
  return t.row_chunks > 1 ? (t.colsum_only ? kColsumGroup : (t.sel_p >= 0 ? kStageGroup : 1)) : 1;
}

// rows r, r + NW, ... < r1 of 8 columns (NW = warps of the block): four rows are loaded before the first is used
template <typename AT, int ACT, int NW>
__device__ __forceinline__ void actbwd_rows(const AT* __restrict__ dy, const AT* __restrict__ z, AT* __restrict__ dz, int n_out, int c,
                                            int r, int r1, float (&sum)[8]) {
  for (; r + 3 * NW < r1; r += 4 * NW) {
    float g[4][8], zz[4][8];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint64_t i = (uint64_t)(r + u * NW) * n_out + c;
      load8<AT>(dy + i, g[u]);
      if (ACT != PM_ACT_NONE) load8<AT>(z + i, zz[u]);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (ACT != PM_ACT_NONE) {
#pragma unroll
        for (int k = 0; k < 8; ++k) g[u][k] = round_as<AT>(__fmul_rn(g[u][k], act_grad(zz[u][k], ACT)));
        store8<AT>(dz + (uint64_t)(r + u * NW) * n_out + c, g[u]);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) sum[k] = __fadd_rn(sum[k], g[u][k]);
    }
  }
  for (; r < r1; r += NW) {
    const uint64_t i = (uint64_t)r * n_out + c;
    float g[8];
    load8<AT>(dy + i, g);
    if (ACT != PM_ACT_NONE) {
      float zz[8];
      load8<AT>(z + i, zz);
#pragma unroll
      for (int k = 0; k < 8; ++k) g[k] = round_as<AT>(__fmul_rn(g[k], act_grad(zz[k], ACT)));
      store8<AT>(dz + i, g);
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) sum[k] = __fadd_rn(sum[k], g[k]);
  }
}

// NW warps per block: 8 in a grouped launch over all stages; 16 in a launch of one stage (microbatch-major order),
// which has fewer blocks and needs more loads in flight per block
template <typename AT, int NW>
__global__ void __launch_bounds__(NW * 32) actbwd_kernel(TickArgs t, int lvl) {
  const int* start = t.act_start + (size_t)lvl * (t.P + 1);
  int lo = 0, hi = t.P - 1;                                 // stage of this column block: largest p with start[p] <= its index
  const int blk = (int)blockIdx.x + t.act_first[lvl];
  if (t.sel_p >= 0) lo = hi = t.sel_p;                     // a launch of one stage: no search
  while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (start[mid] <= blk) lo = mid; else hi = mid - 1; }
  const int p = lo;
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.b_mb < 0 || lvl >= s.n_lin) return;
  const LinDev& L = s.lin[lvl];
  const int c0 = (blk - start[p]) * kActColsV;
  if (c0 >= L.n_out) return;
  // a launch that only sums columns, or a launch of one stage, gives a block several row chunks (fewer, longer-lived
  // blocks); a block's sum is one partial row, and the finishing pass adds as many rows as the launch had blocks
  const int cg = act_chunk_group(t);
  const int chunk = blockIdx.y * cg;
  const int r0 = chunk * t.chunk_rows, r1 = min(t.T, r0 + cg * t.chunk_rows);
  if (r0 >= t.T) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int c = c0 + 8 * lane;
  const uint64_t n = (uint64_t)t.T * L.n_out;
  const AT* dy = (lvl < s.n_lin - 1) ? ws_ptr<AT>(t, s.dh)
                 : (feeds_attention(s.post) ? ws_ptr<AT>(t, s.dy) : gin_read<AT>(t, s, d));
  const bool has_act = bwd_act(L) != PM_ACT_NONE;           // without an activation (or with one applied upstream) dz = dy: nothing is stored
  if (t.colsum_only && has_act) return;
  // the pre-activation stash, or for a ReLU without one the stashed output (same sign pattern)
  const AT* z = !has_act ? dy
                : !(L.flags & LF_ACT_FROM_Y) ? ring_ptr<AT>(t, L.z_ring, d.b_slot, n)
                : (lvl < s.n_lin - 1 ? ring_ptr<AT>(t, L.h_ring, d.b_slot, n) : ring_ptr<AT>(t, t.st[p + 1].x_ring, d.b_next_xslot, n));
  AT* dz = ws_ptr<AT>(t, s.dz);
  const bool vec = (L.n_out & 7) == 0;                      // vector path needs 8-element alignment of every row
  float sum[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (vec) {
    if (c < L.n_out) {
      if (!has_act) actbwd_rows<AT, PM_ACT_NONE, NW>(dy, z, dz, L.n_out, c, r0 + warp, r1, sum);
      else if (L.act == PM_ACT_RELU) actbwd_rows<AT, PM_ACT_RELU, NW>(dy, z, dz, L.n_out, c, r0 + warp, r1, sum);
      else actbwd_rows<AT, PM_ACT_GELU, NW>(dy, z, dz, L.n_out, c, r0 + warp, r1, sum);
    }
  } else {
    for (int r = r0 + warp; r < r1; r += NW) {
      const uint64_t i = (uint64_t)r * L.n_out + c;
#pragma unroll
      for (int k = 0; k < 8; ++k)
        if (c + k < L.n_out) {
          float v = has_act ? round_as<AT>(__fmul_rn(to_f<AT>(dy[i + k]), act_grad(to_f<AT>(z[i + k]), L.act))) : to_f<AT>(dy[i + k]);
          if (has_act) dz[i + k] = from_f<AT>(v);
          sum[k] = __fadd_rn(sum[k], v);
        }
    }
  }
  __shared__ float red[NW][kActColsV];
#pragma unroll
  for (int k = 0; k < 8; ++k) red[warp][8 * lane + k] = sum[k];
  __syncthreads();
  const int cc = c0 + threadIdx.x;
  if (threadIdx.x < kActColsV && cc < L.n_out) {
    float a = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) a = __fadd_rn(a, red[w][threadIdx.x]);
    if (t.row_chunks == 1) t.a.grad[L.b_off + cc] = d.accum ? __fadd_rn(t.a.grad[L.b_off + cc], a) : a;
    else ws_ptr<float>(t, t.colred_off)[((uint64_t)p * t.row_chunks + blockIdx.y) * (2 * (uint64_t)t.max_dim) + cc] = a;   // partial rows are dense: one per block
  }
}

// adds the per-row-chunk partial column sums: db of Linear lvl.  A block owns 32 columns; warp w adds the partials of
// chunks w, w + 8, ... in ascending order (all of its loads are issued before the first addition: the partials sit a
// row of the buffer apart, so every load is a separate round trip), then the eight per-warp sums are added in warp
// order.  The order is fixed, so the result is reproducible.
constexpr int kFinCols = 32, kFinMaxPer = 32;            // columns per block; partials per warp held in registers at a time

__global__ void __launch_bounds__(256) bias_finish_kernel(TickArgs t, int lvl) {
  // the grid follows the list of 256-column blocks of the activation-backward launch (kActColsV / kFinCols blocks
  // here per entry there), so no block falls outside its Linear's columns however unequal the widths are
  constexpr int kPer = kActColsV / kFinCols;
  const int* __restrict__ start = t.act_start + (size_t)lvl * (t.P + 1);
  const int blk = (int)(blockIdx.x / kPer) + t.act_first[lvl];
  int lo = 0, hi = t.P - 1;
  if (t.sel_p >= 0) lo = hi = t.sel_p;
  while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (start[mid] <= blk) lo = mid; else hi = mid - 1; }
  const int p = lo;
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.b_mb < 0 || lvl >= s.n_lin) return;
  const LinDev& L = s.lin[lvl];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cb = (blk - start[p]) * kActColsV + (int)(blockIdx.x % kPer) * kFinCols;
  const int c = cb + lane;
  if (cb >= L.n_out) return;
  const uint64_t ps = 2 * (uint64_t)t.max_dim;
  const float* part = ws_ptr<float>(t, t.colred_off) + (uint64_t)p * t.row_chunks * ps + (c < L.n_out ? c : 0);
  // partial rows the activation-backward launch of this Linear wrote: one per block of that launch
  const int cg = t.fin_deferred ? (t.row_chunks > 1 ? (bwd_act(L) != PM_ACT_NONE ? kStageGroup : kColsumGroup) : 1) : act_chunk_group(t);
  const int n_rows = (t.row_chunks + cg - 1) / cg;
  float sum = 0.f;
  for (int k0 = warp; k0 < n_rows; k0 += 8 * kFinMaxPer) {
    float v[kFinMaxPer];
#pragma unroll
    for (int u = 0; u < kFinMaxPer; ++u) { const int k = k0 + 8 * u; v[u] = k < n_rows ? part[(uint64_t)k * ps] : 0.f; }
#pragma unroll
    for (int u = 0; u < kFinMaxPer; ++u) if (k0 + 8 * u < n_rows) sum = __fadd_rn(sum, v[u]);
  }
  __shared__ float red[8][kFinCols];
  red[warp][lane] = sum;
  __syncthreads();
  if (warp == 0 && c < L.n_out) {
    float a = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) a = __fadd_rn(a, red[w][lane]);
    t.a.grad[L.b_off + c] = d.accum ? __fadd_rn(t.a.grad[L.b_off + c], a) : a;
  }
}

int actbwd_launches(const TickArgs& t) { return (t.row_chunks == 1 || t.defer_finish) ? 1 : 2; }

int deferred_finish_launches(const TickArgs& t) { return (t.row_chunks > 1 ? t.max_lin : 0) + ln_finish_launches(t); }
cudaError_t launch_deferred_finish(const TickArgs& t, int dtype, cudaStream_t stream) {
  (void)dtype;
  if (t.row_chunks > 1) {
    TickArgs tf = t;
    tf.fin_deferred = 1;
    for (int lvl = 0; lvl < t.max_lin; ++lvl)
      if (t.act_blocks[lvl] > 0) bias_finish_kernel<<<t.act_blocks[lvl] * (kActColsV / kFinCols), 256, 0, stream>>>(tf, lvl);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return launch_ln_finish(t, stream);
}

cudaError_t launch_actbwd(const TickArgs& t, int dtype, int lvl, cudaStream_t stream) {
  if (t.act_blocks[lvl] == 0) return cudaSuccess;
  const int cg = act_chunk_group(t);
  dim3 grid(t.act_blocks[lvl], (t.row_chunks + cg - 1) / cg);
  if (t.sel_p >= 0 && t.row_chunks > 1) {
    if (dtype == PM_F32) actbwd_kernel<float, 16><<<grid, 16 * 32, 0, stream>>>(t, lvl);
    else actbwd_kernel<__nv_bfloat16, 16><<<grid, 16 * 32, 0, stream>>>(t, lvl);
  } else {
    if (dtype == PM_F32) actbwd_kernel<float, kActWarps><<<grid, kActWarps * 32, 0, stream>>>(t, lvl);
    else actbwd_kernel<__nv_bfloat16, kActWarps><<<grid, kActWarps * 32, 0, stream>>>(t, lvl);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess || t.row_chunks == 1 || t.defer_finish) return e;
  bias_finish_kernel<<<t.act_blocks[lvl] * (kActColsV / kFinCols), 256, 0, stream>>>(t, lvl);
  return cudaGetLastError();
}

// ---- fp32 SIMT grouped GEMM ------------------------------------------------------------------------
// C[M,N] = sum_k A(m,k) B(k,n), 64x64 tile per block, 16-deep k steps, 4x4 outputs per thread,
// k ascending with fused multiply-add in fp32.
//   mode 0 forward:  A = x [T,in],        B(k,n) = W[n,k]            -> z = C + b, y = act(z)
//   mode 1 dgrad:    A = dz [T,out],      B(k,n) = W[k,n]-gap*delta  -> dx = C
//   mode 2 wgrad:    A(m,k) = dz[k,m],    B(k,n) = x[k,n]            -> dW = C
constexpr int BM = 64, BN = 64, BK = 16;

template <typename AT, typename WT, int MODE>
__global__ void __launch_bounds__(256) simt_gemm_kernel(TickArgs t, int lvl) {
  const int p = stage_of_block(t, blockIdx.z);
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (lvl >= s.n_lin) return;
  if (MODE == 0 ? d.f_mb < 0 : d.b_mb < 0) return;
  if (MODE == 1 && p == 0 && lvl == 0 && s.pre != PRE_EMBED) return;   // raw network inputs need no gradient
  const LinDev& L = s.lin[lvl];
  const int T = t.T;
  int M, N, K;
  if (MODE == 0) { M = T; N = L.n_out; K = L.n_in; }
  else if (MODE == 1) { M = T; N = L.n_in; K = L.n_out; }
  else { M = L.n_out; N = L.n_in; K = T; }
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  if (m0 >= M || n0 >= N) return;

  const uint64_t n_xin = (uint64_t)T * L.n_in, n_xout = (uint64_t)T * L.n_out;
  // operand sources
  const AT* xin = lin_input<AT>(t, s, d, lvl, MODE == 0);   // this Linear's input activation (forward or backward slot)
  const AT* dz = dz_src<AT>(t, s, d, lvl);
  const WT* wf = fwd_weights<WT>(t, s, d, L.w_off);       // forward operand: the weights of the version the forward reads
  const float* wm = t.a.w + L.w_off;
  const float* dl = t.a.delta + L.w_off;
  const float gapf = (float)s.gap;
  const bool corr = d.use_delta != 0;

  __shared__ float As[BK][BM + 1];
  __shared__ float Bs[BK][BN + 1];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < K; k0 += BK) {
    // A tile
    if (MODE == 2) {            // m contiguous: A(m,k) = dz[k*out + m]
      int kk = tid >> 4, mm = (tid & 15) * 4;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int m = m0 + mm + j, k = k0 + kk;
        As[kk][mm + j] = (m < M && k < K) ? to_f<AT>(dz[(uint64_t)k * L.n_out + m]) : 0.f;
      }
    } else {                    // k contiguous
      int mm = tid >> 2, kk = (tid & 3) * 4;
      const AT* src = MODE == 0 ? xin : dz;
      const int ld = MODE == 0 ? L.n_in : L.n_out;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int m = m0 + mm, k = k0 + kk + j;
        As[kk + j][mm] = (m < M && k < K) ? to_f<AT>(src[(uint64_t)m * ld + k]) : 0.f;
      }
    }
    // B tile
    if (MODE == 0) {            // k contiguous: B(k,n) = W[n*in + k]
      int nn = tid >> 2, kk = (tid & 3) * 4;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int n = n0 + nn, k = k0 + kk + j;
        Bs[kk + j][nn] = (n < N && k < K) ? to_f<WT>(wf[(uint64_t)n * L.n_in + k]) : 0.f;
      }
    } else {                    // n contiguous
      int kk = tid >> 4, nn = (tid & 15) * 4;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int n = n0 + nn + j, k = k0 + kk;
        float v = 0.f;
        if (n < N && k < K) {
          uint64_t idx = (uint64_t)k * L.n_in + n;
          if (MODE == 1 && t.stash) {   // weight stashing: the queued version the forward read, as the operand type holds it
            v = to_f<WT>(wf[idx]);
          } else if (MODE == 1) {      // T2: w - (tau_fwd - tau_bkwd) * delta, then rounded as the operand type holds it
            float wv = wm[idx];
            if (corr) wv = __fsub_rn(wv, __fmul_rn(gapf, dl[idx]));
            v = round_as<WT>(wv);
          } else {
            v = to_f<AT>(xin[idx]);
          }
        }
        Bs[kk][nn + j] = v;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }

  // epilogue
  if (MODE == 0) {
    AT* zout = (L.flags & LF_WRITE_Z) ? ring_ptr<AT>(t, L.z_ring, d.f_slot, n_xout) : nullptr;
    AT* yout = y_dest<AT>(t, p, s, d, lvl);
    float* lout = (L.flags & LF_OUT_F32) ? ws_ptr<float>(t, t.yout_off) + (uint64_t)(d.tick & 1) * n_xout : nullptr;
    const float* bias = fwd_small<AT>(t, s, d, L.b_off, L.b_soff);
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
        if (m < M && n < N) {
          const float pre_act = __fadd_rn(acc[i][j], bias[n]);
          if (lout) lout[(uint64_t)m * N + n] = pre_act;          // logits stay fp32
          AT zv = from_f<AT>(pre_act);
          if (zout) zout[(uint64_t)m * N + n] = zv;
          if (yout) yout[(uint64_t)m * N + n] = from_f<AT>(act_fwd(to_f<AT>(zv), L.act));
        }
      }
  } else if (MODE == 1) {
    AT* dx = (lvl == 0 && s.pre == PRE_NONE) ? gin_write_prev<AT>(t, p, d) : ws_ptr<AT>(t, s.dh);
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
        if (m < M && n < N) dx[(uint64_t)m * N + n] = from_f<AT>(acc[i][j]);
      }
  } else {
    float* dW = t.a.grad + L.w_off;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
        if (m < M && n < N) dW[(uint64_t)m * N + n] = d.accum ? __fadd_rn(dW[(uint64_t)m * N + n], acc[i][j]) : acc[i][j];
      }
  }
}

template <typename AT, typename WT>
static cudaError_t launch_simt_t(const TickArgs& t, int mode, int lvl, cudaStream_t stream) {
  const int mt = mode == 2 ? t.max_dim : t.T;
  dim3 grid((t.max_dim + BN - 1) / BN, (mt + BM - 1) / BM, t.sel_p >= 0 ? 1 : t.P);
  if (mode == 0) simt_gemm_kernel<AT, WT, 0><<<grid, 256, 0, stream>>>(t, lvl);
  else if (mode == 1) simt_gemm_kernel<AT, WT, 1><<<grid, 256, 0, stream>>>(t, lvl);
  else simt_gemm_kernel<AT, WT, 2><<<grid, 256, 0, stream>>>(t, lvl);
  return cudaGetLastError();
}

cudaError_t launch_simt_gemm(const TickArgs& t, int dtype, int mode, int lvl, cudaStream_t stream) {
  if (dtype == PM_F32) return launch_simt_t<float, float>(t, mode, lvl, stream);
  return launch_simt_t<__nv_bfloat16, __nv_bfloat16>(t, mode, lvl, stream);
}

}  // namespace pm

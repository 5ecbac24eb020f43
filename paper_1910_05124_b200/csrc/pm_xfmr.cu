// Transformer pieces of a pipeline tick: embedding, LayerNorm, multi-head attention, residual add and
// cross-entropy, forward and backward.  Every kernel is grouped over the stages (blockIdx.y) and acts only
// on stages that carry the op and are active this tick.
//
// Which weight value is read where (Section 2.1: forward pass reads the forward weights, backward pass the
// backward weights): the embedding table and the LayerNorm gain/bias are read in the forward pass; the
// backward pass reads only the LayerNorm gain, in dx_hat = dy * gain, and takes it T2-corrected
// (gain - gap * delta).  Parameter gradients use stashed forward quantities only.
#include <algorithm>
#include "pm_tick.cuh"
#include "pm_ptx.cuh"

namespace pm {

constexpr float LN_EPS = 1e-5f;

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

// ---- pre-op forward: embedding or LayerNorm, one warp per row ------------------------------------------------
//   embedding: u = table[id] * sqrt(d) + PE[position]     (table in the GEMM operand type)
//   LayerNorm: mean, biased variance, rstd = 1/sqrt(var + eps) in fp32; u = xhat * gain + bias (fp32 master values)
// If the stage emits a skip tensor (attention / skip_out) u is also written to the next stage's skip buffer.
// LayerNorm of one row of exactly NP * 256 columns by one warp: the row is read once and stays in registers
template <typename AT, int NP>
__device__ __forceinline__ void ln_fwd_row(const TickArgs& t, const StageDev& s, const StageDyn& d, const AT* x, const float* g,
                                           const float* b, AT* u, AT* skip, int row, int lane) {
  constexpr int dm = NP * 256;
  float xr[NP][8];
#pragma unroll
  for (int q = 0; q < NP; ++q) load8<AT>(x + q * 256 + lane * 8, xr[q]);
  float sum = 0.f, sq = 0.f;
#pragma unroll
  for (int q = 0; q < NP; ++q)
#pragma unroll
    for (int k = 0; k < 8; ++k) sum += xr[q][k];
  const float mu = warp_sum(sum) / (float)dm;
#pragma unroll
  for (int q = 0; q < NP; ++q)
#pragma unroll
    for (int k = 0; k < 8; ++k) { const float v = xr[q][k] - mu; sq += v * v; }
  const float rstd = 1.0f / sqrtf(warp_sum(sq) / (float)dm + LN_EPS);
#pragma unroll
  for (int q = 0; q < NP; ++q) {
    const int c = q * 256 + lane * 8;
    float gv[8], bv[8], o[8];
    load8<float>(g + c, gv);
    load8<float>(b + c, bv);
#pragma unroll
    for (int k = 0; k < 8; ++k) o[k] = __fadd_rn(__fmul_rn(__fmul_rn(xr[q][k] - mu, rstd), gv[k]), bv[k]);
    store8<AT>(u + c, o);
    if (skip) store8<AT>(skip + c, o);
  }
  if (lane == 0) {
    float* st = ring_at<float>(t, s.stat_ring, d.f_slot, (uint64_t)t.T * 2) + (uint64_t)row * 2;
    st[0] = mu; st[1] = rstd;
  }
}

template <typename AT>
__global__ void __launch_bounds__(256) pre_fwd_kernel(TickArgs t) {
  const int p = t.pre_ids[blockIdx.y];
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.f_mb < 0 || s.pre == PRE_NONE) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * 8 + warp;
  if (row >= t.T) return;
  const int dm = s.d_in;
  const uint64_t n = (uint64_t)t.T * dm;
  AT* u = ring_at<AT>(t, s.u_ring, d.f_slot, n) + (uint64_t)row * dm;
  const StageDev& sk_dst = t.st[p + s.skip_hop];             // the residual stage that will add this stage's input
  AT* skip = emits_skip(s) ? ws_at<AT>(t, sk_dst.skip_in) + (uint64_t)d.skip_wslot * n + (uint64_t)row * dm : nullptr;
  const bool vec = (dm & 7) == 0;                            // 8 consecutive columns per lane, 256 per pass
  if (s.pre == PRE_EMBED) {
    const int32_t id = ring_at<int32_t>(t, s.ids_ring, (int)(d.f_mb % s.ids_depth), (uint64_t)t.T)[row];
    const AT* e = fwd_weights<AT>(t, s, d, s.tab_off) + (uint64_t)id * dm;
    const float* pe = ws_at<float>(t, t.pe_off) + (uint64_t)(row % s.seq_len) * dm;
    const float sc = sqrtf((float)dm);
    if (vec) {
      for (int c = lane * 8; c < dm; c += 256) {
        float ev[8], pv[8], o[8];
        load8<AT>(e + c, ev);
        load8<float>(pe + c, pv);
#pragma unroll
        for (int k = 0; k < 8; ++k) o[k] = __fadd_rn(__fmul_rn(ev[k], sc), pv[k]);
        store8<AT>(u + c, o);
        if (skip) store8<AT>(skip + c, o);
      }
    } else {
      for (int c = lane; c < dm; c += 32) {
        AT v = from_f<AT>(__fadd_rn(__fmul_rn(to_f<AT>(e[c]), sc), pe[c]));
        u[c] = v;
        if (skip) skip[c] = v;
      }
    }
    return;
  }
  const AT* x = (s.from_memory ? mem_at<AT>(t, d.f_mb) : ring_at<AT>(t, s.x_ring, d.f_xslot, n)) + (uint64_t)row * dm;
  const float* g = fwd_small<AT>(t, s, d, s.g_off, s.g_soff);
  const float* b = fwd_small<AT>(t, s, d, s.beta_off, s.beta_soff);
  float sum = 0.f, sq = 0.f;
  if (vec && dm == 512) { ln_fwd_row<AT, 2>(t, s, d, x, g, b, u, skip, row, lane); return; }
  if (vec && dm == 1024) { ln_fwd_row<AT, 4>(t, s, d, x, g, b, u, skip, row, lane); return; }
  if (vec && dm == 256) { ln_fwd_row<AT, 1>(t, s, d, x, g, b, u, skip, row, lane); return; }
  if (vec) {
    for (int c = lane * 8; c < dm; c += 256) {
      float xv[8];
      load8<AT>(x + c, xv);
#pragma unroll
      for (int k = 0; k < 8; ++k) sum += xv[k];
    }
    const float mu = warp_sum(sum) / (float)dm;
    for (int c = lane * 8; c < dm; c += 256) {
      float xv[8];
      load8<AT>(x + c, xv);
#pragma unroll
      for (int k = 0; k < 8; ++k) { const float v = xv[k] - mu; sq += v * v; }
    }
    const float rstd = 1.0f / sqrtf(warp_sum(sq) / (float)dm + LN_EPS);
    for (int c = lane * 8; c < dm; c += 256) {
      float xv[8], gv[8], bv[8], o[8];
      load8<AT>(x + c, xv);
      load8<float>(g + c, gv);
      load8<float>(b + c, bv);
#pragma unroll
      for (int k = 0; k < 8; ++k) o[k] = __fadd_rn(__fmul_rn(__fmul_rn(xv[k] - mu, rstd), gv[k]), bv[k]);
      store8<AT>(u + c, o);
      if (skip) store8<AT>(skip + c, o);
    }
    if (lane == 0) {
      float* st = ring_at<float>(t, s.stat_ring, d.f_slot, (uint64_t)t.T * 2) + (uint64_t)row * 2;
      st[0] = mu; st[1] = rstd;
    }
    return;
  }
  for (int c = lane; c < dm; c += 32) sum += to_f<AT>(x[c]);
  const float mu = warp_sum(sum) / (float)dm;
  for (int c = lane; c < dm; c += 32) { float v = to_f<AT>(x[c]) - mu; sq += v * v; }
  const float rstd = 1.0f / sqrtf(warp_sum(sq) / (float)dm + LN_EPS);
  for (int c = lane; c < dm; c += 32) {
    AT v = from_f<AT>(__fadd_rn(__fmul_rn(__fmul_rn(to_f<AT>(x[c]) - mu, rstd), g[c]), b[c]));
    u[c] = v;
    if (skip) skip[c] = v;
  }
  if (lane == 0) {
    float* st = ring_at<float>(t, s.stat_ring, d.f_slot, (uint64_t)t.T * 2) + (uint64_t)row * 2;
    st[0] = mu; st[1] = rstd;
  }
}

cudaError_t launch_pre_fwd(const TickArgs& t, int dtype, cudaStream_t stream) {
  dim3 grid((t.T + 7) / 8, t.n_pre);
  if (dtype == PM_F32) pre_fwd_kernel<float><<<grid, 256, 0, stream>>>(t);
  else pre_fwd_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(t);
  return cudaGetLastError();
}

// ---- residual add: next stage's input = skip + y --------------------------------------------------------------
template <typename AT>
__global__ void __launch_bounds__(256) residual_kernel(TickArgs t) {
  const int p = t.res_ids[blockIdx.y];
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.f_mb < 0 || s.post != POST_RESIDUAL) return;
  const uint64_t n = (uint64_t)t.T * s.d_out_main;
  const AT* skip = ws_at<AT>(t, s.skip_in) + (uint64_t)d.skip_rslot * n;   // written skip_depth - 1 ticks ago
  const AT* y = ws_at<AT>(t, s.ytmp);
  // the stage that emits the memory writes only there: the next stage embeds its own token stream
  AT* out = s.emit_memory ? mem_at<AT>(t, d.f_mb) : ring_at<AT>(t, t.st[p + 1].x_ring, d.f_next_xslot, n);
  // buffers start on 256-byte boundaries and slots are n elements apart: groups of eight are aligned when 8 | n
  const uint64_t n8 = (n % 8 == 0) ? n / 8 : 0;
  // a block takes runs of 4 x 256 groups of eight: thread t the groups base + t, + 256, + 512, + 768, all loads first
  for (uint64_t base = (uint64_t)blockIdx.x * 1024; base < n8; base += (uint64_t)gridDim.x * 1024) {
    float a[4][8], b[4][8];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint64_t i = min(base + u * 256 + threadIdx.x, n8 - 1);
      load8<AT>(skip + 8 * i, a[u]);
      load8<AT>(y + 8 * i, b[u]);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint64_t i = base + u * 256 + threadIdx.x;
      if (i < n8) {
#pragma unroll
        for (int j = 0; j < 8; ++j) a[u][j] = __fadd_rn(a[u][j], b[u][j]);
        store8<AT>(out + 8 * i, a[u]);
      }
    }
  }
  for (uint64_t i = 8 * n8 + (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x)
    out[i] = from_f<AT>(__fadd_rn(to_f<AT>(skip[i]), to_f<AT>(y[i])));
}

// ---- multi-head self-attention, one block per (sequence, head) -----------------------------------------------
// s = q k^T / sqrt(d_k); p~ = exp(s - rowmax); l = sum p~ (unrounded); O = (round(p~) V) / l.
// Whole score matrix in shared memory (S <= 128): the softmax is exact over the full row.
struct AttnShape { int S, dk, d; };

template <typename AT>
__global__ void __launch_bounds__(256) attention_fwd_kernel(TickArgs t) {
  const int p = stage_of_block(t, blockIdx.y);
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.f_mb < 0 || (s.post != POST_ATTENTION && s.post != POST_CROSS_ATTENTION)) return;
  const bool cross = s.post == POST_CROSS_ATTENTION;        // q = the stage's main input, the Linear gave [k | v]
  const int causal = s.causal;
  const int S = s.seq_len, H = s.n_heads, dm = s.d_out_main, dk = dm / H;
  const int n_seq = t.T / S;
  if ((int)blockIdx.x >= n_seq * H) return;
  const int b = blockIdx.x / H, h = blockIdx.x % H;
  extern __shared__ float sm[];
  const int ld = dk + 2, lp = S + 1;   // operands are kept in the activation type, scores in fp32
  float* Pm = sm;                      // [S][S+1]
  float* Ls = Pm + S * lp;             // [S]
  AT* Q = reinterpret_cast<AT*>(Ls + S);   // [S][dk+2]
  AT* K = Q + S * ld;
  AT* V = K + S * ld;
  const int wz = cross ? 2 * dm : 3 * dm;                    // row length of the Linear's output
  const AT* zb = ring_at<AT>(t, s.lin[0].z_ring, d.f_slot, (uint64_t)t.T * wz) + (uint64_t)b * S * wz + h * dk;
  const AT* qb = cross ? ring_at<AT>(t, s.x_ring, d.f_xslot, (uint64_t)t.T * dm) + (uint64_t)b * S * dm + h * dk : zb;
  const int wq = cross ? dm : wz, ko = cross ? 0 : dm;
  for (int i = threadIdx.x; i < S * dk; i += blockDim.x) {
    const int r = i / dk, c = i % dk;
    const AT* row = zb + (uint64_t)r * wz;
    Q[r * ld + c] = qb[(uint64_t)r * wq + c];
    K[r * ld + c] = row[ko + c];
    V[r * ld + c] = row[ko + dm + c];
  }
  __syncthreads();
  const float scale = 1.0f / sqrtf((float)dk);
  for (int i = threadIdx.x; i < S * S; i += blockDim.x) {
    const int r = i / S, c = i % S;
    float acc = 0.f;
    for (int k = 0; k < dk; ++k) acc = fmaf(to_f<AT>(Q[r * ld + k]), to_f<AT>(K[c * ld + k]), acc);
    Pm[r * lp + c] = (causal && c > r) ? -INFINITY : acc * scale;
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int r = warp; r < S; r += 8) {
    float mx = -INFINITY;
    for (int c = lane; c < S; c += 32) mx = fmaxf(mx, Pm[r * lp + c]);
    mx = warp_max(mx);
    float sum = 0.f;
    for (int c = lane; c < S; c += 32) {
      float e = expf(Pm[r * lp + c] - mx);
      sum += e;
      Pm[r * lp + c] = round_as<AT>(e);
    }
    sum = warp_sum(sum);
    if (lane == 0) Ls[r] = sum;
  }
  __syncthreads();
  const uint64_t no = (uint64_t)t.T * dm;
  AT* out = ring_at<AT>(t, t.st[p + 1].x_ring, d.f_next_xslot, no) + (uint64_t)b * S * dm + h * dk;
  for (int i = threadIdx.x; i < S * dk; i += blockDim.x) {
    const int r = i / dk, c = i % dk;
    float acc = 0.f;
    for (int j = 0; j < S; ++j) acc = fmaf(Pm[r * lp + j], to_f<AT>(V[j * ld + c]), acc);
    out[(uint64_t)r * dm + c] = from_f<AT>(acc / Ls[r]);
  }
}

static size_t attn_fwd_smem(int S, int dk, size_t esz) { return sizeof(float) * ((size_t)S * (S + 1) + S) + esz * 3 * (size_t)S * (dk + 2); }
static size_t attn_bwd_smem(int S, int dk, size_t esz) { return sizeof(float) * (2 * (size_t)S * (S + 1) + S) + esz * 4 * (size_t)S * (dk + 2); }

size_t attention_smem_bytes(int S, int dk, int dtype) { return attn_bwd_smem(S, dk, dtype == PM_F32 ? 4 : 2); }

cudaError_t launch_post_fwd(const TickArgs& t, int dtype, cudaStream_t stream, bool skip_attention) {
  int S = 0, dk = 0, nblk = 0;
  bool any_res = false, any_att = false;
  // the shapes are uniform over stages in the supported workloads; the host keeps the maxima in TickArgs
  S = t.att_S; dk = t.att_dk; nblk = t.att_blocks; any_att = t.att_blocks > 0 && !skip_attention; any_res = t.any_residual != 0 && !t.res_fused;
  cudaError_t e = cudaSuccess;
  if (any_att) {
    dim3 grid(nblk, t.sel_p >= 0 ? 1 : t.P);
    if (dtype == PM_F32) attention_fwd_kernel<float><<<grid, 256, attn_fwd_smem(S, dk, 4), stream>>>(t);
    else attention_fwd_kernel<__nv_bfloat16><<<grid, 256, attn_fwd_smem(S, dk, 2), stream>>>(t);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  if (any_res) {
    dim3 grid(t.sel_p >= 0 ? 592 : 64, t.n_res);          // a launch of one stage brings all the blocks itself
    if (dtype == PM_F32) residual_kernel<float><<<grid, 256, 0, stream>>>(t);
    else residual_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(t);
    e = cudaGetLastError();
  }
  return e;
}

// ---- attention backward ------------------------------------------------------------------------------------------
// P recomputed as in the forward pass.  dV = round(P)^T dO; dP = dO V^T; dS = round(P * (dP - rowsum(dP * P)));
// dQ = dS K / sqrt(d_k); dK = dS^T Q / sqrt(d_k).  Results go to the stage's dy buffer as [dq | dk | dv].
template <typename AT>
__global__ void __launch_bounds__(256) attention_bwd_kernel(TickArgs t) {
  const int p = stage_of_block(t, blockIdx.y);
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.b_mb < 0 || (s.post != POST_ATTENTION && s.post != POST_CROSS_ATTENTION)) return;
  const bool cross = s.post == POST_CROSS_ATTENTION;
  const int causal = s.causal;
  const int S = s.seq_len, H = s.n_heads, dm = s.d_out_main, dk = dm / H;
  const int n_seq = t.T / S;
  if ((int)blockIdx.x >= n_seq * H) return;
  const int b = blockIdx.x / H, h = blockIdx.x % H;
  extern __shared__ float sm[];
  const int ld = dk + 2, lp = S + 1;
  float* Pm = sm;                      // [S][S+1] softmax probabilities (fp32)
  float* Dm = Pm + S * lp;             // [S][S+1] dP, then dS
  float* Ls = Dm + S * lp;
  AT* Q = reinterpret_cast<AT*>(Ls + S);   // operands in the activation type, [S][dk+2]
  AT* K = Q + S * ld;
  AT* V = K + S * ld;
  AT* dO = V + S * ld;
  const int wz = cross ? 2 * dm : 3 * dm;
  const AT* zb = ring_at<AT>(t, s.lin[0].z_ring, d.b_slot, (uint64_t)t.T * wz) + (uint64_t)b * S * wz + h * dk;
  const AT* qb = cross ? ring_at<AT>(t, s.x_ring, d.b_xslot, (uint64_t)t.T * dm) + (uint64_t)b * S * dm + h * dk : zb;
  const int wq = cross ? dm : wz, ko = cross ? 0 : dm;
  const AT* go = gin_read<AT>(t, s, d) + (uint64_t)b * S * dm + h * dk;
  for (int i = threadIdx.x; i < S * dk; i += blockDim.x) {
    const int r = i / dk, c = i % dk;
    const AT* row = zb + (uint64_t)r * wz;
    Q[r * ld + c] = qb[(uint64_t)r * wq + c];
    K[r * ld + c] = row[ko + c];
    V[r * ld + c] = row[ko + dm + c];
    dO[r * ld + c] = go[(uint64_t)r * dm + c];
  }
  __syncthreads();
  const float scale = 1.0f / sqrtf((float)dk);
  for (int i = threadIdx.x; i < S * S; i += blockDim.x) {
    const int r = i / S, c = i % S;
    float acc = 0.f, accd = 0.f;
    for (int k = 0; k < dk; ++k) {
      acc = fmaf(to_f<AT>(Q[r * ld + k]), to_f<AT>(K[c * ld + k]), acc);
      accd = fmaf(to_f<AT>(dO[r * ld + k]), to_f<AT>(V[c * ld + k]), accd);
    }
    Pm[r * lp + c] = (causal && c > r) ? -INFINITY : acc * scale;
    Dm[r * lp + c] = accd;                                     // dP
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int r = warp; r < S; r += 8) {
    float mx = -INFINITY;
    for (int c = lane; c < S; c += 32) mx = fmaxf(mx, Pm[r * lp + c]);
    mx = warp_max(mx);
    float sum = 0.f;
    for (int c = lane; c < S; c += 32) { float e = expf(Pm[r * lp + c] - mx); sum += e; Pm[r * lp + c] = e; }
    sum = warp_sum(sum);
    float dsum = 0.f;
    for (int c = lane; c < S; c += 32) { float pr = Pm[r * lp + c] / sum; Pm[r * lp + c] = pr; dsum += Dm[r * lp + c] * pr; }
    dsum = warp_sum(dsum);
    for (int c = lane; c < S; c += 32) Dm[r * lp + c] = round_as<AT>(Pm[r * lp + c] * (Dm[r * lp + c] - dsum));   // dS
  }
  __syncthreads();
  // self-attention: dy = [dq | dk | dv]; cross-attention: dy = [dk | dv] and dq goes to the previous stage's mailbox
  AT* dy = ws_at<AT>(t, s.dy) + (uint64_t)b * S * wz + h * dk;
  AT* dqb = cross ? gin_write_prev<AT>(t, p, d) + (uint64_t)b * S * dm + h * dk : dy;
  for (int i = threadIdx.x; i < S * dk; i += blockDim.x) {
    const int r = i / dk, c = i % dk;
    float aq = 0.f, ak = 0.f, av = 0.f;
    for (int j = 0; j < S; ++j) {
      aq = fmaf(Dm[r * lp + j], to_f<AT>(K[j * ld + c]), aq);            // dQ[r] = sum_j dS[r][j] K[j]
      ak = fmaf(Dm[j * lp + r], to_f<AT>(Q[j * ld + c]), ak);            // dK[r] = sum_j dS[j][r] Q[j]
      av = fmaf(round_as<AT>(Pm[j * lp + r]), to_f<AT>(dO[j * ld + c]), av);   // dV[r] = sum_j P[j][r] dO[j]
    }
    AT* row = dy + (uint64_t)r * wz;
    dqb[(uint64_t)r * wq + c] = from_f<AT>(aq * scale);
    row[ko + c] = from_f<AT>(ak * scale);
    row[ko + dm + c] = from_f<AT>(av);
  }
}

cudaError_t launch_post_bwd(const TickArgs& t, int dtype, cudaStream_t stream) {
  if (t.att_blocks <= 0) return cudaSuccess;
  dim3 grid(t.att_blocks, t.sel_p >= 0 ? 1 : t.P);
  if (dtype == PM_F32) attention_bwd_kernel<float><<<grid, 256, attn_bwd_smem(t.att_S, t.att_dk, 4), stream>>>(t);
  else attention_bwd_kernel<__nv_bfloat16><<<grid, 256, attn_bwd_smem(t.att_S, t.att_dk, 2), stream>>>(t);
  return cudaGetLastError();
}

cudaError_t attention_set_smem_limits(int S, int dk, int dtype) {
  cudaError_t e;
  if (dtype == PM_F32) {
    e = cudaFuncSetAttribute((const void*)attention_fwd_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_fwd_smem(S, dk, 4));
    if (e == cudaSuccess) e = cudaFuncSetAttribute((const void*)attention_bwd_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_bwd_smem(S, dk, 4));
  } else {
    e = cudaFuncSetAttribute((const void*)attention_fwd_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_fwd_smem(S, dk, 2));
    if (e == cudaSuccess) e = cudaFuncSetAttribute((const void*)attention_bwd_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_bwd_smem(S, dk, 2));
  }
  return e;
}

// ---- loss reduction shared by the cross-entropy kernels ----
// per-token loss of this block's row; the last block to arrive adds all of them in a fixed order (strided per-thread
// partials over the first 256 threads, then a fixed tree).  Called by every thread of the block.
__device__ __forceinline__ void ce_finish(const TickArgs& t, const StageDyn& d, int row, float mx, float sum, float logit_tgt) {
  float* rowloss = ws_at<float>(t, t.rowloss_off);
  unsigned int* counter = reinterpret_cast<unsigned int*>(ws_at<float>(t, t.lossred_off) + 64);
  __shared__ bool last;
  if (threadIdx.x == 0) {
    rowloss[row] = (mx + logf(sum)) - logit_tgt;
    __threadfence();
    last = atomicAdd(counter, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (last) {
    __threadfence();
    __shared__ float tree[256];
    if (threadIdx.x < 256) {
      float a = 0.f;
      for (int r = threadIdx.x; r < t.T; r += 256) a += reinterpret_cast<volatile float*>(rowloss)[r];
      tree[threadIdx.x] = a;
    }
    __syncthreads();
    for (int off = 128; off > 0; off >>= 1) {
      if ((int)threadIdx.x < off) tree[threadIdx.x] += tree[threadIdx.x + off];
      __syncthreads();
    }
    if (threadIdx.x == 0) {
      ws_at<float>(t, t.loss_off)[d.b_mb % t.loss_cap] = tree[0] / (float)t.T;
      *counter = 0;
    }
  }
}

// fp32 activations take the exact exponential and a true division; with bf16 activations the gradient is rounded to 8
// bits anyway, so the exponential is the hardware base-2 one (relative error ~2^-21 |x|) and the division a product
// with the reciprocal of the row sum.  The loss itself uses the fp32 sum of these exponentials either way.
template <typename AT> __device__ __forceinline__ float ce_exp(float x);
template <> __device__ __forceinline__ float ce_exp<float>(float x) { return expf(x); }
template <> __device__ __forceinline__ float ce_exp<__nv_bfloat16>(float x) { return __expf(x); }
template <typename AT> __device__ __forceinline__ float ce_div(float e, float sum, float rsum);
template <> __device__ __forceinline__ float ce_div<float>(float e, float sum, float) { return e / sum; }
template <> __device__ __forceinline__ float ce_div<__nv_bfloat16>(float e, float, float rsum) { return e * rsum; }

// ---- cross-entropy at the last stage -------------------------------------------------------------------------------
// One block per token: lse = max + log(sum exp(logit - max)); loss_t = lse - logit[target];
// dlogits = (softmax - onehot) / T in the activation type, written where the last stage reads its incoming
// gradient.  The last block to finish adds the per-token losses in a fixed order.
template <typename AT>
__global__ void __launch_bounds__(256) ce_loss_kernel(TickArgs t) {
  const StageDyn& d = t.dyn[t.P - 1];
  if (d.b_mb < 0) return;
  const StageDev& sl = t.st[t.P - 1];
  const int V = t.n_out_last, row = blockIdx.x;
  const uint64_t n = (uint64_t)t.T * V;
  const float* lg = ws_at<float>(t, t.yout_off) + (uint64_t)((d.tick + 1) & 1) * n + (uint64_t)row * V;
  const int32_t tgt = (ws_at<int32_t>(t, t.tgt_off) + (uint64_t)(d.b_mb % (t.P + 1)) * t.T)[row];
  AT* dl = gin_read<AT>(t, sl, d) + (uint64_t)row * V;
  __shared__ float red[8];
  __shared__ float bc;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool in_regs = V <= 8192 && (V & 7) == 0;            // the whole row fits: 4 x 8 values per thread, one read of the logits
  float v[4][8];
  float mx = -INFINITY;
  if (in_regs) {
#pragma unroll
    for (int k = 0; k < 4; ++k) load8<float>(lg + min((k * 256 + (int)threadIdx.x) * 8, V - 8), v[k]);   // all loads first
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if ((k * 256 + (int)threadIdx.x) * 8 < V) {
#pragma unroll
        for (int e = 0; e < 8; ++e) mx = fmaxf(mx, v[k][e]);
      }
  } else if ((V & 3) == 0) {                                 // long rows: three vectorised passes, the re-reads hit L2
    for (int c = threadIdx.x * 4; c < V; c += 4 * blockDim.x) {
      const float4 q = *reinterpret_cast<const float4*>(lg + c);
      mx = fmaxf(fmaxf(mx, fmaxf(q.x, q.y)), fmaxf(q.z, q.w));
    }
  } else {
    for (int c = threadIdx.x; c < V; c += blockDim.x) mx = fmaxf(mx, lg[c]);
  }
  mx = warp_max(mx);
  if (lane == 0) red[warp] = mx;
  __syncthreads();
  if (threadIdx.x == 0) { float m = red[0]; for (int i = 1; i < 8; ++i) m = fmaxf(m, red[i]); bc = m; }
  __syncthreads();
  mx = bc;
  float sum = 0.f;
  if (in_regs) {
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if ((k * 256 + (int)threadIdx.x) * 8 < V) {
#pragma unroll
        for (int e = 0; e < 8; ++e) { v[k][e] = ce_exp<AT>(v[k][e] - mx); sum += v[k][e]; }
      }
  } else if ((V & 3) == 0) {
    for (int c = threadIdx.x * 4; c < V; c += 4 * blockDim.x) {
      const float4 q = *reinterpret_cast<const float4*>(lg + c);
      sum += expf(q.x - mx); sum += expf(q.y - mx); sum += expf(q.z - mx); sum += expf(q.w - mx);
    }
  } else {
    for (int c = threadIdx.x; c < V; c += blockDim.x) sum += expf(lg[c] - mx);
  }
  sum = warp_sum(sum);
  __syncthreads();
  if (lane == 0) red[warp] = sum;
  __syncthreads();
  if (threadIdx.x == 0) { float a = 0.f; for (int i = 0; i < 8; ++i) a += red[i]; bc = a; }
  __syncthreads();
  sum = bc;
  const float invT = t.loss_scale / (float)t.T, rsum = 1.0f / sum;
  if (in_regs) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int c = (k * 256 + threadIdx.x) * 8;
      if (c < V) {
        float o[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          float pr = ce_div<AT>(v[k][e], sum, rsum);
          if (c + e == tgt) pr -= 1.0f;
          o[e] = pr * invT;
        }
        store8<AT>(dl + c, o);
      }
    }
  } else if ((V & 3) == 0) {
    for (int c = threadIdx.x * 4; c < V; c += 4 * blockDim.x) {
      const float4 q = *reinterpret_cast<const float4*>(lg + c);
      float p0 = expf(q.x - mx) / sum, p1 = expf(q.y - mx) / sum, p2 = expf(q.z - mx) / sum, p3 = expf(q.w - mx) / sum;
      if (tgt == c) p0 -= 1.0f;
      if (tgt == c + 1) p1 -= 1.0f;
      if (tgt == c + 2) p2 -= 1.0f;
      if (tgt == c + 3) p3 -= 1.0f;
      dl[c] = from_f<AT>(p0 * invT); dl[c + 1] = from_f<AT>(p1 * invT);
      dl[c + 2] = from_f<AT>(p2 * invT); dl[c + 3] = from_f<AT>(p3 * invT);
    }
  } else {
    for (int c = threadIdx.x; c < V; c += blockDim.x) {
      float pr = expf(lg[c] - mx) / sum;
      if (c == tgt) pr -= 1.0f;
      dl[c] = from_f<AT>(pr * invT);
    }
  }
  ce_finish(t, d, row, mx, sum, lg[tgt]);
}

// Rows longer than the register path holds (a vocabulary of tens of thousands): 512 threads read the fp32 row once
// into shared memory (four float4 in flight per thread), the exponentials replace it there, and the gradient is
// written from them as 8-byte (bf16) or 16-byte (fp32) vectors.
constexpr int kCeLongThreads = 1024;
template <typename AT> __device__ __forceinline__ void store4(AT* p, float a, float b, float c, float e);
template <> __device__ __forceinline__ void store4<float>(float* p, float a, float b, float c, float e) { *reinterpret_cast<float4*>(p) = make_float4(a, b, c, e); }
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p, float a, float b, float c, float e) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, e);
  *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
}

template <typename AT>
__global__ void __launch_bounds__(kCeLongThreads) ce_loss_long_kernel(TickArgs t) {
  const StageDyn& d = t.dyn[t.P - 1];
  if (d.b_mb < 0) return;
  const StageDev& sl = t.st[t.P - 1];
  const int V = t.n_out_last, row = blockIdx.x, n4 = V >> 2;
  const uint64_t n = (uint64_t)t.T * V;
  const float* lg = ws_at<float>(t, t.yout_off) + (uint64_t)((d.tick + 1) & 1) * n + (uint64_t)row * V;
  const float4* lg4 = reinterpret_cast<const float4*>(lg);
  const int32_t tgt = (ws_at<int32_t>(t, t.tgt_off) + (uint64_t)(d.b_mb % (t.P + 1)) * t.T)[row];
  AT* dl = gin_read<AT>(t, sl, d) + (uint64_t)row * V;
  extern __shared__ float4 rowbuf[];                         // [V / 4]
  __shared__ float red[kCeLongThreads / 32];
  __shared__ float bc[3];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float mx = -INFINITY;
  for (int i = threadIdx.x; i < n4; i += 4 * kCeLongThreads) {
    float4 q[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) q[u] = __ldcs(lg4 + min(i + u * kCeLongThreads, n4 - 1));
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (i + u * kCeLongThreads < n4) {
        rowbuf[i + u * kCeLongThreads] = q[u];
        mx = fmaxf(fmaxf(mx, fmaxf(q[u].x, q[u].y)), fmaxf(q[u].z, q[u].w));
      }
  }
  mx = warp_max(mx);
  if (lane == 0) red[warp] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = red[0];
    for (int i = 1; i < kCeLongThreads / 32; ++i) m = fmaxf(m, red[i]);
    bc[0] = m;
    bc[2] = reinterpret_cast<const float*>(rowbuf)[tgt];      // the target's logit, before the exponentials replace the row
  }
  __syncthreads();
  mx = bc[0];
  const float logit_tgt = bc[2];
  float sum = 0.f;
  for (int i = threadIdx.x; i < n4; i += kCeLongThreads) {
    float4 q = rowbuf[i];
    q.x = ce_exp<AT>(q.x - mx); q.y = ce_exp<AT>(q.y - mx); q.z = ce_exp<AT>(q.z - mx); q.w = ce_exp<AT>(q.w - mx);
    sum += q.x; sum += q.y; sum += q.z; sum += q.w;
    rowbuf[i] = q;
  }
  sum = warp_sum(sum);
  if (lane == 0) red[warp] = sum;
  __syncthreads();
  if (threadIdx.x == 0) { float a = 0.f; for (int i = 0; i < kCeLongThreads / 32; ++i) a += red[i]; bc[1] = a; }
  __syncthreads();
  sum = bc[1];
  const float invT = t.loss_scale / (float)t.T, rsum = 1.0f / sum;
  for (int i = threadIdx.x; i < n4; i += kCeLongThreads) {
    const float4 q = rowbuf[i];
    const int c = 4 * i;
    float p0 = ce_div<AT>(q.x, sum, rsum), p1 = ce_div<AT>(q.y, sum, rsum), p2 = ce_div<AT>(q.z, sum, rsum), p3 = ce_div<AT>(q.w, sum, rsum);
    if (tgt == c) p0 -= 1.0f;
    if (tgt == c + 1) p1 -= 1.0f;
    if (tgt == c + 2) p2 -= 1.0f;
    if (tgt == c + 3) p3 -= 1.0f;
    store4<AT>(dl + c, p0 * invT, p1 * invT, p2 * invT, p3 * invT);
  }
  ce_finish(t, d, row, mx, sum, logit_tgt);
}

cudaError_t launch_ce_loss(const TickArgs& t, int dtype, cudaStream_t stream) {
  const int V = t.n_out_last;
  const size_t row_bytes = sizeof(float) * (size_t)V;
  if (V > 8192 && (V & 3) == 0 && row_bytes <= 200 * 1024) {
    static bool attr_set[2] = {false, false};
    const int which = dtype == PM_F32 ? 0 : 1;
    if (!attr_set[which]) {
      cudaError_t e = dtype == PM_F32
          ? cudaFuncSetAttribute((const void*)ce_loss_long_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)
          : cudaFuncSetAttribute((const void*)ce_loss_long_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
      if (e != cudaSuccess) return e;
      attr_set[which] = true;
    }
    if (dtype == PM_F32) ce_loss_long_kernel<float><<<t.T, kCeLongThreads, row_bytes, stream>>>(t);
    else ce_loss_long_kernel<__nv_bfloat16><<<t.T, kCeLongThreads, row_bytes, stream>>>(t);
    return cudaGetLastError();
  }
  if (dtype == PM_F32) ce_loss_kernel<float><<<t.T, 256, 0, stream>>>(t);
  else ce_loss_kernel<__nv_bfloat16><<<t.T, 256, 0, stream>>>(t);
  return cudaGetLastError();
}

// ---- pre-op backward --------------------------------------------------------------------------------------------
// du_total = du (dgrad output of the first Linear) + gradient of the skip tensor the stage emitted, if any.
template <typename AT>
__device__ __forceinline__ float du_total(const AT* du, const AT* gs, uint64_t i) {
  float v = to_f<AT>(du[i]);
  if (gs) v = __fadd_rn(v, to_f<AT>(gs[i]));
  return v;
}

// LayerNorm input gradient, one warp per row:
//   dxhat = du_total * gain_b (gain_b = gain - gap*delta: T2);  dx = rstd * (dxhat - mean(dxhat) - xhat * mean(dxhat*xhat))
template <typename AT>
__global__ void __launch_bounds__(256) ln_bwd_dx_kernel(TickArgs t) {
  const int p = t.ln_ids[blockIdx.y + t.ln_li0];
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.b_mb < 0 || s.pre != PRE_LN || p == 0) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * 8 + warp;
  if (row >= t.T) return;
  const int dm = s.d_in;
  const uint64_t n = (uint64_t)t.T * dm, ro = (uint64_t)row * dm;
  if (s.from_memory) return;                                 // memory stages take the fused kernel (widths are multiples of 8)
  const AT* du = ws_at<AT>(t, s.dh);
  const AT* gs = emits_skip(s) ? gskip_read<AT>(t, p, d) : nullptr;
  const AT* x = ring_at<AT>(t, s.x_ring, d.b_xslot, n) + ro;
  const float* st = ring_at<float>(t, s.stat_ring, d.b_slot, (uint64_t)t.T * 2) + (uint64_t)row * 2;
  const float mu = st[0], rstd = st[1];
  const float* g = t.stash ? fwd_small<AT>(t, s, d, s.g_off, s.g_soff) : t.a.w + s.g_off;   // stashing: the gain of the queued version
  const float* dl = t.a.delta + s.g_off;
  const float gapf = (float)s.gap;
  const bool corr = d.use_delta != 0 && !t.stash;          // a version read from the queue is used as it is
  AT* out = gin_write_prev<AT>(t, p, d) + ro;
  float s1 = 0.f, s2 = 0.f;
  if ((dm & 7) == 0 && dm <= 2048) {                         // 8 columns per lane per pass, values kept in registers
    float dxh[8][8], xh[8][8];
    int np = 0;
    for (int c = lane * 8; c < dm; c += 256, ++np) {
      float xv[8], dv[8], gv[8];
      load8<AT>(x + c, xv);
      load8<AT>(du + ro + c, dv);
      load8<float>(g + c, gv);
      if (gs) { float sv[8]; load8<AT>(gs + ro + c, sv);
#pragma unroll
        for (int k = 0; k < 8; ++k) dv[k] = __fadd_rn(dv[k], sv[k]); }
      if (corr) { float cv[8]; load8<float>(dl + c, cv);
#pragma unroll
        for (int k = 0; k < 8; ++k) gv[k] = __fsub_rn(gv[k], __fmul_rn(gapf, cv[k])); }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        xh[np][k] = (xv[k] - mu) * rstd;
        dxh[np][k] = dv[k] * gv[k];
        s1 += dxh[np][k]; s2 += dxh[np][k] * xh[np][k];
      }
    }
    s1 = warp_sum(s1) / (float)dm;
    s2 = warp_sum(s2) / (float)dm;
    np = 0;
    for (int c = lane * 8; c < dm; c += 256, ++np) {
      float o[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) o[k] = rstd * (dxh[np][k] - s1 - xh[np][k] * s2);
      store8<AT>(out + c, o);
    }
    return;
  }
  for (int c = lane; c < dm; c += 32) {
    float gb = g[c];
    if (corr) gb = __fsub_rn(gb, __fmul_rn(gapf, dl[c]));
    const float xh = (to_f<AT>(x[c]) - mu) * rstd;
    const float dxh = du_total<AT>(du, gs, ro + c) * gb;
    s1 += dxh; s2 += dxh * xh;
  }
  s1 = warp_sum(s1) / (float)dm;
  s2 = warp_sum(s2) / (float)dm;
  for (int c = lane; c < dm; c += 32) {
    float gb = g[c];
    if (corr) gb = __fsub_rn(gb, __fmul_rn(gapf, dl[c]));
    const float xh = (to_f<AT>(x[c]) - mu) * rstd;
    const float dxh = du_total<AT>(du, gs, ro + c) * gb;
    out[c] = from_f<AT>(rstd * (dxh - s1 - xh * s2));
  }
}

// LayerNorm parameter gradients: dgain[c] = sum_rows du_total * xhat, dbias[c] = sum_rows du_total.
// A block owns 256 columns (8 per lane) and 256 rows; warp w takes rows w, w+8, ... ascending; per-warp partials are added in
// warp order, per-block partials in block order by ln_param_finish_kernel.
constexpr int kLnCols = 256;                         // columns per block: 8 per lane

template <typename AT>
__global__ void __launch_bounds__(256) ln_bwd_param_kernel(TickArgs t) {
  const int p = t.ln_ids[blockIdx.z + t.ln_li0];
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.b_mb < 0 || s.pre != PRE_LN) return;
  const int dm = s.d_in;
  const int c0 = blockIdx.x * kLnCols;
  if (c0 >= dm) return;
  const int chunk = blockIdx.y;
  const int r0 = chunk * t.chunk_rows, r1 = min(t.T, r0 + t.chunk_rows);
  if (r0 >= t.T) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint64_t n = (uint64_t)t.T * dm;
  const AT* du = ws_at<AT>(t, s.dh);
  const AT* gs = emits_skip(s) ? gskip_read<AT>(t, p, d) : nullptr;
  const AT* x = ring_at<AT>(t, s.x_ring, d.b_xslot, n);
  const float* st = ring_at<float>(t, s.stat_ring, d.b_slot, (uint64_t)t.T * 2);
  const bool vec = (dm & 7) == 0;
  const int c = c0 + lane * 8;
  float ag[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, ab[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int r = r0 + warp; r < r1; r += 8) {
    const float mu = st[2 * r], rstd = st[2 * r + 1];
    const uint64_t i = (uint64_t)r * dm + c;
    if (vec) {
      if (c < dm) {
        float dv[8], xv[8];
        load8<AT>(du + i, dv);
        load8<AT>(x + i, xv);
        if (gs) { float sv[8]; load8<AT>(gs + i, sv);
#pragma unroll
          for (int k = 0; k < 8; ++k) dv[k] = __fadd_rn(dv[k], sv[k]); }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          ag[k] = __fadd_rn(ag[k], __fmul_rn(dv[k], (xv[k] - mu) * rstd));
          ab[k] = __fadd_rn(ab[k], dv[k]);
        }
      }
    } else {
#pragma unroll
      for (int k = 0; k < 8; ++k)
        if (c + k < dm) {
          const float v = du_total<AT>(du, gs, i + k);
          ag[k] = __fadd_rn(ag[k], __fmul_rn(v, (to_f<AT>(x[i + k]) - mu) * rstd));
          ab[k] = __fadd_rn(ab[k], v);
        }
    }
  }
  __shared__ float rg[8][kLnCols], rb[8][kLnCols];
#pragma unroll
  for (int k = 0; k < 8; ++k) { rg[warp][lane * 8 + k] = ag[k]; rb[warp][lane * 8 + k] = ab[k]; }
  __syncthreads();
  const int cc = c0 + threadIdx.x;
  if (cc < dm) {
    float a = 0.f, b2 = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) { a = __fadd_rn(a, rg[w][threadIdx.x]); b2 = __fadd_rn(b2, rb[w][threadIdx.x]); }
    if (t.row_chunks == 1) {
      t.a.grad[s.g_off + cc] = d.accum ? __fadd_rn(t.a.grad[s.g_off + cc], a) : a;
      t.a.grad[s.beta_off + cc] = d.accum ? __fadd_rn(t.a.grad[s.beta_off + cc], b2) : b2;
    } else {
      float* part = ws_at<float>(t, t.colred_off) + ((uint64_t)p * t.row_chunks + chunk) * (2 * (uint64_t)t.max_dim);
      part[cc] = a;
      part[t.max_dim + cc] = b2;
    }
  }
}

__global__ void __launch_bounds__(256) ln_param_finish_kernel(TickArgs t) {
  const int p = t.ln_ids[blockIdx.y + t.ln_li0];
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.b_mb < 0 || s.pre != PRE_LN) return;
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= s.d_in) return;
  const float* part = ws_at<float>(t, t.colred_off) + (uint64_t)p * t.row_chunks * (2 * (uint64_t)t.max_dim);
  float a = 0.f, b2 = 0.f;
  for (int k = 0; k < t.row_chunks; ++k) {
    a = __fadd_rn(a, part[(uint64_t)k * 2 * t.max_dim + c]);
    b2 = __fadd_rn(b2, part[(uint64_t)k * 2 * t.max_dim + t.max_dim + c]);
  }
  t.a.grad[s.g_off + c] = d.accum ? __fadd_rn(t.a.grad[s.g_off + c], a) : a;
  t.a.grad[s.beta_off + c] = d.accum ? __fadd_rn(t.a.grad[s.beta_off + c], b2) : b2;
}

// Fused LayerNorm backward (widths that are multiples of 8, at most WPR*NP*256): one pass over du, x and the skip
// gradient produces dx and the partial column sums of dgain, dbias.  A block owns ln_chunk_rows rows; WPR warps
// share a row (each NP*256 of its columns; with WPR = 2 the two row sums meet in shared memory behind a 64-thread
// named barrier, first half + second half), the 8 / WPR warp groups take rows g, g + 8 / WPR, ... in ascending
// order; a lane owns 8 consecutive columns per 256-column group; per-warp partials are added in warp order,
// per-block partials in block order by ln_fused_finish_kernel.
template <typename AT, int NP, int WPR>
__global__ void __launch_bounds__(256, NP <= 2 ? 2 : 1) ln_bwd_fused_kernel(TickArgs t) {
  const int li = blockIdx.y + t.ln_li0, p = t.ln_ids[li];
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.b_mb < 0) return;
  const int chunk = blockIdx.x;
  const int r0 = chunk * t.ln_chunk_rows, r1 = min(t.T, r0 + t.ln_chunk_rows);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int dm = s.d_in;
  const uint64_t n = (uint64_t)t.T * dm;
  const AT* du = ws_at<AT>(t, s.dh);
  const AT* gs = emits_skip(s) ? gskip_read<AT>(t, p, d) : nullptr;
  const AT* x = s.from_memory ? mem_at<AT>(t, d.b_mb) : ring_at<AT>(t, s.x_ring, d.b_xslot, n);
  const float* st = ring_at<float>(t, s.stat_ring, d.b_slot, (uint64_t)t.T * 2);
  // dx goes to the previous stage's mailbox; a stage that normalises the memory adds it to the memory gradient of
  // its microbatch (the last such stage runs first and stores); the first stage has no predecessor
  AT* out = s.from_memory ? gmem_at<AT>(t, d) : (p > 0 ? gin_write_prev<AT>(t, p, d) : nullptr);
  const bool accumulate = s.from_memory && !s.mem_first;
  const float gapf = (float)s.gap;
  const bool corr = d.use_delta != 0 && !t.stash;          // a version read from the queue is used as it is
  const int half = WPR == 2 ? (warp & 1) : 0, rw = WPR == 2 ? (warp >> 1) : warp;
  const int cbase = half * NP * 256;                         // first column of this warp's share of a row
  __shared__ float xs[2][4][2][2];                           // [row parity][warp pair][half][s1, s2]
  extern __shared__ float lnred[];                           // [8 warps][2][NP*256] at the end; before that the staged rows
  // Staging (launches of one stage, which have one block or two per SM and few rows in flight otherwise): every row of
  // the block's x, du and skip gradient is requested at once with 16-byte asynchronous copies; the row loop then
  // reads shared memory, so a block pays one round trip to memory instead of one per row.
  const bool stage = t.ln_stage != 0;
  AT* stg = reinterpret_cast<AT*>(lnred);
  const uint64_t rstride = (uint64_t)t.ln_chunk_rows * dm;   // elements of one staged array
  if (stage) {
    const int per_row = dm * (int)sizeof(AT) / 16, total = (r1 - r0) * per_row;
    const bool with_gs = gs != nullptr;
    for (int i = threadIdx.x; i < total; i += 256) {
      const int rr = i / per_row, cc = i - rr * per_row;
      const uint64_t go = ((uint64_t)(r0 + rr) * dm) * sizeof(AT) + (uint64_t)cc * 16, so = ((uint64_t)rr * dm) * sizeof(AT) + (uint64_t)cc * 16;
      cp_async16(reinterpret_cast<char*>(stg) + so, reinterpret_cast<const char*>(x) + go);
      cp_async16(reinterpret_cast<char*>(stg + rstride) + so, reinterpret_cast<const char*>(du) + go);
      if (with_gs) cp_async16(reinterpret_cast<char*>(stg + 2 * rstride) + so, reinterpret_cast<const char*>(gs) + go);
    }
    cp_async_wait_all();
    __syncthreads();
  }
  float gb[NP][8], ag[NP][8], ab[NP][8];
#pragma unroll
  for (int q = 0; q < NP; ++q) {
    const int c = cbase + q * 256 + lane * 8;
#pragma unroll
    for (int k = 0; k < 8; ++k) { gb[q][k] = 0.f; ag[q][k] = 0.f; ab[q][k] = 0.f; }
    if (c < dm) {
      load8<float>((t.stash ? fwd_small<AT>(t, s, d, s.g_off, s.g_soff) : t.a.w + s.g_off) + c, gb[q]);   // stashing: the queued version's gain
      if (corr) { float cv[8]; load8<float>(t.a.delta + s.g_off + c, cv);
#pragma unroll
        for (int k = 0; k < 8; ++k) gb[q][k] = __fsub_rn(gb[q][k], __fmul_rn(gapf, cv[k])); }     // gain - (tau_fwd - tau_bkwd) * delta
    }
  }
  const bool has_gs = gs != nullptr;
  if (!has_gs) gs = du;                                      // keeps the loads below free of branches; the value is not used
  int par = 0;
  for (int r = r0 + rw; r < r1; r += 8 / WPR, par ^= 1) {
    const float mu = st[2 * r], rstd = st[2 * r + 1];
    const uint64_t ro = (uint64_t)r * dm;
    float xh[NP][8], dxh[NP][8];
    float s1 = 0.f, s2 = 0.f;
    // every load of the row is issued before the first use
    float xa[NP][8], da[NP][8], sa[NP][8];
    const uint64_t so = (uint64_t)(r - r0) * dm;
    const AT* xr = stage ? stg + so : x + ro;
    const AT* dr = stage ? stg + rstride + so : du + ro;
    const AT* sr = stage ? (has_gs ? stg + 2 * rstride + so : dr) : gs + ro;
#pragma unroll
    for (int q = 0; q < NP; ++q) {
      const int c = min(cbase + q * 256 + lane * 8, dm - 8);
      load8<AT>(xr + c, xa[q]);
      load8<AT>(dr + c, da[q]);
      load8<AT>(sr + c, sa[q]);
    }
#pragma unroll
    for (int q = 0; q < NP; ++q) {
      const int c = cbase + q * 256 + lane * 8;
      if (c < dm) {
        float (&xv)[8] = xa[q];
        float (&dv)[8] = da[q];
        if (has_gs) {
#pragma unroll
          for (int k = 0; k < 8; ++k) dv[k] = __fadd_rn(dv[k], sa[q][k]); }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          xh[q][k] = (xv[k] - mu) * rstd;
          dxh[q][k] = dv[k] * gb[q][k];
          s1 += dxh[q][k]; s2 += dxh[q][k] * xh[q][k];
          ag[q][k] = __fadd_rn(ag[q][k], __fmul_rn(dv[k], xh[q][k]));
          ab[q][k] = __fadd_rn(ab[q][k], dv[k]);
        }
      } else {
#pragma unroll
        for (int k = 0; k < 8; ++k) { xh[q][k] = 0.f; dxh[q][k] = 0.f; }
      }
    }
    s1 = warp_sum(s1);
    s2 = warp_sum(s2);
    if (WPR == 2) {
      // the slot alternates with the row: a warp that runs ahead writes the other slot, and cannot come back to
      // this one before its partner has passed the next row's barrier
      if (lane == 0) { xs[par][rw][half][0] = s1; xs[par][rw][half][1] = s2; }
      switch (rw) {                                          // barrier numbers as immediates: the kernel reserves five, not all sixteen
        case 0: asm volatile("bar.sync 1, 64;" ::: "memory"); break;
        case 1: asm volatile("bar.sync 2, 64;" ::: "memory"); break;
        case 2: asm volatile("bar.sync 3, 64;" ::: "memory"); break;
        default: asm volatile("bar.sync 4, 64;" ::: "memory"); break;
      }
      s1 = xs[par][rw][0][0] + xs[par][rw][1][0];
      s2 = xs[par][rw][0][1] + xs[par][rw][1][1];
    }
    s1 /= (float)dm;
    s2 /= (float)dm;
    if (out) {
#pragma unroll
      for (int q = 0; q < NP; ++q) {
        const int c = cbase + q * 256 + lane * 8;
        if (c < dm) {
          float o[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) o[k] = rstd * (dxh[q][k] - s1 - xh[q][k] * s2);
          if (accumulate) {
            float prev[8];
            load8<AT>(out + ro + c, prev);
#pragma unroll
            for (int k = 0; k < 8; ++k) o[k] = __fadd_rn(prev[k], round_as<AT>(o[k]));
          }
          store8<AT>(out + ro + c, o);
        }
      }
    }
  }
  if (stage) __syncthreads();                                // the staged rows are not read any more: the buffer takes the partial sums
#pragma unroll
  for (int q = 0; q < NP; ++q)
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      lnred[(warp * 2 + 0) * (NP * 256) + q * 256 + lane * 8 + k] = ag[q][k];
      lnred[(warp * 2 + 1) * (NP * 256) + q * 256 + lane * 8 + k] = ab[q][k];
    }
  __syncthreads();
  float* part = ws_at<float>(t, t.lnred_off) + ((uint64_t)li * t.ln_chunks + chunk) * (2 * (uint64_t)t.max_ln_dim);
  for (int c = threadIdx.x; c < dm; c += 256) {
    float a = 0.f, b2 = 0.f;
    const int hf = WPR == 2 ? c / (NP * 256) : 0, lc = c - hf * (NP * 256);   // the warps that hold this column, in warp order
#pragma unroll
    for (int w = 0; w < 8; ++w)
      if (WPR == 1 || (w & 1) == hf) { a = __fadd_rn(a, lnred[(w * 2 + 0) * (NP * 256) + lc]); b2 = __fadd_rn(b2, lnred[(w * 2 + 1) * (NP * 256) + lc]); }
    part[c] = a;
    part[t.max_ln_dim + c] = b2;
  }
}

// Adds the per-block partials of dgain, dbias.  A block owns 32 columns; warp w adds the partials of chunks w, w + 8, ...
// in ascending order (its loads are issued before the first addition: partials of one column sit a buffer row apart,
// so each is a separate round trip), then the eight per-warp sums are added in warp order: a fixed order.
constexpr int kLnFinCols = 32, kLnFinPer = 16;

__global__ void __launch_bounds__(256) ln_fused_finish_kernel(TickArgs t) {
  const int li = blockIdx.y + t.ln_li0, p = t.ln_ids[li];
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.b_mb < 0) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (blockIdx.x * kLnFinCols >= s.d_in) return;
  const int c = blockIdx.x * kLnFinCols + lane;
  const uint64_t ps = 2 * (uint64_t)t.max_ln_dim;
  const float* part = ws_at<float>(t, t.lnred_off) + (uint64_t)li * t.ln_chunks * ps + (c < s.d_in ? c : 0);
  float a = 0.f, b2 = 0.f;
  for (int k0 = warp; k0 < t.ln_chunks; k0 += 8 * kLnFinPer) {
    float va[kLnFinPer], vb[kLnFinPer];
#pragma unroll
    for (int u = 0; u < kLnFinPer; ++u) {
      const int k = k0 + 8 * u;
      va[u] = k < t.ln_chunks ? part[(uint64_t)k * ps] : 0.f;
      vb[u] = k < t.ln_chunks ? part[(uint64_t)k * ps + t.max_ln_dim] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < kLnFinPer; ++u) if (k0 + 8 * u < t.ln_chunks) { a = __fadd_rn(a, va[u]); b2 = __fadd_rn(b2, vb[u]); }
  }
  __shared__ float red[2][8][kLnFinCols];
  red[0][warp][lane] = a; red[1][warp][lane] = b2;
  __syncthreads();
  if (warp == 0 && c < s.d_in) {
    float ga = 0.f, gb = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) { ga = __fadd_rn(ga, red[0][w][lane]); gb = __fadd_rn(gb, red[1][w][lane]); }
    t.a.grad[s.g_off + c] = d.accum ? __fadd_rn(t.a.grad[s.g_off + c], ga) : ga;
    t.a.grad[s.beta_off + c] = d.accum ? __fadd_rn(t.a.grad[s.beta_off + c], gb) : gb;
  }
}

template <typename AT, int NP, int WPR>
static cudaError_t launch_ln_fused(const TickArgs& t, cudaStream_t stream) {
  size_t smem = (size_t)8 * 2 * NP * 256 * sizeof(float);
  // launches of one stage stage their rows in shared memory when two such blocks fit on an SM
  const size_t stage_bytes = (size_t)3 * t.ln_chunk_rows * t.max_ln_dim * sizeof(AT);
  TickArgs ta = t;
  ta.ln_stage = (t.sel_p >= 0 && stage_bytes <= 100 * 1024 && (t.max_ln_dim * sizeof(AT)) % 16 == 0) ? 1 : 0;
  if (ta.ln_stage) smem = std::max(smem, stage_bytes);
  static size_t attr_bytes = 48 * 1024;
  if (smem > attr_bytes) {
    cudaError_t e = cudaFuncSetAttribute((const void*)ln_bwd_fused_kernel<AT, NP, WPR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_bytes = smem;
  }
  ln_bwd_fused_kernel<AT, NP, WPR><<<dim3(t.ln_chunks, t.n_ln), 256, smem, stream>>>(ta);
  if (!t.defer_finish) ln_fused_finish_kernel<<<dim3((t.max_ln_dim + kLnFinCols - 1) / kLnFinCols, t.n_ln), 256, 0, stream>>>(t);
  return cudaGetLastError();
}

// Embedding gradient: dTable[v] = sqrt(d) * sum over tokens t with id[t] == v (ascending t) of du_total[t].
// A block owns up to kEmbRows vocabulary rows (row v belongs to block v mod the number of blocks, so that the
// frequent ids of a Zipf distribution are spread over the blocks) and a slice of the columns.  It reads the
// microbatch's token ids once (16 consecutive tokens per thread) and compacts the tokens that fall into its rows
// into a list in ascending token order (a prefix sum over the per-thread counts).  A row with few tokens is summed
// by one warp; a row with many by all eight, each adding a contiguous segment of the row's tokens in order, the
// eight partial sums then added in warp order.  Several tokens are gathered at a time so that their loads are in
// flight together.  Every row is written (zeros included) and the order of the additions is fixed.
constexpr int kEmbRows = 256;                         // a block's columns: 32 lanes x CPL (4, 8 or 16) columns per lane
constexpr int kEmbHeavy = 24;                         // tokens per row from which the block shares the row

template <typename AT> __device__ __forceinline__ void load4(const AT* p, float (&v)[4]);
template <> __device__ __forceinline__ void load4<float>(const float* p, float (&v)[4]) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
}
template <> __device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[4]) {
  const uint2 q = *reinterpret_cast<const uint2*>(p);
  const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&q.x));
  const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&q.y));
  v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
}

template <typename AT, int CPL> __device__ __forceinline__ void load_cols(const AT* p, float (&v)[CPL]) {
  if constexpr (CPL == 4) load4<AT>(p, v);
  else {
#pragma unroll
    for (int h = 0; h < CPL / 8; ++h) {
      float w[8];
      load8<AT>(p + 8 * h, w);
#pragma unroll
      for (int e = 0; e < 8; ++e) v[8 * h + e] = w[e];
    }
  }
}

// adds the rows of the tokens sub[k_lo .. k_hi-1] (ascending token order) to acc; 32 / CPL tokens are gathered at a time
template <typename AT, int CPL>
__device__ __forceinline__ void embed_gather(const int32_t* sub, int k_lo, int k_hi, const AT* du, const AT* gs,
                                             int dm, int col, float sc, float (&acc)[CPL]) {
  constexpr int NB = 32 / CPL;
  for (int k = k_lo; k < k_hi; k += NB) {
    uint64_t ro[NB];
#pragma unroll
    for (int u = 0; u < NB; ++u) ro[u] = (uint64_t)sub[min(k + u, k_hi - 1)] * dm + col;   // slots past the end repeat the last token (not added)
    float val[NB][CPL], sv[NB][CPL];
#pragma unroll
    for (int u = 0; u < NB; ++u) load_cols<AT, CPL>(du + ro[u], val[u]);                 // all loads first (no branch between them)
    if (gs) {
#pragma unroll
      for (int u = 0; u < NB; ++u) load_cols<AT, CPL>(gs + ro[u], sv[u]);
#pragma unroll
      for (int u = 0; u < NB; ++u)
#pragma unroll
        for (int e = 0; e < CPL; ++e) val[u][e] = __fadd_rn(val[u][e], sv[u][e]);
    }
#pragma unroll
    for (int u = 0; u < NB; ++u)
      if (k + u < k_hi) {
#pragma unroll
        for (int e = 0; e < CPL; ++e) acc[e] = __fadd_rn(acc[e], __fmul_rn(val[u][e], sc));
      }
  }
}

template <typename AT, int CPL>
__global__ void __launch_bounds__(256) embed_bwd_kernel(TickArgs t) {
  constexpr int kEmbCols = 32 * CPL;
  const int p = t.embed_ids[blockIdx.y];
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.b_mb < 0) return;
  // rows are dealt to the blocks round-robin (row v belongs to block v mod gridDim.x, a power of two): the frequent
  // ids of a Zipf distribution, which sit next to each other at the start of the vocabulary, land in different blocks
  const int nb_shift = __ffs((int)gridDim.x) - 1, nb_mask = (int)gridDim.x - 1, blk = (int)blockIdx.x;
  const int dm = s.d_in;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int col = blockIdx.z * kEmbCols + lane * CPL;        // this lane's columns
  if (blk >= s.vocab || blockIdx.z * kEmbCols >= dm) return;
  const int n_rows = (s.vocab - blk + nb_mask) >> nb_shift;  // rows blk, blk + gridDim.x, ... (at most kEmbRows)
  extern __shared__ int32_t hits[];                          // [T] (token << 8 | row within the block), ascending token
  __shared__ int warp_cnt[2][8];
  __shared__ int row_cnt[kEmbRows], row_start[kEmbRows];
  int32_t* sub = hits + t.T;                                 // [T] token indices grouped by row, ascending inside a row
  float (*part)[kEmbCols] = reinterpret_cast<float (*)[kEmbCols]>(sub + t.T);   // [8][kEmbCols] shared rows: per-warp partial sums
  for (int i = threadIdx.x; i < kEmbRows; i += 256) row_cnt[i] = 0;
  __syncthreads();
  const int32_t* ids = ring_at<int32_t>(t, s.ids_ring, (int)(d.b_mb % s.ids_depth), (uint64_t)t.T);
  int nh = 0;                                                // hits so far (the same value in every thread)
  for (int tb0 = 0; tb0 < t.T; tb0 += 16 * 256) {            // 4096 tokens per pass: thread i takes tokens 16 i .. 16 i + 15
    int rel[16];
    const int tok0 = tb0 + 16 * (int)threadIdx.x;
    if (tok0 + 16 <= t.T && (t.T & 3) == 0) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int4 q = __ldg(reinterpret_cast<const int4*>(ids + tok0) + k);
        rel[4 * k] = q.x; rel[4 * k + 1] = q.y; rel[4 * k + 2] = q.z; rel[4 * k + 3] = q.w;
      }
    } else {
#pragma unroll
      for (int k = 0; k < 16; ++k) rel[k] = tok0 + k < t.T ? __ldg(ids + tok0 + k) : -1;
    }
#pragma unroll
    for (int k = 0; k < 16; ++k) rel[k] = (rel[k] >= 0 && (rel[k] & nb_mask) == blk) ? (rel[k] >> nb_shift) : -1;   // row inside this block
    int mine = 0;
#pragma unroll
    for (int k = 0; k < 16; ++k) mine += (rel[k] >= 0 && rel[k] < kEmbRows) ? 1 : 0;
    // exclusive prefix of the per-thread counts over the block: shuffle scan per warp, then the warp totals
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += v; }
    if (lane == 31) warp_cnt[0][warp] = incl;
    __syncthreads();
    int base = nh, tot = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) { const int cw = warp_cnt[0][w]; if (w < warp) base += cw; tot += cw; }
    int pos = base + incl - mine;
#pragma unroll
    for (int k = 0; k < 16; ++k)
      if (rel[k] >= 0 && rel[k] < kEmbRows) { hits[pos++] = ((tok0 + k) << 8) | rel[k]; atomicAdd(&row_cnt[rel[k]], 1); }
    nh += tot;
    __syncthreads();                                         // warp_cnt is reused by the next pass
  }
  __syncthreads();
  {                                                          // exclusive prefix of the row counts (kEmbRows = 256 = one per thread)
    const int mine = row_cnt[threadIdx.x];
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += v; }
    if (lane == 31) warp_cnt[1][warp] = incl;
    __syncthreads();
    int base = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) if (w < warp) base += warp_cnt[1][w];
    row_start[threadIdx.x] = base + incl - mine;
  }
  __syncthreads();
  // the list, grouped by row: warp w scans it once for each of its rows and copies the matching tokens in order
  for (int rr = warp; rr < n_rows; rr += 8) {
    if (row_cnt[rr] == 0) continue;
    int seen = row_start[rr];
    for (int hb = 0; hb < nh; hb += 32) {
      const int hv = hb + lane < nh ? hits[hb + lane] : -1;
      const bool m = hv >= 0 && (hv & 255) == rr;
      const unsigned bal = __ballot_sync(0xffffffffu, m);
      if (m) sub[seen + __popc(bal & ((1u << lane) - 1u))] = hv >> 8;
      seen += __popc(bal);
    }
  }
  __syncthreads();
  const AT* du = ws_at<AT>(t, s.dh);
  const AT* gs = emits_skip(s) ? gskip_read<AT>(t, p, d) : nullptr;
  const float sc = sqrtf((float)dm);
  const bool col_ok = col < dm;                              // widths are multiples of CPL
  const int col_ld = col_ok ? col : dm - CPL;                  // every lane takes part in the warp-wide steps; lanes beyond the width load a valid address
  // ---- rows with many tokens: the whole block per row
  for (int rr = 0; rr < n_rows; ++rr) {
    const int cnt = row_cnt[rr];
    if (cnt < kEmbHeavy) continue;                           // uniform over the block
    const int k_lo = (int)((long long)cnt * warp / 8), k_hi = (int)((long long)cnt * (warp + 1) / 8);
    float acc[CPL];
#pragma unroll
    for (int e = 0; e < CPL; ++e) acc[e] = 0.f;
    embed_gather<AT, CPL>(sub + row_start[rr], k_lo, k_hi, du, gs, dm, col_ld, sc, acc);
#pragma unroll
    for (int e = 0; e < CPL; ++e) part[warp][lane * CPL + e] = acc[e];
    __syncthreads();
    for (int c = threadIdx.x; c < kEmbCols && blockIdx.z * kEmbCols + c < dm; c += 256) {
      float a = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) a = __fadd_rn(a, part[w][c]);
      float* gp = t.a.grad + s.tab_off + (uint64_t)((rr << nb_shift) + blk) * dm + blockIdx.z * kEmbCols + c;
      *gp = d.accum ? __fadd_rn(*gp, a) : a;
    }
    __syncthreads();
  }
  // ---- the other rows: one warp per row
  for (int rr = warp; rr < n_rows; rr += 8) {
    const int v = (rr << nb_shift) + blk;
    const int cnt = row_cnt[rr];
    if (cnt >= kEmbHeavy) continue;
    float acc[CPL];
#pragma unroll
    for (int e = 0; e < CPL; ++e) acc[e] = 0.f;
    if (cnt > 0) embed_gather<AT, CPL>(sub + row_start[rr], 0, cnt, du, gs, dm, col_ld, sc, acc);
    if (col_ok) {
#pragma unroll
      for (int e = 0; e < CPL; e += 4) {
        float4* gp = reinterpret_cast<float4*>(t.a.grad + s.tab_off + (uint64_t)v * dm + col + e);
        float4 o = make_float4(acc[e], acc[e + 1], acc[e + 2], acc[e + 3]);
        if (d.accum) { const float4 q = *gp; o = make_float4(__fadd_rn(q.x, o.x), __fadd_rn(q.y, o.y), __fadd_rn(q.z, o.z), __fadd_rn(q.w, o.w)); }
        *gp = o;
      }
    }
  }
}

int pre_bwd_launches(const TickArgs& t) {
  const int fin = t.defer_finish ? 0 : 1;
  return (t.any_ln ? (t.ln_fused ? 1 + fin : (t.row_chunks == 1 ? 2 : 2 + fin)) : 0) + (t.any_embed ? 1 : 0);
}

// the LayerNorm finishing pass on its own (grouped over the stages of ln_ids)
int ln_finish_launches(const TickArgs& t) { return t.any_ln && (t.ln_fused || t.row_chunks > 1) ? 1 : 0; }
cudaError_t launch_ln_finish(const TickArgs& t, cudaStream_t stream) {
  if (!t.any_ln) return cudaSuccess;
  if (t.ln_fused) ln_fused_finish_kernel<<<dim3((t.max_ln_dim + kLnFinCols - 1) / kLnFinCols, t.n_ln), 256, 0, stream>>>(t);
  else if (t.row_chunks > 1) ln_param_finish_kernel<<<dim3((t.max_ln_dim + 255) / 256, t.n_ln), 256, 0, stream>>>(t);
  return cudaGetLastError();
}

cudaError_t launch_pre_bwd(const TickArgs& t, int dtype, cudaStream_t stream) {
  cudaError_t e = cudaSuccess;
  if (t.any_ln && t.ln_fused) {
    if (dtype == PM_F32) e = t.max_ln_dim <= 256 ? launch_ln_fused<float, 1, 1>(t, stream) : (t.max_ln_dim <= 512 ? launch_ln_fused<float, 2, 1>(t, stream) : launch_ln_fused<float, 2, 2>(t, stream));
    else e = t.max_ln_dim <= 256 ? launch_ln_fused<__nv_bfloat16, 1, 1>(t, stream) : (t.max_ln_dim <= 512 ? launch_ln_fused<__nv_bfloat16, 2, 1>(t, stream) : launch_ln_fused<__nv_bfloat16, 2, 2>(t, stream));
    if (e != cudaSuccess) return e;
  } else if (t.any_ln) {
    dim3 g1((t.T + 7) / 8, t.n_ln), g2((t.max_ln_dim + kLnCols - 1) / kLnCols, t.row_chunks, t.n_ln);
    if (dtype == PM_F32) { ln_bwd_dx_kernel<float><<<g1, 256, 0, stream>>>(t); ln_bwd_param_kernel<float><<<g2, 256, 0, stream>>>(t); }
    else { ln_bwd_dx_kernel<__nv_bfloat16><<<g1, 256, 0, stream>>>(t); ln_bwd_param_kernel<__nv_bfloat16><<<g2, 256, 0, stream>>>(t); }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (t.row_chunks > 1 && !t.defer_finish) {
      dim3 g3((t.max_ln_dim + 255) / 256, t.n_ln);
      ln_param_finish_kernel<<<g3, 256, 0, stream>>>(t);
      e = cudaGetLastError();
      if (e != cudaSuccess) return e;
    }
  }
  if (t.any_embed) {
    // columns per lane: wide models are cut into column slices so that a row with many tokens is spread over blocks
    const int dm = t.max_embed_dim;
    const int cpl = (dm % 16 == 0 && dm <= 512) ? 16 : (dm % 8 == 0 ? 8 : 4);
    const int slices = (dm + 32 * cpl - 1) / (32 * cpl);
    int n_blk = 1;                                           // a power of two with at most kEmbRows rows per block ...
    while (n_blk * kEmbRows < t.max_vocab) n_blk <<= 1;
    while (n_blk * slices * t.n_embed < 2 * 148 && t.max_vocab / n_blk > 32) n_blk <<= 1;   // ... and enough blocks for a small vocabulary
    dim3 g(n_blk, t.n_embed, slices);
    // the hit list, the same tokens grouped by row, and the per-warp partial sums of a shared row
    const size_t smem = 2 * sizeof(int32_t) * (size_t)t.T + sizeof(float) * 8 * 32 * (size_t)cpl;
    auto go = [&](auto kernel) -> cudaError_t {
      if (smem + 1024 > 48 * 1024) {                         // static shared memory counts towards the default limit
        cudaError_t ea = cudaFuncSetAttribute((const void*)kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (ea != cudaSuccess) return ea;
      }
      kernel<<<g, 256, smem, stream>>>(t);
      return cudaGetLastError();
    };
    if (dtype == PM_F32) e = cpl == 16 ? go(embed_bwd_kernel<float, 16>) : (cpl == 8 ? go(embed_bwd_kernel<float, 8>) : go(embed_bwd_kernel<float, 4>));
    else e = cpl == 16 ? go(embed_bwd_kernel<__nv_bfloat16, 16>) : (cpl == 8 ? go(embed_bwd_kernel<__nv_bfloat16, 8>) : go(embed_bwd_kernel<__nv_bfloat16, 4>));
  }
  return e;
}

}  // namespace pm

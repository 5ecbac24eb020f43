// Multi-head self-attention on the tensor cores (tcgen05 + TMEM + TMA), forward and backward, for
// sequences of 128 tokens and heads of width 64 (bf16).  One CTA of 128 threads handles one (sequence, head):
// thread r owns query row r = TMEM lane r, so the softmax needs no cross-thread traffic.
//
// forward :  S = Q K^T (128x128x64)  ->  p~ = exp(S/8 - rowmax), l = sum p~  ->  O = (bf16(p~) V) / l  (128x64x128);
//            P overwrites Q and K, O the columns of S: 50 KB and 128 tensor-memory columns, four CTAs per SM
// backward:  S = Q K^T, dP = dO V^T  ->  P = softmax, D = rowsum(dP*P), dS = bf16(P*(dP - D)), Pb = bf16(P)
//            dV = Pb^T dO,  dQ = dS K / 8,  dK = dS^T Q / 8   (each 128x64x128)
// Q, K, V, dO arrive by TMA as 128-byte-swizzled [128 rows x 64] tiles; the same tile serves as a K-major
// operand (rows x d_k) or as an MN-major operand (k-rows x 64) depending on the product.  P and dS are
// written by the threads as two [128 x 64-key] swizzled tiles, read K-major (P V, dS K) or MN-major (P^T dO,
// dS^T Q).  exp is the fast ex2-based intrinsic (relative error ~1e-7, far below the bf16 rounding of P).
// Every mbarrier wait is bounded.
#include <string>
#include <vector>

#include "pm_ptx.cuh"
#include "pm_tick.cuh"

namespace pm {

constexpr int AT_S = 128, AT_DK = 64;
constexpr int AT_TILE = AT_S * AT_DK * 2;          // 16 KB: one [128 x 64] bf16 tile
constexpr int AT_FWD_SMEM = 3 * AT_TILE + 1024 + 128;                       // Q|P0, K|P1, V: four CTAs per SM
constexpr int AT_BWD_SMEM = 5 * AT_TILE + 1024 + 128 + 3 * 2 * AT_S * 4;   // Q, K, dO, V|P0|dS0, P1|dS1, row-statistics exchange: two CTAs per SM
constexpr int AT_TMEM_COLS = 256;

// per attention stage: the tensor holding q (the Linear's [q | k | v] output, or for cross-attention the stage's main
// input ring), the tensor holding k, v (the Linear's output), and the incoming-gradient mailbox
enum { AMAP_Q = 0, AMAP_KV = 1, AMAP_DO = 2, AMAPS_PER_STAGE = 3 };

__device__ __forceinline__ void issue_k64(uint32_t tmem_d, uint32_t a, uint32_t b, uint32_t idesc, bool a_kmajor, bool b_kmajor,
                                          uint32_t a_lbo, uint32_t b_lbo, bool acc_first) {
  // one 64-deep k slab: four MMAs of depth 16
#pragma unroll
  for (int k16 = 0; k16 < 4; ++k16) {
    const uint64_t da = a_kmajor ? make_desc(a + k16 * 32, 16, 1024) : make_desc(a + k16 * 2048, a_lbo, 1024);
    const uint64_t db = b_kmajor ? make_desc(b + k16 * 32, 16, 1024) : make_desc(b + k16 * 2048, b_lbo, 1024);
    tc_mma_bf16(tmem_d, da, db, idesc, (acc_first || k16 > 0) ? 1u : 0u);
  }
}

// write 8 consecutive bf16 (16 bytes) of row r, column chunk j (0..15) into a pair of [128 x 64] swizzled tiles
__device__ __forceinline__ void put_chunk(uint8_t* tiles, int r, int j, uint4 v) {
  *reinterpret_cast<uint4*>(tiles + (j >> 3) * AT_TILE + r * 128 + (((j & 7) ^ (r & 7)) << 4)) = v;
}

struct AttnCommon {
  uint32_t sbase; uint8_t* sptr; uint32_t bar_load, bar_mma; uint32_t* tmem_slot; volatile int* abort_flag;
};

__device__ __forceinline__ AttnCommon attn_setup(uint8_t* smem_raw, int tile_bytes, uint32_t tmem_cols = AT_TMEM_COLS) {
  AttnCommon c;
  const uint32_t raw = smem_u32(smem_raw);
  c.sbase = (raw + 1023u) & ~1023u;
  c.sptr = smem_raw + (c.sbase - raw);
  c.bar_load = c.sbase + tile_bytes;
  c.bar_mma = c.bar_load + 8;
  c.tmem_slot = reinterpret_cast<uint32_t*>(c.sptr + tile_bytes + 16);
  c.abort_flag = reinterpret_cast<volatile int*>(c.tmem_slot + 1);
  if (threadIdx.x == 0) {
    mbar_init(c.bar_load, 1);
    mbar_init(c.bar_mma, 1);
    *c.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if ((threadIdx.x >> 5) == 0) {
    __syncwarp();
    tmem_alloc(smem_u32(c.tmem_slot), tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  return c;
}

__device__ __forceinline__ void attn_teardown(const AttnCommon& c, uint32_t tmem_base, uint32_t tmem_cols = AT_TMEM_COLS) {
  tc_fence_before();
  __syncthreads();
  if ((threadIdx.x >> 5) == 0) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, tmem_cols);
  }
}

// all threads: wait for an MMA batch; returns false (uniformly) if any thread gave up
__device__ __forceinline__ bool wait_mma(const AttnCommon& c, uint32_t parity, int* status, int code) {
  bool ok = mbar_wait(c.bar_mma, parity, c.abort_flag, status, code);
  ok = __syncthreads_and(ok);
  tc_fence_after();
  return ok;
}

__device__ __forceinline__ void attn_store32(__nv_bfloat16* dst, const uint32_t (&o)[32], float sc) {
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    float f[8];
#pragma unroll
    for (int e2 = 0; e2 < 8; ++e2) f[e2] = __uint_as_float(o[g * 8 + e2]) * sc;
    *reinterpret_cast<uint4*>(dst + g * 8) = make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
  }
}

__global__ void __launch_bounds__(128, 4) attn_fwd_tc_kernel(TickArgs t, const CUtensorMap* __restrict__ maps, const int* __restrict__ stage_ids, int* status) {
  const int p = stage_ids[blockIdx.y];
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.f_mb < 0 || !feeds_attention(s.post)) return;
  const bool cross = s.post == POST_CROSS_ATTENTION;         // q = the stage's main input; the Linear gave [k | v]
  const int causal = s.causal;
  const int H = s.n_heads, dm = s.d_out_main;
  if ((int)blockIdx.x >= (t.T / AT_S) * H) return;
  const int b = blockIdx.x / H, h = blockIdx.x % H;
  extern __shared__ uint8_t smem_raw[];
  const AttnCommon c = attn_setup(smem_raw, 3 * AT_TILE, 128);
  const uint32_t tmem_base = *c.tmem_slot;
  const uint32_t sQ = c.sbase, sK = sQ + AT_TILE, sV = sK + AT_TILE, sP = sQ;   // P overwrites Q and K once S = Q K^T is done
  uint8_t* pP = c.sptr;
  const CUtensorMap* lm = maps + (size_t)p * AMAPS_PER_STAGE;
  const int r = threadIdx.x;                                 // query row = TMEM lane
  const int warp = r >> 5;

  if (r == 0) {
    const int ko = cross ? 0 : dm;                           // column of k inside the Linear's output
    mbar_arrive_expect_tx(c.bar_load, 3 * AT_TILE);
    tma_load_3d(sQ, lm + AMAP_Q, c.bar_load, h * AT_DK, b * AT_S, cross ? d.f_xslot : d.f_slot);
    tma_load_3d(sK, lm + AMAP_KV, c.bar_load, ko + h * AT_DK, b * AT_S, d.f_slot);
    tma_load_3d(sV, lm + AMAP_KV, c.bar_load, ko + dm + h * AT_DK, b * AT_S, d.f_slot);
    if (mbar_wait(c.bar_load, 0, c.abort_flag, status, 11)) {
      tc_fence_after();
      issue_k64(tmem_base, sQ, sK, make_idesc_mn(128, 128, 0, 0), true, true, 0, 0, false);   // S = Q K^T
      tc_commit(c.bar_mma);
    }
  }
  if (wait_mma(c, 0, status, 12)) {
    const float scale = 0.125f;                              // 1 / sqrt(64)
    const uint32_t lane_addr = tmem_base + ((uint32_t)(warp * 32) << 16);
    float mx = -INFINITY;
#pragma unroll 1
    for (int cc = 0; cc < 4; ++cc) {
      uint32_t v[32];
      tmem_ld32(lane_addr + cc * 32, v);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (!causal || cc * 32 + j <= r) mx = fmaxf(mx, __uint_as_float(v[j]) * scale);
    }
    float l = 0.f;
#pragma unroll 1
    for (int cc = 0; cc < 4; ++cc) {
      uint32_t v[32];
      tmem_ld32(lane_addr + cc * 32, v);
      tmem_ld_wait();
      float e[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        e[j] = (!causal || cc * 32 + j <= r) ? __expf(__uint_as_float(v[j]) * scale - mx) : 0.f;
        l += e[j];
      }
#pragma unroll
      for (int g = 0; g < 4; ++g)
        put_chunk(pP, r, cc * 4 + g, make_uint4(pack_bf16(e[g * 8], e[g * 8 + 1]), pack_bf16(e[g * 8 + 2], e[g * 8 + 3]),
                                                 pack_bf16(e[g * 8 + 4], e[g * 8 + 5]), pack_bf16(e[g * 8 + 6], e[g * 8 + 7])));
    }
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    if (r == 0) {
      tc_fence_after();
      const uint32_t idesc = make_idesc_mn(128, 64, 0, 1);   // O = P V : A = P K-major, B = V MN-major (k = key rows)
      issue_k64(tmem_base, sP, sV, idesc, true, false, 0, 8192, false);            // O takes the columns S has left
      issue_k64(tmem_base, sP + AT_TILE, sV + 4 * 2048, idesc, true, false, 0, 8192, true);
      tc_commit(c.bar_mma);
    }
    if (wait_mma(c, 1, status, 13)) {
      uint32_t o0[32], o1[32];
      tmem_ld32(lane_addr, o0);
      tmem_ld32(lane_addr + 32, o1);
      tmem_ld_wait();
      const float inv = 1.0f / l;
      __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(t.ring + t.st[p + 1].x_ring) + (size_t)d.f_next_xslot * ((size_t)t.T * dm) +
                           (size_t)(b * AT_S + r) * dm + h * AT_DK;
#pragma unroll
      for (int g = 0; g < 8; ++g) {
        const uint32_t* src = g < 4 ? o0 + (g & 3) * 8 : o1 + (g & 3) * 8;
        float f[8];
#pragma unroll
        for (int e2 = 0; e2 < 8; ++e2) f[e2] = __uint_as_float(src[e2]) * inv;
        *reinterpret_cast<uint4*>(out + g * 8) = make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
      }
    }
  }
  attn_teardown(c, tmem_base, 128);
}

// Backward: 256 threads, two per query row (thread r + 128*hf owns keys 64*hf .. 64*hf+63 of row r), two CTAs per SM.
// Shared memory holds five tiles: Q, K, dO, and V | X, where P (two 64-key tiles) overwrites V and X once
// dP = dO V^T is done, and dS overwrites P once dV = P^T dO is done.  The exponentials are computed once and
// stay in registers; dP is read from tensor memory twice (for D, then for dS).  Row statistics of the two halves
// meet in a small exchange buffer.  Accumulators: S at columns 0..127, dP at 128..255; then dV at 0..63,
// dQ at 64..127, dK at 128..191.
constexpr int AT_BWD_THREADS = 256;
constexpr int AT_BWD_TILES = 5;
constexpr int AT_XCH_BYTES = 3 * 2 * AT_S * 4;

__global__ void __launch_bounds__(AT_BWD_THREADS, 2) attn_bwd_tc_kernel(TickArgs t, const CUtensorMap* __restrict__ maps, const int* __restrict__ stage_ids, int* status) {
  const int p = stage_ids[blockIdx.y];
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.b_mb < 0 || !feeds_attention(s.post)) return;
  const bool cross = s.post == POST_CROSS_ATTENTION;
  const int causal = s.causal;
  const int H = s.n_heads, dm = s.d_out_main;
  if ((int)blockIdx.x >= (t.T / AT_S) * H) return;
  const int b = blockIdx.x / H, h = blockIdx.x % H;
  extern __shared__ uint8_t smem_raw[];
  const AttnCommon c = attn_setup(smem_raw, AT_BWD_TILES * AT_TILE);
  const uint32_t tmem_base = *c.tmem_slot;
  const uint32_t sQ = c.sbase, sK = sQ + AT_TILE, sdO = sK + AT_TILE, sV = sdO + AT_TILE, sP = sV;   // P and dS: tiles 3 and 4
  uint8_t* pP = c.sptr + 3 * AT_TILE;
  float* xch = reinterpret_cast<float*>(c.sptr + AT_BWD_TILES * AT_TILE + 128);                      // [3][2][128]
  const CUtensorMap* lm = maps + (size_t)p * AMAPS_PER_STAGE;
  const int tid = threadIdx.x;
  const int r = tid & 127, hf = tid >> 7;                    // query row (TMEM lane), key half
  const int warp = tid >> 5;

  if (tid == 0) {
    const int ko = cross ? 0 : dm;
    mbar_arrive_expect_tx(c.bar_load, 4 * AT_TILE);
    tma_load_3d(sQ, lm + AMAP_Q, c.bar_load, h * AT_DK, b * AT_S, cross ? d.b_xslot : d.b_slot);
    tma_load_3d(sK, lm + AMAP_KV, c.bar_load, ko + h * AT_DK, b * AT_S, d.b_slot);
    tma_load_3d(sV, lm + AMAP_KV, c.bar_load, ko + dm + h * AT_DK, b * AT_S, d.b_slot);
    tma_load_3d(sdO, lm + AMAP_DO, c.bar_load, h * AT_DK, b * AT_S, gin_slot_read(s, d));
    if (mbar_wait(c.bar_load, 0, c.abort_flag, status, 14)) {
      tc_fence_after();
      const uint32_t idesc = make_idesc_mn(128, 128, 0, 0);
      issue_k64(tmem_base, sQ, sK, idesc, true, true, 0, 0, false);          // S  = Q K^T
      issue_k64(tmem_base + 128, sdO, sV, idesc, true, true, 0, 0, false);   // dP = dO V^T
      tc_commit(c.bar_mma);
    }
  }
  if (wait_mma(c, 0, status, 15)) {
    const float scale = 0.125f;
    const uint32_t lane_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t colS = (uint32_t)(hf * 64), colP = 128u + (uint32_t)(hf * 64);
    float e[64];
    float mx = -INFINITY;
#pragma unroll
    for (int cc = 0; cc < 2; ++cc) {
      uint32_t v[32];
      tmem_ld32(lane_addr + colS + cc * 32, v);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        e[cc * 32 + j] = (!causal || hf * 64 + cc * 32 + j <= r) ? __uint_as_float(v[j]) * scale : -INFINITY;
        mx = fmaxf(mx, e[cc * 32 + j]);
      }
    }
    xch[hf * AT_S + r] = mx;
    __syncthreads();
    mx = fmaxf(xch[r], xch[AT_S + r]);
    float l = 0.f;
#pragma unroll
    for (int j = 0; j < 64; ++j) { e[j] = __expf(e[j] - mx); l += e[j]; }
    xch[2 * AT_S + hf * AT_S + r] = l;
    __syncthreads();
    l = xch[2 * AT_S + r] + xch[3 * AT_S + r];
    const float inv = 1.0f / l;
#pragma unroll
    for (int j = 0; j < 64; ++j) e[j] *= inv;                // P (unrounded)
    float D = 0.f;
#pragma unroll
    for (int cc = 0; cc < 2; ++cc) {
      uint32_t g[32];
      tmem_ld32(lane_addr + colP + cc * 32, g);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j) D += __uint_as_float(g[j]) * e[cc * 32 + j];
    }
    xch[4 * AT_S + hf * AT_S + r] = D;
#pragma unroll
    for (int q = 0; q < 8; ++q)
      put_chunk(pP, r, hf * 8 + q, make_uint4(pack_bf16(e[q * 8], e[q * 8 + 1]), pack_bf16(e[q * 8 + 2], e[q * 8 + 3]),
                                               pack_bf16(e[q * 8 + 4], e[q * 8 + 5]), pack_bf16(e[q * 8 + 6], e[q * 8 + 7])));
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    D = xch[4 * AT_S + r] + xch[5 * AT_S + r];
    const uint32_t i_mm = make_idesc_mn(128, 64, 1, 1), i_km = make_idesc_mn(128, 64, 0, 1);
    if (tid == 0) {
      tc_fence_after();
      // dV = P^T dO : A = P read MN-major (m = key, k = query row; the second 64-key group one tile on), B = dO MN-major
      issue_k64(tmem_base, sP, sdO, i_mm, false, false, AT_TILE, 8192, false);
      issue_k64(tmem_base, sP + 4 * 2048, sdO + 4 * 2048, i_mm, false, false, AT_TILE, 8192, true);
      tc_commit(c.bar_mma);
    }
    if (wait_mma(c, 1, status, 16)) {
      // dS = bf16(P * (dP - D)) over the P tiles (dV has finished reading them)
#pragma unroll
      for (int cc = 0; cc < 2; ++cc) {
        uint32_t g[32];
        tmem_ld32(lane_addr + colP + cc * 32, g);
        tmem_ld_wait();
        float ds[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) ds[j] = e[cc * 32 + j] * (__uint_as_float(g[j]) - D);
#pragma unroll
        for (int q = 0; q < 4; ++q)
          put_chunk(pP, r, hf * 8 + cc * 4 + q, make_uint4(pack_bf16(ds[q * 8], ds[q * 8 + 1]), pack_bf16(ds[q * 8 + 2], ds[q * 8 + 3]),
                                                            pack_bf16(ds[q * 8 + 4], ds[q * 8 + 5]), pack_bf16(ds[q * 8 + 6], ds[q * 8 + 7])));
      }
      fence_async_smem();
      tc_fence_before();
      __syncthreads();
      if (tid == 0) {
        tc_fence_after();
        // dQ = dS K : A = dS K-major (k = key), B = K MN-major (k = key rows)
        issue_k64(tmem_base + 64, sP, sK, i_km, true, false, 0, 8192, false);
        issue_k64(tmem_base + 64, sP + AT_TILE, sK + 4 * 2048, i_km, true, false, 0, 8192, true);
        // dK = dS^T Q : A = dS read MN-major (m = key, k = query row), B = Q MN-major
        issue_k64(tmem_base + 128, sP, sQ, i_mm, false, false, AT_TILE, 8192, false);
        issue_k64(tmem_base + 128, sP + 4 * 2048, sQ + 4 * 2048, i_mm, false, false, AT_TILE, 8192, true);
        tc_commit(c.bar_mma);
      }
      // self-attention: the stage's dy buffer receives [dq | dk | dv]; cross-attention: dy = [dk | dv] and dq goes
      // to the previous stage's gradient mailbox.  This thread stores 32 of the 64 head columns.
      const int wz = cross ? 2 * dm : 3 * dm, ko = cross ? 0 : dm;
      __nv_bfloat16* dy = reinterpret_cast<__nv_bfloat16*>(t.ws + s.dy) + (size_t)(b * AT_S + r) * wz + h * AT_DK + hf * 32;
      __nv_bfloat16* dq = cross ? gin_write_prev<__nv_bfloat16>(t, p, d) + (size_t)(b * AT_S + r) * dm + h * AT_DK + hf * 32 : dy;
      {
        uint32_t o[32];
        tc_fence_after();
        tmem_ld32(lane_addr + hf * 32, o);                   // dV while dQ and dK are being computed
        tmem_ld_wait();
        attn_store32(dy + ko + dm, o, 1.0f);
      }
      if (wait_mma(c, 0, status, 17)) {
        uint32_t o[32];
        tmem_ld32(lane_addr + 64 + hf * 32, o);
        tmem_ld_wait();
        attn_store32(dq, o, scale);
        tmem_ld32(lane_addr + 128 + hf * 32, o);
        tmem_ld_wait();
        attn_store32(dy + ko, o, scale);
      }
    }
  }
  attn_teardown(c, tmem_base);
}

// ---- sequences of 256 tokens -------------------------------------------------------------------------------------
// Forward: one CTA of 256 threads per (sequence, head, block of 128 query rows); thread r + 128*hf owns keys
// 128*hf .. 128*hf+127 of query row r.  Shared memory holds K (two tiles), Q, one spare tile and V (two tiles);
// P (four 64-key tiles) overwrites K, Q and the spare once S = Q K^T (128 x 256 x 64) is done.  S occupies tensor
// memory columns 0..255, O = P V (128 x 64 x 256) then lands on columns 0..63.  Under the causal mask the first
// query block only multiplies against the first 128 keys.
constexpr int AT2_S = 256;
constexpr int AT2_FWD_TILES = 6;
constexpr int AT2_FWD_SMEM = AT2_FWD_TILES * AT_TILE + 1024 + 128 + 2 * 2 * AT_S * 4;

__global__ void __launch_bounds__(256, 2) attn_fwd_tc256_kernel(TickArgs t, const CUtensorMap* __restrict__ maps, const int* __restrict__ stage_ids, int* status) {
  const int p = stage_ids[blockIdx.y];
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.f_mb < 0 || !feeds_attention(s.post)) return;
  const bool cross = s.post == POST_CROSS_ATTENTION;
  const int causal = s.causal;
  const int H = s.n_heads, dm = s.d_out_main;
  if ((int)blockIdx.x >= (t.T / AT2_S) * H * 2) return;
  const int qb = blockIdx.x & 1, bh = blockIdx.x >> 1;
  const int b = bh / H, h = bh % H;
  extern __shared__ uint8_t smem_raw[];
  const AttnCommon c = attn_setup(smem_raw, AT2_FWD_TILES * AT_TILE, 256);
  const uint32_t tmem_base = *c.tmem_slot;
  const uint32_t sK = c.sbase, sQ = sK + 2 * AT_TILE, sV = sK + 4 * AT_TILE, sP = sK;
  uint8_t* pP = c.sptr;
  float* xch = reinterpret_cast<float*>(c.sptr + AT2_FWD_TILES * AT_TILE + 128);   // [2][2][128]
  const CUtensorMap* lm = maps + (size_t)p * AMAPS_PER_STAGE;
  const int tid = threadIdx.x;
  const int r = tid & 127, hf = tid >> 7, warp = tid >> 5;
  const int row0 = b * AT2_S;
  const bool half_only = causal && qb == 0;                  // keys 128.. are all masked for the first query block

  if (tid == 0) {
    const int ko = cross ? 0 : dm;
    mbar_arrive_expect_tx(c.bar_load, 5 * AT_TILE);
    tma_load_3d(sQ, lm + AMAP_Q, c.bar_load, h * AT_DK, row0 + qb * AT_S, cross ? d.f_xslot : d.f_slot);
    tma_load_3d(sK, lm + AMAP_KV, c.bar_load, ko + h * AT_DK, row0, d.f_slot);
    tma_load_3d(sK + AT_TILE, lm + AMAP_KV, c.bar_load, ko + h * AT_DK, row0 + AT_S, d.f_slot);
    tma_load_3d(sV, lm + AMAP_KV, c.bar_load, ko + dm + h * AT_DK, row0, d.f_slot);
    tma_load_3d(sV + AT_TILE, lm + AMAP_KV, c.bar_load, ko + dm + h * AT_DK, row0 + AT_S, d.f_slot);
    if (mbar_wait(c.bar_load, 0, c.abort_flag, status, 21)) {
      tc_fence_after();
      issue_k64(tmem_base, sQ, sK, make_idesc_mn(128, half_only ? 128 : 256, 0, 0), true, true, 0, 0, false);   // S = Q K^T
      tc_commit(c.bar_mma);
    }
  }
  if (wait_mma(c, 0, status, 22)) {
    const float scale = 0.125f;
    const uint32_t lane_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t colS = (uint32_t)(hf * 128);
    const int qpos = qb * AT_S + r;                          // position of this query inside its sequence
    const bool dead = half_only && hf == 1;                  // nothing of this half is kept
    float mx = -INFINITY;
    if (!dead) {
#pragma unroll 1
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t v[32];
        tmem_ld32(lane_addr + colS + cc * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (!causal || hf * 128 + cc * 32 + j <= qpos) mx = fmaxf(mx, __uint_as_float(v[j]) * scale);
      }
    }
    xch[hf * AT_S + r] = mx;
    __syncthreads();
    mx = fmaxf(xch[r], xch[AT_S + r]);
    float l = 0.f;
    if (!dead) {
#pragma unroll 1
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t v[32];
        tmem_ld32(lane_addr + colS + cc * 32, v);
        tmem_ld_wait();
        float e[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          e[j] = (!causal || hf * 128 + cc * 32 + j <= qpos) ? __expf(__uint_as_float(v[j]) * scale - mx) : 0.f;
          l += e[j];
        }
#pragma unroll
        for (int g = 0; g < 4; ++g)
          put_chunk(pP, r, hf * 16 + cc * 4 + g, make_uint4(pack_bf16(e[g * 8], e[g * 8 + 1]), pack_bf16(e[g * 8 + 2], e[g * 8 + 3]),
                                                             pack_bf16(e[g * 8 + 4], e[g * 8 + 5]), pack_bf16(e[g * 8 + 6], e[g * 8 + 7])));
      }
    }
    xch[2 * AT_S + hf * AT_S + r] = l;
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    l = xch[2 * AT_S + r] + xch[3 * AT_S + r];
    if (tid == 0) {
      tc_fence_after();
      const uint32_t idesc = make_idesc_mn(128, 64, 0, 1);   // O = P V : A = P K-major, B = V MN-major (k = key rows)
      const int n_slab = half_only ? 2 : 4;
      for (int c4 = 0; c4 < n_slab; ++c4)
        issue_k64(tmem_base, sP + c4 * AT_TILE, sV + (c4 >> 1) * AT_TILE + (c4 & 1) * 4 * 2048, idesc, true, false, 0, 8192, c4 > 0);
      tc_commit(c.bar_mma);
    }
    if (wait_mma(c, 1, status, 23)) {
      uint32_t o[32];
      tmem_ld32(lane_addr + hf * 32, o);
      tmem_ld_wait();
      __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(t.ring + t.st[p + 1].x_ring) + (size_t)d.f_next_xslot * ((size_t)t.T * dm) +
                           (size_t)(row0 + qpos) * dm + h * AT_DK + hf * 32;
      attn_store32(out, o, 1.0f / l);
    }
  }
  attn_teardown(c, tmem_base, 256);
}

// Backward: one CTA of 512 threads per (sequence, head), looping over the two blocks of 128 query rows; thread
// r + 128*qt owns keys 64*qt .. 64*qt+63 of query row r of the current block.  Shared memory: Q_i, dO_i, K (two tiles),
// V (two tiles, reloaded per block) which P (four 64-key tiles) overwrites once dP = dO V^T is done, and dS (four
// tiles).  Tensor memory: columns 0..255 hold S_i, then dP_i, then dQ_i (0..63); 256..383 accumulate dK and
// 384..511 dV over the two query blocks (lane = key inside a block of 128 keys, 64 columns per key block).
constexpr int AT2_BWD_THREADS = 512;
constexpr int AT2_BWD_TILES = 12;
constexpr int AT2_XCH_BYTES = 3 * 4 * AT_S * 4;
constexpr int AT2_BWD_SMEM = AT2_BWD_TILES * AT_TILE + 1024 + 128 + AT2_XCH_BYTES;

__global__ void __launch_bounds__(AT2_BWD_THREADS, 1) attn_bwd_tc256_kernel(TickArgs t, const CUtensorMap* __restrict__ maps, const int* __restrict__ stage_ids, int* status) {
  const int p = stage_ids[blockIdx.y];
  const StageDyn& d = t.dyn[p];
  const StageDev& s = t.st[p];
  if (d.b_mb < 0 || !feeds_attention(s.post)) return;
  const bool cross = s.post == POST_CROSS_ATTENTION;
  const int causal = s.causal;
  const int H = s.n_heads, dm = s.d_out_main;
  if ((int)blockIdx.x >= (t.T / AT2_S) * H) return;
  const int b = blockIdx.x / H, h = blockIdx.x % H;
  extern __shared__ uint8_t smem_raw[];
  const AttnCommon c = attn_setup(smem_raw, AT2_BWD_TILES * AT_TILE, 512);
  const uint32_t tmem_base = *c.tmem_slot;
  const uint32_t sQ = c.sbase, sdO = sQ + AT_TILE, sK = sQ + 2 * AT_TILE, sV = sQ + 4 * AT_TILE, sP = sV, sdS = sQ + 8 * AT_TILE;
  uint8_t* pP = c.sptr + 4 * AT_TILE;
  uint8_t* pdS = c.sptr + 8 * AT_TILE;
  float* xch = reinterpret_cast<float*>(c.sptr + AT2_BWD_TILES * AT_TILE + 128);   // [3][4][128]
  const CUtensorMap* lm = maps + (size_t)p * AMAPS_PER_STAGE;
  const int tid = threadIdx.x;
  const int r = tid & 127, qt = tid >> 7, warp = tid >> 5;
  const uint32_t lane_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
  const int row0 = b * AT2_S;
  const int wz = cross ? 2 * dm : 3 * dm, ko = cross ? 0 : dm;
  const float scale = 0.125f;
  const uint32_t i_s = make_idesc_mn(128, 256, 0, 0), i_mm = make_idesc_mn(128, 64, 1, 1), i_km = make_idesc_mn(128, 64, 0, 1);
  __nv_bfloat16* dyb = reinterpret_cast<__nv_bfloat16*>(t.ws + s.dy);
  uint32_t ph = 0;
  bool ok = true;

#pragma unroll 1
  for (int i = 0; i < 2; ++i) {
    if (tid == 0) {
      mbar_arrive_expect_tx(c.bar_load, (i == 0 ? 6 : 4) * AT_TILE);
      tma_load_3d(sQ, lm + AMAP_Q, c.bar_load, h * AT_DK, row0 + i * AT_S, cross ? d.b_xslot : d.b_slot);
      tma_load_3d(sdO, lm + AMAP_DO, c.bar_load, h * AT_DK, row0 + i * AT_S, gin_slot_read(s, d));
      if (i == 0) {
        tma_load_3d(sK, lm + AMAP_KV, c.bar_load, ko + h * AT_DK, row0, d.b_slot);
        tma_load_3d(sK + AT_TILE, lm + AMAP_KV, c.bar_load, ko + h * AT_DK, row0 + AT_S, d.b_slot);
      }
      tma_load_3d(sV, lm + AMAP_KV, c.bar_load, ko + dm + h * AT_DK, row0, d.b_slot);
      tma_load_3d(sV + AT_TILE, lm + AMAP_KV, c.bar_load, ko + dm + h * AT_DK, row0 + AT_S, d.b_slot);
      if (mbar_wait(c.bar_load, (uint32_t)(i & 1), c.abort_flag, status, 24)) {
        tc_fence_after();
        issue_k64(tmem_base, sQ, sK, i_s, true, true, 0, 0, false);             // S_i = Q_i K^T
        tc_commit(c.bar_mma);
      }
    }
    ok = wait_mma(c, ph, status, 25);
    ph ^= 1u;
    if (!ok) break;
    const int qpos = i * AT_S + r;
    float e[64];
    float mx = -INFINITY;
#pragma unroll
    for (int cc = 0; cc < 2; ++cc) {
      uint32_t v[32];
      tmem_ld32(lane_addr + qt * 64 + cc * 32, v);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        e[cc * 32 + j] = (!causal || qt * 64 + cc * 32 + j <= qpos) ? __uint_as_float(v[j]) * scale : -INFINITY;
        mx = fmaxf(mx, e[cc * 32 + j]);
      }
    }
    xch[qt * AT_S + r] = mx;
    tc_fence_before();
    __syncthreads();                                          // every thread holds its part of S_i: dP_i may take its place
    if (tid == 0) {
      tc_fence_after();
      issue_k64(tmem_base, sdO, sV, i_s, true, true, 0, 0, false);              // dP_i = dO_i V^T
      tc_commit(c.bar_mma);
    }
    mx = fmaxf(fmaxf(xch[r], xch[AT_S + r]), fmaxf(xch[2 * AT_S + r], xch[3 * AT_S + r]));
    float l = 0.f;
#pragma unroll
    for (int j = 0; j < 64; ++j) { e[j] = __expf(e[j] - mx); l += e[j]; }
    xch[4 * AT_S + qt * AT_S + r] = l;
    __syncthreads();
    l = (xch[4 * AT_S + r] + xch[5 * AT_S + r]) + (xch[6 * AT_S + r] + xch[7 * AT_S + r]);
    const float inv = 1.0f / l;
#pragma unroll
    for (int j = 0; j < 64; ++j) e[j] *= inv;                // P (unrounded)
    ok = wait_mma(c, ph, status, 26);                        // dP_i is there, V has been read
    ph ^= 1u;
    if (!ok) break;
    float D = 0.f;
#pragma unroll
    for (int cc = 0; cc < 2; ++cc) {
      uint32_t g[32];
      tmem_ld32(lane_addr + qt * 64 + cc * 32, g);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j) D += __uint_as_float(g[j]) * e[cc * 32 + j];
    }
    xch[8 * AT_S + qt * AT_S + r] = D;
#pragma unroll
    for (int q = 0; q < 8; ++q)
      put_chunk(pP, r, qt * 8 + q, make_uint4(pack_bf16(e[q * 8], e[q * 8 + 1]), pack_bf16(e[q * 8 + 2], e[q * 8 + 3]),
                                               pack_bf16(e[q * 8 + 4], e[q * 8 + 5]), pack_bf16(e[q * 8 + 6], e[q * 8 + 7])));
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    D = (xch[8 * AT_S + r] + xch[9 * AT_S + r]) + (xch[10 * AT_S + r] + xch[11 * AT_S + r]);
    if (tid == 0) {
      tc_fence_after();
      // dV += P^T dO_i per block of 128 keys: A = P read MN-major (m = key, two 64-key tiles; k = query row), B = dO MN-major
      for (int kb = 0; kb < 2; ++kb) {
        issue_k64(tmem_base + 384 + 64 * kb, sP + 2 * kb * AT_TILE, sdO, i_mm, false, false, AT_TILE, 8192, i > 0);
        issue_k64(tmem_base + 384 + 64 * kb, sP + 2 * kb * AT_TILE + 4 * 2048, sdO + 4 * 2048, i_mm, false, false, AT_TILE, 8192, true);
      }
    }
    // dS = bf16(P * (dP - D))
#pragma unroll
    for (int cc = 0; cc < 2; ++cc) {
      uint32_t g[32];
      tmem_ld32(lane_addr + qt * 64 + cc * 32, g);
      tmem_ld_wait();
      float ds[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) ds[j] = e[cc * 32 + j] * (__uint_as_float(g[j]) - D);
#pragma unroll
      for (int q = 0; q < 4; ++q)
        put_chunk(pdS, r, qt * 8 + cc * 4 + q, make_uint4(pack_bf16(ds[q * 8], ds[q * 8 + 1]), pack_bf16(ds[q * 8 + 2], ds[q * 8 + 3]),
                                                           pack_bf16(ds[q * 8 + 4], ds[q * 8 + 5]), pack_bf16(ds[q * 8 + 6], ds[q * 8 + 7])));
    }
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      // dQ_i = dS K : A = dS K-major (k = key), B = K MN-major (k = key rows)
      for (int c4 = 0; c4 < 4; ++c4)
        issue_k64(tmem_base, sdS + c4 * AT_TILE, sK + (c4 >> 1) * AT_TILE + (c4 & 1) * 4 * 2048, i_km, true, false, 0, 8192, c4 > 0);
      // dK += dS^T Q_i per block of 128 keys: A = dS read MN-major, B = Q MN-major
      for (int kb = 0; kb < 2; ++kb) {
        issue_k64(tmem_base + 256 + 64 * kb, sdS + 2 * kb * AT_TILE, sQ, i_mm, false, false, AT_TILE, 8192, i > 0);
        issue_k64(tmem_base + 256 + 64 * kb, sdS + 2 * kb * AT_TILE + 4 * 2048, sQ + 4 * 2048, i_mm, false, false, AT_TILE, 8192, true);
      }
      tc_commit(c.bar_mma);
    }
    ok = wait_mma(c, ph, status, 27);                        // everything issued so far is done
    ph ^= 1u;
    if (!ok) break;
    if (qt < 2) {
      // self-attention: dy = [dq | dk | dv]; cross-attention: dq goes to the previous stage's gradient mailbox
      __nv_bfloat16* dq = (cross ? gin_write_prev<__nv_bfloat16>(t, p, d) + (size_t)(row0 + qpos) * dm
                                 : dyb + (size_t)(row0 + qpos) * wz) + h * AT_DK + qt * 32;
      uint32_t o[32];
      tmem_ld32(lane_addr + qt * 32, o);
      tmem_ld_wait();
      attn_store32(dq, o, scale);
    }
    tc_fence_before();
    __syncthreads();                                          // columns 0..63 and the Q, dO, V tiles are free again
  }
  if (ok) {
    const int kb = qt & 1, which = qt >> 1;                   // which: 0 = dK (scaled), 1 = dV
    __nv_bfloat16* dst = dyb + (size_t)(row0 + kb * AT_S + r) * wz + h * AT_DK + (which ? ko + dm : ko);
    const uint32_t col = 256u + (uint32_t)(which * 128 + kb * 64);
    tc_fence_after();
#pragma unroll
    for (int cc = 0; cc < 2; ++cc) {
      uint32_t o[32];
      tmem_ld32(lane_addr + col + cc * 32, o);
      tmem_ld_wait();
      attn_store32(dst + cc * 32, o, which ? 1.0f : scale);
    }
  }
  attn_teardown(c, tmem_base, 512);
}

// ---- host side --------------------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct AttnPlan {
  const CUtensorMap* d_maps = nullptr;
  const int* d_stage_ids = nullptr;      // the stages that end in attention, in pipeline order
  int n_att = 0;
  int* d_status = nullptr;
  std::vector<int> h_ids;                // host copy of the stage list
};

static uint64_t attn_maps_bytes(int n_stages) { return (uint64_t)n_stages * AMAPS_PER_STAGE * sizeof(CUtensorMap); }
uint64_t attn_workspace_bytes(int n_stages) { return 256 + attn_maps_bytes(n_stages) + ((uint64_t)n_stages * sizeof(int) + 255) / 256 * 256; }

bool attn_tc_supported(int dtype, int S, int dk) { return dtype == PM_BF16 && (S == AT_S || S == AT2_S) && dk == AT_DK; }

pm_status attn_plan_create(AttnPlan** out, const TickArgs& t, const std::vector<StageDev>& st, void* ws_region, cudaStream_t stream, std::string& err) {
  *out = nullptr;
  void* fnp = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t ce = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fnp, cudaEnableDefault, &qres);
  if (ce != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fnp) { err = "cuTensorMapEncodeTiled is not available from this driver"; return PM_ERR_CUDA; }
  EncodeTiledFn fn = (EncodeTiledFn)fnp;
  std::vector<CUtensorMap> maps((size_t)t.P * AMAPS_PER_STAGE);
  memset(maps.data(), 0, maps.size() * sizeof(CUtensorMap));
  std::vector<int> ids;
  for (int p = 0; p < t.P; ++p) if (feeds_attention(st[p].post)) ids.push_back(p);
  const cuuint64_t T = (cuuint64_t)t.T;
  for (int p = 0; p < t.P; ++p) {
    const StageDev& s = st[p];
    if (!feeds_attention(s.post)) continue;
    const bool cross = s.post == POST_CROSS_ATTENTION;
    const cuuint64_t dz = (cuuint64_t)s.lin[0].n_out, dm = (cuuint64_t)s.d_out_main;
    cuuint32_t box[3] = {AT_DK, AT_S, 1}, es[3] = {1, 1, 1};
    auto enc = [&](int which, void* base, cuuint64_t width, cuuint64_t slots, const char* what) -> bool {
      cuuint64_t dims[3] = {width, T, slots}, strides[2] = {width * 2, T * width * 2};
      CUresult r = fn(&maps[(size_t)p * AMAPS_PER_STAGE + which], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides,
                      box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) { err = std::string("cuTensorMapEncodeTiled (attention ") + what + ") failed with code " + std::to_string((int)r); return false; }
      return true;
    };
    if (!enc(AMAP_KV, t.ring + s.lin[0].z_ring, dz, (cuuint64_t)s.depth, "k, v")) return PM_ERR_CUDA;
    if (cross) { if (!enc(AMAP_Q, t.ring + s.x_ring, dm, (cuuint64_t)s.xdepth, "q")) return PM_ERR_CUDA; }
    else if (!enc(AMAP_Q, t.ring + s.lin[0].z_ring, dz, (cuuint64_t)s.depth, "q")) return PM_ERR_CUDA;
    if (!enc(AMAP_DO, t.ws + s.gin, dm, (cuuint64_t)s.gin_depth, "dO")) return PM_ERR_CUDA;
  }
  char* region = (char*)ws_region;
  cudaError_t e = cudaMemcpyAsync(region + 256, maps.data(), maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice, stream);
  if (e == cudaSuccess && !ids.empty()) e = cudaMemcpyAsync(region + 256 + attn_maps_bytes(t.P), ids.data(), ids.size() * sizeof(int), cudaMemcpyHostToDevice, stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(region, 0, 256, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (e == cudaSuccess) e = cudaFuncSetAttribute((const void*)attn_fwd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, AT_FWD_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute((const void*)attn_bwd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, AT_BWD_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute((const void*)attn_fwd_tc256_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, AT2_FWD_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute((const void*)attn_bwd_tc256_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, AT2_BWD_SMEM);
  if (e != cudaSuccess) { err = std::string("attention plan: ") + cudaGetErrorString(e); return PM_ERR_CUDA; }
  AttnPlan* plan = new AttnPlan();
  plan->d_status = (int*)region;
  plan->d_maps = (const CUtensorMap*)(region + 256);
  plan->d_stage_ids = (const int*)(region + 256 + attn_maps_bytes(t.P));
  plan->n_att = (int)ids.size();
  plan->h_ids = ids;
  *out = plan;
  return PM_OK;
}

void attn_plan_destroy(AttnPlan* plan) { delete plan; }
int* attn_status_word(AttnPlan* plan) { return plan ? plan->d_status : nullptr; }

cudaError_t attn_tc_launch(AttnPlan* plan, const TickArgs& t, bool forward, cudaStream_t stream) {
  if (plan->n_att == 0) return cudaSuccess;
  int n_att = plan->n_att;
  const int* ids = plan->d_stage_ids;
  if (t.sel_p >= 0) {                                 // one stage only: its entry of the stage list
    int idx = -1;
    for (int i = 0; i < plan->n_att; ++i) if (plan->h_ids[(size_t)i] == t.sel_p) idx = i;
    if (idx < 0) return cudaSuccess;
    ids += idx; n_att = 1;
  }
  dim3 grid(t.att_blocks, n_att);                     // att_blocks = (sequence, head) pairs
  if (t.att_S == AT2_S) {
    if (forward) attn_fwd_tc256_kernel<<<dim3(2 * t.att_blocks, n_att), 256, AT2_FWD_SMEM, stream>>>(t, plan->d_maps, ids, plan->d_status);
    else attn_bwd_tc256_kernel<<<grid, AT2_BWD_THREADS, AT2_BWD_SMEM, stream>>>(t, plan->d_maps, ids, plan->d_status);
    return cudaGetLastError();
  }
  if (forward) attn_fwd_tc_kernel<<<grid, 128, AT_FWD_SMEM, stream>>>(t, plan->d_maps, ids, plan->d_status);
  else attn_bwd_tc_kernel<<<grid, AT_BWD_THREADS, AT_BWD_SMEM, stream>>>(t, plan->d_maps, ids, plan->d_status);
  return cudaGetLastError();
}

}  // namespace pm

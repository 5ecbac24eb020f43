// bf16 grouped GEMMs of the pipeline on the 5th-generation tensor cores.
//
// One launch covers every stage that is active in this tick.  The kernel is persistent: one CTA per SM
// walks a flattened list of 128x128 output tiles (stage, row tile, column tile).  Operands are staged in
// shared memory in the 128-byte-swizzled canonical layouts, the accumulators live in tensor memory
// (two buffers of 128 lanes x 128 fp32 columns, so the epilogue of one tile overlaps the main loop of
// the next), one elected thread issues tcgen05.mma, and eight warps drain the accumulators with
// tcgen05.ld.
//
//   mode 0 forward  D[T,out]  = x[T,in] * W[out,in]^T      A K-major (TMA), B K-major (TMA, bf16 shadow)
//                   z = bf16(D + b) -> ring,  y = bf16(act(z)) -> next consumer
//   mode 1 dgrad    D[T,in]   = dz[T,out] * Wc[out,in]     A K-major (TMA); the fp32 master weights and the
//                   T2 accumulator delta arrive by TMA in a staging ring, four transform warps turn them
//                   into the MN-major bf16 operand bf16(w - gap*delta) (Section 3.2): the corrected
//                   weights exist only in shared memory
//   mode 2 wgrad    D[out,in] = dz[T,out]^T * x[T,in]      A MN-major (TMA), B MN-major (TMA), fp32 out
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer + TMEM owner, (mode 1: warps 2..5 = operand
// transform,) last eight warps = epilogue (two per TMEM lane group, each taking 64 of the 128 columns).
// Every wait on an mbarrier is bounded; on expiry the CTA records a code in a status word, stops
// issuing work, waits (bounded) for its copies in flight, frees its tensor memory and returns.
#include <cuda.h>

#include <algorithm>

#include "pm_ptx.cuh"
#include "pm_umma.cuh"
#include "pm_update_math.cuh"

namespace pm {

constexpr int TILE_M = 128, TILE_N = 128, TILE_K = 64;     // bf16: 64 elements = one 128-byte swizzle row
constexpr int A_BYTES = TILE_M * TILE_K * 2;               // 16 KB
constexpr int B_BYTES = TILE_N * TILE_K * 2;               // 16 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int STG_HALF_BYTES = TILE_K * TILE_N * 4;        // one fp32 [64 x 128] tile: 32 KB
constexpr int STG_BYTES = 2 * STG_HALF_BYTES;              // w tile + delta tile
constexpr int ACC_COLS = 128, TMEM_COLS = 2 * ACC_COLS;
constexpr int N_EPI_WARPS = 8;

template <int MODE> struct Cfg {                           // MODE 0 forward, 2 wgrad, 1 dgrad against a QUEUED weight version (weight
                                                           // stashing, tau_bkwd = tau_fwd: a plain bf16 operand; the corrected dgrad has kernels of its own)
  static constexpr int kStages = 4;                        // operand ring depth
  static constexpr int kThreads = 32 * (2 + N_EPI_WARPS);
  static constexpr int kOutWarpBytes = 8192;               // per epilogue warp: two boxes of 32 rows x 128 B
  static constexpr int kOutBytes = N_EPI_WARPS * kOutWarpBytes;
  static constexpr int kTileBytes = kStages * STAGE_BYTES + kOutBytes;
  static constexpr int kSmemBytes = kTileBytes + 1024 /*alignment slack*/ + 512 /*barriers*/;
};

enum { MAP_ACT_K = 0, MAP_W_K = 1, MAP_DZ_K = 2, MAP_DZ_MN = 3, MAP_ACT_MN = 4, MAP_W_F32 = 5, MAP_D_F32 = 6,
       MAP_Z_OUT = 7, MAP_Y_OUT = 8, MAP_DX_OUT = 9, MAP_DW_OUT = 10, MAP_W_F32Q = 11, MAP_D_F32Q = 12, MAP_W_F32H = 13, MAP_D_F32H = 14, MAP_W_MN = 15, MAPS_PER_LINEAR = 16 };

// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 128, operand majors as given.
__device__ __forceinline__ uint32_t make_idesc(int a_mn_major, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
         ((uint32_t)(TILE_N >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
}

// forward epilogue for 8 columns: z = bf16(acc + bias), y = bf16(act(z)); the activation is a template parameter so
// that Linears without GELU never pay for erff
template <int ACT>
__device__ __forceinline__ void epi_zy8(const float (&pf)[8], uint8_t* zdst, uint8_t* ydst) {
  float zf[8], yf[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    zf[e] = __bfloat162float(__float2bfloat16_rn(pf[e]));
    yf[e] = ACT == PM_ACT_RELU ? fmaxf(zf[e], 0.0f) : (ACT == PM_ACT_GELU ? act_fwd(zf[e], PM_ACT_GELU) : zf[e]);
  }
  *reinterpret_cast<uint4*>(zdst) = make_uint4(pack_bf16(zf[0], zf[1]), pack_bf16(zf[2], zf[3]), pack_bf16(zf[4], zf[5]), pack_bf16(zf[6], zf[7]));
  *reinterpret_cast<uint4*>(ydst) = make_uint4(pack_bf16(yf[0], yf[1]), pack_bf16(yf[2], yf[3]), pack_bf16(yf[4], yf[5]), pack_bf16(yf[6], yf[7]));
}

// State of one epilogue warp's staging buffer (two slots of 4 KB) across blocks.
struct EpiState {
  bool stored = false;        // a TMA store of this warp may still be reading the staging buffer
  bool prev_both = false;     // the previous block used both slots
  uint32_t slot = 0;          // slot the next single-output block writes
};

// The PipeMare update of one 32-row x 64-column block of a Linear matrix, applied to the weight gradient while it is
// still on chip (r0, r1: the block's accumulators, lane = row).  The block goes through the warp's staging buffer
// once, in the layout the dW store uses, and comes back with a lane owning four consecutive columns of a row, so
// that every access to the master weights, the moments and delta is a full 128-byte line per eight lanes.  Per
// element the arithmetic is upd_one's, i.e. exactly what the stand-alone update kernel does with a stored gradient.
template <int OPT>
__device__ __forceinline__ void epi_update_block(const TickArgs& t, const StageDyn& d, const LinDev& L, int M, int N, int mrow, int nb,
                                                 const uint32_t (&r0)[32], const uint32_t (&r1)[32], uint8_t* obuf, int lane) {
  const uint32_t row_off = (uint32_t)lane * 128, sw = (uint32_t)(lane & 7);
  __syncwarp();                                                   // the previous block's reads of the buffer are done
#pragma unroll
  for (int g = 0; g < 8; ++g) {                                   // two boxes of 32 fp32 columns, 16-byte chunks swizzled by row
    *reinterpret_cast<uint4*>(obuf + row_off + (((uint32_t)g ^ sw) << 4)) = make_uint4(r0[g * 4], r0[g * 4 + 1], r0[g * 4 + 2], r0[g * 4 + 3]);
    *reinterpret_cast<uint4*>(obuf + 4096 + row_off + (((uint32_t)g ^ sw) << 4)) = make_uint4(r1[g * 4], r1[g * 4 + 1], r1[g * 4 + 2], r1[g * 4 + 3]);
  }
  __syncwarp();
  UpdScalars sc;
  sc.alpha = d.alpha; sc.gamma = d.gamma; sc.omg = d.one_minus_gamma; sc.bc1 = d.bc1; sc.bc2 = d.bc2; sc.use_delta = d.use_delta;
  sc.lp_shift = d.lp_shift; sc.rc_shift = d.rc_uslot >= 0 ? d.rc_shift : -1; sc.rc_gap = d.rc_gap;
  const bool need_dl = sc.use_delta || sc.rc_shift >= 0;
  const float beta1 = t.upd_beta1, beta2 = t.upd_beta2, eps = t.upd_eps;
  const float omb1 = __fsub_rn(1.0f, beta1), omb2 = __fsub_rn(1.0f, beta2);
  const int rr0 = lane >> 3, ch = lane & 7;                       // row within a group of four, 16-byte chunk of the 32-column box
  constexpr int NB = 4;                                           // row groups whose loads are in flight together
#pragma unroll 1
  for (int it0 = 0; it0 < 16; it0 += NB) {                        // 16 = 2 boxes x 8 groups of four rows
    float4 g4[NB], w4[NB], m4[NB], s4[NB], d4[NB];
    uint64_t e[NB];
    bool on[NB];
#pragma unroll
    for (int u = 0; u < NB; ++u) {
      const int it = it0 + u, box = it >> 3, rr = (it & 7) * 4 + rr0;
      const int row = mrow + rr, col = nb + box * 32 + ch * 4;
      on[u] = row < M && col < N;
      e[u] = L.w_off + (uint64_t)row * (uint64_t)N + (uint64_t)col;
      g4[u] = *reinterpret_cast<const float4*>(obuf + box * 4096 + rr * 128 + (((uint32_t)ch ^ (uint32_t)(rr & 7)) << 4));
      if (on[u]) {
        w4[u] = __ldcs(reinterpret_cast<const float4*>(t.a.w + e[u]));
        m4[u] = __ldcs(reinterpret_cast<const float4*>(t.a.m + e[u]));
        if (need_dl) d4[u] = __ldcs(reinterpret_cast<const float4*>(t.a.delta + e[u]));
        if (OPT == PM_ADAM) s4[u] = __ldcs(reinterpret_cast<const float4*>(t.a.s + e[u]));
      }
    }
#pragma unroll
    for (int u = 0; u < NB; ++u) {
      if (!on[u]) continue;
      float4 wn;
      wn.x = upd_one<OPT>(g4[u].x, w4[u].x, m4[u].x, s4[u].x, d4[u].x, sc, beta1, beta2, omb1, omb2, eps);
      wn.y = upd_one<OPT>(g4[u].y, w4[u].y, m4[u].y, s4[u].y, d4[u].y, sc, beta1, beta2, omb1, omb2, eps);
      wn.z = upd_one<OPT>(g4[u].z, w4[u].z, m4[u].z, s4[u].z, d4[u].z, sc, beta1, beta2, omb1, omb2, eps);
      wn.w = upd_one<OPT>(g4[u].w, w4[u].w, m4[u].w, s4[u].w, d4[u].w, sc, beta1, beta2, omb1, omb2, eps);
      __stcs(reinterpret_cast<float4*>(t.a.w + e[u]), wn);
      __stcs(reinterpret_cast<float4*>(t.a.m + e[u]), m4[u]);
      if (OPT == PM_ADAM) __stcs(reinterpret_cast<float4*>(t.a.s + e[u]), s4[u]);
      if (sc.use_delta) __stcs(reinterpret_cast<float4*>(t.a.delta + e[u]), d4[u]);
      {
        __nv_bfloat162 lo2 = __floats2bfloat162_rn(wn.x, wn.y), hi2 = __floats2bfloat162_rn(wn.z, wn.w);
        uint2 pk; pk.x = *reinterpret_cast<uint32_t*>(&lo2); pk.y = *reinterpret_cast<uint32_t*>(&hi2);
        *reinterpret_cast<uint2*>(t.upd_lp + (sc.lp_shift + (int64_t)e[u])) = pk;              // re-read by a later forward: default caching
      }
      if (sc.rc_shift >= 0) {                                     // corrected recompute weights of the new version (T2 for recompute)
        const float gp = sc.rc_gap;
        __nv_bfloat162 lo2 = __floats2bfloat162_rn(__fsub_rn(wn.x, __fmul_rn(gp, d4[u].x)), __fsub_rn(wn.y, __fmul_rn(gp, d4[u].y)));
        __nv_bfloat162 hi2 = __floats2bfloat162_rn(__fsub_rn(wn.z, __fmul_rn(gp, d4[u].z)), __fsub_rn(wn.w, __fmul_rn(gp, d4[u].w)));
        uint2 pk; pk.x = *reinterpret_cast<uint32_t*>(&lo2); pk.y = *reinterpret_cast<uint32_t*>(&hi2);
        *reinterpret_cast<uint2*>(t.upd_lp + (sc.rc_shift + (int64_t)e[u])) = pk;
      }
    }
  }
}

// One epilogue block of the forward (MODE 0) or wgrad (MODE 2) GEMM: 32 rows x 64 accumulator columns held in
// r0, r1 go through this warp's swizzled staging buffer to one or two TMA stores (full 128-byte rows; rows and
// columns beyond the tensor are clipped).  Called by a whole warp; lane = row within the block.
// A block with one bf16 output (a Linear without activation) fills one 4 KB slot and alternates slots, so it
// only waits for the store issued two blocks ago; blocks with two outputs (z and y, or 64 fp32 columns) use both.
// bias4: the bias of columns 4*l .. 4*l+3 of the warp's column range in lane l (MODE 0), fetched before the
// accumulator was awaited; bias_lane0: the lane holding this block's first four columns.
template <int MODE>
__device__ __forceinline__ void epi_block(const TickArgs& t, const CUtensorMap* lm, const StageDev& s, const StageDyn& d, const LinDev& L,
                                          int p, int lvl, int N, int mrow, int nb, const uint32_t (&r0)[32], const uint32_t (&r1)[32],
                                          uint8_t* obuf, uint32_t obuf_s, int lane, const float4 bias4, int bias_lane0, EpiState& es,
                                          uint4 (&skq)[8], const __nv_bfloat16* next_skip = nullptr, int next_cols = 0, int yslot_pre = -1) {
  if (MODE == 2 && t.fuse_upd) {                                  // the update is applied here; nothing is stored to the grad arena
    if (t.upd_opt == PM_SGDM) epi_update_block<PM_SGDM>(t, d, L, L.n_out, N, mrow, nb, r0, r1, obuf, lane);
    else epi_update_block<PM_ADAM>(t, d, L, L.n_out, N, mrow, nb, r0, r1, obuf, lane);
    return;
  }
  const uint32_t row_off = (uint32_t)lane * 128;
  const uint32_t sw = (uint32_t)(lane & 7);
  const bool f32out = MODE == 0 && (L.flags & LF_OUT_F32) != 0;
  const bool both = MODE == 2 || f32out || ((L.flags & LF_WRITE_Z) && (L.flags & LF_WRITE_Y));
  if (lane == 0 && es.stored) {                                   // earlier stores must have finished reading what is overwritten
    if (both || es.prev_both) tma_store_wait_read(); else tma_store_wait_read_1();
  }
  __syncwarp();
  const uint32_t so = both ? 0u : es.slot * 4096u;                // slot of a single-output block
  if (MODE == 0) {
    const int act = L.act;
    // A stage that ends in a residual add writes the sum itself: out = bf16(skip + bf16(acc + b)), straight into the
    // next stage's input (or the memory ring); the skip tensor was sent by the emitting stage skip_depth - 1 ticks ago.
    const bool resid = s.post == POST_RESIDUAL;                     // skq: this lane's 64 skip values (see load_skip64)
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      float bb[8];
      {
        const int src = bias_lane0 + 2 * g;
        bb[0] = __shfl_sync(0xffffffffu, bias4.x, src); bb[1] = __shfl_sync(0xffffffffu, bias4.y, src);
        bb[2] = __shfl_sync(0xffffffffu, bias4.z, src); bb[3] = __shfl_sync(0xffffffffu, bias4.w, src);
        bb[4] = __shfl_sync(0xffffffffu, bias4.x, src + 1); bb[5] = __shfl_sync(0xffffffffu, bias4.y, src + 1);
        bb[6] = __shfl_sync(0xffffffffu, bias4.z, src + 1); bb[7] = __shfl_sync(0xffffffffu, bias4.w, src + 1);
      }
      float pf[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) pf[e] = __fadd_rn(__uint_as_float(g < 4 ? r0[(g & 3) * 8 + e] : r1[(g & 3) * 8 + e]), bb[e]);
      if (f32out) {
        // fp32 logits: two 32-column boxes per warp, eight 16-byte chunks per row each
        uint8_t* box = obuf + (g >> 2) * 4096;
        *reinterpret_cast<float4*>(box + row_off + ((((uint32_t)(g & 3) * 2) ^ sw) << 4)) = make_float4(pf[0], pf[1], pf[2], pf[3]);
        *reinterpret_cast<float4*>(box + row_off + ((((uint32_t)(g & 3) * 2 + 1) ^ sw) << 4)) = make_float4(pf[4], pf[5], pf[6], pf[7]);
      } else {
        const uint32_t off = row_off + (((uint32_t)g ^ sw) << 4);
        if (!both) {                                                // one output: no activation (z = y = bf16(acc + b)), or a ReLU whose z is not kept
          if (resid) {
            const uint32_t w[4] = {skq[g].x, skq[g].y, skq[g].z, skq[g].w};
            // the registers just read take the NEXT block's skip values (same row, 64 columns on): their latency hides
            // behind the rest of this block instead of standing in front of the next one
            if (next_skip) skq[g] = 8 * g < next_cols ? __ldg(reinterpret_cast<const uint4*>(next_skip + 8 * g)) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 sk = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[e]));
              pf[2 * e] = __fadd_rn(sk.x, __bfloat162float(__float2bfloat16_rn(pf[2 * e])));
              pf[2 * e + 1] = __fadd_rn(sk.y, __bfloat162float(__float2bfloat16_rn(pf[2 * e + 1])));
            }
          }
          if (act == PM_ACT_RELU) {
#pragma unroll
            for (int e = 0; e < 8; ++e) pf[e] = fmaxf(pf[e], 0.0f);   // bf16(max(x, 0)) = max(bf16(x), 0)
          }
          *reinterpret_cast<uint4*>(obuf + so + off) = make_uint4(pack_bf16(pf[0], pf[1]), pack_bf16(pf[2], pf[3]), pack_bf16(pf[4], pf[5]), pack_bf16(pf[6], pf[7]));
        }
        else if (act == PM_ACT_NONE) epi_zy8<PM_ACT_NONE>(pf, obuf + off, obuf + 4096 + off);
        else if (act == PM_ACT_RELU) epi_zy8<PM_ACT_RELU>(pf, obuf + off, obuf + 4096 + off);
        else epi_zy8<PM_ACT_GELU>(pf, obuf + off, obuf + 4096 + off);
      }
    }
  } else if (MODE == 1) {
#pragma unroll
    for (int g = 0; g < 8; ++g) {                                 // dx: one bf16 output, 64 columns per row
      float f[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(g < 4 ? r0[(g & 3) * 8 + e] : r1[(g & 3) * 8 + e]);
      *reinterpret_cast<uint4*>(obuf + so + row_off + (((uint32_t)g ^ sw) << 4)) =
          make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
    }
  } else {
#pragma unroll
    for (int g = 0; g < 8; ++g) {                                 // two boxes of 32 fp32 columns
      *reinterpret_cast<uint4*>(obuf + row_off + (((uint32_t)g ^ sw) << 4)) = make_uint4(r0[g * 4], r0[g * 4 + 1], r0[g * 4 + 2], r0[g * 4 + 3]);
      *reinterpret_cast<uint4*>(obuf + 4096 + row_off + (((uint32_t)g ^ sw) << 4)) = make_uint4(r1[g * 4], r1[g * 4 + 1], r1[g * 4 + 2], r1[g * 4 + 3]);
    }
  }
  fence_async_smem();                                             // staging writes -> visible to the TMA engine
  __syncwarp();
  if (lane == 0) {
    if (MODE == 0) {
      // (the caller may have formed the slot before it waited for the accumulator: it is the same for every block of a tile)
      const int yslot = yslot_pre >= 0 ? yslot_pre : (lvl < s.n_lin - 1 ? d.f_slot
                        : (s.emit_memory ? (int)(d.f_mb % t.mem_depth) : (p < t.P - 1 ? d.f_next_xslot : (int)(d.tick & 1))));
      if (f32out) {
        tma_store_3d(lm + MAP_Y_OUT, obuf_s, nb, mrow, (int)(d.tick & 1));
        if (nb + 32 < N) tma_store_3d(lm + MAP_Y_OUT, obuf_s + 4096, nb + 32, mrow, (int)(d.tick & 1));
      } else if (!both) {
        if (L.flags & LF_WRITE_Z) tma_store_3d(lm + MAP_Z_OUT, obuf_s + so, nb, mrow, d.f_slot);
        else if (L.flags & LF_WRITE_Y) tma_store_3d(lm + MAP_Y_OUT, obuf_s + so, nb, mrow, yslot);
      } else {
        tma_store_3d(lm + MAP_Z_OUT, obuf_s, nb, mrow, d.f_slot);
        tma_store_3d(lm + MAP_Y_OUT, obuf_s + 4096, nb, mrow, yslot);
      }
    } else if (MODE == 1) {
      // to the previous stage's gradient mailbox, or this stage's own scratch when a pre-op stands before the Linear
      tma_store_3d(lm + MAP_DX_OUT, obuf_s + so, nb, mrow, (lvl == 0 && s.pre == PRE_NONE) ? d.prev_wslot : 0);
    } else {
      if (d.accum) {                                                // a later microbatch of the minibatch: dW adds to the arena
        tma_reduce_add_2d(lm + MAP_DW_OUT, obuf_s, nb, mrow);
        if (nb + 32 < N) tma_reduce_add_2d(lm + MAP_DW_OUT, obuf_s + 4096, nb + 32, mrow);
      } else {
        tma_store_2d(lm + MAP_DW_OUT, obuf_s, nb, mrow);
        if (nb + 32 < N) tma_store_2d(lm + MAP_DW_OUT, obuf_s + 4096, nb + 32, mrow);
      }
    }
    tma_store_commit();
  }
  es.stored = true;
  es.prev_both = both;
  if (!both) es.slot ^= 1u;
}

// The 64 skip-tensor values of row `row`, columns nb .. nb+63, that a residual stage's epilogue adds (zeros outside
// the tensor and for other stages).  Issued before the accumulator is awaited, so the loads overlap the main loop.
__device__ __forceinline__ void load_skip64(const TickArgs& t, const StageDev& s, const StageDyn& d, int N, int row, int nb, uint4 (&skq)[8]) {
  const bool on = s.post == POST_RESIDUAL && row < t.T;
  const __nv_bfloat16* skrow = ws_at<__nv_bfloat16>(t, s.skip_in) + (uint64_t)d.skip_rslot * ((uint64_t)t.T * N) + (uint64_t)row * N + nb;
#pragma unroll
  for (int g = 0; g < 8; ++g)                                       // columns are multiples of 8
    skq[g] = (on && nb + 8 * g < N) ? __ldg(reinterpret_cast<const uint4*>(skrow + 8 * g)) : make_uint4(0u, 0u, 0u, 0u);
}

// dgrad epilogue of a stage whose predecessor's ReLU backward is fused here (StageDev::mask_dx): the 64 values of this
// stage's own stashed input x (row `row`, columns nb .. nb+63, the slot of the microbatch in backward) whose sign
// decides which entries of dx survive: dz_prev = dx where x > 0 (x = ReLU(z_prev) > 0 exactly where z_prev > 0), else 0.
__device__ __forceinline__ uint64_t load_mask_bits64(const TickArgs& t, const StageDev& s, const StageDyn& d, int N, int row, int nb) {
  // Bit i is set where x[row, nb + i] > 0.  The 64 values are compressed to bits BEFORE the accumulator is read from
  // tensor memory, so that they never share the register file with it (the kernel runs at 96 registers per thread).
  if (row >= t.T) return 0ull;
  const __nv_bfloat16* xrow = ring_at<__nv_bfloat16>(t, s.x_ring, d.b_xslot, (uint64_t)t.T * N) + (uint64_t)row * N + nb;
  uint4 xq[8];
#pragma unroll
  for (int g = 0; g < 8; ++g)
    xq[g] = (nb + 8 * g < N) ? __ldg(reinterpret_cast<const uint4*>(xrow + 8 * g)) : make_uint4(0u, 0u, 0u, 0u);
  uint64_t mk = 0ull;
#pragma unroll
  for (int g = 0; g < 8; ++g) {
    const uint32_t w[4] = {xq[g].x, xq[g].y, xq[g].z, xq[g].w};
    uint32_t bits = 0u;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const uint32_t lo = w[e] & 0xFFFFu, hi = w[e] >> 16;
      bits |= (uint32_t)(!(lo & 0x8000u) && (lo & 0x7FFFu) != 0u) << (2 * e);
      bits |= (uint32_t)(!(hi & 0x8000u) && (hi & 0x7FFFu) != 0u) << (2 * e + 1);
    }
    mk |= (uint64_t)bits << (8 * g);
  }
  return mk;
}
// zeroes f[e] where bit e of `bits` is clear
__device__ __forceinline__ void apply_mask8(float (&f)[8], uint32_t bits) {
#pragma unroll
  for (int e = 0; e < 8; ++e) if (!((bits >> e) & 1u)) f[e] = 0.0f;
}

// bias of columns n .. n+3 (zero beyond the tensor); n is a multiple of four
__device__ __forceinline__ float4 load_bias4(const float* bias, int n, int N) {
  return n < N ? __ldg(reinterpret_cast<const float4*>(bias + n)) : make_float4(0.f, 0.f, 0.f, 0.f);
}

// ---- tile walk ---------------------------------------------------------------------------------------
// tile_start[p] .. tile_start[p+1] are the flattened tile ids of stage p for this (mode, level).
struct Tile { int p, m0, n0, M, N, K, n_kb; bool valid; };
// the tile a CTA's slot holds: from the launch's order list, or, in a launch of one stage (its tiles in ascending
// order), from the launch arguments alone, so that no role starts with a chain of dependent global loads
__device__ __forceinline__ int tile_at(const TickArgs& t, const int* __restrict__ order, int slot) {
  return t.sel_p >= 0 ? t.sel_tile0 + slot : order[slot];
}

template <int MODE>
__device__ __forceinline__ Tile decode_tile(const TickArgs& t, const int* __restrict__ tile_start, int lvl, int tile) {
  Tile r;
  const int lo = t.sel_p >= 0 ? t.sel_p : tile_start[t.P + 1 + tile];                           // the stage of this tile: table behind the P + 1 starts
  r.p = lo;
  const StageDyn& d = t.dyn[lo];
  const StageDev& s = t.st[lo];
  r.valid = lvl < s.n_lin && (MODE == 0 ? d.f_mb >= 0 : d.b_mb >= 0) && !(MODE == 1 && lo == 0 && lvl == 0 && s.pre != PRE_EMBED);
  const LinDev& L = s.lin[lvl < s.n_lin ? lvl : 0];
  if (MODE == 0) { r.M = t.T; r.N = L.n_out; r.K = L.n_in; }
  else if (MODE == 1) { r.M = t.T; r.N = L.n_in; r.K = L.n_out; }
  else { r.M = L.n_out; r.N = L.n_in; r.K = t.T; }
  const int tiles_n = (r.N + TILE_N - 1) / TILE_N;
  const int local = tile - (t.sel_p >= 0 ? t.sel_tile0 : tile_start[lo]);
  r.m0 = (local / tiles_n) * TILE_M;
  r.n0 = (local % tiles_n) * TILE_N;
  r.n_kb = (r.K + TILE_K - 1) / TILE_K;
  return r;
}

struct Ring {                       // position in a ring of mbarrier-guarded slots
  int idx; uint32_t phase;
  __device__ __forceinline__ void advance(int n) { if (++idx == n) { idx = 0; phase ^= 1u; } }
};

// ---- the kernel --------------------------------------------------------------------------------------
template <int MODE>
__global__ void __launch_bounds__(Cfg<MODE>::kThreads, 1)
umma_gemm_kernel(TickArgs t, const CUtensorMap* __restrict__ maps, const int* __restrict__ tile_start, const int* __restrict__ order, int n_slots, int lvl, int* status) {
  using C = Cfg<MODE>;
  constexpr int NS = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;                      // swizzled tiles need 1024-byte alignment
  uint8_t* tiles_ptr = smem_raw + (tiles - raw);
  const uint32_t outs = tiles + NS * STAGE_BYTES;                     // epilogue staging for TMA stores
  uint8_t* outs_ptr = tiles_ptr + NS * STAGE_BYTES;
  const uint32_t bars = tiles + C::kTileBytes;
  // barrier block: full[NS] empty[NS] tfull[2] tempty[2], then tmem base word and abort flag
  const uint32_t bar_full = bars, bar_empty = bar_full + 8 * NS, bar_tfull = bar_empty + 8 * NS, bar_tempty = bar_tfull + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tiles_ptr + C::kTileBytes + 8 * (2 * NS + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NS; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar_tfull + 8 * i, 1); mbar_init(bar_tempty + 8 * i, N_EPI_WARPS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    __syncwarp();
    tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      Ring op{0, 0};
      int issued_op = 0;
      bool ok = true;
      for (int slot = blockIdx.x; slot < n_slots && ok; slot += gridDim.x) {
        const int tile = tile_at(t, order, slot);
        if (tile < 0) continue;
        const Tile tl = decode_tile<MODE>(t, tile_start, lvl, tile);
        if (!tl.valid) continue;
        const StageDyn& d = t.dyn[tl.p];
        const CUtensorMap* lm = maps + ((size_t)tl.p * PM_MAX_LINEARS + lvl) * MAPS_PER_LINEAR;
        // dz operand: the dz scratch, or (no activation) the incoming gradient itself, which for the last Linear of a
        // stage without attention is the rotating mailbox slot written during the previous tick
        const StageDev& sd_ = t.st[tl.p];
        const int dz_slot = (bwd_act(sd_.lin[lvl]) == PM_ACT_NONE && lvl == sd_.n_lin - 1 && !feeds_attention(sd_.post)) ? dz_mailbox_slot(t, sd_, d) : 0;
        if (MODE == 0) { tma_prefetch_desc(lm + MAP_ACT_K); tma_prefetch_desc(lm + MAP_W_K); }
        else if (MODE == 1) { tma_prefetch_desc(lm + MAP_DZ_K); tma_prefetch_desc(lm + MAP_W_MN); }
        else { tma_prefetch_desc(lm + MAP_DZ_MN); tma_prefetch_desc(lm + MAP_ACT_MN); }
        for (int kb = 0; kb < tl.n_kb; ++kb) {
          const int k0 = kb * TILE_K;
          if (!mbar_wait(bar_empty + 8 * op.idx, op.phase ^ 1, abort_flag, status, 1)) { ok = false; break; }
          const uint32_t sa = tiles + op.idx * STAGE_BYTES, sb = sa + A_BYTES, fb = bar_full + 8 * op.idx;
          if (MODE == 0) {
            mbar_arrive_expect_tx(fb, A_BYTES + B_BYTES);
            tma_load_3d(sa, lm + MAP_ACT_K, fb, k0, tl.m0, (lvl == 0 && t.st[tl.p].pre == PRE_NONE) ? d.f_xslot : d.f_slot);
            tma_load_3d(sb, lm + MAP_W_K, fb, k0, tl.n0, d.f_vslot);
          } else if (MODE == 1) {
            // dx = dz W_v: dz K-major, the queued version v of the weights (the one the microbatch's forward read) as the
            // MN-major operand, two 64-column runs
            mbar_arrive_expect_tx(fb, A_BYTES + B_BYTES);
            tma_load_3d(sa, lm + MAP_DZ_K, fb, k0, tl.m0, dz_slot);
            tma_load_3d(sb, lm + MAP_W_MN, fb, tl.n0, k0, d.f_vslot);
            tma_load_3d(sb + B_BYTES / 2, lm + MAP_W_MN, fb, tl.n0 + 64, k0, d.f_vslot);
          } else {
            mbar_arrive_expect_tx(fb, A_BYTES + B_BYTES);
            const int slot = (lvl == 0 && t.st[tl.p].pre == PRE_NONE) ? d.b_xslot : d.b_slot;
            tma_load_3d(sa, lm + MAP_DZ_MN, fb, tl.m0, k0, dz_slot);
            tma_load_3d(sa + A_BYTES / 2, lm + MAP_DZ_MN, fb, tl.m0 + 64, k0, dz_slot);
            tma_load_3d(sb, lm + MAP_ACT_MN, fb, tl.n0, k0, slot);
            tma_load_3d(sb + B_BYTES / 2, lm + MAP_ACT_MN, fb, tl.n0 + 64, k0, slot);
          }
          op.advance(NS); ++issued_op;
        }
      }
      if (*abort_flag) {
        // copies already issued still land in this CTA's shared memory: wait for them (bounded) before leaving
        for (int back = 1; back <= NS && back <= issued_op; ++back) {
          const int it = issued_op - back;
          const long long t0 = clock64();
          while (!mbar_try_wait(bar_full + 8 * (it % NS), (uint32_t)(it / NS) & 1u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc = make_idesc(MODE == 2, MODE != 0);
      // K-major: 16 elements = 32 bytes along the swizzled row.  MN-major: 16 k-rows of 128 bytes.
      const uint64_t dba = MODE == 2 ? desc_base(A_BYTES / 2, 1024) : desc_base(16, 1024);
      const uint64_t dbb = MODE == 0 ? desc_base(16, 1024) : desc_base(B_BYTES / 2, 1024);
      const uint32_t ka = MODE == 2 ? 2048 : 32, kb_ = MODE == 0 ? 32 : 2048;
      Ring op{0, 0}, acc{0, 0};
      bool ok = true;
      for (int slot = blockIdx.x; slot < n_slots && ok; slot += gridDim.x) {
        const int tile = tile_at(t, order, slot);
        if (tile < 0) continue;
        const Tile tl = decode_tile<MODE>(t, tile_start, lvl, tile);
        if (!tl.valid) continue;
        if (!mbar_wait(bar_tempty + 8 * acc.idx, acc.phase ^ 1, abort_flag, status, 6)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_acc = tmem_base + (uint32_t)(acc.idx * ACC_COLS);
        for (int kb = 0; kb < tl.n_kb; ++kb) {
          if (!mbar_wait(bar_full + 8 * op.idx, op.phase, abort_flag, status, 2)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = tiles + op.idx * STAGE_BYTES, sb = sa + A_BYTES;
#pragma unroll
          for (int k16 = 0; k16 < TILE_K / 16; ++k16)
            tc_mma_bf16(tmem_acc, desc_at(dba, sa + k16 * ka), desc_at(dbb, sb + k16 * kb_), idesc, (kb > 0 || k16 > 0) ? 1u : 0u);
          tc_commit(bar_empty + 8 * op.idx);      // frees the operand slot once these MMAs have read it
          op.advance(NS);
        }
        if (ok) tc_commit(bar_tfull + 8 * acc.idx);   // accumulator complete
        acc.advance(2);
      }
    }
  } else {
    // ---------------- epilogue: 8 warps, warp%4 = TMEM lane group, two warps per group split the columns ----------------
    // Each warp drains a 32-row x 64-column block, writes it into its own swizzled staging buffer and lets
    // the TMA engine store it (full 128-byte rows; rows and columns beyond the tensor are clipped).
    const int q = warp & 3;
    const int ew = warp - 2;                                          // 0..7
    const int half = ew >> 2;                                         // 0: columns 0..63, 1: columns 64..127
    uint8_t* obuf = outs_ptr + ew * C::kOutWarpBytes;
    const uint32_t obuf_s = outs + ew * C::kOutWarpBytes;
    const uint32_t row_off = (uint32_t)lane * 128;
    const uint32_t sw = (uint32_t)(lane & 7);
    Ring acc{0, 0};
    bool ok = true;
    EpiState es;
    for (int slot = blockIdx.x; slot < n_slots && ok; slot += gridDim.x) {
      const int tile = tile_at(t, order, slot);
      if (tile < 0) continue;
      const Tile tl = decode_tile<MODE>(t, tile_start, lvl, tile);
      if (!tl.valid) continue;
      const StageDyn& d = t.dyn[tl.p];
      const StageDev& s = t.st[tl.p];
      const LinDev& L = s.lin[lvl];
      const CUtensorMap* lm = maps + ((size_t)tl.p * PM_MAX_LINEARS + lvl) * MAPS_PER_LINEAR;
      const int mrow = tl.m0 + q * 32;                                // first row of this warp's block
      const int nb = tl.n0 + half * 64;
      // bias of this warp's 64 columns, four per lane in lanes 0..15, on its way while the accumulator completes
      const float4 bias4 = (MODE == 0 && lane < 16) ? load_bias4(fwd_small<__nv_bfloat16>(t, s, d, L.b_off, L.b_soff), nb + 4 * lane, tl.N) : make_float4(0.f, 0.f, 0.f, 0.f);
      uint4 skq[8];
      if (MODE == 0) load_skip64(t, s, d, tl.N, mrow + lane, nb, skq);
      bool ready = mbar_wait(bar_tfull + 8 * acc.idx, acc.phase, abort_flag, status, 4);
      ready = __all_sync(0xffffffffu, ready);                         // tcgen05.ld needs the whole warp
      if (!ready) { ok = false; break; }
      tc_fence_after();
      uint32_t r0[32], r1[32];
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc.idx * ACC_COLS + half * 64);
      tmem_ld32(taddr, r0);
      tmem_ld32(taddr + 32, r1);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8 * acc.idx);           // the accumulator buffer may be overwritten now
      __syncwarp();
      acc.advance(2);
      if (mrow >= tl.M || nb >= tl.N) continue;                       // nothing of this block is inside the tensor
      epi_block<MODE>(t, lm, s, d, L, tl.p, lvl, tl.N, mrow, nb, r0, r1, obuf, obuf_s, lane, bias4, 0, es, skq);
    }
    if (lane == 0 && es.stored) tma_store_wait_all();                    // global writes complete before the CTA retires
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ---- CTA-pair GEMM: 256 x 256 output tiles ---------------------------------------------------------------
// The same forward / wgrad products on tiles of 256 x 256 computed by two CTAs of a cluster with one
// tcgen05.mma.cta_group::2 per 16 k-columns.  Each CTA loads its 128 rows of A and its 128 of the 256
// columns of B, so a CTA ingests 32 KB per 128x256x64 product: half the shared-memory fill per FLOP of the
// single-CTA kernel, whose tensor pipe waits on that fill.  Roles per CTA: warp 0 = TMA producer (loads
// land in its own shared memory and are counted on the leader's `full` barrier), warp 1 = TMEM owner and,
// in the leader (cluster rank 0), MMA issuer; eight epilogue warps drain the CTA's own 128 accumulator
// rows (two warps per lane group, 128 columns each, in two blocks of 64).  tcgen05.commit arrives on the
// `empty` / `tfull` barriers of both CTAs; the epilogue warps of both arrive on the leader's `tempty`.
// Used when every GEMM of the launch has at least 256 rows and columns; smaller shapes keep the kernel above.
constexpr int P2_TILE = 256;
constexpr int P2_STAGES = 5;
constexpr int P2_ACC_COLS = 256;                                      // two accumulators fill the 512 TMEM columns
constexpr int P2_THREADS = 32 * (2 + N_EPI_WARPS);
constexpr int P2_TILE_BYTES = P2_STAGES * STAGE_BYTES + N_EPI_WARPS * 8192;
constexpr int P2_SMEM_BYTES = P2_TILE_BYTES + 1024 + 512;

template <int MODE>
__device__ __forceinline__ Tile decode_pair_tile(const TickArgs& t, const int* __restrict__ tile_start, int lvl, int tile) {
  Tile r;
  const int lo = t.sel_p >= 0 ? t.sel_p : tile_start[t.P + 1 + tile];                           // the stage of this tile: table behind the P + 1 starts
  r.p = lo;
  const StageDyn& d = t.dyn[lo];
  const StageDev& s = t.st[lo];
  r.valid = lvl < s.n_lin && (MODE == 0 ? d.f_mb >= 0 : d.b_mb >= 0) && !(MODE == 1 && lo == 0 && lvl == 0 && s.pre != PRE_EMBED);
  const LinDev& L = s.lin[lvl < s.n_lin ? lvl : 0];
  if (MODE == 0) { r.M = t.T; r.N = L.n_out; r.K = L.n_in; }
  else if (MODE == 1) { r.M = t.T; r.N = L.n_in; r.K = L.n_out; }
  else { r.M = L.n_out; r.N = L.n_in; r.K = t.T; }
  const int tiles_n = (r.N + P2_TILE - 1) / P2_TILE;
  const int local = tile - (t.sel_p >= 0 ? t.sel_tile0 : tile_start[lo]);
  r.m0 = (local / tiles_n) * P2_TILE;
  r.n0 = (local % tiles_n) * P2_TILE;
  r.n_kb = (r.K + TILE_K - 1) / TILE_K;
  return r;
}

template <int MODE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(P2_THREADS, 1)
umma_pair_gemm_kernel(TickArgs t, const CUtensorMap* __restrict__ maps, const int* __restrict__ tile_start, const int* __restrict__ order, int n_slots, int lvl, int* status) {
  constexpr int NS = P2_STAGES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;                      // same offset in both CTAs of the pair
  uint8_t* tiles_ptr = smem_raw + (tiles - raw);
  const uint32_t outs = tiles + NS * STAGE_BYTES;
  uint8_t* outs_ptr = tiles_ptr + NS * STAGE_BYTES;
  const uint32_t bars = tiles + P2_TILE_BYTES;
  // barrier block: full[NS] (used in the leader) empty[NS] tfull[2] tempty[2] (leader), tmem base word, abort flag
  const uint32_t bar_full = bars, bar_empty = bar_full + 8 * NS, bar_tfull = bar_empty + 8 * NS, bar_tempty = bar_tfull + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tiles_ptr + P2_TILE_BYTES + 8 * (2 * NS + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();                            // 0 = leader
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NS; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar_tfull + 8 * i, 1); mbar_init(bar_tempty + 8 * i, 2 * N_EPI_WARPS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    __syncwarp();
    tmem_alloc_pair(smem_u32(tmem_slot), 2 * P2_ACC_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  cluster_sync_all();                                                 // barriers of both CTAs are initialised
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer (both CTAs) ----------------
    if (lane == 0) {
      Ring op{0, 0};
      int issued_op = 0;
      bool ok = true;
      for (int slot = pair; slot < n_slots && ok; slot += n_pairs) {
        const int tile = tile_at(t, order, slot);
        if (tile < 0) continue;
        const Tile tl = decode_pair_tile<MODE>(t, tile_start, lvl, tile);
        if (!tl.valid) continue;
        const StageDyn& d = t.dyn[tl.p];
        const StageDev& sd_ = t.st[tl.p];
        const CUtensorMap* lm = maps + ((size_t)tl.p * PM_MAX_LINEARS + lvl) * MAPS_PER_LINEAR;
        const int dz_slot = (bwd_act(sd_.lin[lvl]) == PM_ACT_NONE && lvl == sd_.n_lin - 1 && !feeds_attention(sd_.post)) ? dz_mailbox_slot(t, sd_, d) : 0;
        if (MODE == 0) { tma_prefetch_desc(lm + MAP_ACT_K); tma_prefetch_desc(lm + MAP_W_K); }
        else if (MODE == 1) { tma_prefetch_desc(lm + MAP_DZ_K); tma_prefetch_desc(lm + MAP_W_MN); }
        else { tma_prefetch_desc(lm + MAP_DZ_MN); tma_prefetch_desc(lm + MAP_ACT_MN); }
        const int ma = tl.m0 + rank * TILE_M, nbh = tl.n0 + rank * TILE_N;   // this CTA's rows of A and of B
        // ring slots of the operands: read here, once per tile (the k-block loop is the critical path of the kernel and
        // every wait in it makes the compiler re-read what lives in memory)
        const int aslot = (lvl == 0 && sd_.pre == PRE_NONE) ? d.f_xslot : d.f_slot;
        const int xslot = (lvl == 0 && sd_.pre == PRE_NONE) ? d.b_xslot : d.b_slot;
        const int vslot = d.f_vslot;                                  // weight version the forward reads
        const int n_kb = tl.n_kb;
        for (int kb = 0; kb < n_kb; ++kb) {
          const int k0 = kb * TILE_K;
          if (!mbar_wait(bar_empty + 8 * op.idx, op.phase ^ 1, abort_flag, status, 31)) { ok = false; break; }
          const uint32_t sa = tiles + op.idx * STAGE_BYTES, sb = sa + A_BYTES;
          if (rank == 0) mbar_arrive_expect_tx(bar_full + 8 * op.idx, 2 * (A_BYTES + B_BYTES));   // the bytes of both CTAs
          const uint32_t fb = mapa_shared(bar_full + 8 * op.idx, 0);
          if (MODE == 0) {
            tma_load_3d_pair(sa, lm + MAP_ACT_K, fb, k0, ma, aslot);
            tma_load_3d_pair(sb, lm + MAP_W_K, fb, k0, nbh, vslot);
          } else if (MODE == 1) {
            tma_load_3d_pair(sa, lm + MAP_DZ_K, fb, k0, ma, dz_slot);
            tma_load_3d_pair(sb, lm + MAP_W_MN, fb, nbh, k0, vslot);
            tma_load_3d_pair(sb + B_BYTES / 2, lm + MAP_W_MN, fb, nbh + 64, k0, vslot);
          } else {
            tma_load_3d_pair(sa, lm + MAP_DZ_MN, fb, ma, k0, dz_slot);
            tma_load_3d_pair(sa + A_BYTES / 2, lm + MAP_DZ_MN, fb, ma + 64, k0, dz_slot);
            tma_load_3d_pair(sb, lm + MAP_ACT_MN, fb, nbh, k0, xslot);
            tma_load_3d_pair(sb + B_BYTES / 2, lm + MAP_ACT_MN, fb, nbh + 64, k0, xslot);
          }
          op.advance(NS); ++issued_op;
        }
      }
      if (*abort_flag) {
        // copies already issued still land in this CTA's shared memory: give them time (bounded) before leaving
        if (rank == 0) {
          for (int back = 1; back <= NS && back <= issued_op; ++back) {
            const int it = issued_op - back;
            const long long t0 = clock64();
            while (!mbar_try_wait(bar_full + 8 * (it % NS), (uint32_t)(it / NS) & 1u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
          }
        }
        // rank 1's copies are counted on the same barriers of the leader (the expected bytes are those of both CTAs), and
        // no CTA of the pair leaves before the cluster barrier at the end of the kernel, which the leader reaches only
        // after these waits: rank 1 needs no wait of its own
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (leader CTA only) ----------------
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = make_idesc_mn(P2_TILE, P2_TILE, MODE == 2, MODE != 0);
      const uint64_t dba = MODE == 2 ? desc_base(A_BYTES / 2, 1024) : desc_base(16, 1024);
      const uint64_t dbb = MODE == 0 ? desc_base(16, 1024) : desc_base(B_BYTES / 2, 1024);
      const uint32_t ka = MODE == 2 ? 2048 : 32, kb_ = MODE == 0 ? 32 : 2048;
      Ring op{0, 0}, acc{0, 0};
      bool ok = true;
      for (int slot = pair; slot < n_slots && ok; slot += n_pairs) {
        const int tile = tile_at(t, order, slot);
        if (tile < 0) continue;
        const Tile tl = decode_pair_tile<MODE>(t, tile_start, lvl, tile);
        if (!tl.valid) continue;
        if (!mbar_wait(bar_tempty + 8 * acc.idx, acc.phase ^ 1, abort_flag, status, 36)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_acc = tmem_base + (uint32_t)(acc.idx * P2_ACC_COLS);
        for (int kb = 0; kb < tl.n_kb; ++kb) {
          if (!mbar_wait(bar_full + 8 * op.idx, op.phase, abort_flag, status, 32)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = tiles + op.idx * STAGE_BYTES, sb = sa + A_BYTES;
#pragma unroll
          for (int k16 = 0; k16 < TILE_K / 16; ++k16)
            tc_mma_bf16_pair(tmem_acc, desc_at(dba, sa + k16 * ka), desc_at(dbb, sb + k16 * kb_), idesc, (kb > 0 || k16 > 0) ? 1u : 0u);
          tc_commit_pair(bar_empty + 8 * op.idx, 3);                  // frees the operand slot in both CTAs
          op.advance(NS);
        }
        if (ok) tc_commit_pair(bar_tfull + 8 * acc.idx, 3);           // accumulator complete, both CTAs
        acc.advance(2);
      }
    }
  } else {
    // ---------------- epilogue: 8 warps per CTA, warp%4 = TMEM lane group, two warps per group split the 256 columns ----------------
    const int q = warp & 3;
    const int ew = warp - 2;                                          // 0..7
    const int half = ew >> 2;                                         // 0: columns 0..127, 1: columns 128..255
    uint8_t* obuf = outs_ptr + ew * 8192;
    const uint32_t obuf_s = outs + ew * 8192;
    Ring acc{0, 0};
    bool ok = true;
    EpiState es;
    for (int slot = pair; slot < n_slots && ok; slot += n_pairs) {
      const int tile = tile_at(t, order, slot);
      if (tile < 0) continue;
      const Tile tl = decode_pair_tile<MODE>(t, tile_start, lvl, tile);
      if (!tl.valid) continue;
      const StageDyn& d = t.dyn[tl.p];
      const StageDev& s = t.st[tl.p];
      const LinDev& L = s.lin[lvl];
      const CUtensorMap* lm = maps + ((size_t)tl.p * PM_MAX_LINEARS + lvl) * MAPS_PER_LINEAR;
      const int mrow = tl.m0 + rank * TILE_M + q * 32;                // first row of this warp's blocks
      // bias of this warp's 128 columns, four per lane, on its way while the accumulator completes
      const float4 bias4 = MODE == 0 ? load_bias4(fwd_small<__nv_bfloat16>(t, s, d, L.b_off, L.b_soff), tl.n0 + half * 128 + 4 * lane, tl.N) : make_float4(0.f, 0.f, 0.f, 0.f);
      uint4 skq[8];                                                   // skip values of the 64-column block in hand (residual stages)
      if (MODE == 0) load_skip64(t, s, d, tl.N, mrow + lane, tl.n0 + half * 128, skq);
      // ring slot of the forward output, formed while the accumulator completes (the elected lane needs it for its stores)
      const int yslot_pre = MODE != 0 ? -1 : (lvl < s.n_lin - 1 ? d.f_slot
                            : (s.emit_memory ? (int)(d.f_mb % t.mem_depth) : (tl.p < t.P - 1 ? d.f_next_xslot : (int)(d.tick & 1))));
      bool ready = mbar_wait(bar_tfull + 8 * acc.idx, acc.phase, abort_flag, status, 34);
      ready = __all_sync(0xffffffffu, ready);                         // tcgen05.ld needs the whole warp
      if (!ready) { ok = false; break; }
      tc_fence_after();
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {
        const int nb = tl.n0 + half * 128 + c * 64;
        uint32_t r0[32], r1[32];
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc.idx * P2_ACC_COLS + half * 128 + c * 64);
        tmem_ld32(taddr, r0);
        tmem_ld32(taddr + 32, r1);
        tmem_ld_wait();
        if (c == 1) tc_fence_before();
        __syncwarp();
        if (c == 1 && lane == 0) mbar_arrive_cluster(mapa_shared(bar_tempty + 8 * acc.idx, 0));   // this warp has read its part of the accumulator
        __syncwarp();
        if (mrow >= tl.M || nb >= tl.N) continue;                     // nothing of this block is inside the tensor
        // a residual stage: block 0 refills the skip registers with block 1's values as it consumes them
        const __nv_bfloat16* nxt = nullptr;
        if (MODE == 0 && c == 0 && s.post == POST_RESIDUAL && mrow + lane < t.T && nb + 64 < tl.N)
          nxt = ws_at<__nv_bfloat16>(t, s.skip_in) + (uint64_t)d.skip_rslot * ((uint64_t)t.T * tl.N) + (uint64_t)(mrow + lane) * tl.N + nb + 64;
        epi_block<MODE>(t, lm, s, d, L, tl.p, lvl, tl.N, mrow, nb, r0, r1, obuf, obuf_s, lane, bias4, c * 16, es, skq, nxt, tl.N - (nb + 64), yslot_pre);
      }
      acc.advance(2);
    }
    if (lane == 0 && es.stored) tma_store_wait_all();                    // global writes complete before the CTA retires
  }
  tc_fence_before();
  cluster_sync_all();                                                 // no barrier or shared memory of a CTA is touched after this
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 2 * P2_ACC_COLS);
  }
}

// ---- dgrad with reuse of the corrected operand -----------------------------------------------------------
// D[T,in] = dz[T,out] * Wc[out,in].  With thousands of rows the fp32 w and delta tiles (64 KB per k-block) and
// their conversion would be repeated for every 128-row tile; here one CTA computes up to four 128-row tiles
// against the SAME converted tile: per k-block the staging ring receives w and delta once, the transform warps
// write bf16(w - gap*delta) once, and the MMA warp issues one product per row tile into its own accumulator
// (4 x 128 TMEM columns).  Traffic per 128x128x64 product drops from 80 KB to 32 KB.
constexpr int DG_MG = 4;                                   // row tiles per B tile
constexpr int DG_NA = 3, DG_NB = 2, DG_NG = 2;             // A ring, B (converted) ring, fp32 staging ring
constexpr int DG_EPI_WARPS = 4;
constexpr int DG_XF_WARPS = 8;                             // transform warps: 32 of the 64 k-rows per half
constexpr int DG_THREADS = 32 * (2 + DG_XF_WARPS + DG_EPI_WARPS);
constexpr int DG_TILE_BYTES = DG_NG * STG_BYTES + DG_NB * B_BYTES + DG_NA * A_BYTES + DG_EPI_WARPS * 4096;
constexpr int DG_SMEM_BYTES = DG_TILE_BYTES + 1024 + 512;

struct DgTile { int p, m0, n0, n_m, M, N, K, n_kb; bool valid; };

__device__ __forceinline__ DgTile decode_dgrad(const TickArgs& t, const int* __restrict__ tile_start, int lvl, int tile) {
  DgTile r;
  const int lo = t.sel_p >= 0 ? t.sel_p : tile_start[t.P + 1 + tile];                           // the stage of this tile: table behind the P + 1 starts
  r.p = lo;
  const StageDyn& d = t.dyn[lo];
  const StageDev& s = t.st[lo];
  r.valid = lvl < s.n_lin && d.b_mb >= 0 && !(lo == 0 && lvl == 0 && s.pre != PRE_EMBED);
  const LinDev& L = s.lin[lvl < s.n_lin ? lvl : 0];
  r.M = t.T; r.N = L.n_in; r.K = L.n_out;
  const int tiles_n = (r.N + TILE_N - 1) / TILE_N;
  const int tiles_m = (r.M + TILE_M - 1) / TILE_M;
  const int local = tile - (t.sel_p >= 0 ? t.sel_tile0 : tile_start[lo]);
  const int mg = local / tiles_n;
  r.m0 = mg * DG_MG * TILE_M;
  r.n0 = (local % tiles_n) * TILE_N;
  r.n_m = min(DG_MG, tiles_m - mg * DG_MG);
  r.n_kb = (r.K + TILE_K - 1) / TILE_K;
  return r;
}

__global__ void __launch_bounds__(DG_THREADS, 1)
umma_dgrad_kernel(TickArgs t, const CUtensorMap* __restrict__ maps, const int* __restrict__ tile_start, const int* __restrict__ order, int n_slots, int lvl, int* status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t stg = base;                                          // [DG_NG][w 32 KB | delta 32 KB]
  const uint32_t sB = stg + DG_NG * STG_BYTES;                        // [DG_NB][16 KB] converted operand
  const uint32_t sA = sB + DG_NB * B_BYTES;                           // [DG_NA][16 KB] dz tiles
  const uint32_t sO = sA + DG_NA * A_BYTES;                           // [4][4 KB] epilogue staging
  uint8_t* stg_ptr = base_ptr;
  uint8_t* sB_ptr = base_ptr + DG_NG * STG_BYTES;
  uint8_t* sO_ptr = sB_ptr + DG_NB * B_BYTES + DG_NA * A_BYTES;
  const uint32_t bars = base + DG_TILE_BYTES;
  const uint32_t bar_sfull = bars, bar_sempty = bar_sfull + 8 * DG_NG, bar_bfull = bar_sempty + 8 * DG_NG,
                 bar_bempty = bar_bfull + 8 * DG_NB, bar_afull = bar_bempty + 8 * DG_NB, bar_aempty = bar_afull + 8 * DG_NA,
                 bar_tfull = bar_aempty + 8 * DG_NA, bar_tempty = bar_tfull + 8;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + DG_TILE_BYTES + 8 * (2 * DG_NG + 2 * DG_NB + 2 * DG_NA + 2));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < DG_NG; ++i) { mbar_init(bar_sfull + 8 * i, 1); mbar_init(bar_sempty + 8 * i, DG_XF_WARPS); }
    for (int i = 0; i < DG_NB; ++i) { mbar_init(bar_bfull + 8 * i, DG_XF_WARPS); mbar_init(bar_bempty + 8 * i, 1); }
    for (int i = 0; i < DG_NA; ++i) { mbar_init(bar_afull + 8 * i, 1); mbar_init(bar_aempty + 8 * i, 1); }
    mbar_init(bar_tfull, 1);
    mbar_init(bar_tempty, DG_EPI_WARPS);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    __syncwarp();
    tmem_alloc(smem_u32(tmem_slot), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    // Two cursors walk the same (tile, k-block) sequence: the fp32 staging loads run one k-block ahead of the dz
    // loads, so that the load + conversion of the next weight tile overlaps the products of the current one.
    if (lane == 0) {
      struct Cursor { int tile, kb; DgTile tl; bool done; };
      auto seek = [&](Cursor& c) {                                    // move to the next valid tile at or after c.tile
        for (; c.tile < n_slots; c.tile += gridDim.x) {              // c.tile walks the slots of the order array
          const int tile = tile_at(t, order, c.tile);
          if (tile < 0) continue;
          c.tl = decode_dgrad(t, tile_start, lvl, tile);
          if (c.tl.valid) { c.kb = 0; c.done = false; return; }
        }
        c.done = true;
      };
      auto step = [&](Cursor& c) { if (++c.kb >= c.tl.n_kb) { c.tile += gridDim.x; seek(c); } };
      Cursor cs{(int)blockIdx.x, 0, DgTile{}, false}, ca{(int)blockIdx.x, 0, DgTile{}, false};
      seek(cs); seek(ca);
      Ring sg{0, 0}, ar{0, 0};
      int issued_sg = 0, issued_a = 0;
      bool ok = true;
      auto issue_staging = [&](const Cursor& c) {
        const StageDyn& d = t.dyn[c.tl.p];
        const CUtensorMap* lm = maps + ((size_t)c.tl.p * PM_MAX_LINEARS + lvl) * MAPS_PER_LINEAR;
        if (!mbar_wait(bar_sempty + 8 * sg.idx, sg.phase ^ 1, abort_flag, status, 21)) { ok = false; return; }
        const uint32_t sw = stg + sg.idx * STG_BYTES, fb = bar_sfull + 8 * sg.idx;
        const bool corr = d.use_delta != 0;
        mbar_arrive_expect_tx(fb, corr ? STG_BYTES : STG_HALF_BYTES);
        tma_load_2d(sw, lm + MAP_W_F32, fb, c.tl.n0, c.kb * TILE_K);
        if (corr) tma_load_2d(sw + STG_HALF_BYTES, lm + MAP_D_F32, fb, c.tl.n0, c.kb * TILE_K);
        sg.advance(DG_NG); ++issued_sg;
      };
      if (!cs.done) { issue_staging(cs); step(cs); }
      while (!ca.done && ok) {
        if (!cs.done) { issue_staging(cs); step(cs); if (!ok) break; }
        const StageDyn& d = t.dyn[ca.tl.p];
        const StageDev& sd_ = t.st[ca.tl.p];
        const CUtensorMap* lm = maps + ((size_t)ca.tl.p * PM_MAX_LINEARS + lvl) * MAPS_PER_LINEAR;
        const int dz_slot = (bwd_act(sd_.lin[lvl]) == PM_ACT_NONE && lvl == sd_.n_lin - 1 && !feeds_attention(sd_.post)) ? dz_mailbox_slot(t, sd_, d) : 0;
        for (int mi = 0; mi < ca.tl.n_m; ++mi) {
          if (!mbar_wait(bar_aempty + 8 * ar.idx, ar.phase ^ 1, abort_flag, status, 22)) { ok = false; break; }
          const uint32_t fa = bar_afull + 8 * ar.idx;
          mbar_arrive_expect_tx(fa, A_BYTES);
          tma_load_3d(sA + ar.idx * A_BYTES, lm + MAP_DZ_K, fa, ca.kb * TILE_K, ca.tl.m0 + mi * TILE_M, dz_slot);
          ar.advance(DG_NA); ++issued_a;
        }
        step(ca);
      }
      if (*abort_flag) {
        for (int back = 1; back <= DG_NG && back <= issued_sg; ++back) {
          const int it = issued_sg - back;
          const long long t0 = clock64();
          while (!mbar_try_wait(bar_sfull + 8 * (it % DG_NG), (uint32_t)(it / DG_NG) & 1u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        }
        for (int back = 1; back <= DG_NA && back <= issued_a; ++back) {
          const int it = issued_a - back;
          const long long t0 = clock64();
          while (!mbar_try_wait(bar_afull + 8 * (it % DG_NA), (uint32_t)(it / DG_NA) & 1u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc = make_idesc(0, 1);
      const uint64_t dba = desc_base(16, 1024), dbb = desc_base(B_BYTES / 2, 1024);
      Ring br{0, 0}, ar{0, 0};
      uint32_t tphase = 0;
      bool ok = true;
      for (int slot = blockIdx.x; slot < n_slots && ok; slot += gridDim.x) {
        const int tile = tile_at(t, order, slot);
        if (tile < 0) continue;
        const DgTile tl = decode_dgrad(t, tile_start, lvl, tile);
        if (!tl.valid) continue;
        if (!mbar_wait(bar_tempty, tphase ^ 1, abort_flag, status, 23)) { ok = false; break; }
        tc_fence_after();
        for (int kb = 0; kb < tl.n_kb && ok; ++kb) {
          if (!mbar_wait(bar_bfull + 8 * br.idx, br.phase, abort_flag, status, 24)) { ok = false; break; }
          const uint32_t sb = sB + br.idx * B_BYTES;
          for (int mi = 0; mi < tl.n_m; ++mi) {
            if (!mbar_wait(bar_afull + 8 * ar.idx, ar.phase, abort_flag, status, 25)) { ok = false; break; }
            tc_fence_after();
            const uint32_t sa = sA + ar.idx * A_BYTES;
#pragma unroll
            for (int k16 = 0; k16 < TILE_K / 16; ++k16)
              tc_mma_bf16(tmem_base + (uint32_t)(mi * ACC_COLS), desc_at(dba, sa + k16 * 32), desc_at(dbb, sb + k16 * 2048),
                          idesc, (kb > 0 || k16 > 0) ? 1u : 0u);
            tc_commit(bar_aempty + 8 * ar.idx);
            ar.advance(DG_NA);
          }
          if (ok) tc_commit(bar_bempty + 8 * br.idx);
          br.advance(DG_NB);
        }
        if (ok) tc_commit(bar_tfull);
        tphase ^= 1;
      }
    }
  } else if (warp < 2 + DG_XF_WARPS) {
    // ---------------- operand transform: fp32 w, delta in staging -> bf16(w - gap*delta), MN-major ----------------
    const int tt = (threadIdx.x - 64) & 127;                          // position within a group of four warps
    const int hsel = (threadIdx.x - 64) >> 7;                         // which half of the 64 k-rows this group converts
    const int c = tt & 15, rb = tt >> 4;
    const uint32_t dst_in_tile = (uint32_t)(c >> 3) * (B_BYTES / 2) + (uint32_t)rb * 128 + (uint32_t)(((c & 7) ^ rb) << 4);
    const uint32_t src_in_tile = (uint32_t)rb * (TILE_N * 4) + (uint32_t)c * 32;
    Ring br{0, 0}, sg{0, 0};
    bool ok = true;
    for (int slot = blockIdx.x; slot < n_slots && ok; slot += gridDim.x) {
      const int tile = tile_at(t, order, slot);
      if (tile < 0) continue;
      const DgTile tl = decode_dgrad(t, tile_start, lvl, tile);
      if (!tl.valid) continue;
      const float gapf = (float)t.st[tl.p].gap;
      const bool corr = t.dyn[tl.p].use_delta != 0;
      for (int kb = 0; kb < tl.n_kb; ++kb) {
        bool go = mbar_wait(bar_sfull + 8 * sg.idx, sg.phase, abort_flag, status, 26);
        go = go && mbar_wait(bar_bempty + 8 * br.idx, br.phase ^ 1, abort_flag, status, 27);
        go = __all_sync(0xffffffffu, go);
        if (!go) { ok = false; break; }
        const uint8_t* src = stg_ptr + sg.idx * STG_BYTES + src_in_tile;
        uint8_t* dst = sB_ptr + br.idx * B_BYTES + dst_in_tile;
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          const int j = hsel * 4 + jj;
          const float4 w0 = *reinterpret_cast<const float4*>(src + j * 8 * TILE_N * 4);
          const float4 w1 = *reinterpret_cast<const float4*>(src + j * 8 * TILE_N * 4 + 16);
          float v[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
          if (corr) {
            const float4 d0 = *reinterpret_cast<const float4*>(src + STG_HALF_BYTES + j * 8 * TILE_N * 4);
            const float4 d1 = *reinterpret_cast<const float4*>(src + STG_HALF_BYTES + j * 8 * TILE_N * 4 + 16);
            const float dd[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = __fsub_rn(v[e], __fmul_rn(gapf, dd[e]));   // w - (tau_fwd - tau_bkwd) * delta
          }
          *reinterpret_cast<uint4*>(dst + j * 1024) =
              make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) { mbar_arrive(bar_bfull + 8 * br.idx); mbar_arrive(bar_sempty + 8 * sg.idx); }
        br.advance(DG_NB); sg.advance(DG_NG);
      }
    }
  } else {
    // ---------------- epilogue: one warp per TMEM lane group, 64 columns at a time through a swizzled staging buffer ----------------
    const int q = warp & 3;
    const int ew = warp - 2 - DG_XF_WARPS;
    uint8_t* obuf = sO_ptr + ew * 4096;
    const uint32_t obuf_s = sO + ew * 4096;
    const uint32_t row_off = (uint32_t)lane * 128, sw = (uint32_t)(lane & 7);
    uint32_t tphase = 0;
    bool ok = true, stored = false;
    for (int slot = blockIdx.x; slot < n_slots && ok; slot += gridDim.x) {
      const int tile = tile_at(t, order, slot);
      if (tile < 0) continue;
      const DgTile tl = decode_dgrad(t, tile_start, lvl, tile);
      if (!tl.valid) continue;
      const StageDyn& d = t.dyn[tl.p];
      const StageDev& s = t.st[tl.p];
      const CUtensorMap* lm = maps + ((size_t)tl.p * PM_MAX_LINEARS + lvl) * MAPS_PER_LINEAR;
      bool ready = mbar_wait(bar_tfull, tphase, abort_flag, status, 28);
      ready = __all_sync(0xffffffffu, ready);
      if (!ready) { ok = false; break; }
      tc_fence_after();
      const int dslot = (lvl == 0 && s.pre == PRE_NONE) ? d.prev_wslot : 0;
      const bool masked = lvl == 0 && s.mask_dx != 0;              // the previous stage's ReLU backward is applied here
      for (int mi = 0; mi < tl.n_m; ++mi) {
        const int mrow = tl.m0 + mi * TILE_M + q * 32;
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
          const int nb = tl.n0 + half * 64;
          uint32_t r0[32], r1[32];
          const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(mi * ACC_COLS + half * 64);
          const uint64_t mk = masked ? load_mask_bits64(t, s, d, tl.N, mrow + lane, nb) : ~0ull;
          tmem_ld32(taddr, r0);
          tmem_ld32(taddr + 32, r1);
          tmem_ld_wait();
          if (mrow >= tl.M || nb >= tl.N) continue;
          if (lane == 0 && stored) tma_store_wait_read();
          __syncwarp();
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            float f[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(g < 4 ? r0[(g & 3) * 8 + e] : r1[(g & 3) * 8 + e]);
            if (masked) apply_mask8(f, (uint32_t)(mk >> (8 * g)) & 0xFFu);
            *reinterpret_cast<uint4*>(obuf + row_off + (((uint32_t)g ^ sw) << 4)) =
                make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) { tma_store_3d(lm + MAP_DX_OUT, obuf_s, nb, mrow, dslot); tma_store_commit(); }
          stored = true;
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty);                         // all four accumulators have been read
      tphase ^= 1;
    }
    if (lane == 0 && stored) tma_store_wait_all();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// ---- dgrad on CTA pairs ------------------------------------------------------------------------------------
// The same product and the same on-the-fly correction on tiles of 256 rows x 256 columns per CTA pair
// (tcgen05.mma.cta_group::2, M = 256, N = 256: the width at which the tensor pipe runs at its full rate; an MMA
// costs at least ~84 cycles whatever its width, so 128-column tiles cap it at 77 %).  Each CTA stages the fp32 w
// and delta of ITS 128 columns in slabs of 32 k-rows (2 x 16 KB per slab, three slabs in flight), converts them to
// bf16(w - gap*delta) in its own shared memory, and loads its 128 rows of dz.  Up to two 256-row tiles share one
// converted tile (then the two 256-column accumulators fill the tensor memory and the epilogue drains the first
// while the MMAs of the second finish; the next group's MMAs start on an accumulator as soon as it is drained);
// a Linear with few tiles takes one row tile per group and alternates between the two accumulators.
// Barriers: staging (sfull / sempty) is local to a CTA; the converted tile (bfull) and the dz tiles (afull) are
// counted in the leader, which issues the MMAs; tcgen05.commit releases slots (bempty, aempty) and publishes
// accumulators (tfull) in both CTAs; the epilogue warps of both arrive on the leader's tempty.
constexpr int DP_TILE_M = 256, DP_TILE_N = 256, DP_HALF_N = 128;
constexpr int DP_MG = 2;                                   // 256-row tiles per converted tile (at most)
constexpr int DP_SLAB_K = 32;                              // k-rows per fp32 staging slab
constexpr int DP_NG = 3, DP_NB = 2, DP_NA = 4;             // fp32 slab ring, converted ring, dz ring (two k-blocks of dz in flight)
constexpr int DP_STG_HALF = DP_SLAB_K * DP_HALF_N * 4;     // one fp32 [32 x 128] slab: 16 KB
constexpr int DP_STG_BYTES = 2 * DP_STG_HALF;              // w slab + delta slab
constexpr int DP_B_BYTES = TILE_K * DP_HALF_N * 2;         // converted [64 k x 128 n] bf16: 16 KB (two 64-column runs of 8 KB)
constexpr int DP_ACC_COLS = DP_TILE_N;                     // 256 columns per accumulator; two fill the tensor memory
constexpr int DP_XF_WARPS = 8, DP_EPI_WARPS = 8;
constexpr int DP_THREADS = 32 * (3 + DP_XF_WARPS + DP_EPI_WARPS);   // staging producer, MMA issuer, transform, epilogue, dz producer
constexpr int DP_TILE_BYTES = DP_NG * DP_STG_BYTES + DP_NB * DP_B_BYTES + DP_NA * A_BYTES + DP_EPI_WARPS * 4096;
constexpr int DP_SMEM_BYTES = DP_TILE_BYTES + 1024 + 512;
static_assert(DP_SMEM_BYTES <= 227 * 1024, "pair dgrad kernel: shared memory");

// Row tiles per group for a Linear with these dimensions: two, unless that leaves fewer than `split_below` groups
// (a launch that covers one stage only must still bring a tile group for most CTA pairs).
__host__ __device__ inline int dgrad_pair_mg(int T, int n_in, int split_below) {
  const int tiles_n = (n_in + DP_TILE_N - 1) / DP_TILE_N, tiles_m = (T + DP_TILE_M - 1) / DP_TILE_M;
  return (((tiles_m + DP_MG - 1) / DP_MG) * tiles_n < split_below) ? 1 : DP_MG;
}

__device__ __forceinline__ DgTile decode_dgrad_pair(const TickArgs& t, const int* __restrict__ tile_start, int lvl, int tile) {
  DgTile r;
  const int lo = t.sel_p >= 0 ? t.sel_p : tile_start[t.P + 1 + tile];                           // the stage of this tile: table behind the P + 1 starts
  r.p = lo;
  const StageDyn& d = t.dyn[lo];
  const StageDev& s = t.st[lo];
  r.valid = lvl < s.n_lin && d.b_mb >= 0 && !(lo == 0 && lvl == 0 && s.pre != PRE_EMBED);
  const LinDev& L = s.lin[lvl < s.n_lin ? lvl : 0];
  r.M = t.T; r.N = L.n_in; r.K = L.n_out;
  const int mgr = dgrad_pair_mg(r.M, r.N, t.dgrad_split_below);
  const int tiles_n = (r.N + DP_TILE_N - 1) / DP_TILE_N;
  const int tiles_m = (r.M + DP_TILE_M - 1) / DP_TILE_M;
  const int local = tile - (t.sel_p >= 0 ? t.sel_tile0 : tile_start[lo]);
  const int mg = local / tiles_n;
  r.m0 = mg * mgr * DP_TILE_M;
  r.n0 = (local % tiles_n) * DP_TILE_N;
  r.n_m = min(mgr, tiles_m - mg * mgr);
  r.n_kb = (r.K + TILE_K - 1) / TILE_K;
  return r;
}

// Which accumulator (0 | 1: tensor-memory columns 0..255 | 256..511) a row tile of a group uses, and how often each
// has been used so far (the barrier phases follow from the counts).  The MMA issuer and the epilogue warps walk the
// same tile sequence and keep identical copies.
struct DpAcc {
  uint32_t uses[2];
  int next1;                                                         // accumulator of the next single-row-tile group
  __device__ __forceinline__ int buf(int mi, int n_m) const { return n_m == 2 ? mi : next1; }
  __device__ __forceinline__ void done_group(int n_m) { if (n_m == 2) { ++uses[0]; ++uses[1]; } else { ++uses[next1]; next1 ^= 1; } }
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(DP_THREADS, 1)
umma_dgrad_pair_kernel(TickArgs t, const CUtensorMap* __restrict__ maps, const int* __restrict__ tile_start, const int* __restrict__ order, int n_slots, int lvl, int* status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t stg = base;                                          // [DP_NG][w 16 KB | delta 16 KB] fp32 slabs of 32 k-rows x 128 columns
  const uint32_t sB = stg + DP_NG * DP_STG_BYTES;                     // [DP_NB][16 KB] converted operand (this CTA's 128 columns, 64 k-rows)
  const uint32_t sA = sB + DP_NB * DP_B_BYTES;                        // [DP_NA][16 KB] dz tiles (this CTA's 128 rows, 64 k-columns)
  const uint32_t sO = sA + DP_NA * A_BYTES;                           // [8][4 KB] epilogue staging
  uint8_t* stg_ptr = base_ptr;
  uint8_t* sB_ptr = base_ptr + DP_NG * DP_STG_BYTES;
  uint8_t* sO_ptr = sB_ptr + DP_NB * DP_B_BYTES + DP_NA * A_BYTES;
  const uint32_t bars = base + DP_TILE_BYTES;
  const uint32_t bar_sfull = bars, bar_sempty = bar_sfull + 8 * DP_NG, bar_bfull = bar_sempty + 8 * DP_NG,
                 bar_bempty = bar_bfull + 8 * DP_NB, bar_afull = bar_bempty + 8 * DP_NB, bar_aempty = bar_afull + 8 * DP_NA,
                 bar_tfull = bar_aempty + 8 * DP_NA, bar_tempty = bar_tfull + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + DP_TILE_BYTES + 8 * (2 * DP_NG + 2 * DP_NB + 2 * DP_NA + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();                            // 0 = leader
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int i = 0; i < DP_NG; ++i) { mbar_init(bar_sfull + 8 * i, 1); mbar_init(bar_sempty + 8 * i, DP_XF_WARPS); }
    for (int i = 0; i < DP_NB; ++i) { mbar_init(bar_bfull + 8 * i, 2 * 2 * DP_XF_WARPS); mbar_init(bar_bempty + 8 * i, 1); }   // two slabs x two CTAs x eight warps
    for (int i = 0; i < DP_NA; ++i) { mbar_init(bar_afull + 8 * i, 1); mbar_init(bar_aempty + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar_tfull + 8 * i, 1); mbar_init(bar_tempty + 8 * i, 2 * DP_EPI_WARPS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    __syncwarp();
    tmem_alloc_pair(smem_u32(tmem_slot), 2 * DP_ACC_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // Two producer threads, each with its own cursor over the same (tile, k-block) sequence: warp 0 feeds the fp32
  // slab ring (w, delta), the last warp the dz ring.  Everything that is fixed for a tile is read once when the
  // cursor reaches the tile; the loops hold nothing but barrier waits and copies.
  struct Cursor { int tile, kb; DgTile tl; bool done; const CUtensorMap* lm; bool corr; int dz_slot; };
  auto seek = [&](Cursor& c) {
    for (; c.tile < n_slots; c.tile += n_pairs) {
      const int tile = tile_at(t, order, c.tile);
      if (tile < 0) continue;
      c.tl = decode_dgrad_pair(t, tile_start, lvl, tile);
      if (c.tl.valid) {
        const StageDyn& d = t.dyn[c.tl.p];
        const StageDev& sd_ = t.st[c.tl.p];
        c.lm = maps + ((size_t)c.tl.p * PM_MAX_LINEARS + lvl) * MAPS_PER_LINEAR;
        c.corr = d.use_delta != 0;
        c.dz_slot = (bwd_act(sd_.lin[lvl]) == PM_ACT_NONE && lvl == sd_.n_lin - 1 && !feeds_attention(sd_.post)) ? dz_mailbox_slot(t, sd_, d) : 0;
        c.kb = 0; c.done = false;
        return;
      }
    }
    c.done = true;
  };
  auto step = [&](Cursor& c) { if (++c.kb >= c.tl.n_kb) { c.tile += n_pairs; seek(c); } };

  if (warp == 0) {
    // ---------------- TMA producer of the fp32 slab ring (both CTAs): two slabs of 32 k-rows per k-block ----------------
    if (lane == 0) {
      Cursor cs{pair, 0, DgTile{}, false, nullptr, false, 0};
      seek(cs);
      Ring sg{0, 0};
      int issued_sg = 0;
      bool ok = true;
      while (!cs.done && ok) {
        const int ncol = cs.tl.n0 + rank * DP_HALF_N;
        for (int h = 0; h < TILE_K / DP_SLAB_K; ++h) {
          if (!mbar_wait(bar_sempty + 8 * sg.idx, sg.phase ^ 1, abort_flag, status, 41)) { ok = false; break; }
          const uint32_t sw = stg + sg.idx * DP_STG_BYTES, fb = bar_sfull + 8 * sg.idx;
          mbar_arrive_expect_tx(fb, cs.corr ? DP_STG_BYTES : DP_STG_HALF);
          tma_load_2d(sw, cs.lm + MAP_W_F32Q, fb, ncol, cs.kb * TILE_K + h * DP_SLAB_K);
          if (cs.corr) tma_load_2d(sw + DP_STG_HALF, cs.lm + MAP_D_F32Q, fb, ncol, cs.kb * TILE_K + h * DP_SLAB_K);
          sg.advance(DP_NG); ++issued_sg;
        }
        step(cs);
      }
      if (*abort_flag) {                                              // copies already issued still land here: wait (bounded)
        for (int back = 1; back <= DP_NG && back <= issued_sg; ++back) {
          const int it = issued_sg - back;
          const long long t0 = clock64();
          while (!mbar_try_wait(bar_sfull + 8 * (it % DP_NG), (uint32_t)(it / DP_NG) & 1u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        }
      }
    }
  } else if (warp == 2 + DP_XF_WARPS + DP_EPI_WARPS) {
    // ---------------- TMA producer of the dz ring (both CTAs) ----------------
    if (lane == 0) {
      Cursor ca{pair, 0, DgTile{}, false, nullptr, false, 0};
      seek(ca);
      Ring ar{0, 0};
      int issued_a = 0;
      bool ok = true;
      while (!ca.done && ok) {
        for (int mi = 0; mi < ca.tl.n_m; ++mi) {
          if (!mbar_wait(bar_aempty + 8 * ar.idx, ar.phase ^ 1, abort_flag, status, 42)) { ok = false; break; }
          if (rank == 0) mbar_arrive_expect_tx(bar_afull + 8 * ar.idx, 2 * A_BYTES);       // the rows of both CTAs
          tma_load_3d_pair(sA + ar.idx * A_BYTES, ca.lm + MAP_DZ_K, mapa_shared(bar_afull + 8 * ar.idx, 0),
                           ca.kb * TILE_K, ca.tl.m0 + mi * DP_TILE_M + rank * TILE_M, ca.dz_slot);
          ar.advance(DP_NA); ++issued_a;
        }
        step(ca);
      }
      if (*abort_flag) {
        if (rank == 0) {
          for (int back = 1; back <= DP_NA && back <= issued_a; ++back) {
            const int it = issued_a - back;
            const long long t0 = clock64();
            while (!mbar_try_wait(bar_afull + 8 * (it % DP_NA), (uint32_t)(it / DP_NA) & 1u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
          }
        }
        // rank 1's copies are counted on the same barriers of the leader (the expected bytes are those of both CTAs), and
        // no CTA of the pair leaves before the cluster barrier at the end of the kernel, which the leader reaches only
        // after these waits: rank 1 needs no wait of its own
      }
    }
  }
  else if (warp == 1) {
    // ---------------- MMA issuer (leader CTA only) ----------------
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = make_idesc_mn(DP_TILE_M, DP_TILE_N, 0, 1);
      const uint64_t dba = desc_base(16, 1024), dbb = desc_base(DP_B_BYTES / 2, 1024);   // B: two 64-column runs per CTA, 8 KB apart
      Ring br{0, 0}, ar{0, 0};
      DpAcc acc{{0u, 0u}, 0};
      bool ok = true;
      for (int slot = pair; slot < n_slots && ok; slot += n_pairs) {
        const int tile = tile_at(t, order, slot);
        if (tile < 0) continue;
        const DgTile tl = decode_dgrad_pair(t, tile_start, lvl, tile);
        if (!tl.valid) continue;
        const int n_m = tl.n_m, n_kb = tl.n_kb;
        for (int kb = 0; kb < n_kb && ok; ++kb) {
          if (!mbar_wait(bar_bfull + 8 * br.idx, br.phase, abort_flag, status, 44)) { ok = false; break; }
          const uint32_t sb = sB + br.idx * DP_B_BYTES;
          uint32_t sa[DP_MG], abar[DP_MG];
          for (int mi = 0; mi < n_m; ++mi) {
            if (!mbar_wait(bar_afull + 8 * ar.idx, ar.phase, abort_flag, status, 45)) { ok = false; break; }
            sa[mi] = sA + ar.idx * A_BYTES;
            abar[mi] = bar_aempty + 8 * ar.idx;
            ar.advance(DP_NA);
          }
          if (!ok) break;
          tc_fence_after();
          // one row tile after the other: the first k-block of a group waits for each accumulator to be drained just
          // before its first product, and the last k-block publishes the first accumulator while the products of
          // the second are still running
          for (int mi = 0; mi < n_m && ok; ++mi) {
            const int b = acc.buf(mi, n_m);
            if (kb == 0) {
              if (!mbar_wait(bar_tempty + 8 * b, (acc.uses[b] & 1u) ^ 1u, abort_flag, status, 43)) { ok = false; break; }
              tc_fence_after();
            }
            const uint32_t tmem_acc = tmem_base + (uint32_t)(b * DP_ACC_COLS);
#pragma unroll
            for (int k16 = 0; k16 < TILE_K / 16; ++k16)
              tc_mma_bf16_pair(tmem_acc, desc_at(dba, sa[mi] + k16 * 32), desc_at(dbb, sb + k16 * 2048), idesc, (kb > 0 || k16 > 0) ? 1u : 0u);
            tc_commit_pair(abar[mi], 3);                              // this dz tile may be overwritten in both CTAs
            if (kb == n_kb - 1) tc_commit_pair(bar_tfull + 8 * b, 3);  // accumulator complete, both CTAs
          }
          if (ok) tc_commit_pair(bar_bempty + 8 * br.idx, 3);
          br.advance(DP_NB);
        }
        acc.done_group(n_m);
      }
    }
  } else if (warp < 2 + DP_XF_WARPS) {
    // ---------------- operand transform (both CTAs): fp32 w, delta [32 k][128 n] -> bf16(w - gap*delta), MN-major ----------------
    // thread: four consecutive columns (c4) of rows rbase + 8 j; reads are contiguous float4, stores 8 bytes into the swizzled atom.
    // Two slabs (k-rows 0..31 and 32..63) fill one converted tile.
    const int tt = threadIdx.x - 64;                                  // 0..255
    const int c4 = tt & 31, rbase = tt >> 5;                          // 0..31 (four columns each), 0..7
    const int run = c4 >> 4, cc = (c4 & 15);                          // 64-column run of the tile, position inside it (units of four columns)
    const uint32_t leader_bfull = mapa_shared(bar_bfull, 0);
    Ring br{0, 0}, sg{0, 0};
    bool ok = true;
    for (int slot = pair; slot < n_slots && ok; slot += n_pairs) {
      const int tile = tile_at(t, order, slot);
      if (tile < 0) continue;
      const DgTile tl = decode_dgrad_pair(t, tile_start, lvl, tile);
      if (!tl.valid) continue;
      const float gapf = (float)t.st[tl.p].gap;
      const bool corr = t.dyn[tl.p].use_delta != 0;
      for (int kb = 0; kb < tl.n_kb && ok; ++kb) {
        for (int h = 0; h < TILE_K / DP_SLAB_K; ++h) {
          bool go = mbar_wait(bar_sfull + 8 * sg.idx, sg.phase, abort_flag, status, 46);
          if (h == 0) go = go && mbar_wait(bar_bempty + 8 * br.idx, br.phase ^ 1, abort_flag, status, 47);
          go = __all_sync(0xffffffffu, go);
          if (!go) { ok = false; break; }
          const uint8_t* src = stg_ptr + sg.idx * DP_STG_BYTES;
          uint8_t* dst = sB_ptr + br.idx * DP_B_BYTES + run * (DP_B_BYTES / 2);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int rs = rbase + 8 * j;                             // row of the slab
            const int r = h * DP_SLAB_K + rs;                         // k-row of the tile
            const float4 w = *reinterpret_cast<const float4*>(src + rs * (DP_HALF_N * 4) + c4 * 16);
            float v[4] = {w.x, w.y, w.z, w.w};
            if (corr) {
              const float4 dl = *reinterpret_cast<const float4*>(src + DP_STG_HALF + rs * (DP_HALF_N * 4) + c4 * 16);
              v[0] = __fsub_rn(v[0], __fmul_rn(gapf, dl.x)); v[1] = __fsub_rn(v[1], __fmul_rn(gapf, dl.y));   // w - (tau_fwd - tau_bkwd) * delta
              v[2] = __fsub_rn(v[2], __fmul_rn(gapf, dl.z)); v[3] = __fsub_rn(v[3], __fmul_rn(gapf, dl.w));
            }
            const uint32_t off = (uint32_t)(r >> 3) * 1024 + (uint32_t)(r & 7) * 128 + ((((uint32_t)cc >> 1) ^ (uint32_t)(r & 7)) << 4) + ((uint32_t)cc & 1) * 8;
            *reinterpret_cast<uint2*>(dst + off) = make_uint2(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]));
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) { mbar_arrive_cluster(leader_bfull + 8 * br.idx); mbar_arrive(bar_sempty + 8 * sg.idx); }
          sg.advance(DP_NG);
        }
        br.advance(DP_NB);
      }
    }
  }
  else {
    // ---------------- epilogue (both CTAs): 8 warps, warp%4 = TMEM lane group, two warps per group split the 256 columns ----------------
    const int q = warp & 3;
    const int ew = warp - 2 - DP_XF_WARPS;                            // 0..7
    const int half = ew >> 2;                                         // 0: columns 0..127 of the tile, 1: columns 128..255
    uint8_t* obuf = sO_ptr + ew * 4096;
    const uint32_t obuf_s = sO + ew * 4096;
    const uint32_t row_off = (uint32_t)lane * 128, sw = (uint32_t)(lane & 7);
    const uint32_t leader_tempty = mapa_shared(bar_tempty, 0);
    DpAcc acc{{0u, 0u}, 0};
    bool ok = true, stored = false;
    for (int slot = pair; slot < n_slots && ok; slot += n_pairs) {
      const int tile = tile_at(t, order, slot);
      if (tile < 0) continue;
      const DgTile tl = decode_dgrad_pair(t, tile_start, lvl, tile);
      if (!tl.valid) continue;
      const StageDyn& d = t.dyn[tl.p];
      const StageDev& s = t.st[tl.p];
      const CUtensorMap* lm = maps + ((size_t)tl.p * PM_MAX_LINEARS + lvl) * MAPS_PER_LINEAR;
      const int dslot = (lvl == 0 && s.pre == PRE_NONE) ? d.prev_wslot : 0;
      const bool masked = lvl == 0 && s.mask_dx != 0;              // the previous stage's ReLU backward is applied here
#pragma unroll 1
      for (int mi = 0; mi < tl.n_m && ok; ++mi) {
        const int b = acc.buf(mi, tl.n_m);
        bool ready = mbar_wait(bar_tfull + 8 * b, acc.uses[b] & 1u, abort_flag, status, 48);
        ready = __all_sync(0xffffffffu, ready);
        if (!ready) { ok = false; break; }
        tc_fence_after();
        const int mrow = tl.m0 + mi * DP_TILE_M + rank * TILE_M + q * 32;
#pragma unroll 1
        for (int c = 0; c < 2; ++c) {
          const int nb = tl.n0 + half * 128 + c * 64;
          uint32_t r0[32], r1[32];
          const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * DP_ACC_COLS + half * 128 + c * 64);
          const uint64_t mk = masked ? load_mask_bits64(t, s, d, tl.N, mrow + lane, nb) : ~0ull;
          tmem_ld32(taddr, r0);
          tmem_ld32(taddr + 32, r1);
          tmem_ld_wait();
          if (c == 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_tempty + 8 * b);   // this warp has read its part of this accumulator
          }
          if (mrow >= tl.M || nb >= tl.N) continue;
          if (lane == 0 && stored) tma_store_wait_read();
          __syncwarp();
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            float f[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(g < 4 ? r0[(g & 3) * 8 + e] : r1[(g & 3) * 8 + e]);
            if (masked) apply_mask8(f, (uint32_t)(mk >> (8 * g)) & 0xFFu);
            *reinterpret_cast<uint4*>(obuf + row_off + (((uint32_t)g ^ sw) << 4)) =
                make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) { tma_store_3d(lm + MAP_DX_OUT, obuf_s, nb, mrow, dslot); tma_store_commit(); }
          stored = true;
        }
      }
      acc.done_group(tl.n_m);
    }
    if (lane == 0 && stored) tma_store_wait_all();
  }
  tc_fence_before();
  cluster_sync_all();                                                 // no barrier or shared memory of a CTA is touched after this
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 2 * DP_ACC_COLS);
  }
}

// ---- dgrad on CTA pairs, 128-column tiles ----------------------------------------------------------------------
// Used where a launch covers ONE stage whose input is narrow (microbatch-major order): with 256-column tiles such a
// Linear has too few tile groups for the CTA pairs, and a single row tile per group doubles the fp32 traffic per
// FLOP beyond what L2 delivers.  Here a tile is half as wide, so twice as many groups exist.
// The same product and the same on-the-fly correction on tiles of 256 rows x 128 columns per CTA pair
// (tcgen05.mma.cta_group::2, M = 256, N = 128).  Each CTA stages the fp32 w and delta of ITS 64 columns
// (2 x 16 KB per k-block), converts them to bf16(w - gap*delta) in its own shared memory, and loads its 128
// rows of dz; two 256-row tiles share one converted tile, so a CTA ingests 64 KB per 2 x (128x128x64) of its
// own products, as the single-CTA kernel does, but the accumulators (2 x 128 columns) are double-buffered and
// the eight epilogue warps drain one group while the next is computed.  Barriers: staging (sfull / sempty)
// is local to a CTA; the converted tile (bfull) and the dz tiles (afull) are counted in the leader, which
// issues the MMAs; tcgen05.commit releases slots (bempty, aempty) and publishes accumulators (tfull) in both
// CTAs; the epilogue warps of both arrive on the leader's tempty.
constexpr int D1_TILE_M = 256, D1_TILE_N = 128, D1_HALF_N = 64;
constexpr int D1_MG = 2;                                   // 256-row tiles per converted tile
constexpr int D1_PF = 4;                                   // k-blocks of fp32 w and delta asked of L2 ahead of the staging ring
constexpr int D1_NG = 2, D1_NB = 2, D1_NA = 7;             // fp32 staging ring, converted ring, dz ring (3.5 k-blocks of dz in flight)
constexpr int D1_STG_HALF = TILE_K * D1_HALF_N * 4;        // one fp32 [64 x 64] tile: 16 KB
constexpr int D1_STG_BYTES = 2 * D1_STG_HALF;
constexpr int D1_B_BYTES = TILE_K * D1_HALF_N * 2;         // converted [64 k x 64 n] bf16: 8 KB
constexpr int D1_ACC_COLS = D1_MG * D1_TILE_N;             // 256 columns per accumulator buffer
constexpr int D1_XF_WARPS = 8, D1_EPI_WARPS = 8;
constexpr int D1_THREADS = 32 * (4 + D1_XF_WARPS + D1_EPI_WARPS);   // staging producer, MMA issuer, transform, epilogue, dz producer, second MMA issuer
constexpr int D1_TILE_BYTES = D1_NG * D1_STG_BYTES + D1_NB * D1_B_BYTES + D1_NA * A_BYTES + D1_EPI_WARPS * 4096;
constexpr int D1_SMEM_BYTES = D1_TILE_BYTES + 1024 + 512;

__device__ __forceinline__ DgTile decode_dgrad_pair128(const TickArgs& t, const int* __restrict__ tile_start, int lvl, int tile) {
  DgTile r;
  const int lo = t.sel_p >= 0 ? t.sel_p : tile_start[t.P + 1 + tile];                           // the stage of this tile: table behind the P + 1 starts
  r.p = lo;
  const StageDyn& d = t.dyn[lo];
  const StageDev& s = t.st[lo];
  r.valid = lvl < s.n_lin && d.b_mb >= 0 && !(lo == 0 && lvl == 0 && s.pre != PRE_EMBED);
  const LinDev& L = s.lin[lvl < s.n_lin ? lvl : 0];
  r.M = t.T; r.N = L.n_in; r.K = L.n_out;
  const int tiles_n = (r.N + D1_TILE_N - 1) / D1_TILE_N;
  const int tiles_m = (r.M + D1_TILE_M - 1) / D1_TILE_M;
  const int local = tile - (t.sel_p >= 0 ? t.sel_tile0 : tile_start[lo]);
  const int mg = local / tiles_n;
  r.m0 = mg * D1_MG * D1_TILE_M;
  r.n0 = (local % tiles_n) * D1_TILE_N;
  r.n_m = min(D1_MG, tiles_m - mg * D1_MG);
  r.n_kb = (r.K + TILE_K - 1) / TILE_K;
  return r;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(D1_THREADS, 1)
umma_dgrad_pair128_kernel(TickArgs t, const CUtensorMap* __restrict__ maps, const int* __restrict__ tile_start, const int* __restrict__ order, int n_slots, int lvl, int* status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t stg = base;                                          // [D1_NG][w 16 KB | delta 16 KB]
  const uint32_t sB = stg + D1_NG * D1_STG_BYTES;                     // [D1_NB][8 KB] converted operand (this CTA's 64 columns)
  const uint32_t sA = sB + D1_NB * D1_B_BYTES;                        // [D1_NA][16 KB] dz tiles (this CTA's 128 rows)
  const uint32_t sO = sA + D1_NA * A_BYTES;                           // [8][4 KB] epilogue staging
  uint8_t* stg_ptr = base_ptr;
  uint8_t* sB_ptr = base_ptr + D1_NG * D1_STG_BYTES;
  uint8_t* sO_ptr = sB_ptr + D1_NB * D1_B_BYTES + D1_NA * A_BYTES;
  const uint32_t bars = base + D1_TILE_BYTES;
  const uint32_t bar_sfull = bars, bar_sempty = bar_sfull + 8 * D1_NG, bar_bfull = bar_sempty + 8 * D1_NG,
                 bar_bempty = bar_bfull + 8 * D1_NB, bar_afull = bar_bempty + 8 * D1_NB, bar_aempty = bar_afull + 8 * D1_NA,
                 bar_tfull = bar_aempty + 8 * D1_NA, bar_tempty = bar_tfull + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + D1_TILE_BYTES + 8 * (2 * D1_NG + 2 * D1_NB + 2 * D1_NA + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();                            // 0 = leader
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int i = 0; i < D1_NG; ++i) { mbar_init(bar_sfull + 8 * i, 1); mbar_init(bar_sempty + 8 * i, D1_XF_WARPS); }
    for (int i = 0; i < D1_NB; ++i) { mbar_init(bar_bfull + 8 * i, 2 * D1_XF_WARPS); mbar_init(bar_bempty + 8 * i, D1_MG); }   // released by both MMA issuers
    for (int i = 0; i < D1_NA; ++i) { mbar_init(bar_afull + 8 * i, 1); mbar_init(bar_aempty + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar_tfull + 8 * i, D1_MG); mbar_init(bar_tempty + 8 * i, 2 * D1_EPI_WARPS); }   // published by both MMA issuers
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    __syncwarp();
    tmem_alloc_pair(smem_u32(tmem_slot), 2 * D1_ACC_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // Two producer threads, each with its own cursor over the same (tile, k-block) sequence: warp 0 feeds the fp32
  // staging ring (w, delta), the last warp the dz ring.  Their k-block loops are the critical path of the kernel
  // (a handful of extra loads in them cost 3 %), so everything that is fixed for a tile is read once when the
  // cursor reaches the tile and the loops hold nothing but barrier waits and copies.
  struct Cursor { int tile, kb; DgTile tl; bool done; const CUtensorMap* lm; bool corr; int dz_slot; };
  auto seek = [&](Cursor& c) {
    for (; c.tile < n_slots; c.tile += n_pairs) {
      const int tile = tile_at(t, order, c.tile);
      if (tile < 0) continue;
      c.tl = decode_dgrad_pair128(t, tile_start, lvl, tile);
      if (c.tl.valid) {
        const StageDyn& d = t.dyn[c.tl.p];
        const StageDev& sd_ = t.st[c.tl.p];
        c.lm = maps + ((size_t)c.tl.p * PM_MAX_LINEARS + lvl) * MAPS_PER_LINEAR;
        c.corr = d.use_delta != 0;
        c.dz_slot = (bwd_act(sd_.lin[lvl]) == PM_ACT_NONE && lvl == sd_.n_lin - 1 && !feeds_attention(sd_.post)) ? dz_mailbox_slot(t, sd_, d) : 0;
        c.kb = 0; c.done = false;
        return;
      }
    }
    c.done = true;
  };
  auto step = [&](Cursor& c) { if (++c.kb >= c.tl.n_kb) { c.tile += n_pairs; seek(c); } };

  if (warp == 0) {
    // ---------------- TMA producer of the fp32 staging ring (both CTAs) ----------------
    if (lane == 0) {
      Cursor cs{pair, 0, DgTile{}, false, nullptr, false, 0};
      seek(cs);
      Cursor cp = cs;                                                 // runs D1_PF k-blocks ahead and asks L2 for them
      auto prefetch = [&]() {
        if (cp.done) return;
        if (cp.tl.m0 == 0) {                                          // the pairs of one row group ask for all: the others run beside them
          tma_prefetch_2d(cp.lm + MAP_W_F32H, cp.tl.n0 + rank * D1_HALF_N, cp.kb * TILE_K);
          if (cp.corr) tma_prefetch_2d(cp.lm + MAP_D_F32H, cp.tl.n0 + rank * D1_HALF_N, cp.kb * TILE_K);
        }
        step(cp);
      };
      for (int i = 0; i < D1_NG; ++i) step(cp);                       // the first D1_NG k-blocks are loaded at once
      for (int i = 0; i < D1_PF; ++i) prefetch();
      Ring sg{0, 0};
      int issued_sg = 0;
      while (!cs.done) {
        prefetch();
        if (!mbar_wait(bar_sempty + 8 * sg.idx, sg.phase ^ 1, abort_flag, status, 41)) break;
        const uint32_t sw = stg + sg.idx * D1_STG_BYTES, fb = bar_sfull + 8 * sg.idx;
        mbar_arrive_expect_tx(fb, cs.corr ? D1_STG_BYTES : D1_STG_HALF);
        tma_load_2d(sw, cs.lm + MAP_W_F32H, fb, cs.tl.n0 + rank * D1_HALF_N, cs.kb * TILE_K);
        if (cs.corr) tma_load_2d(sw + D1_STG_HALF, cs.lm + MAP_D_F32H, fb, cs.tl.n0 + rank * D1_HALF_N, cs.kb * TILE_K);
        sg.advance(D1_NG); ++issued_sg;
        step(cs);
      }
      if (*abort_flag) {                                              // copies already issued still land here: wait (bounded)
        for (int back = 1; back <= D1_NG && back <= issued_sg; ++back) {
          const int it = issued_sg - back;
          const long long t0 = clock64();
          while (!mbar_try_wait(bar_sfull + 8 * (it % D1_NG), (uint32_t)(it / D1_NG) & 1u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        }
      }
    }
  } else if (warp == 2 + D1_XF_WARPS + D1_EPI_WARPS) {
    // ---------------- TMA producer of the dz ring (both CTAs) ----------------
    if (lane == 0) {
      Cursor ca{pair, 0, DgTile{}, false, nullptr, false, 0};
      seek(ca);
      Ring ar{0, 0};
      int issued_a = 0;
      bool ok = true;
      while (!ca.done && ok) {
        for (int mi = 0; mi < ca.tl.n_m; ++mi) {
          if (!mbar_wait(bar_aempty + 8 * ar.idx, ar.phase ^ 1, abort_flag, status, 42)) { ok = false; break; }
          if (rank == 0) mbar_arrive_expect_tx(bar_afull + 8 * ar.idx, 2 * A_BYTES);       // the rows of both CTAs
          tma_load_3d_pair(sA + ar.idx * A_BYTES, ca.lm + MAP_DZ_K, mapa_shared(bar_afull + 8 * ar.idx, 0),
                           ca.kb * TILE_K, ca.tl.m0 + mi * D1_TILE_M + rank * TILE_M, ca.dz_slot);
          ar.advance(D1_NA); ++issued_a;
        }
        step(ca);
      }
      if (*abort_flag) {
        if (rank == 0) {
          for (int back = 1; back <= D1_NA && back <= issued_a; ++back) {
            const int it = issued_a - back;
            const long long t0 = clock64();
            while (!mbar_try_wait(bar_afull + 8 * (it % D1_NA), (uint32_t)(it / D1_NA) & 1u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
          }
        }
        // rank 1's copies are counted on the same barriers of the leader (the expected bytes are those of both CTAs), and
        // no CTA of the pair leaves before the cluster barrier at the end of the kernel, which the leader reaches only
        // after these waits: rank 1 needs no wait of its own
      }
    }
  } else if (warp == 1 || warp == 3 + D1_XF_WARPS + D1_EPI_WARPS) {
    // ---------------- MMA issuers (leader CTA only): one thread per row tile of a group ----------------
    // Issuing an MMA, its commits and the barrier polls in front of them cost the issuing thread about 1400 cycles per
    // k-block of two row tiles, of which the tensor pipe works 512: one thread cannot keep the pipe busy.  The two row tiles
    // of a group have accumulators of their own, so their MMAs need no order between them: thread `me` waits for the
    // shared converted tile and for ITS dz tile, issues its four MMAs and commits its dz slot; both threads commit the
    // converted slot and the accumulator buffer (those barriers count two arrivals).
    if (lane == 0 && rank == 0) {
      const int me = warp == 1 ? 0 : 1;
      const uint32_t idesc = make_idesc_mn(D1_TILE_M, D1_TILE_N, 0, 1);
      const uint64_t dba = desc_base(16, 1024), dbb = desc_base(D1_B_BYTES, 1024);   // B: one 64-column run per CTA
      Ring br{0, 0}, ar{0, 0}, acc{0, 0};
      bool ok = true;
      for (int slot = pair; slot < n_slots && ok; slot += n_pairs) {
        const int tile = tile_at(t, order, slot);
        if (tile < 0) continue;
        const DgTile tl = decode_dgrad_pair128(t, tile_start, lvl, tile);
        if (!tl.valid) continue;
        if (!mbar_wait(bar_tempty + 8 * acc.idx, acc.phase ^ 1, abort_flag, status, 43)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_acc = tmem_base + (uint32_t)(acc.idx * D1_ACC_COLS + me * D1_TILE_N);
        const bool mine = me < tl.n_m;                               // a group at the end of the rows may hold one tile only
        for (int kb = 0; kb < tl.n_kb && ok; ++kb) {
          if (!mbar_wait(bar_bfull + 8 * br.idx, br.phase, abort_flag, status, 44)) { ok = false; break; }
          const uint32_t sb = sB + br.idx * D1_B_BYTES;
          // the dz slots of this k-block sit in ring order, row tile 0 first; this thread's is the me-th
          Ring mr = ar;
          if (me == 1) mr.advance(D1_NA);
          for (int mi = 0; mi < tl.n_m; ++mi) ar.advance(D1_NA);
          if (mine) {
            if (!mbar_wait(bar_afull + 8 * mr.idx, mr.phase, abort_flag, status, 45)) { ok = false; break; }
            tc_fence_after();
            const uint32_t sa = sA + mr.idx * A_BYTES;
#pragma unroll
            for (int k16 = 0; k16 < TILE_K / 16; ++k16)
              tc_mma_bf16_pair(tmem_acc, desc_at(dba, sa + k16 * 32), desc_at(dbb, sb + k16 * 2048), idesc, (kb > 0 || k16 > 0) ? 1u : 0u);
            tc_commit_pair(bar_aempty + 8 * mr.idx, 3);
          }
          tc_commit_pair(bar_bempty + 8 * br.idx, 3);                 // with no MMA of this thread outstanding it arrives at once
          br.advance(D1_NB);
        }
        if (ok) tc_commit_pair(bar_tfull + 8 * acc.idx, 3);
        acc.advance(2);
      }
    }
  } else if (warp < 2 + D1_XF_WARPS) {
    // ---------------- operand transform (both CTAs): fp32 w, delta [64 k][64 n] -> bf16(w - gap*delta), MN-major ----------------
    // thread: four consecutive columns (c4) of rows r0 + 16 j; reads are contiguous float4, stores 8 bytes into the swizzled atom
    const int tt = threadIdx.x - 64;                                  // 0..255
    const int c4 = tt & 15, rbase = tt >> 4;                          // 0..15, 0..15
    const uint32_t leader_bfull = mapa_shared(bar_bfull, 0);
    Ring br{0, 0}, sg{0, 0};
    bool ok = true;
    for (int slot = pair; slot < n_slots && ok; slot += n_pairs) {
      const int tile = tile_at(t, order, slot);
      if (tile < 0) continue;
      const DgTile tl = decode_dgrad_pair128(t, tile_start, lvl, tile);
      if (!tl.valid) continue;
      const float gapf = (float)t.st[tl.p].gap;
      const bool corr = t.dyn[tl.p].use_delta != 0;
      for (int kb = 0; kb < tl.n_kb; ++kb) {
        bool go = mbar_wait(bar_sfull + 8 * sg.idx, sg.phase, abort_flag, status, 46);
        go = __all_sync(0xffffffffu, go);
        if (!go) { ok = false; break; }
        // the staged fp32 values go to registers and the staging slot back to its producer at once: the wait for a free
        // converted slot and the stores into it are then off the slot's round trip (copy latency + this read)
        const uint8_t* src = stg_ptr + sg.idx * D1_STG_BYTES;
        float4 w[4], dl[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int r = rbase + 16 * j;                               // k-row
          w[j] = *reinterpret_cast<const float4*>(src + r * (D1_HALF_N * 4) + c4 * 16);
          if (corr) dl[j] = *reinterpret_cast<const float4*>(src + D1_STG_HALF + r * (D1_HALF_N * 4) + c4 * 16);
        }
        uint2 o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float v[4] = {w[j].x, w[j].y, w[j].z, w[j].w};
          if (corr) {
            v[0] = __fsub_rn(v[0], __fmul_rn(gapf, dl[j].x)); v[1] = __fsub_rn(v[1], __fmul_rn(gapf, dl[j].y));   // w - (tau_fwd - tau_bkwd) * delta
            v[2] = __fsub_rn(v[2], __fmul_rn(gapf, dl[j].z)); v[3] = __fsub_rn(v[3], __fmul_rn(gapf, dl[j].w));
          }
          o[j] = make_uint2(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]));
        }
        __syncwarp();                                                 // every lane's values have arrived (they were used above)
        if (lane == 0) mbar_arrive(bar_sempty + 8 * sg.idx);
        go = mbar_wait(bar_bempty + 8 * br.idx, br.phase ^ 1, abort_flag, status, 47);
        go = __all_sync(0xffffffffu, go);
        if (!go) { ok = false; break; }
        uint8_t* dst = sB_ptr + br.idx * D1_B_BYTES;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int r = rbase + 16 * j;
          const uint32_t off = (uint32_t)(r >> 3) * 1024 + (uint32_t)(r & 7) * 128 + ((((uint32_t)c4 >> 1) ^ (uint32_t)(r & 7)) << 4) + ((uint32_t)c4 & 1) * 8;
          *reinterpret_cast<uint2*>(dst + off) = o[j];
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(leader_bfull + 8 * br.idx);
        br.advance(D1_NB); sg.advance(D1_NG);
      }
    }
  } else {
    // ---------------- epilogue (both CTAs): 8 warps, warp%4 = TMEM lane group, two warps per group split the 128 columns ----------------
    const int q = warp & 3;
    const int ew = warp - 2 - D1_XF_WARPS;                            // 0..7
    const int half = ew >> 2;
    uint8_t* obuf = sO_ptr + ew * 4096;
    const uint32_t obuf_s = sO + ew * 4096;
    const uint32_t row_off = (uint32_t)lane * 128, sw = (uint32_t)(lane & 7);
    const uint32_t leader_tempty = mapa_shared(bar_tempty, 0);
    Ring acc{0, 0};
    bool ok = true, stored = false;
    for (int slot = pair; slot < n_slots && ok; slot += n_pairs) {
      const int tile = tile_at(t, order, slot);
      if (tile < 0) continue;
      const DgTile tl = decode_dgrad_pair128(t, tile_start, lvl, tile);
      if (!tl.valid) continue;
      const StageDyn& d = t.dyn[tl.p];
      const StageDev& s = t.st[tl.p];
      const CUtensorMap* lm = maps + ((size_t)tl.p * PM_MAX_LINEARS + lvl) * MAPS_PER_LINEAR;
      bool ready = mbar_wait(bar_tfull + 8 * acc.idx, acc.phase, abort_flag, status, 48);
      ready = __all_sync(0xffffffffu, ready);
      if (!ready) { ok = false; break; }
      tc_fence_after();
      const int dslot = (lvl == 0 && s.pre == PRE_NONE) ? d.prev_wslot : 0;
      const bool masked = lvl == 0 && s.mask_dx != 0;              // the previous stage's ReLU backward is applied here
      const int nb = tl.n0 + half * 64;
#pragma unroll 1
      for (int mi = 0; mi < tl.n_m; ++mi) {
        const int mrow = tl.m0 + mi * D1_TILE_M + rank * TILE_M + q * 32;
        uint32_t r0[32], r1[32];
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc.idx * D1_ACC_COLS + mi * D1_TILE_N + half * 64);
        const uint64_t mk = masked ? load_mask_bits64(t, s, d, tl.N, mrow + lane, nb) : ~0ull;
        tmem_ld32(taddr, r0);
        tmem_ld32(taddr + 32, r1);
        tmem_ld_wait();
        if (mi == tl.n_m - 1) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(leader_tempty + 8 * acc.idx);   // this warp has read its part of both accumulators
        }
        if (mrow >= tl.M || nb >= tl.N) continue;
        if (lane == 0 && stored) tma_store_wait_read();
        __syncwarp();
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          float f[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(g < 4 ? r0[(g & 3) * 8 + e] : r1[(g & 3) * 8 + e]);
          if (masked) apply_mask8(f, (uint32_t)(mk >> (8 * g)) & 0xFFu);
          *reinterpret_cast<uint4*>(obuf + row_off + (((uint32_t)g ^ sw) << 4)) =
              make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) { tma_store_3d(lm + MAP_DX_OUT, obuf_s, nb, mrow, dslot); tma_store_commit(); }
        stored = true;
      }
      acc.advance(2);
    }
    if (lane == 0 && stored) tma_store_wait_all();
  }
  tc_fence_before();
  cluster_sync_all();                                                 // no barrier or shared memory of a CTA is touched after this
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 2 * D1_ACC_COLS);
  }
}

// ---- host side -----------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct UmmaPlan {
  const CUtensorMap* d_maps = nullptr;
  const int* d_tile_start = nullptr;     // per (mode, level) at ts_off: [P+1] starts, then the stage of each tile
  size_t ts_off[5][PM_MAX_LINEARS] = {};
  const int* d_orders = nullptr;         // concatenated order arrays
  int* d_status = nullptr;
  int n_slots[5][PM_MAX_LINEARS] = {};
  int grid[5][PM_MAX_LINEARS] = {};
  bool pair[5][PM_MAX_LINEARS] = {};     // launch uses the CTA-pair kernel (256 x 256 tiles)
  size_t order_off[5][PM_MAX_LINEARS] = {};
  int P = 0;
  // launches of one stage (microbatch-major order): the stage's tiles in ascending order are a slice of the identity list
  std::vector<int> h_tile_start;         // host copy of the tile starts
  const int* d_identity = nullptr;       // 0, 1, 2, ...
  int max_ctas = 148;
};

// Tile tables of every (mode, level): the flattened tile ids per stage, and the order in which the persistent
// CTAs walk them.  CTA b takes order[b], order[b + G], ...: the lists are a longest-processing-time-first
// assignment (weight = k-blocks x row tiles + a constant per tile), so that one very deep GEMM (a vocabulary
// projection next to d_model-sized layers) does not leave most SMs idle.  Unused slots hold -1.
struct TileTables {
  std::vector<int> tile_start;           // per (mode, level): [P+1] starts, then the stage of each tile
  size_t ts_off[5][PM_MAX_LINEARS] = {};
  std::vector<int> orders;
  int n_slots[5][PM_MAX_LINEARS] = {};
  int grid[5][PM_MAX_LINEARS] = {};
  bool pair[5][PM_MAX_LINEARS] = {};
  size_t order_off[5][PM_MAX_LINEARS] = {};
  int max_tiles = 0;                     // most tiles of any (mode, level)
};

static int device_sms() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
    cudaGetLastError();
    return 148;
  }
  return sms;
}

// PM_UMMA_PAIR=0 in the environment keeps every launch on the single-CTA kernels (for comparisons).
static bool pair_kernels_allowed() {
  const char* v = getenv("PM_UMMA_PAIR");
  return !(v && v[0] == '0');
}

static TileTables build_tile_tables(int T, const std::vector<StageDev>& st, int sms, int dgrad_split_below) {
  const int P = (int)st.size();
  const bool allow_pair = pair_kernels_allowed();
  TileTables tt;
  auto cdiv = [](int a, int b) { return (a + b - 1) / b; };
  for (int mode = 0; mode < 5; ++mode)                      // 3: dgrad once more, on 128-column pair tiles (launches of one narrow stage);
                                                            // 4: dgrad as a plain GEMM against a queued weight version (weight stashing)
    for (int l = 0; l < PM_MAX_LINEARS; ++l) {
      // block of this (mode, level): P + 1 tile starts, then the stage of every tile (one load instead of a search)
      tt.ts_off[mode][l] = tt.tile_start.size();
      std::vector<int> ts_block((size_t)P + 1, 0);
      int* ts = ts_block.data();
      std::vector<std::pair<long long, int>> work;          // (weight, tile id)
      // forward and wgrad launches whose GEMMs all have at least 256 rows and columns run on CTA pairs
      bool pair = allow_pair && sms >= 2;
      int n_lin_here = 0;
      for (int p = 0; p < P && pair; ++p)
        if (l < st[p].n_lin) {
          const LinDev& L = st[p].lin[l];
          ++n_lin_here;
          if ((mode == 2 ? L.n_out : T) < P2_TILE || (mode == 0 ? L.n_out : L.n_in) < P2_TILE) pair = false;
          if ((mode == 1 || mode == 3 || mode == 4) && p == 0 && l == 0 && st[p].pre != PRE_EMBED) --n_lin_here;   // the first Linear of the network has no input gradient
        }
      pair = pair && n_lin_here > 0;
      tt.pair[mode][l] = pair;
      if (mode == 3 && !pair) { tt.n_slots[mode][l] = 0; tt.grid[mode][l] = 0; tt.order_off[mode][l] = tt.orders.size();
                                tt.tile_start.insert(tt.tile_start.end(), (size_t)P + 1, 0); continue; }
      const bool dg = mode == 1 || mode == 3;
      const int tile_m = pair ? P2_TILE : TILE_M, tile_n = pair ? (mode == 1 ? DP_TILE_N : (mode == 3 ? D1_TILE_N : P2_TILE)) : TILE_N;
      const int mg_rows_fixed = pair ? (mode == 3 ? D1_MG : DP_MG) : DG_MG;   // dgrad: row tiles sharing one converted weight tile
      int acc = 0;
      for (int p = 0; p < P; ++p) {
        ts[p] = acc;
        if (l < st[p].n_lin) {
          const LinDev& L = st[p].lin[l];
          const int M = mode == 2 ? L.n_out : T, N = mode == 0 ? L.n_out : L.n_in, K = mode == 0 ? L.n_in : ((dg || mode == 4) ? L.n_out : T);
          const int tm = cdiv(M, tile_m), tn = cdiv(N, tile_n), n_kb = cdiv(K, TILE_K);
          const int mg_rows = (pair && mode == 1) ? dgrad_pair_mg(T, L.n_in, dgrad_split_below) : mg_rows_fixed;
          const int groups = dg ? cdiv(tm, mg_rows) : tm;
          for (int g = 0; g < groups; ++g) {
            const int n_m = dg ? std::min(mg_rows, tm - g * mg_rows) : 1;
            for (int n = 0; n < tn; ++n) work.push_back({(long long)n_kb * n_m + 3 * n_m, acc + g * tn + n});
          }
          acc += groups * tn;
        }
      }
      ts[P] = acc;
      tt.max_tiles = std::max(tt.max_tiles, acc);
      tt.tile_start.insert(tt.tile_start.end(), ts_block.begin(), ts_block.end());
      for (int p = 0; p < P; ++p) tt.tile_start.insert(tt.tile_start.end(), (size_t)(ts_block[p + 1] - ts_block[p]), p);
      const int G = std::max(1, std::min(acc, pair ? sms / 2 : sms));     // persistent CTAs, or CTA pairs
      tt.grid[mode][l] = pair ? 2 * G : G;
      tt.order_off[mode][l] = tt.orders.size();
      if (acc == 0) { tt.n_slots[mode][l] = 0; continue; }
      std::stable_sort(work.begin(), work.end(), [](const std::pair<long long, int>& a, const std::pair<long long, int>& b) { return a.first > b.first; });
      std::vector<std::vector<int>> lists(G);
      std::vector<long long> load(G, 0);
      for (const auto& w : work) {
        int best = 0;
        for (int b = 1; b < G; ++b) if (load[b] < load[best]) best = b;
        lists[best].push_back(w.second);
        load[best] += w.first;
      }
      size_t max_len = 0;
      for (const auto& li : lists) max_len = std::max(max_len, li.size());
      tt.n_slots[mode][l] = (int)(max_len * G);
      tt.orders.resize(tt.orders.size() + max_len * G, -1);
      int* ord = tt.orders.data() + tt.order_off[mode][l];
      for (int b = 0; b < G; ++b)
        for (size_t k = 0; k < lists[b].size(); ++k) ord[k * G + b] = lists[b][k];
    }
  return tt;
}

static uint64_t maps_bytes(int P) { return (uint64_t)P * PM_MAX_LINEARS * MAPS_PER_LINEAR * sizeof(CUtensorMap); }
static uint64_t ints_bytes(size_t n) { return ((uint64_t)n * sizeof(int) + 255) / 256 * 256; }

uint64_t umma_workspace_bytes(int T, const std::vector<StageDev>& st, int dgrad_split_below) {
  const TileTables tt = build_tile_tables(T, st, device_sms(), dgrad_split_below);
  return 256 + maps_bytes((int)st.size()) + ints_bytes(tt.tile_start.size()) + ints_bytes(tt.orders.size()) + ints_bytes((size_t)tt.max_tiles);
}

static bool encode(EncodeTiledFn fn, CUtensorMap* m, int kind, void* base, int rank, const uint64_t* dims,
                   const uint64_t* strides_bytes, const uint32_t* box, std::string& err) {
  cuuint64_t gd[3]; cuuint64_t gs[2]; cuuint32_t bx[3]; cuuint32_t es[3] = {1, 1, 1};
  for (int i = 0; i < rank; ++i) { gd[i] = dims[i]; bx[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) gs[i] = strides_bytes[i];
  CUresult r = fn(m, kind >= 2 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, base, gd, gs, bx, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, kind == 3 ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { err = "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r); return false; }
  return true;
}

pm_status umma_plan_create(UmmaPlan** out, const TickArgs& t, const std::vector<StageDev>& st, void* ws_region, cudaStream_t stream, std::string& err) {
  *out = nullptr;
  void* fnp = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t ce = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fnp, cudaEnableDefault, &qres);
  if (ce != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fnp) { err = "cuTensorMapEncodeTiled is not available from this driver"; return PM_ERR_CUDA; }
  EncodeTiledFn fn = (EncodeTiledFn)fnp;
  const int P = t.P;
  std::vector<CUtensorMap> maps((size_t)P * PM_MAX_LINEARS * MAPS_PER_LINEAR);
  memset(maps.data(), 0, maps.size() * sizeof(CUtensorMap));
  UmmaPlan* plan = new UmmaPlan();
  plan->P = P;
  const uint64_t T = (uint64_t)t.T;
  for (int p = 0; p < P; ++p) {
    const StageDev& s = st[p];
    for (int l = 0; l < s.n_lin; ++l) {
      const LinDev& L = s.lin[l];
      CUtensorMap* m = maps.data() + ((size_t)p * PM_MAX_LINEARS + l) * MAPS_PER_LINEAR;
      // input activation of this Linear: ring [slots][T][n_in]
      const bool in_is_x = l == 0 && s.pre == PRE_NONE;
      char* act_base = t.ring + (l > 0 ? s.lin[l - 1].h_ring : (in_is_x ? s.x_ring : s.u_ring));
      const uint64_t slots = in_is_x ? (uint64_t)s.xdepth : (uint64_t)s.depth;
      const uint64_t n_in = (uint64_t)L.n_in, n_out = (uint64_t)L.n_out;
      bool okm = true;
      {
        uint64_t dims[3] = {n_in, T, slots}, strides[2] = {n_in * 2, T * n_in * 2};
        uint32_t box_k[3] = {TILE_K, TILE_M, 1}, box_mn[3] = {64, TILE_K, 1};
        okm = okm && encode(fn, m + MAP_ACT_K, 0, act_base, 3, dims, strides, box_k, err);
        okm = okm && encode(fn, m + MAP_ACT_MN, 0, act_base, 3, dims, strides, box_mn, err);
      }
      {
        uint64_t dims[2] = {n_in, n_out}, strides[1] = {n_in * 2}, strides4[1] = {n_in * 4};
        uint32_t box[2] = {TILE_K, TILE_N}, box4[2] = {TILE_N, TILE_K};
        {
          // forward operand: the bf16 copy of w; in microbatch-major order one copy per version the forward can reach
          uint64_t dims3[3] = {n_in, n_out, 1}, strides3[2] = {n_in * 2, n_in * n_out * 2};
          uint32_t box3[3] = {TILE_K, TILE_N, 1};
          void* wbase = (void*)(t.a.w_lp + L.w_off);
          if (t.mb_major) {
            dims3[2] = (uint64_t)(s.vdepth + s.rdepth); strides3[1] = (s.end - s.begin) * 2;
            wbase = (void*)(reinterpret_cast<__nv_bfloat16*>(t.ring + s.v_ring) + (L.w_off - s.begin));
          }
          okm = okm && encode(fn, m + MAP_W_K, 0, wbase, 3, dims3, strides3, box3, err);
          uint32_t box3mn[3] = {64, TILE_K, 1};                         // the same copies as an MN-major operand (dgrad against a queued version)
          okm = okm && encode(fn, m + MAP_W_MN, 0, wbase, 3, dims3, strides3, box3mn, err);
        }
        okm = okm && encode(fn, m + MAP_W_F32, 3, (void*)(t.a.w + L.w_off), 2, dims, strides4, box4, err);
        okm = okm && encode(fn, m + MAP_D_F32, 3, (void*)(t.a.delta + L.w_off), 2, dims, strides4, box4, err);
        uint32_t box4q[2] = {DP_HALF_N, DP_SLAB_K};                     // CTA-pair dgrad: slabs of 32 k-rows x 128 columns per CTA
        okm = okm && encode(fn, m + MAP_W_F32Q, 3, (void*)(t.a.w + L.w_off), 2, dims, strides4, box4q, err);
        okm = okm && encode(fn, m + MAP_D_F32Q, 3, (void*)(t.a.delta + L.w_off), 2, dims, strides4, box4q, err);
        uint32_t box4h[2] = {64, TILE_K};                               // 128-column pair dgrad: 64 columns per CTA
        okm = okm && encode(fn, m + MAP_W_F32H, 3, (void*)(t.a.w + L.w_off), 2, dims, strides4, box4h, err);
        okm = okm && encode(fn, m + MAP_D_F32H, 3, (void*)(t.a.delta + L.w_off), 2, dims, strides4, box4h, err);
      }
      {
        // dz operand (same rule as dz_src): dz scratch | dh scratch | attention's dy | rotating incoming-gradient mailbox
        char* dzb; uint64_t dz_slots = 1;
        if (bwd_act(L) != PM_ACT_NONE) dzb = t.ws + s.dz;
        else if (l < s.n_lin - 1) dzb = t.ws + s.dh;
        else if (feeds_attention(s.post)) dzb = t.ws + s.dy;
        else if (s.emit_memory) { dzb = t.ws + t.gmem_off; dz_slots = (uint64_t)t.gmem_depth; }
        else { dzb = t.ws + s.gin; dz_slots = (uint64_t)s.gin_depth; }
        uint64_t dims[3] = {n_out, T, dz_slots}, strides[2] = {n_out * 2, T * n_out * 2};
        uint32_t box_k[3] = {TILE_K, TILE_M, 1}, box_mn[3] = {64, TILE_K, 1};
        okm = okm && encode(fn, m + MAP_DZ_K, 0, dzb, 3, dims, strides, box_k, err);
        okm = okm && encode(fn, m + MAP_DZ_MN, 0, dzb, 3, dims, strides, box_mn, err);
      }
      {
        // outputs: 32-row boxes of one 128-byte swizzle row (64 bf16 or 32 fp32 columns)
        uint32_t box_bf[3] = {64, 32, 1}, box_f32[2] = {32, 32};
        uint64_t zd[3] = {n_out, T, (uint64_t)s.depth}, zs[2] = {n_out * 2, T * n_out * 2};
        if (L.flags & LF_WRITE_Z) okm = okm && encode(fn, m + MAP_Z_OUT, 1, t.ring + L.z_ring, 3, zd, zs, box_bf, err);
        if (L.flags & LF_OUT_F32) {
          uint64_t ld[3] = {n_out, T, 2}, ls[2] = {n_out * 4, T * n_out * 4};
          uint32_t box3[3] = {32, 32, 1};
          okm = okm && encode(fn, m + MAP_Y_OUT, 2, t.ws + t.yout_off, 3, ld, ls, box3, err);
        } else if (L.flags & LF_WRITE_Y) {
          char* ybase; uint64_t yslots;
          if (l < s.n_lin - 1) { ybase = t.ring + L.h_ring; yslots = (uint64_t)s.depth; }
          else if (s.emit_memory) { ybase = t.ring + t.mem_ring; yslots = (uint64_t)t.mem_depth; }   // the residual sum is the memory
          else if (p < P - 1) { ybase = t.ring + st[p + 1].x_ring; yslots = (uint64_t)st[p + 1].xdepth; }
          else { ybase = t.ws + t.yout_off; yslots = 2; }
          uint64_t yd[3] = {n_out, T, yslots};
          okm = okm && encode(fn, m + MAP_Y_OUT, 1, ybase, 3, yd, zs, box_bf, err);
        }
        if (!(p == 0 && l == 0 && s.pre != PRE_EMBED)) {
          const bool to_prev = l == 0 && s.pre == PRE_NONE;
          char* xbase = to_prev ? t.ws + st[p - 1].gin : t.ws + s.dh;
          uint64_t xd[3] = {n_in, T, (uint64_t)(to_prev ? st[p - 1].gin_depth : 1)}, xs[2] = {n_in * 2, T * n_in * 2};
          okm = okm && encode(fn, m + MAP_DX_OUT, 1, xbase, 3, xd, xs, box_bf, err);
        }
        uint64_t wd[2] = {n_in, n_out}, wst[1] = {n_in * 4};
        okm = okm && encode(fn, m + MAP_DW_OUT, 2, (void*)(t.a.grad + L.w_off), 2, wd, wst, box_f32, err);
      }
      if (!okm) { delete plan; return PM_ERR_CUDA; }
    }
  }
  const TileTables tt = build_tile_tables(t.T, st, device_sms(), t.dgrad_split_below);
  for (int mode = 0; mode < 5; ++mode)
    for (int l = 0; l < PM_MAX_LINEARS; ++l) {
      plan->n_slots[mode][l] = tt.n_slots[mode][l];
      plan->grid[mode][l] = tt.grid[mode][l];
      plan->pair[mode][l] = tt.pair[mode][l];
      plan->order_off[mode][l] = tt.order_off[mode][l];
      plan->ts_off[mode][l] = tt.ts_off[mode][l];
    }
  char* region = (char*)ws_region;
  cudaError_t e = cudaMemcpyAsync(region + 256, maps.data(), maps_bytes(P), cudaMemcpyHostToDevice, stream);
  char* ts_dev = region + 256 + maps_bytes(P);
  char* ord_dev = ts_dev + ints_bytes(tt.tile_start.size());
  if (e == cudaSuccess) e = cudaMemcpyAsync(ts_dev, tt.tile_start.data(), tt.tile_start.size() * sizeof(int), cudaMemcpyHostToDevice, stream);
  if (e == cudaSuccess && !tt.orders.empty()) e = cudaMemcpyAsync(ord_dev, tt.orders.data(), tt.orders.size() * sizeof(int), cudaMemcpyHostToDevice, stream);
  char* id_dev = ord_dev + ints_bytes(tt.orders.size());
  std::vector<int> identity((size_t)tt.max_tiles);
  for (int i = 0; i < tt.max_tiles; ++i) identity[(size_t)i] = i;
  if (e == cudaSuccess && tt.max_tiles > 0) e = cudaMemcpyAsync(id_dev, identity.data(), identity.size() * sizeof(int), cudaMemcpyHostToDevice, stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(region, 0, 256, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) { err = std::string("tensor map upload: ") + cudaGetErrorString(e); delete plan; return PM_ERR_CUDA; }
  e = cudaFuncSetAttribute((const void*)umma_gemm_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<0>::kSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute((const void*)umma_dgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DG_SMEM_BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute((const void*)umma_gemm_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<2>::kSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute((const void*)umma_gemm_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<1>::kSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute((const void*)umma_pair_gemm_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, P2_SMEM_BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute((const void*)umma_pair_gemm_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, P2_SMEM_BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute((const void*)umma_pair_gemm_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, P2_SMEM_BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute((const void*)umma_dgrad_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DP_SMEM_BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute((const void*)umma_dgrad_pair128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, D1_SMEM_BYTES);
  if (e != cudaSuccess) { err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); delete plan; return PM_ERR_CUDA; }
  plan->d_status = (int*)region;
  plan->d_maps = (const CUtensorMap*)(region + 256);
  plan->d_tile_start = (const int*)ts_dev;
  plan->d_orders = (const int*)ord_dev;
  plan->d_identity = (const int*)id_dev;
  plan->h_tile_start = tt.tile_start;
  plan->max_ctas = device_sms();
  *out = plan;
  return PM_OK;
}

void umma_plan_destroy(UmmaPlan* plan) { delete plan; }

// ---- self-test of the bounded wait ---------------------------------------------------------------------------
// One CTA, one thread: waits on an mbarrier on which nothing ever arrives, through the same bounded wait the GEMM
// kernels use, with the cycle limit given as an argument.  No tensor memory is allocated and no copy is in flight, so
// giving up is safe: the wait returns false, the abort flag and the status word are set, the kernel ends.
__global__ void wait_timeout_probe_kernel(int* status, long long limit_cycles, int* returned) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  const uint32_t b = smem_u32(&bar);
  mbar_init(b, 1);
  abort_flag = 0;
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  const bool ok = mbar_try_wait(b, 0) || mbar_wait_slow(b, 0, &abort_flag, status, 99, limit_cycles);
  *returned = ok ? 1 : (abort_flag ? 2 : 3);         // 2: gave up and raised the abort flag
}

cudaError_t umma_wait_timeout_probe(UmmaPlan* plan, long long limit_cycles, int* d_returned, cudaStream_t stream) {
  wait_timeout_probe_kernel<<<1, 1, 0, stream>>>(plan->d_status, limit_cycles, d_returned);
  return cudaGetLastError();
}
cudaError_t umma_clear_status(UmmaPlan* plan, cudaStream_t stream) { return cudaMemsetAsync(plan->d_status, 0, sizeof(int), stream); }

int* umma_status_word(UmmaPlan* plan) { return plan ? plan->d_status : nullptr; }

cudaError_t umma_launch(UmmaPlan* plan, const TickArgs& t, int mode, int lvl, cudaStream_t stream) {
  int n_slots = plan->n_slots[mode][lvl];
  if (n_slots == 0) return cudaSuccess;
  int grid = plan->grid[mode][lvl];                                   // one persistent CTA per SM
  const int* ts = plan->d_tile_start + plan->ts_off[mode][lvl];
  const int* ord = plan->d_orders + plan->order_off[mode][lvl];
  int tile0 = 0;
  bool narrow = false;                                                // dgrad of one narrow stage: 128-column tiles
  if (t.sel_p >= 0 && mode == 1 && plan->pair[1][lvl] && plan->pair[3][lvl]) {
    const int* h1 = plan->h_tile_start.data() + plan->ts_off[1][lvl];
    narrow = h1[t.sel_p + 1] - h1[t.sel_p] < 64;                      // too few 256-column tile groups for the CTA pairs
    if (narrow) { mode = 3; ts = plan->d_tile_start + plan->ts_off[3][lvl]; }
  }
  if (t.sel_p >= 0) {                                                 // the tiles of one stage, in ascending order
    const int* hts = plan->h_tile_start.data() + plan->ts_off[mode][lvl];
    const int first = hts[t.sel_p];
    n_slots = hts[t.sel_p + 1] - first;
    if (n_slots == 0) return cudaSuccess;
    ord = plan->d_identity + first;
    tile0 = first;
    const bool pr = plan->pair[mode][lvl];
    const int G = std::max(1, std::min(n_slots, pr ? plan->max_ctas / 2 : plan->max_ctas));
    grid = pr ? 2 * G : G;
  }
  TickArgs ta = t;
  ta.sel_tile0 = tile0;
  if (plan->pair[mode][lvl]) {
    if (mode == 0) umma_pair_gemm_kernel<0><<<grid, P2_THREADS, P2_SMEM_BYTES, stream>>>(ta, plan->d_maps, ts, ord, n_slots, lvl, plan->d_status);
    else if (mode == 1) umma_dgrad_pair_kernel<<<grid, DP_THREADS, DP_SMEM_BYTES, stream>>>(ta, plan->d_maps, ts, ord, n_slots, lvl, plan->d_status);
    else if (mode == 3) umma_dgrad_pair128_kernel<<<grid, D1_THREADS, D1_SMEM_BYTES, stream>>>(ta, plan->d_maps, ts, ord, n_slots, lvl, plan->d_status);
    else if (mode == 4) umma_pair_gemm_kernel<1><<<grid, P2_THREADS, P2_SMEM_BYTES, stream>>>(ta, plan->d_maps, ts, ord, n_slots, lvl, plan->d_status);
    else umma_pair_gemm_kernel<2><<<grid, P2_THREADS, P2_SMEM_BYTES, stream>>>(ta, plan->d_maps, ts, ord, n_slots, lvl, plan->d_status);
    return cudaGetLastError();
  }
  if (mode == 0) umma_gemm_kernel<0><<<grid, Cfg<0>::kThreads, Cfg<0>::kSmemBytes, stream>>>(ta, plan->d_maps, ts, ord, n_slots, lvl, plan->d_status);
  else if (mode == 1) umma_dgrad_kernel<<<grid, DG_THREADS, DG_SMEM_BYTES, stream>>>(ta, plan->d_maps, ts, ord, n_slots, lvl, plan->d_status);
  else if (mode == 4) umma_gemm_kernel<1><<<grid, Cfg<1>::kThreads, Cfg<1>::kSmemBytes, stream>>>(ta, plan->d_maps, ts, ord, n_slots, lvl, plan->d_status);
  else umma_gemm_kernel<2><<<grid, Cfg<2>::kThreads, Cfg<2>::kSmemBytes, stream>>>(ta, plan->d_maps, ts, ord, n_slots, lvl, plan->d_status);
  return cudaGetLastError();
}

}  // namespace pm

// Tensor-core projection kernel for sm_100a (the Linear operator of
// Section 3.2.2 re-designed for Blackwell): TMA feeds a ring of 128-byte
// swizzled shared-memory stages, one thread issues tcgen05.mma with FP32
// accumulators in tensor memory, four warps read the accumulators back with
// tcgen05.ld and apply the fused epilogue (Section 3.3.1).
//
// Orientation: the WEIGHT rows are the M = 128 side of the MMA and the tokens
// are the N side (16 .. 256), so one kernel covers prefill (N = 128 / 256) and
// batched decode (N = 16 .. 64).  Both operands are stored with the contraction
// index contiguous, which is the K-major layout TMA + tcgen05 want; the caller's
// weights are never copied or re-laid out.  An accumulator row (one output
// feature) lives in one TMEM lane = one epilogue thread; its columns are tokens.
//
// Persistent CTAs, one per SM.  Work is a list of segments (tile, k-block range):
//   mode 0 (prefill)  whole tiles, round-robin over CTAs, grouped raster
//   mode 1 (decode)   "stream-K": the (tile, k-block) space is cut into equal
//                     contiguous ranges so that every SM streams the same
//                     number of weight bytes whatever the shape (the paper's
//                     small-M path splits only N; with 128-row tiles that
//                     would leave most SMs idle).  A tile that spans several
//                     CTAs is finished by the last CTA to arrive, which adds
//                     the FP32 partials in a fixed order (deterministic).
// Two accumulator buffers in tensor memory let the epilogue of segment j
// overlap the MMAs of segment j+1.  The epilogue stages a chunk of the tile in
// shared memory and writes it out with 16-byte, fully coalesced stores.
//
// Roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA
// issuer, warps 2..5 = epilogue (warp w may touch TMEM lanes 32*(w%4)..+31).
// Every mbarrier wait is bounded; on expiry the status word gets
// THINFER_ETIMEOUT and the CTA tears down instead of hanging.
#pragma once
#include "epilogue.cuh"

namespace thinfer {

constexpr int kTcBM = 128;  // output features per tile
constexpr int kTcBK = 64;   // contraction elements per stage (128 bytes)
constexpr int kTcThreads = 192;
#ifndef THINFER_TC_MAX_STAGES
#define THINFER_TC_MAX_STAGES 8
#endif
constexpr int kTcMaxStages = THINFER_TC_MAX_STAGES;  // ring depth cap (small token tiles would allow more)
constexpr int kTcGroup = 8;          // feature tiles per raster group (keeps a weight panel and the activations in L2)

struct TcGemmArgs {
  int n_feat[3];  // rows of each weight matrix (QKV: q, k, v; SWIGLU: ffn for gate and for up; else one)
  int tiles[3];   // 128-row tiles per matrix
  int rows;       // tokens
  int k;          // contraction length
  int mode;       // 0 = whole tiles round-robin, 1 = stream-K
  int units_per_cta;  // stream-K: (tile, k-block) units per CTA
  float* partial_ws;  // stream-K: [n_tiles + grid][NA*BN][128] FP32 partial accumulators
  int* tile_counters; // stream-K: [n_tiles][2] arrival counters (claimed, parked), zero between launches
  unsigned long long* dbg;  // optional trace slots
  const float* sumsq_in;  // folded RMSNorm (see EpiArgs): per-tile sums of squares of the token operand, or nullptr
  int norm_dim;           // length of the normalised rows
  float norm_eps;
  int static_finisher;  // stream-K inside a cooperative launch: the CTA that holds the head of a tile finishes it
  int* status;        // device-visible status word
  EpiArgs e;
};

__host__ __device__ constexpr int tc_num_a(int epi) { return epi == EPI_SWIGLU ? 2 : 1; }
__host__ __device__ constexpr int tc_stage_bytes(int bn, int epi) { return tc_num_a(epi) * kTcBM * 128 + bn * 128; }
// epilogue staging: CW tokens x 128 features x 4 bytes
__host__ __device__ constexpr int tc_stage_out_bytes(int bn) { return (bn >= 32 ? 32 : 16) * kTcBM * 4; }
// Kernels that allocate tensor memory run one CTA per SM on this part (the occupancy query returns 1 for
// them whatever their register and shared-memory footprint), so the ring simply takes what one CTA can have.
__host__ __device__ constexpr int tc_ring_budget(int bn) { return 200000 - tc_stage_out_bytes(bn) + 16384; }
__host__ __device__ constexpr int tc_stages(int bn, int epi) {
  return (tc_ring_budget(bn) / tc_stage_bytes(bn, epi)) > kTcMaxStages ? kTcMaxStages : (tc_ring_budget(bn) / tc_stage_bytes(bn, epi));
}
__host__ __device__ constexpr int tc_acc_cols(int bn, int epi) { return tc_num_a(epi) * bn; }
__host__ __device__ constexpr int tc_tmem_cols(int bn, int epi) {
  int need = 2 * tc_acc_cols(bn, epi), c = 32;
  while (c < need) c <<= 1;
  return c;
}
__host__ __device__ constexpr int tc_smem_bytes(int bn, int epi) {
  return tc_stages(bn, epi) * tc_stage_bytes(bn, epi) + tc_stage_out_bytes(bn) + 1024 /*alignment slack*/ + 512 /*barriers, 1/rms*/;
}
__host__ __device__ constexpr bool tc_epi_fp32_stage(int epi) {
  return epi == EPI_RESID || epi == EPI_PLAIN_F32 || epi == EPI_SWIGLU_IL || epi == EPI_QKV_ROPE;
}
// output features per tile: the interleaved gate/up tile produces 64 (its 128 rows are 64 gate + 64 up rows)
__host__ __device__ constexpr int tc_tile_feats(int epi) { return epi == EPI_SWIGLU_IL ? 64 : kTcBM; }

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

struct TcSeg {
  int tile, kb0, kb1;
};

// The j-th segment of this CTA; false when there is none.  Every role walks the same sequence.
struct TcSegIter {
  int mode, n_tiles, nkb, next_tile, stride;
  long long u, u_end;
  TcSegIter() = default;
  __device__ TcSegIter(const TcGemmArgs& a, int n_tiles_, int nkb_) {
    mode = a.mode;
    n_tiles = n_tiles_;
    nkb = nkb_;
    next_tile = blockIdx.x;
    stride = gridDim.x;
    const long long total = static_cast<long long>(n_tiles_) * nkb_;
    u = static_cast<long long>(blockIdx.x) * a.units_per_cta;
    u_end = u + a.units_per_cta;
    if (u_end > total) u_end = total;
  }
  __device__ bool next(TcSeg& s) {
    if (mode == 0) {
      if (next_tile >= n_tiles) return false;
      s.tile = next_tile;
      s.kb0 = 0;
      s.kb1 = nkb;
      next_tile += stride;
      return true;
    }
    if (u >= u_end) return false;
    s.tile = static_cast<int>(u / nkb);
    s.kb0 = static_cast<int>(u - static_cast<long long>(s.tile) * nkb);
    const long long left = u_end - u;
    s.kb1 = (nkb - s.kb0 < left) ? nkb : s.kb0 + static_cast<int>(left);
    u += s.kb1 - s.kb0;
    return true;
  }
};

struct TcTile {
  int mat, feat0, feat_off, tok0;
};

template <int BN, int EPI>
__device__ __forceinline__ TcTile tc_tile_coords(const TcGemmArgs& a, int tile, int n_ft, int n_tt) {
  const int per_group = kTcGroup * n_tt;
  const int gid = tile / per_group;
  const int first_ft = gid * kTcGroup;
  const int gsz = min(kTcGroup, n_ft - first_ft);
  const int in_group = tile - gid * per_group;
  int ft = first_ft + in_group % gsz;
  TcTile t;
  t.tok0 = (in_group / gsz) * BN;
  t.mat = 0;
  t.feat_off = 0;
  if (EPI == EPI_QKV_ROPE) {
    if (ft >= a.tiles[0]) {
      ft -= a.tiles[0];
      t.mat = 1;
      t.feat_off = a.n_feat[0];
      if (ft >= a.tiles[1]) {
        ft -= a.tiles[1];
        t.mat = 2;
        t.feat_off += a.n_feat[1];
      }
    }
  }
  t.feat0 = ft * tc_tile_feats(EPI);
  return t;
}

// ---- epilogue of one chunk of CW token columns --------------------------------------------
// Phase A: thread `row` (one output feature) applies the element-wise part and writes its CW
// values to the staging tile [token][feature].  Phase B: the 128 threads copy the staged tile
// out in 16-byte pieces (8 features of one token), fully coalesced.
template <int EPI, int CW>
__device__ __forceinline__ void tc_emit_chunk(const TcGemmArgs& a, const TcTile& t, uint8_t* stage, int row, int ethread,
                                              const float (&v)[CW], const float (&v2)[CW], int tok_base) {
  const EpiArgs& e = a.e;
  constexpr bool F32 = tc_epi_fp32_stage(EPI);
  half_t* st16 = reinterpret_cast<half_t*>(stage);
  float* st32 = reinterpret_cast<float*>(stage);

  // RESID: the residual pieces this thread adds in phase B are requested now, so that their latency runs
  // under phase A and the barrier instead of once per piece (the stores below may alias the loads as far
  // as the compiler knows, so it would not move them up by itself)
  constexpr int kPieces = (CW * 16 + 127) / 128;
  uint4 rx[EPI == EPI_RESID ? kPieces : 1];
  if (EPI == EPI_RESID && (e.ld_out & 7) == 0) {
#pragma unroll
    for (int it = 0; it < kPieces; ++it) {
      const int idx = ethread + it * 128;
      const int c = idx >> 4, piece = idx & 15;
      const int r = tok_base + c, n0 = t.feat0 + piece * 8;
      rx[it] = make_uint4(0, 0, 0, 0);
      if (idx < CW * 16 && r < a.rows && a.n_feat[t.mat] - n0 >= 8) {
        const half_t* src = e.resid + static_cast<size_t>(r) * e.ld_out + n0;
        rx[it] = a.static_finisher ? __ldcg(reinterpret_cast<const uint4*>(src))  // written earlier in the same kernel
                                   : *reinterpret_cast<const uint4*>(src);        // written by an earlier kernel
      }
    }
  }

  // ---------------- phase A
  {
#pragma unroll
    for (int c = 0; c < CW; ++c) {
      if (F32) st32[c * kTcBM + row] = v[c];
      else if (EPI == EPI_SWIGLU) st16[c * kTcBM + row] = f_to_h(silu_f(v[c]) * v2[c]);
      else st16[c * kTcBM + row] = f_to_h(v[c]);
    }
  }
  epi_bar();

  // ---------------- phase B
  const int n_feat = a.n_feat[t.mat];
  if (EPI == EPI_SWIGLU_IL) {
    // rows 0..63 of the tile are gate features f0..f0+63, rows 64..127 the up rows of the same features
#pragma unroll
    for (int idx = ethread; idx < CW * 8; idx += 128) {
      const int c = idx >> 3, piece = idx & 7;
      const int r = tok_base + c;
      const int n0 = t.feat0 + piece * 8;
      if (r < a.rows && n0 < n_feat) {
        const float* g = st32 + c * kTcBM + piece * 8;
        const float* u = g + 64;
        half_t* dst = reinterpret_cast<half_t*>(e.out) + static_cast<size_t>(r) * e.ld_out + n0;
        if (n_feat - n0 >= 8 && (e.ld_out & 7) == 0) {
          uint4 o;
          o.x = pack2(silu_f(g[0]) * u[0], silu_f(g[1]) * u[1]);
          o.y = pack2(silu_f(g[2]) * u[2], silu_f(g[3]) * u[3]);
          o.z = pack2(silu_f(g[4]) * u[4], silu_f(g[5]) * u[5]);
          o.w = pack2(silu_f(g[6]) * u[6], silu_f(g[7]) * u[7]);
          *reinterpret_cast<uint4*>(dst) = o;
        } else {
          for (int j = 0; j < min(8, n_feat - n0); ++j) dst[j] = f_to_h(silu_f(g[j]) * u[j]);
        }
      }
    }
    epi_bar();
    return;
  }
#pragma unroll
  for (int it = 0; it < kPieces; ++it) {
    const int idx = ethread + it * 128;
    if (idx >= CW * 16) break;
    const int c = idx >> 4, piece = idx & 15;
    const int r = tok_base + c;
    const int n0 = t.feat0 + piece * 8;  // first feature of the piece inside its matrix
    const bool live = r < a.rows && n0 < n_feat;
    const int valid = min(8, n_feat - n0);
    float sq = 0.f;
    if (live) {
    if (EPI == EPI_QKV_ROPE) {
      const int b = r / e.seq_len, s = r - b * e.seq_len;
      const int h = n0 / e.head_dim, i = n0 - h * e.head_dim;
      half_t* dst;
      if (t.mat == 0) dst = e.q_out + ((static_cast<size_t>(b) * e.n_q_heads + h) * e.seq_len + s) * e.head_dim + i;
      else dst = (t.mat == 1 ? e.k_cache : e.v_cache) +
                 ((static_cast<size_t>(b) * e.n_kv_heads + h) * e.t_max + e.pos0 + s +
                  (e.pos_arr != nullptr ? e.pos_arr[b] : 0)) * e.head_dim + i;
      // the 8 staged FP32 sums are 4 rotation pairs (2j, 2j+1) of one head: their cos / sin are 4 consecutive
      // table entries, two 16-byte loads per piece (Algorithm 1; V rows are stored as they are)
      const float* src = st32 + c * kTcBM + piece * 8;
      float y[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) y[j] = src[j];
      if (t.mat != 2) {
        const int pos = e.pos0 + s + (e.pos_arr != nullptr ? e.pos_arr[b] : 0);
        const size_t o = static_cast<size_t>(pos) * (e.head_dim >> 1) + (i >> 1);
        const float4 cs = __ldg(reinterpret_cast<const float4*>(e.rope_cos + o));
        const float4 sn = __ldg(reinterpret_cast<const float4*>(e.rope_sin + o));
        const float c4[4] = {cs.x, cs.y, cs.z, cs.w}, s4[4] = {sn.x, sn.y, sn.z, sn.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float x0 = y[2 * j], x1 = y[2 * j + 1];
          y[2 * j] = fmaf(-x1, s4[j], x0 * c4[j]);
          y[2 * j + 1] = fmaf(x0, s4[j], x1 * c4[j]);
        }
      }
      uint4 o16;
      o16.x = pack2(y[0], y[1]);
      o16.y = pack2(y[2], y[3]);
      o16.z = pack2(y[4], y[5]);
      o16.w = pack2(y[6], y[7]);
      *reinterpret_cast<uint4*>(dst) = o16;
    } else {
      const size_t off = static_cast<size_t>(r) * e.ld_out + n0;
      const bool vec = valid == 8 && (e.ld_out & 7) == 0;
      if (EPI == EPI_PLAIN_F32) {
        float* dst = reinterpret_cast<float*>(e.out) + off;
        const float* src = st32 + c * kTcBM + piece * 8;
        if (vec) {
          reinterpret_cast<float4*>(dst)[0] = reinterpret_cast<const float4*>(src)[0];
          reinterpret_cast<float4*>(dst)[1] = reinterpret_cast<const float4*>(src)[1];
        } else {
          for (int j = 0; j < valid; ++j) dst[j] = src[j];
        }
      } else if (EPI == EPI_RESID) {
        half_t* dst = reinterpret_cast<half_t*>(e.out) + off;
        const float* src = st32 + c * kTcBM + piece * 8;
        if (vec) {
          float x[8];
          unpack8(rx[it], x);  // requested before phase A
          uint4 o;
          o.x = pack2(x[0] + src[0], x[1] + src[1]);
          o.y = pack2(x[2] + src[2], x[3] + src[3]);
          o.z = pack2(x[4] + src[4], x[5] + src[5]);
          o.w = pack2(x[6] + src[6], x[7] + src[7]);
          *reinterpret_cast<uint4*>(dst) = o;
          if (e.outg != nullptr) {  // folded RMSNorm of the next sub-layer (gain here, 1/rms there)
            float y[8], g[8];
            unpack8(o, y);
            unpack8(ldg_cached(e.gain_next + n0), g);
            uint4 og;
            og.x = pack2(y[0] * g[0], y[1] * g[1]);
            og.y = pack2(y[2] * g[2], y[3] * g[3]);
            og.z = pack2(y[4] * g[4], y[5] * g[5]);
            og.w = pack2(y[6] * g[6], y[7] * g[7]);
            *reinterpret_cast<uint4*>(e.outg + off) = og;
#pragma unroll
            for (int j = 0; j < 8; ++j) sq = fmaf(y[j], y[j], sq);
          }
        } else {
          for (int j = 0; j < valid; ++j) {
            const half_t yh = f_to_h(h_to_f(__ldcg(e.resid + off + j)) + src[j]);
            dst[j] = yh;
            if (e.outg != nullptr) {
              const float y = h_to_f(yh);
              e.outg[off + j] = f_to_h(y * h_to_f(e.gain_next[n0 + j]));
              sq = fmaf(y, y, sq);
            }
          }
        }
      } else {  // PLAIN_F16, SWIGLU
        half_t* dst = reinterpret_cast<half_t*>(e.out) + off;
        const half_t* src = st16 + c * kTcBM + piece * 8;
        if (vec) {
          *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
        } else {
          for (int j = 0; j < valid; ++j) dst[j] = src[j];
        }
      }
    }
    }  // live
    if (EPI == EPI_RESID && e.outg != nullptr) {
      // the 16 pieces of one token sit in 16 consecutive lanes: add their squares, lane 0 of the group
      // records the tile's contribution (every lane takes part in the shuffles)
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
      if (piece == 0 && r < a.rows) e.sumsq[(t.feat0 / kTcBM) * 64 + r] = sq;
    }
  }
  epi_bar();
}

template <int CW>
__device__ __forceinline__ void tc_load_acc(uint32_t taddr, float (&f)[CW]) {
  uint32_t r[CW];
  if constexpr (CW == 32) tmem_ld32(taddr, r);
  else tmem_ld16(taddr, r);
  tmem_ld_wait();
#pragma unroll
  for (int c = 0; c < CW; ++c) f[c] = __uint_as_float(r[c]);
}

// ---- epilogue of one segment ------------------------------------------------------------------
// Reads the accumulator buffer of the segment from tensor memory.  A whole tile is finished
// directly; a partial one (stream-K) is parked in the workspace and finished by the last CTA to
// arrive, which adds the partials in slot order.  `col_scale` (shared memory, one factor per token
// column of the tile, or nullptr) multiplies the finished sums before the element-wise part: the
// 1/rms of a folded RMSNorm.  Called by the 128 epilogue threads.
template <int BN, int EPI>
__device__ __forceinline__ void tc_epilogue_segment(const TcGemmArgs& a, const TcSeg& sg, const TcTile& t, uint32_t acc,
                                                    uint64_t* tempty, uint8_t* stage_out, int* flag, int row,
                                                    int ethread, int lane, int nkb, const float* col_scale) {
  constexpr int NA = tc_num_a(EPI);
  constexpr int ACC_COLS = tc_acc_cols(BN, EPI);
  constexpr int CW = BN >= 32 ? 32 : 16;
  const bool whole = sg.kb0 == 0 && sg.kb1 == nkb;
  if (whole) {
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += CW) {
      float v[CW], v2[CW];
      tc_load_acc<CW>(acc + c0, v);
      if (NA == 2) tc_load_acc<CW>(acc + BN + c0, v2);
      if (c0 + CW >= BN) {  // accumulator fully read: hand it back to the MMA warp
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty);
      }
      if (col_scale != nullptr) {
#pragma unroll
        for (int c = 0; c < CW; ++c) {
          v[c] *= col_scale[c0 + c];
          if (NA == 2) v2[c] *= col_scale[c0 + c];
        }
      }
      tc_emit_chunk<EPI, CW>(a, t, stage_out, row, ethread, v, v2, t.tok0 + c0);
    }
    return;
  }
  // stream-K: the tile is split over CTAs first_cta .. last_cta; one of them (the finisher) adds the FP32
  // partial accumulators of the others to its own, in CTA order, and runs the element-wise epilogue.
  const long long first_unit = static_cast<long long>(sg.tile) * nkb;
  const int first_cta = static_cast<int>(first_unit / a.units_per_cta);
  const int last_cta = static_cast<int>((first_unit + nkb - 1) / a.units_per_cta);
  const int n_seg = last_cta - first_cta + 1;
  const int mine = static_cast<int>(blockIdx.x) - first_cta;
  float* slot = a.partial_ws + static_cast<size_t>(sg.tile + blockIdx.x) * (ACC_COLS * kTcBM);
  int* claimed = a.tile_counters + 2 * sg.tile;  // CTAs that have reached their epilogue of this tile
  int* parked = claimed + 1;                     // CTAs whose partial is complete in the workspace

  // Adds the parked partials of segments [s_begin, s_end) for chunk c0, in order; the loads of up to four
  // segments are in flight together (one L2 round trip instead of one per segment).
  auto add_partials = [&](int s_begin, int s_end, int c0, float (&v)[CW], float (&v2)[CW]) {
    constexpr int PB = CW == 16 ? 4 : 1;
    for (int s0 = s_begin; s0 < s_end; s0 += PB) {
      float p[PB][CW], p2[PB][CW];
#pragma unroll
      for (int u = 0; u < PB; ++u) {
        const bool on = s0 + u < s_end;
        const float* src = a.partial_ws + static_cast<size_t>(sg.tile + first_cta + (on ? s0 + u : s_begin)) * (ACC_COLS * kTcBM);
#pragma unroll
        for (int c = 0; c < CW; ++c) {
          p[u][c] = on ? __ldcg(src + (c0 + c) * kTcBM + row) : 0.f;
          if (NA == 2) p2[u][c] = on ? __ldcg(src + (BN + c0 + c) * kTcBM + row) : 0.f;
        }
      }
#pragma unroll
      for (int u = 0; u < PB; ++u) {
#pragma unroll
        for (int c = 0; c < CW; ++c) {
          v[c] += p[u][c];
          if (NA == 2) v2[c] += p2[u][c];
        }
      }
    }
  };

  if (!a.static_finisher) {
    // Everybody parks its partial at once and claims a ticket while the stores drain; whoever holds the last
    // ticket adds all slots in CTA order (its own included) once they are all marked complete.
#pragma unroll 1
    for (int c0 = 0; c0 < ACC_COLS; c0 += CW) {
      float v[CW];
      tc_load_acc<CW>(acc + c0, v);
#pragma unroll
      for (int c = 0; c < CW; ++c) slot[(c0 + c) * kTcBM + row] = v[c];
    }
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(tempty);
    int ticket = 0;
    if (ethread == 0) ticket = atomicAdd(claimed, 1);  // travels while the other threads' fences complete
    __threadfence();
    epi_bar();
    if (ethread == 0) {
      atomicAdd(parked, 1);
      int ok = ticket == n_seg - 1 ? 1 : 0;
      if (ok) {  // last ticket: wait (bounded) until every slot is complete
        const uint64_t t0 = global_ns();
        uint32_t polls = 0;
        for (;;) {
          int seen;
          asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(parked) : "memory");
          if (seen >= n_seg) break;
          if ((++polls & 0xffu) == 0u && global_ns() - t0 > kWaitLimitNs) {
            if (a.status != nullptr) *reinterpret_cast<volatile int*>(a.status) = kErrTimeout;
            ok = 0;
            break;
          }
        }
      }
      *flag = ok;
    }
    epi_bar();
    if (*reinterpret_cast<volatile int*>(flag) == 0) return;
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += CW) {
      float v[CW], v2[CW];
#pragma unroll
      for (int c = 0; c < CW; ++c) v[c] = v2[c] = 0.f;
      add_partials(0, n_seg, c0, v, v2);
      if (col_scale != nullptr) {
#pragma unroll
        for (int c = 0; c < CW; ++c) {
          v[c] *= col_scale[c0 + c];
          if (NA == 2) v2[c] *= col_scale[c0 + c];
        }
      }
      tc_emit_chunk<EPI, CW>(a, t, stage_out, row, ethread, v, v2, t.tok0 + c0);
    }
    if (ethread == 0) {  // ready for the next launch
      *claimed = 0;
      *parked = 0;
    }
    return;
  }

  // Cooperative launch (all CTAs resident): the CTA that holds the head of the tile finishes it - the head is
  // the LAST segment it works on, every other segment is the FIRST one of another CTA, parked long ago.
  const bool finisher = sg.kb0 == 0;
  if (!finisher) {
#pragma unroll 1
    for (int c0 = 0; c0 < ACC_COLS; c0 += CW) {
      float v[CW];
      tc_load_acc<CW>(acc + c0, v);
#pragma unroll
      for (int c = 0; c < CW; ++c) slot[(c0 + c) * kTcBM + row] = v[c];
    }
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(tempty);
    __threadfence();
    epi_bar();
    if (ethread == 0) atomicAdd(parked, 1);
    return;
  }

  // finisher: the others have claimed before (or are known to be ahead); wait for their partials (bounded)
  if (ethread == 0) {
    const uint64_t t0 = global_ns();
    uint32_t polls = 0;
    int ok = 1;
    for (;;) {
      int seen;
      asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(parked) : "memory");
      if (seen >= n_seg - 1) break;
      if ((++polls & 0xffu) == 0u && global_ns() - t0 > kWaitLimitNs) {
        if (a.status != nullptr) *reinterpret_cast<volatile int*>(a.status) = kErrTimeout;
        ok = 0;
        break;
      }
    }
    *flag = ok;
  }
  epi_bar();
  const bool ok = *reinterpret_cast<volatile int*>(flag) != 0;
#pragma unroll 1
  for (int c0 = 0; c0 < BN; c0 += CW) {
    float own[CW], own2[CW], v[CW], v2[CW];
    tc_load_acc<CW>(acc + c0, own);
    if (NA == 2) tc_load_acc<CW>(acc + BN + c0, own2);
    if (c0 + CW >= BN) {
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty);
    }
    if (ok) {
      // sum in CTA order whoever finishes: the result does not depend on arrival order
#pragma unroll
      for (int c = 0; c < CW; ++c) v[c] = v2[c] = 0.f;
      add_partials(0, mine, c0, v, v2);
#pragma unroll
      for (int c = 0; c < CW; ++c) {
        v[c] += own[c];
        if (NA == 2) v2[c] += own2[c];
      }
      add_partials(mine + 1, n_seg, c0, v, v2);
      if (col_scale != nullptr) {
#pragma unroll
        for (int c = 0; c < CW; ++c) {
          v[c] *= col_scale[c0 + c];
          if (NA == 2) v2[c] *= col_scale[c0 + c];
        }
      }
      tc_emit_chunk<EPI, CW>(a, t, stage_out, row, ethread, v, v2, t.tok0 + c0);
    }
  }
  if (ethread == 0) {  // ready for the next unit / launch
    *claimed = 0;
    *parked = 0;
  }
}

template <int BN, int EPI>
__global__ void __launch_bounds__(kTcThreads, 1)
    tc_gemm_kernel(const __grid_constant__ CUtensorMap tm_w0, const __grid_constant__ CUtensorMap tm_w1,
                   const __grid_constant__ CUtensorMap tm_w2, const __grid_constant__ CUtensorMap tm_x,
                   const TcGemmArgs a) {
  constexpr int NA = tc_num_a(EPI);
  constexpr int STAGES = tc_stages(BN, EPI);
  constexpr int STAGE_BYTES = tc_stage_bytes(BN, EPI);
  constexpr int A_BYTES = kTcBM * 128;
  constexpr int ACC_COLS = tc_acc_cols(BN, EPI);
  constexpr int TMEM_COLS = tc_tmem_cols(BN, EPI);
  constexpr int CW = BN >= 32 ? 32 : 16;
  constexpr uint32_t IDESC = idesc_f16(kTcBM, BN, 0, 0);
  static_assert(2 * ACC_COLS <= 512, "two accumulator buffers must fit in tensor memory");

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* stage_out = smem + STAGES * STAGE_BYTES;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(stage_out + tc_stage_out_bytes(BN));
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* tfull_bar = empty_bar + STAGES;   // [2] accumulator ready for the epilogue
  uint64_t* tempty_bar = tfull_bar + 2;       // [2] accumulator drained by the epilogue
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(tempty_bar + 2);
  int* flag = reinterpret_cast<int*>(tmem_holder + 1);
  float* rstd_sm = reinterpret_cast<float*>(flag + 1);  // [BN] 1/rms per token column when the norm is folded

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_ft = a.tiles[0] + a.tiles[1] + a.tiles[2];
  const int n_tt = (a.rows + BN - 1) / BN;
  const int n_tiles = n_ft * n_tt;
  const int nkb = (a.k + kTcBK - 1) / kTcBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&tfull_bar[i], 1);
      mbar_init(&tempty_bar[i], 4);  // one arrival per epilogue warp
    }
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(tmem_holder, TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_holder);
  pdl_launch_dependents();
  if (a.dbg != nullptr && threadIdx.x == 0) {
    atomicMin(a.dbg + 10, static_cast<unsigned long long>(global_ns()));
    if (blockIdx.x == 0) a.dbg[0] = global_ns();
  }

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_w0);
      tma_prefetch_desc(&tm_x);
      // Weights do not depend on the previous kernel of the step: in decode the first ring-full of
      // weight tiles is requested before the dependency wait, the token tiles follow after it.
      const uint32_t pre = a.mode == 1 ? STAGES : 0;
      {
        TcSegIter it(a, n_tiles, nkb);
        TcSeg sg;
        uint32_t n = 0;
        while (n < pre && it.next(sg)) {
          const TcTile t = tc_tile_coords<BN, EPI>(a, sg.tile, n_ft, n_tt);
          const CUtensorMap* tmw = (EPI == EPI_QKV_ROPE) ? (t.mat == 0 ? &tm_w0 : (t.mat == 1 ? &tm_w1 : &tm_w2)) : &tm_w0;
          for (int kb = sg.kb0; kb < sg.kb1 && n < pre; ++kb, ++n) {
            uint8_t* st = smem + n * STAGE_BYTES;
            mbar_expect_tx(&full_bar[n], STAGE_BYTES);
            tma_load_2d(st, tmw, &full_bar[n], kb * kTcBK, t.feat0);
            if (NA == 2) tma_load_2d(st + A_BYTES, &tm_w1, &full_bar[n], kb * kTcBK, t.feat0);
            if (EPI == EPI_SWIGLU_IL) tma_load_2d(st + A_BYTES / 2, &tm_w1, &full_bar[n], kb * kTcBK, t.feat0);
          }
        }
      }
      pdl_wait();
      if (a.dbg != nullptr) {
        atomicMin(a.dbg + 11, static_cast<unsigned long long>(global_ns()));
        if (blockIdx.x == 0) a.dbg[1] = global_ns();
      }
      TcSegIter it(a, n_tiles, nkb);
      TcSeg sg;
      uint32_t n = 0;  // k-blocks issued so far (ring position)
      bool ok = true;
      while (ok && it.next(sg)) {
        const TcTile t = tc_tile_coords<BN, EPI>(a, sg.tile, n_ft, n_tt);
        const CUtensorMap* tmw = (EPI == EPI_QKV_ROPE) ? (t.mat == 0 ? &tm_w0 : (t.mat == 1 ? &tm_w1 : &tm_w2)) : &tm_w0;
        for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++n) {
          const int s = n % STAGES;
          uint8_t* st = smem + s * STAGE_BYTES;
          if (n >= pre) {
            if (!mbar_wait(&empty_bar[s], ((n / STAGES) & 1) ^ 1u, a.status)) {
              ok = false;
              break;
            }
            mbar_expect_tx(&full_bar[s], STAGE_BYTES);
            tma_load_2d(st, tmw, &full_bar[s], kb * kTcBK, t.feat0);
            if (NA == 2) tma_load_2d(st + A_BYTES, &tm_w1, &full_bar[s], kb * kTcBK, t.feat0);
            if (EPI == EPI_SWIGLU_IL) tma_load_2d(st + A_BYTES / 2, &tm_w1, &full_bar[s], kb * kTcBK, t.feat0);
          }
          tma_load_2d(st + NA * A_BYTES, &tm_x, &full_bar[s], kb * kTcBK, t.tok0);
        }
      }
      if (a.dbg != nullptr) {
        atomicMax(a.dbg + 12, static_cast<unsigned long long>(global_ns()));
        if (blockIdx.x == 0) a.dbg[2] = global_ns();
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      TcSegIter it(a, n_tiles, nkb);
      TcSeg sg;
      uint32_t n = 0, j = 0;
      bool ok = true;
      while (ok && it.next(sg)) {
        const uint32_t buf = j & 1, use = j >> 1;
        if (!mbar_wait(&tempty_bar[buf], (use & 1) ^ 1u, a.status)) break;
        tc_fence_after();
        const uint32_t acc = tmem_base + buf * ACC_COLS;
        for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++n) {
          const int s = n % STAGES;
          if (!mbar_wait(&full_bar[s], (n / STAGES) & 1, a.status)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + s * STAGE_BYTES);
          const uint64_t da = smem_desc_sw128(sa, 16, 1024);
          const uint64_t da2 = smem_desc_sw128(sa + A_BYTES, 16, 1024);
          const uint64_t db = smem_desc_sw128(sa + NA * A_BYTES, 16, 1024);
#pragma unroll
          for (int k = 0; k < kTcBK / 16; ++k) {
            const uint32_t accum = (kb != sg.kb0 || k != 0) ? 1u : 0u;
            tc_mma_f16(acc, da + 2 * k, db + 2 * k, IDESC, accum);  // +32 bytes per K=16 step
            if (NA == 2) tc_mma_f16(acc + BN, da2 + 2 * k, db + 2 * k, IDESC, accum);
          }
          tc_commit(&empty_bar[s]);  // frees the stage once these MMAs have read it
        }
        if (ok) tc_commit(&tfull_bar[buf]);
        ++j;
      }
      if (a.dbg != nullptr) atomicMax(a.dbg + 13, static_cast<unsigned long long>(global_ns()));
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    const int row = q * 32 + lane;
    const int ethread = (warp - 2) * 32 + lane;
    const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    pdl_wait();  // residual stream, RoPE positions, stream-K scratch: all written by earlier kernels
    if (a.sumsq_in != nullptr) {
      // one token tile (decode): 1/rms per token from the per-tile sums the previous projection left
      if (ethread < BN) {
        float r = 0.f;
        if (ethread < a.rows) {
          const int parts = (a.norm_dim + kTcBM - 1) / kTcBM;
          float ssum = 0.f;
          for (int p = 0; p < parts; ++p) ssum += __ldcg(a.sumsq_in + p * 64 + ethread);
          r = rsqrtf(ssum / static_cast<float>(a.norm_dim) + a.norm_eps);
        }
        rstd_sm[ethread] = r;
      }
      epi_bar();
    }
    const float* col_scale = a.sumsq_in != nullptr ? rstd_sm : nullptr;
    TcSegIter it(a, n_tiles, nkb);
    TcSeg sg;
    uint32_t j = 0;
    while (it.next(sg)) {
      const uint32_t buf = j & 1, use = j >> 1;
      ++j;
      const TcTile t = tc_tile_coords<BN, EPI>(a, sg.tile, n_ft, n_tt);
      if (EPI == EPI_RESID && BN <= 64 && ethread < 2 * BN) {
        // decode: pull the residual rows this tile may need (two 128-byte lines per token) into L1 while the
        // weights stream, so the end-of-kernel epilogue does not pay an L2 round trip for them
        const int r = t.tok0 + (ethread >> 1);
        if (r < a.rows && t.feat0 + (ethread & 1) * 64 < a.n_feat[0])
          asm volatile("prefetch.global.L1 [%0];" ::"l"(a.e.resid + static_cast<size_t>(r) * a.e.ld_out + t.feat0 + (ethread & 1) * 64));
      }
      if (!mbar_wait(&tfull_bar[buf], use & 1, a.status)) break;
      tc_fence_after();
      const uint32_t acc = lane_base + buf * ACC_COLS;
      if (a.dbg != nullptr && ethread == 0) atomicMax(a.dbg + 14, static_cast<unsigned long long>(global_ns()));
      tc_epilogue_segment<BN, EPI>(a, sg, t, acc, &tempty_bar[buf], stage_out, flag, row, ethread, lane, nkb, col_scale);
    }
    if (a.dbg != nullptr && ethread == 0) atomicMax(a.dbg + 15, static_cast<unsigned long long>(global_ns()));
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
}

}  // namespace thinfer

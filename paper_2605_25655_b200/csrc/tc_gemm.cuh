// Tensor-core projection kernel for sm_100a (the large-M Linear of
// Section 3.2.2, re-designed for Blackwell): TMA feeds a ring of 128-byte
// swizzled shared-memory stages, one thread issues tcgen05.mma with the FP32
// accumulator in tensor memory, four warps read the accumulator back with
// tcgen05.ld and apply the fused epilogue (Section 3.3.1).
//
// Orientation: the WEIGHT rows are the M = 128 side of the MMA and the tokens
// are the N side (16 .. 256), so the same kernel covers prefill (N = 256) and
// batched decode (N = 16).  Both operands are stored with the contraction
// index contiguous, which is exactly the K-major layout TMA + tcgen05 want; no
// copy or re-layout of the caller's weights is made.  An accumulator row (one
// output feature) lives in one TMEM lane = one epilogue thread; its columns are
// the tokens.
//
// Roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA
// issuer, warps 2..5 = epilogue (warp w may touch TMEM lanes 32*(w%4)..+31).
// Every mbarrier wait is bounded; on expiry the status word gets
// THINFER_ETIMEOUT and the CTA tears down instead of hanging.
#pragma once
#include "epilogue.cuh"

namespace thinfer {

constexpr int kTcBM = 128;  // output features per CTA
constexpr int kTcBK = 64;   // contraction elements per stage (128 bytes)
constexpr int kTcThreads = 192;
constexpr int kTcGroup = 8;  // feature tiles per raster group (keeps a weight panel and the activations in L2)

struct TcGemmArgs {
  int n_feat[3];  // rows of each weight matrix (QKV: q, k, v; SWIGLU: ffn for gate and for up; else one)
  int tiles[3];   // 128-row tiles per matrix
  int rows;       // tokens
  int k;          // contraction length
  int* status;    // device-visible status word
  EpiArgs e;
};

__host__ __device__ constexpr int tc_num_a(int epi) { return epi == EPI_SWIGLU ? 2 : 1; }
__host__ __device__ constexpr int tc_stage_bytes(int bn, int epi) { return tc_num_a(epi) * kTcBM * 128 + bn * 128; }
__host__ __device__ constexpr int tc_stages(int bn, int epi) {
  return (200000 / tc_stage_bytes(bn, epi)) > 8 ? 8 : (200000 / tc_stage_bytes(bn, epi));
}
__host__ __device__ constexpr int tc_tmem_cols(int bn, int epi) {
  int need = tc_num_a(epi) * bn, c = 32;
  while (c < need) c <<= 1;
  return c;
}
__host__ __device__ constexpr int tc_smem_bytes(int bn, int epi) {
  return tc_stages(bn, epi) * tc_stage_bytes(bn, epi) + 1024 /*alignment slack*/ + 256 /*barriers*/;
}

// ---- epilogue for one chunk of CW token columns held by this thread (feature n) ----
template <int EPI, int CW>
__device__ __forceinline__ void tc_epilogue_chunk(const TcGemmArgs& a, const float (&acc)[CW], const float (&acc2)[CW],
                                                  int n_cat, bool n_valid, int n_local, int tok_base) {
  const EpiArgs& e = a.e;
  if (EPI == EPI_QKV_ROPE) {
    // per-thread constants: which buffer, which head, which element of the head
    int kind = 0, nn = n_cat;
    if (nn >= e.n_q) {
      nn -= e.n_q;
      kind = 1;
      if (nn >= e.n_kv) {
        nn -= e.n_kv;
        kind = 2;
      }
    }
    const int h = nn / e.head_dim, i = nn - h * e.head_dim;
    const int half = e.head_dim >> 1;
    __half* dst = kind == 0 ? e.q_out : (kind == 1 ? e.k_cache : e.v_cache);
    int b = tok_base / e.seq_len, s = tok_base - b * e.seq_len;
#pragma unroll
    for (int c = 0; c < CW; ++c) {
      float v = acc[c];
      const float partner = __shfl_xor_sync(0xffffffffu, v, 1);  // the other element of the (2j, 2j+1) pair
      const int r = tok_base + c;
      if (n_valid && r < a.rows) {
        const int pos = e.pos0 + s;
        if (kind != 2) {
          const float cs = __ldg(e.rope_cos + static_cast<size_t>(pos) * half + (i >> 1));
          const float sn = __ldg(e.rope_sin + static_cast<size_t>(pos) * half + (i >> 1));
          v = (i & 1) ? fmaf(partner, sn, v * cs) : fmaf(-partner, sn, v * cs);
        }
        const size_t off = kind == 0
                               ? ((static_cast<size_t>(b) * e.n_q_heads + h) * e.seq_len + s) * e.head_dim + i
                               : ((static_cast<size_t>(b) * e.n_kv_heads + h) * e.t_max + pos) * e.head_dim + i;
        dst[off] = __float2half_rn(v);
      }
      if (++s == e.seq_len) {
        s = 0;
        ++b;
      }
    }
  } else {
#pragma unroll
    for (int c = 0; c < CW; ++c) {
      const int r = tok_base + c;
      if (n_valid && r < a.rows) {
        const size_t off = static_cast<size_t>(r) * e.ld_out + n_local;
        if (EPI == EPI_PLAIN_F16) {
          reinterpret_cast<__half*>(e.out)[off] = __float2half_rn(acc[c]);
        } else if (EPI == EPI_PLAIN_F32) {
          reinterpret_cast<float*>(e.out)[off] = acc[c];
        } else if (EPI == EPI_RESID) {
          reinterpret_cast<__half*>(e.out)[off] = __float2half_rn(__half2float(e.resid[off]) + acc[c]);
        } else {  // EPI_SWIGLU: acc = gate, acc2 = up
          reinterpret_cast<__half*>(e.out)[off] = __float2half_rn(silu_f(acc[c]) * acc2[c]);
        }
      }
    }
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
  constexpr int TMEM_COLS = tc_tmem_cols(BN, EPI);
  constexpr int CW = BN >= 32 ? 32 : 16;
  constexpr uint32_t IDESC = idesc_f16(kTcBM, BN, 0, 0);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* acc_bar = empty_bar + STAGES;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_bar + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- tile coordinates (grouped raster: kTcGroup feature tiles x all token tiles) ----
  const int n_ft = a.tiles[0] + a.tiles[1] + a.tiles[2];
  const int n_tt = (a.rows + BN - 1) / BN;
  const int per_group = kTcGroup * n_tt;
  const int gid = blockIdx.x / per_group;
  const int first_ft = gid * kTcGroup;
  const int gsz = min(kTcGroup, n_ft - first_ft);
  const int in_group = blockIdx.x - gid * per_group;
  int ft = first_ft + in_group % gsz;
  const int tt = in_group / gsz;
  int mat = 0, feat_off = 0;
  if (EPI == EPI_QKV_ROPE) {
    if (ft >= a.tiles[0]) {
      ft -= a.tiles[0];
      mat = 1;
      feat_off = a.n_feat[0];
      if (ft >= a.tiles[1]) {
        ft -= a.tiles[1];
        mat = 2;
        feat_off += a.n_feat[1];
      }
    }
  }
  const int feat0 = ft * kTcBM;  // first weight row of this tile inside its matrix
  const int tok0 = tt * BN;
  const int nkb = (a.k + kTcBK - 1) / kTcBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(acc_bar, 1);
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(tmem_holder, TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_holder);

  if (warp == 0) {
    if (lane == 0) {
      const CUtensorMap* tmw = (EPI == EPI_QKV_ROPE) ? (mat == 0 ? &tm_w0 : (mat == 1 ? &tm_w1 : &tm_w2)) : &tm_w0;
      tma_prefetch_desc(tmw);
      tma_prefetch_desc(&tm_x);
      for (int kb = 0; kb < nkb; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        if (!mbar_wait(&empty_bar[s], ph ^ 1u, a.status)) break;
        uint8_t* st = smem + s * STAGE_BYTES;
        mbar_expect_tx(&full_bar[s], STAGE_BYTES);
        tma_load_2d(st, tmw, &full_bar[s], kb * kTcBK, feat0);
        if (NA == 2) tma_load_2d(st + A_BYTES, &tm_w1, &full_bar[s], kb * kTcBK, feat0);
        tma_load_2d(st + NA * A_BYTES, &tm_x, &full_bar[s], kb * kTcBK, tok0);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      for (int kb = 0; kb < nkb; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        if (!mbar_wait(&full_bar[s], ph, a.status)) break;
        tc_fence_after();
        const uint32_t sa = smem_u32(smem + s * STAGE_BYTES);
        const uint64_t da = smem_desc_sw128(sa, 16, 1024);
        const uint64_t da2 = smem_desc_sw128(sa + A_BYTES, 16, 1024);
        const uint64_t db = smem_desc_sw128(sa + NA * A_BYTES, 16, 1024);
#pragma unroll
        for (int k = 0; k < kTcBK / 16; ++k) {
          const uint32_t accum = (kb | k) != 0 ? 1u : 0u;
          tc_mma_f16(tmem_base, da + 2 * k, db + 2 * k, IDESC, accum);  // +32 bytes per K=16 step
          if (NA == 2) tc_mma_f16(tmem_base + BN, da2 + 2 * k, db + 2 * k, IDESC, accum);
        }
        tc_commit(&empty_bar[s]);  // frees the stage once these MMAs have read it
      }
      tc_commit(acc_bar);
    }
  } else {
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    const int row = q * 32 + lane;
    const bool n_valid = feat0 + row < a.n_feat[mat];
    const int n_local = feat0 + row;
    const int n_cat = feat_off + n_local;
    if (mbar_wait(acc_bar, 0, a.status)) {
      tc_fence_after();
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += CW) {
        uint32_t r1[CW], r2[CW];
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + c0;
        if constexpr (CW == 32) {
          tmem_ld32(taddr, r1);
          if (NA == 2) tmem_ld32(taddr + BN, r2);
        } else {
          tmem_ld16(taddr, r1);
          if (NA == 2) tmem_ld16(taddr + BN, r2);
        }
        tmem_ld_wait();
        float f1[CW], f2[CW];
#pragma unroll
        for (int c = 0; c < CW; ++c) {
          f1[c] = __uint_as_float(r1[c]);
          f2[c] = NA == 2 ? __uint_as_float(r2[c]) : 0.f;
        }
        tc_epilogue_chunk<EPI, CW>(a, f1, f2, n_cat, n_valid, n_local, tok0 + c0);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
}

}  // namespace thinfer

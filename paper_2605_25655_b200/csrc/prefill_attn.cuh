// Prefill causal attention on tcgen05 (Eq. 6; the staged scheme of
// Section 3.3.2 with the Q/O row block stationary on chip and K/V streamed):
//
//   Stage 1  S = Q_blk K_j^T     tcgen05.mma, both operands from shared memory,
//                                scores stay in tensor memory
//   Stage 2  scale + softmax     one thread per query row reads its score row
//                                from tensor memory (no cross-thread reduction
//                                needed), FP32, online form across K/V tiles
//   Stage 3  O_blk += P V_j      P is written to shared memory as FP16 in the
//                                128-byte swizzled layout and fed back to
//                                tcgen05.mma; O accumulates in tensor memory
//
// Scores and weights never leave the SM.  One CTA handles TWO blocks of 128
// query rows of one (request, head), each owned by a group of four warps (one
// thread per row; TMEM lane = row; a score row of 64 fits in registers, so it is
// read from tensor memory once).  A ninth warp issues the TMA loads (K/V tiles of
// 64 keys into a ring of three buffers) and the MMAs, interleaving the two
// blocks: S0, S1, PV0, S0', PV1, S1', ... so that while one group is in its
// softmax stage the tensor core works for the other ("ping-pong"; kernels that
// allocate tensor memory run one CTA per SM, so the overlap has to come from
// inside the CTA).  Tiles above the causal diagonal are skipped; only tiles that
// touch it are masked.  The accumulator O is rescaled lazily: only when the row
// maximum grows by more than 2^8 (weights stay <= 256, exact after the final
// division by the row sum).
#pragma once
#include "common.cuh"

namespace thinfer {

constexpr int kAttnBQ = 128;   // query rows per CTA
constexpr int kAttnBK = 64;    // keys per tile
constexpr int kAttnThreads = 288;  // two softmax groups of 128 + the issuing warp

struct AttnPreArgs {
  half_t* out;  // [batch][seq_len][n_q_heads * D]
  int n_q_heads, n_kv_heads, seq_len;
  float scale_log2;  // log2(e) / sqrt(D)
  int* status;
};

__host__ __device__ constexpr int attn_pre_smem_bytes(int d) {
  // 2 x Q (D/64 sub-tiles of 128 rows x 128 B) + 3 x (K + V) (D/64 sub-tiles of 64 keys x 128 B) + 2 x P + barriers
  return (d / 64) * (2 * 16384 + 6 * 8192) + 2 * 16384 + 256;
}

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
    attn_prefill_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                        const __grid_constant__ CUtensorMap tm_v, const AttnPreArgs a) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int SUB = D / 64;                 // 64-wide column blocks of a head
  constexpr int Q_BYTES = SUB * 16384;
  constexpr int KV_SUB = kAttnBK * 128;       // one 64-column block of a K or V tile
  constexpr int KV_BYTES = SUB * KV_SUB;
  constexpr int NBUF = 3;
  constexpr int TMEM_COLS = 512;
  constexpr uint32_t IDESC_S = idesc_f16(128, kAttnBK, 0, 0);  // Q (K-major) x K^T (K-major)
  constexpr uint32_t IDESC_O = idesc_f16(128, D, 0, 1);        // P (K-major) x V (head_dim contiguous)
  constexpr float kLazy = 8.0f;  // rescale O only when the row maximum grows by more than 2^8

  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* sm_q = smem;                        // [2] query blocks
  uint8_t* sm_k = sm_q + 2 * Q_BYTES;          // [NBUF]
  uint8_t* sm_v = sm_k + NBUF * KV_BYTES;      // [NBUF]
  uint8_t* sm_p = sm_v + NBUF * KV_BYTES;      // [2] x 128 rows x 64 keys
  uint64_t* bar_q = reinterpret_cast<uint64_t*>(sm_p + 2 * 16384);
  uint64_t* bar_kv = bar_q + 1;  // [NBUF]
  uint64_t* bar_s = bar_kv + NBUF;  // [2]
  uint64_t* bar_p = bar_s + 2;      // [2]
  uint64_t* bar_o = bar_p + 2;      // [2]
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bar_o + 2);
  if ((smem_u32(smem) & 1023u) != 0u) {  // the swizzled tiles need 1024-byte alignment
    if (threadIdx.x == 0 && a.status != nullptr) *reinterpret_cast<volatile int*>(a.status) = -5;
    return;
  }

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_qt = (a.seq_len + kAttnBQ - 1) / kAttnBQ;
  const int n_pairs = (n_qt + 1) / 2;
  const int pair = n_pairs - 1 - blockIdx.x;  // longest rows first
  const int h = blockIdx.y, b = blockIdx.z;
  const int hk = h / (a.n_q_heads / a.n_kv_heads);
  // causal: block t attends keys 0 .. q0_t + 127 (clipped to the sequence); a block past the sequence has no tiles
  int q0[2], n_kt[2];
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    q0[t] = (2 * pair + t) * kAttnBQ;
    n_kt[t] = q0[t] < a.seq_len ? (min(q0[t] + kAttnBQ, a.seq_len) - 1) / kAttnBK + 1 : 0;
  }
  const int n_all = max(n_kt[0], n_kt[1]);

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1);
    for (int i = 0; i < NBUF; ++i) mbar_init(&bar_kv[i], 1);
    for (int t = 0; t < 2; ++t) {
      mbar_init(&bar_s[t], 1);
      mbar_init(&bar_p[t], 128);
      mbar_init(&bar_o[t], 1);
    }
    fence_barrier_init();
  }
  if (warp == 8) tmem_alloc(tmem_holder, TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_holder);
  // tensor-memory columns: S0 0..63, S1 64..127, O0 128..255, O1 256..383
  const uint32_t TM_S[2] = {0u, 64u}, TM_O[2] = {128u, 256u};

  if (warp == 8) {
    if (lane == 0) {
      auto load_kv = [&](int j) {
        const int buf = j % NBUF;
        mbar_expect_tx(&bar_kv[buf], 2 * KV_BYTES);
#pragma unroll
        for (int sb = 0; sb < SUB; ++sb) {
          tma_load_3d(sm_k + buf * KV_BYTES + sb * KV_SUB, &tm_k, &bar_kv[buf], sb * 64, j * kAttnBK, b * a.n_kv_heads + hk);
          tma_load_3d(sm_v + buf * KV_BYTES + sb * KV_SUB, &tm_v, &bar_kv[buf], sb * 64, j * kAttnBK, b * a.n_kv_heads + hk);
        }
      };
      auto wait_kv = [&](int j) { return mbar_wait(&bar_kv[j % NBUF], (j / NBUF) & 1, a.status); };
      auto issue_s = [&](int t, int j) {  // Stage 1: S_t = Q_t K_j^T
        const int buf = j % NBUF;
#pragma unroll
        for (int sb = 0; sb < SUB; ++sb) {
          const uint64_t dq = smem_desc_sw128(smem_u32(sm_q + t * Q_BYTES + sb * 16384), 16, 1024);
          const uint64_t dk = smem_desc_sw128(smem_u32(sm_k + buf * KV_BYTES + sb * KV_SUB), 16, 1024);
#pragma unroll
          for (int k = 0; k < 4; ++k) tc_mma_f16(tmem_base + TM_S[t], dq + 2 * k, dk + 2 * k, IDESC_S, (sb | k) != 0);
        }
        tc_commit(&bar_s[t]);
      };
      auto issue_pv = [&](int t, int j) {  // Stage 3: O_t += P_t V_j
        const int buf = j % NBUF;
#pragma unroll
        for (int ks = 0; ks < kAttnBK / 16; ++ks) {
          // P: 32 bytes per K=16 step inside the 128-byte row.  V: rows are keys (128 B each = 64 head
          // elements), 16 keys per step; the next 64 head elements are one sub-tile further (leading offset)
          const uint64_t dp = smem_desc_sw128(smem_u32(sm_p + t * 16384) + ks * 32, 16, 1024);
          const uint64_t dv = smem_desc_sw128(smem_u32(sm_v + buf * KV_BYTES) + ks * 2048, KV_SUB, 1024);
          tc_mma_f16(tmem_base + TM_O[t], dp, dv, IDESC_O, (j | ks) != 0);
        }
        tc_commit(&bar_o[t]);
      };
      tma_prefetch_desc(&tm_q);
      tma_prefetch_desc(&tm_k);
      tma_prefetch_desc(&tm_v);
      mbar_expect_tx(bar_q, 2 * Q_BYTES);
#pragma unroll
      for (int t = 0; t < 2; ++t)
#pragma unroll
        for (int sb = 0; sb < SUB; ++sb)
          tma_load_3d(sm_q + t * Q_BYTES + sb * 16384, &tm_q, bar_q, sb * 64, q0[t], b * a.n_q_heads + h);
      load_kv(0);
      if (n_all > 1) load_kv(1);
      bool ok = mbar_wait(bar_q, 0, a.status) && wait_kv(0);
      if (ok) {
        tc_fence_after();
        if (n_kt[0] > 0) issue_s(0, 0);
        if (n_kt[1] > 0) issue_s(1, 0);
      }
      for (int j = 0; j < n_all && ok; ++j) {
        // ring slot of tile j+2 held tile j-1: both of its P V products must have completed
        if (j + 2 < n_all) {
          if (j >= 1) {
            for (int t = 0; t < 2 && ok; ++t)
              if (j - 1 < n_kt[t]) ok = mbar_wait(&bar_o[t], (j - 1) & 1, a.status);
          }
          if (ok) load_kv(j + 2);
        }
        for (int t = 0; t < 2 && ok; ++t) {
          if (j < n_kt[t]) {
            ok = mbar_wait(&bar_p[t], j & 1, a.status);
            if (!ok) break;
            tc_fence_after();
            issue_pv(t, j);
          }
          if (j + 1 < n_kt[t]) {
            ok = wait_kv(j + 1);
            if (!ok) break;
            tc_fence_after();
            issue_s(t, j + 1);
          }
        }
      }
    }
  } else {
    const int t = warp >> 2;                    // which query block this group owns
    const int row = (warp & 3) * 32 + lane;     // query row inside the block = TMEM lane
    const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    uint8_t* sm_pt = sm_p + t * 16384;
    float m = -INFINITY, l = 0.f;  // m: the reference maximum baked into O and l
    bool ok = true;
    for (int j = 0; j < n_kt[t] && ok; ++j) {
      if (!mbar_wait(&bar_s[t], j & 1, a.status)) { ok = false; break; }
      tc_fence_after();
      // Stage 2: the whole score row of this tile in registers (one pass over tensor memory)
      uint32_t r0[32], r1[32];
      tmem_ld32(lane_addr + TM_S[t], r0);
      tmem_ld32(lane_addr + TM_S[t] + 32, r1);
      tmem_ld_wait();
      const int kbase = j * kAttnBK - q0[t];        // key index relative to this block's first row
      const bool masked = kbase + kAttnBK - 1 > 0;  // some key of the tile lies above the diagonal for some row
      // row maximum: four independent chains (a single chain of 64 dependent max operations is all latency)
      float mx;
      {
        float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        if (!masked) {
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            m4[c & 3] = fmaxf(m4[c & 3], __uint_as_float(r0[c]));
            m4[c & 3] = fmaxf(m4[c & 3], __uint_as_float(r1[c]));
          }
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            if (kbase + c <= row) m4[c & 3] = fmaxf(m4[c & 3], __uint_as_float(r0[c]));
            if (kbase + 32 + c <= row) m4[c & 3] = fmaxf(m4[c & 3], __uint_as_float(r1[c]));
          }
        }
        mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
      }
      mx *= a.scale_log2;
      // P of the previous tile must have been consumed and O must be complete before they are touched
      if (j > 0) {
        if (!mbar_wait(&bar_o[t], (j - 1) & 1, a.status)) { ok = false; break; }
        tc_fence_after();
      }
      const bool grow = mx > m + kLazy;  // first tile: m = -inf -> true
      const float alpha = grow ? ex2_approx(m - mx) : 1.0f;
      if (grow) m = mx;
      if (j > 0 && __any_sync(0xffffffffu, grow)) {  // tensor-memory accesses are warp-wide
#pragma unroll 1
        for (int c0 = 0; c0 < D; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(lane_addr + TM_O[t] + c0, r);
          tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 32; ++c) r[c] = __float_as_uint(__uint_as_float(r[c]) * alpha);
          tmem_st32(lane_addr + TM_O[t] + c0, r);
        }
        tmem_st_wait();
      }
      // weights (FP16 for the tensor core), row sum of the rounded weights, P -> shared memory (128-byte swizzle)
      float sum4[4] = {0.f, 0.f, 0.f, 0.f};
      uint8_t* prow = sm_pt + row * 128;
      const float neg_m = -m;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t pk[16];
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          const uint32_t s0 = half == 0 ? r0[c] : r1[c];
          const uint32_t s1 = half == 0 ? r0[c + 1] : r1[c + 1];
          float p0 = ex2_approx(fmaf(__uint_as_float(s0), a.scale_log2, neg_m));
          float p1 = ex2_approx(fmaf(__uint_as_float(s1), a.scale_log2, neg_m));
          if (masked) {
            if (kbase + half * 32 + c > row) p0 = 0.f;
            if (kbase + half * 32 + c + 1 > row) p1 = 0.f;
          }
          const half2_t hp = f2_to_h2(p0, p1);
          const float2 back = h2_to_f2(hp);
          sum4[(c >> 1) & 3] += back.x + back.y;
          pk[c >> 1] = *reinterpret_cast<const uint32_t*>(&hp);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int phys = (half * 4 + i) ^ (row & 7);
          *reinterpret_cast<uint4*>(prow + phys * 16) = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
        }
      }
      const float sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
      l = l * alpha + sum;
      fence_proxy_async_smem();
      tc_fence_before();
      mbar_arrive(&bar_p[t]);
    }
    if (ok && n_kt[t] > 0 && mbar_wait(&bar_o[t], (n_kt[t] - 1) & 1, a.status)) {
      tc_fence_after();
      const float inv = 1.0f / l;
      const int qrow = q0[t] + row;
#pragma unroll 1
      for (int c0 = 0; c0 < D; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(lane_addr + TM_O[t] + c0, r);
        tmem_ld_wait();
        if (qrow < a.seq_len) {
          half_t* dst = a.out + (static_cast<size_t>(b) * a.seq_len + qrow) * (a.n_q_heads * D) + h * D + c0;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 o;
            o.x = pack2(__uint_as_float(r[8 * i]) * inv, __uint_as_float(r[8 * i + 1]) * inv);
            o.y = pack2(__uint_as_float(r[8 * i + 2]) * inv, __uint_as_float(r[8 * i + 3]) * inv);
            o.z = pack2(__uint_as_float(r[8 * i + 4]) * inv, __uint_as_float(r[8 * i + 5]) * inv);
            o.w = pack2(__uint_as_float(r[8 * i + 6]) * inv, __uint_as_float(r[8 * i + 7]) * inv);
            *reinterpret_cast<uint4*>(dst + 8 * i) = o;
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 8) tmem_dealloc(tmem_base, TMEM_COLS);
}

}  // namespace thinfer

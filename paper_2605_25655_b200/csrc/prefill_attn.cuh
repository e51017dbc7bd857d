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
// Scores and weights never leave the SM.  One CTA handles 128 query rows of one
// (request, head); K/V tiles of 128 keys arrive by TMA into a double buffer;
// tiles above the causal diagonal are skipped and only the diagonal tile is
// masked.  Warps 0..3: softmax rows (TMEM lane = row); warp 4: TMA + MMA issue.
#pragma once
#include "common.cuh"

namespace thinfer {

constexpr int kAttnBQ = 128;   // query rows per CTA
constexpr int kAttnBK = 128;   // keys per tile
constexpr int kAttnThreads = 160;

struct AttnPreArgs {
  __half* out;  // [batch][seq_len][n_q_heads * D]
  int n_q_heads, n_kv_heads, seq_len;
  float scale_log2;  // log2(e) / sqrt(D)
  int* status;
};

__host__ __device__ constexpr int attn_pre_smem_bytes(int d) {
  // Q + 2 x K + 2 x V (each D/64 sub-tiles of 128 rows x 128 B) + P (2 sub-tiles) + slack + barriers
  return (d / 64) * 16384 * 5 + 2 * 16384 + 1024 + 256;
}

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
    attn_prefill_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                        const __grid_constant__ CUtensorMap tm_v, const AttnPreArgs a) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int SUB = D / 64;            // 64-wide column blocks of a head
  constexpr int TILE_BYTES = SUB * 16384;
  constexpr int TMEM_COLS = 256;
  constexpr uint32_t TM_S = 0, TM_O = 128;
  constexpr uint32_t IDESC_S = idesc_f16(128, kAttnBK, 0, 0);  // Q (K-major) x K^T (K-major)
  constexpr uint32_t IDESC_O = idesc_f16(128, D, 0, 1);        // P (K-major) x V (head_dim contiguous)

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sm_q = smem;
  uint8_t* sm_k = sm_q + TILE_BYTES;       // 2 buffers
  uint8_t* sm_v = sm_k + 2 * TILE_BYTES;   // 2 buffers
  uint8_t* sm_p = sm_v + 2 * TILE_BYTES;   // 2 sub-tiles of 64 keys
  uint64_t* bar_q = reinterpret_cast<uint64_t*>(sm_p + 2 * 16384);
  uint64_t* bar_kv = bar_q + 1;  // [2]
  uint64_t* bar_s = bar_kv + 2;
  uint64_t* bar_p = bar_s + 1;
  uint64_t* bar_o = bar_p + 1;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bar_o + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_qt = (a.seq_len + kAttnBQ - 1) / kAttnBQ;
  const int qt = n_qt - 1 - blockIdx.x;  // longest rows first
  const int h = blockIdx.y, b = blockIdx.z;
  const int hk = h / (a.n_q_heads / a.n_kv_heads);
  const int q0 = qt * kAttnBQ;
  const int n_kt = qt + 1;  // causal: tiles above the diagonal are never touched

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1);
    mbar_init(&bar_kv[0], 1);
    mbar_init(&bar_kv[1], 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_p, 128);
    mbar_init(bar_o, 1);
    fence_barrier_init();
  }
  if (warp == 4) tmem_alloc(tmem_holder, TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_holder);

  if (warp == 4) {
    if (lane == 0) {
      tma_prefetch_desc(&tm_q);
      tma_prefetch_desc(&tm_k);
      tma_prefetch_desc(&tm_v);
      mbar_expect_tx(bar_q, TILE_BYTES);
#pragma unroll
      for (int sb = 0; sb < SUB; ++sb) tma_load_3d(sm_q + sb * 16384, &tm_q, bar_q, sb * 64, q0, b * a.n_q_heads + h);
      auto load_kv = [&](int j) {
        const int buf = j & 1;
        mbar_expect_tx(&bar_kv[buf], 2 * TILE_BYTES);
#pragma unroll
        for (int sb = 0; sb < SUB; ++sb) {
          tma_load_3d(sm_k + buf * TILE_BYTES + sb * 16384, &tm_k, &bar_kv[buf], sb * 64, j * kAttnBK,
                      b * a.n_kv_heads + hk);
          tma_load_3d(sm_v + buf * TILE_BYTES + sb * 16384, &tm_v, &bar_kv[buf], sb * 64, j * kAttnBK,
                      b * a.n_kv_heads + hk);
        }
      };
      load_kv(0);
      bool ok = mbar_wait(bar_q, 0, a.status);
      for (int j = 0; j < n_kt && ok; ++j) {
        const int buf = j & 1;
        if (j + 1 < n_kt) load_kv(j + 1);  // its buffer was released by the P V product of tile j-1
        if (!mbar_wait(&bar_kv[buf], (j >> 1) & 1, a.status)) break;
        tc_fence_after();
        // Stage 1: S = Q K^T
#pragma unroll
        for (int sb = 0; sb < SUB; ++sb) {
          const uint64_t dq = smem_desc_sw128(smem_u32(sm_q + sb * 16384), 16, 1024);
          const uint64_t dk = smem_desc_sw128(smem_u32(sm_k + buf * TILE_BYTES + sb * 16384), 16, 1024);
#pragma unroll
          for (int k = 0; k < 4; ++k) tc_mma_f16(tmem_base + TM_S, dq + 2 * k, dk + 2 * k, IDESC_S, (sb | k) != 0);
        }
        tc_commit(bar_s);
        // Stage 3 (after the softmax threads have produced P and rescaled O)
        if (!mbar_wait(bar_p, j & 1, a.status)) break;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < kAttnBK / 16; ++ks) {
          // P: sub-tile ks/4 (64 keys), 32 bytes per K=16 step inside the 128-byte row
          const uint64_t dp = smem_desc_sw128(smem_u32(sm_p + (ks >> 2) * 16384) + (ks & 3) * 32, 16, 1024);
          // V: rows are keys (128 B each = 64 head elements); 16 keys per step; the next 64 head
          // elements are TILE 16 KB further (leading byte offset)
          const uint64_t dv = smem_desc_sw128(smem_u32(sm_v + buf * TILE_BYTES) + ks * 2048, 16384, 1024);
          tc_mma_f16(tmem_base + TM_O, dp, dv, IDESC_O, (j | ks) != 0);
        }
        tc_commit(bar_o);
        if (!mbar_wait(bar_o, j & 1, a.status)) break;
      }
    }
  } else {
    const int row = warp * 32 + lane;  // query row inside the block = TMEM lane
    const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
    float m = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kt && ok; ++j) {
      if (!mbar_wait(bar_s, j & 1, a.status)) { ok = false; break; }
      tc_fence_after();
      const bool diag = (j == qt);
      // Stage 2, pass 1: row maximum
      float mx = -INFINITY;
#pragma unroll 1
      for (int c0 = 0; c0 < kAttnBK; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(lane_addr + TM_S + c0, r);
        tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          const float s = __uint_as_float(r[c]);
          if (!diag || c0 + c <= row) mx = fmaxf(mx, s);
        }
      }
      const float m_new = fmaxf(m, mx * a.scale_log2);
      const float alpha = exp2f(m - m_new);  // first tile: m = -inf -> 0
      m = m_new;
      // O of the previous tiles must be complete before it is rescaled, and P free before it is rewritten
      if (j > 0) {
        if (!mbar_wait(bar_o, (j - 1) & 1, a.status)) { ok = false; break; }
        tc_fence_after();
#pragma unroll 1
        for (int c0 = 0; c0 < D; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(lane_addr + TM_O + c0, r);
          tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 32; ++c) r[c] = __float_as_uint(__uint_as_float(r[c]) * alpha);
          tmem_st32(lane_addr + TM_O + c0, r);
        }
        tmem_st_wait();
      }
      // pass 2: weights, row sum, P -> shared memory (FP16, 128-byte swizzle)
      float sum = 0.f;
#pragma unroll 1
      for (int c0 = 0; c0 < kAttnBK; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(lane_addr + TM_S + c0, r);
        tmem_ld_wait();
        uint32_t pk[16];
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          float p0 = exp2f(fmaf(__uint_as_float(r[c]), a.scale_log2, -m));
          float p1 = exp2f(fmaf(__uint_as_float(r[c + 1]), a.scale_log2, -m));
          if (diag && c0 + c > row) p0 = 0.f;
          if (diag && c0 + c + 1 > row) p1 = 0.f;
          // the sum uses the FP16-rounded weights the tensor core will see
          const __half2 hp = __floats2half2_rn(p0, p1);
          const float2 back = __half22float2(hp);
          sum += back.x + back.y;
          pk[c >> 1] = *reinterpret_cast<const uint32_t*>(&hp);
        }
        uint8_t* prow = sm_p + (c0 >> 6) * 16384 + row * 128;
        const int chunk0 = (c0 & 63) >> 3;  // first 16-byte chunk of this 32-key group
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int phys = (chunk0 + i) ^ (row & 7);
          *reinterpret_cast<uint4*>(prow + phys * 16) = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
        }
      }
      l = l * alpha + sum;
      fence_proxy_async_smem();
      tc_fence_before();
      mbar_arrive(bar_p);
    }
    if (ok && mbar_wait(bar_o, (n_kt - 1) & 1, a.status)) {
      tc_fence_after();
      const float inv = 1.0f / l;
      const int qrow = q0 + row;
#pragma unroll 1
      for (int c0 = 0; c0 < D; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(lane_addr + TM_O + c0, r);
        tmem_ld_wait();
        if (qrow < a.seq_len) {
          __half* dst = a.out + (static_cast<size_t>(b) * a.seq_len + qrow) * (a.n_q_heads * D) + h * D + c0;
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
  if (warp == 4) tmem_dealloc(tmem_base, TMEM_COLS);
}

}  // namespace thinfer

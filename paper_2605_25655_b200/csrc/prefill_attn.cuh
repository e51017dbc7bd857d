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
// (request, head); K/V tiles of 64 keys arrive by TMA into a double buffer;
// tiles above the causal diagonal are skipped and only the tiles that touch it
// are masked.  Warps 0..3: softmax rows (TMEM lane = row; a score row of 64 fits
// in registers, so it is read from tensor memory once); warp 4: TMA + MMA issue.
// Sized (113 KB of shared memory, 256 TMEM columns) so that two CTAs share an SM:
// while one is in its softmax stage the tensor core works for the other.
#pragma once
#include "common.cuh"

namespace thinfer {

constexpr int kAttnBQ = 128;   // query rows per CTA
constexpr int kAttnBK = 64;    // keys per tile
constexpr int kAttnThreads = 128;

struct AttnPreArgs {
  __half* out;  // [batch][seq_len][n_q_heads * D]
  int n_q_heads, n_kv_heads, seq_len;
  float scale_log2;  // log2(e) / sqrt(D)
  int* status;
};

__host__ __device__ constexpr int attn_pre_smem_bytes(int d) {
  // Q (D/64 sub-tiles of 128 rows x 128 B) + 2 x K + 1 x V (D/64 sub-tiles of 64 keys x 128 B) + P + barriers
  return (d / 64) * (16384 + 3 * 8192) + 16384 + 256;
}

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 2)
    attn_prefill_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                        const __grid_constant__ CUtensorMap tm_v, const AttnPreArgs a) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int SUB = D / 64;                 // 64-wide column blocks of a head
  constexpr int Q_BYTES = SUB * 16384;
  constexpr int KV_SUB = kAttnBK * 128;       // one 64-column block of a K or V tile
  constexpr int KV_BYTES = SUB * KV_SUB;
  constexpr int TMEM_COLS = 256;
  constexpr uint32_t TM_S = 0, TM_O = 64;
  constexpr uint32_t IDESC_S = idesc_f16(128, kAttnBK, 0, 0);  // Q (K-major) x K^T (K-major)
  constexpr uint32_t IDESC_O = idesc_f16(128, D, 0, 1);        // P (K-major) x V (head_dim contiguous)

  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* sm_q = smem;
  uint8_t* sm_k = sm_q + Q_BYTES;         // 2 buffers: K of the next tile arrives while this one is used
  uint8_t* sm_v = sm_k + 2 * KV_BYTES;    // 1 buffer: V is needed only after the softmax stage
  uint8_t* sm_p = sm_v + KV_BYTES;        // 128 rows x 64 keys
  uint64_t* bar_q = reinterpret_cast<uint64_t*>(sm_p + 16384);
  uint64_t* bar_kv = bar_q + 1;  // [0], [1]: K buffers; [2]: V
  uint64_t* bar_s = bar_kv + 3;
  uint64_t* bar_p = bar_s + 1;
  uint64_t* bar_o = bar_p + 1;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bar_o + 1);
  if ((smem_u32(smem) & 1023u) != 0u) {  // the swizzled tiles need 1024-byte alignment
    if (threadIdx.x == 0 && a.status != nullptr) *reinterpret_cast<volatile int*>(a.status) = -5;
    return;
  }

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool issuer = threadIdx.x == 0;
  const int n_qt = (a.seq_len + kAttnBQ - 1) / kAttnBQ;
  const int qt = n_qt - 1 - blockIdx.x;  // longest rows first
  const int h = blockIdx.y, b = blockIdx.z;
  const int hk = h / (a.n_q_heads / a.n_kv_heads);
  const int q0 = qt * kAttnBQ;
  // causal: keys 0 .. q0+127 (clipped to the sequence); tiles above the diagonal are never touched
  const int last_key = min(q0 + kAttnBQ, a.seq_len) - 1;
  const int n_kt = last_key / kAttnBK + 1;

  if (issuer) {
    mbar_init(bar_q, 1);
    mbar_init(&bar_kv[0], 1);
    mbar_init(&bar_kv[1], 1);
    mbar_init(&bar_kv[2], 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_p, kAttnThreads);
    mbar_init(bar_o, 1);
    fence_barrier_init();
  }
  if (warp == 0) tmem_alloc(tmem_holder, TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_holder);

  auto load_k = [&](int j) {
    const int buf = j & 1;
    mbar_expect_tx(&bar_kv[buf], KV_BYTES);
#pragma unroll
    for (int sb = 0; sb < SUB; ++sb)
      tma_load_3d(sm_k + buf * KV_BYTES + sb * KV_SUB, &tm_k, &bar_kv[buf], sb * 64, j * kAttnBK, b * a.n_kv_heads + hk);
  };
  auto load_v = [&](int j) {
    mbar_expect_tx(&bar_kv[2], KV_BYTES);
#pragma unroll
    for (int sb = 0; sb < SUB; ++sb)
      tma_load_3d(sm_v + sb * KV_SUB, &tm_v, &bar_kv[2], sb * 64, j * kAttnBK, b * a.n_kv_heads + hk);
  };
  if (issuer) {
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    mbar_expect_tx(bar_q, Q_BYTES);
#pragma unroll
    for (int sb = 0; sb < SUB; ++sb) tma_load_3d(sm_q + sb * 16384, &tm_q, bar_q, sb * 64, q0, b * a.n_q_heads + h);
    load_k(0);
  }

  const int row = warp * 32 + lane;  // query row inside the block = TMEM lane
  const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
  float m = -INFINITY, l = 0.f;
  bool ok = true;
  for (int j = 0; j < n_kt && ok; ++j) {
    if (issuer) {
      // V buffer and the other K buffer were released by the products of tile j-1 (complete: bar_o awaited
      // by this thread in the previous iteration)
      load_v(j);
      if (j + 1 < n_kt) load_k(j + 1);
      bool go = j > 0 || mbar_wait(bar_q, 0, a.status);
      go = go && mbar_wait(&bar_kv[j & 1], (j >> 1) & 1, a.status);
      if (go) {
        tc_fence_after();
        // Stage 1: S = Q K^T
#pragma unroll
        for (int sb = 0; sb < SUB; ++sb) {
          const uint64_t dq = smem_desc_sw128(smem_u32(sm_q + sb * 16384), 16, 1024);
          const uint64_t dk = smem_desc_sw128(smem_u32(sm_k + (j & 1) * KV_BYTES + sb * KV_SUB), 16, 1024);
#pragma unroll
          for (int k = 0; k < 4; ++k) tc_mma_f16(tmem_base + TM_S, dq + 2 * k, dk + 2 * k, IDESC_S, (sb | k) != 0);
        }
        tc_commit(bar_s);
      }
    }
    __syncwarp();
    if (!mbar_wait(bar_s, j & 1, a.status)) { ok = false; break; }
    tc_fence_after();
    // Stage 2: the whole score row of this tile in registers (one pass over tensor memory)
    uint32_t r0[32], r1[32];
    tmem_ld32(lane_addr + TM_S, r0);
    tmem_ld32(lane_addr + TM_S + 32, r1);
    tmem_ld_wait();
    const int kbase = j * kAttnBK - q0;           // key index relative to this block's first row
    const bool masked = kbase + kAttnBK - 1 > 0;  // some key of the tile lies above the diagonal for some row
    float mx = -INFINITY;
#pragma unroll
    for (int c = 0; c < 32; ++c) {
      if (!masked || kbase + c <= row) mx = fmaxf(mx, __uint_as_float(r0[c]));
      if (!masked || kbase + 32 + c <= row) mx = fmaxf(mx, __uint_as_float(r1[c]));
    }
    const float m_new = fmaxf(m, mx * a.scale_log2);
    const float alpha = exp2f(m - m_new);  // first tile: m = -inf -> 0
    m = m_new;
    // P of the previous tile must have been consumed and O must be complete before they are touched
    if (j > 0) {
      if (!mbar_wait(bar_o, (j - 1) & 1, a.status)) { ok = false; break; }
      tc_fence_after();
    }
    float sum = 0.f;
    uint8_t* prow = sm_p + row * 128;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      uint32_t pk[16];
#pragma unroll
      for (int c = 0; c < 32; c += 2) {
        const uint32_t s0 = half == 0 ? r0[c] : r1[c];
        const uint32_t s1 = half == 0 ? r0[c + 1] : r1[c + 1];
        float p0 = exp2f(fmaf(__uint_as_float(s0), a.scale_log2, -m));
        float p1 = exp2f(fmaf(__uint_as_float(s1), a.scale_log2, -m));
        if (masked && kbase + half * 32 + c > row) p0 = 0.f;
        if (masked && kbase + half * 32 + c + 1 > row) p1 = 0.f;
        // the sum uses the FP16-rounded weights the tensor core will see
        const __half2 hp = __floats2half2_rn(p0, p1);
        const float2 back = __half22float2(hp);
        sum += back.x + back.y;
        pk[c >> 1] = *reinterpret_cast<const uint32_t*>(&hp);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int phys = (half * 4 + i) ^ (row & 7);
        *reinterpret_cast<uint4*>(prow + phys * 16) = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
      }
    }
    l = l * alpha + sum;
    if (j > 0) {  // rescale O of the previous tiles
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
    fence_proxy_async_smem();
    tc_fence_before();
    mbar_arrive(bar_p);
    if (issuer) {
      // Stage 3: O += P V once every row has written its weights and V has arrived
      bool go = mbar_wait(bar_p, j & 1, a.status) && mbar_wait(&bar_kv[2], j & 1, a.status);
      if (go) {
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < kAttnBK / 16; ++ks) {
          // P: 32 bytes per K=16 step inside the 128-byte row.  V: rows are keys (128 B each = 64 head
          // elements), 16 keys per step; the next 64 head elements are one sub-tile further (leading offset)
          const uint64_t dp = smem_desc_sw128(smem_u32(sm_p) + ks * 32, 16, 1024);
          const uint64_t dv = smem_desc_sw128(smem_u32(sm_v) + ks * 2048, KV_SUB, 1024);
          tc_mma_f16(tmem_base + TM_O, dp, dv, IDESC_O, (j | ks) != 0);
        }
        tc_commit(bar_o);
        // the next iteration reuses the V buffer and a K buffer: wait for this product here
        mbar_wait(bar_o, j & 1, a.status);
      }
    }
    __syncwarp();
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

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, TMEM_COLS);
}

}  // namespace thinfer

// Prefill causal attention on tcgen05 (Eq. 6; the staged scheme of
// Section 3.3.2 with the Q/O row block stationary on chip and K/V streamed):
//
//   Stage 1  S = Q_blk K_j^T     tcgen05.mma, both operands from shared memory,
//                                scores stay in tensor memory
//   Stage 2  scale + softmax     one thread per query row reads its score row
//                                from tensor memory (no cross-thread reduction
//                                needed), FP32, online form across K/V tiles
//   Stage 3  O_blk += P V_j      P is written back to tensor memory as packed
//                                FP16 and is the A operand of tcgen05.mma from
//                                there; O accumulates in tensor memory
//
// Scores and weights never leave the SM.  One CTA handles TWO blocks of 128
// query rows of one (request, head), each owned by a group of four warps (one
// thread per row; TMEM lane = row; a score row of 64 fits in registers, so it is
// read from tensor memory once) and by one MMA-issuing warp of its own; an
// eleventh warp issues the TMA loads (K/V tiles of 64 keys into a ring of three
// buffers shared by the two blocks).  Kernels that allocate tensor memory run
// one CTA per SM, so the overlap of the stages has to come from inside the CTA:
//
//   * the stages of one block are decoupled: as soon as a group has its score
//     row in registers it releases the score columns, and its issuer starts
//     S(j+1) while the group is still in the softmax of tile j; P has two
//     buffers per block, so the softmax of tile j+1 does not wait for P(j) V_j;
//   * the two blocks run independently of each other (each issuer follows the
//     events of its own group), coupled only through the K/V ring.
//
// Tiles above the causal diagonal are skipped; only tiles that touch it are
// masked.  The accumulator O is rescaled lazily: only when the row maximum grows
// by more than 2^8 (weights stay <= 256, exact after the final division by the
// row sum); only then does a group wait for its previous P V product.
#pragma once
#include "common.cuh"

namespace thinfer {

constexpr int kAttnBQ = 128;   // query rows per CTA
constexpr int kAttnBK = 64;    // keys per tile
constexpr int kAttnThreads = 352;  // two softmax groups of 128 + one MMA-issuing warp per group + the loading warp

struct AttnPreArgs {
  half_t* out;  // [batch][seq_len][n_q_heads * D]
  int n_q_heads, n_kv_heads, seq_len;
  int n_items;      // batch * n_q_heads: the (request, head) pairs
  int chunk_items;  // (request, head) pairs whose K and V stay in L2 together
  float scale_log2;  // log2(e) / sqrt(D)
  int* status;
};

__host__ __device__ constexpr int attn_pre_smem_bytes(int d) {
  // 2 x Q (D/64 sub-tiles of 128 rows x 128 B) + 3 x (K + V) (D/64 sub-tiles of 64 keys x 128 B) + barriers
  return (d / 64) * (2 * 16384 + 6 * 8192) + 256;
}

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
    attn_prefill_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                        const __grid_constant__ CUtensorMap tm_v, const AttnPreArgs a) {
  pdl_launch_dependents();
  constexpr int SUB = D / 64;                 // 64-wide column blocks of a head
  constexpr int Q_BYTES = SUB * 16384;
  constexpr int KV_SUB = kAttnBK * 128;       // one 64-column block of a K or V tile
  constexpr int KV_BYTES = SUB * KV_SUB;
  constexpr uint32_t TM_P = 384;              // P buffers: 32 columns (64 packed weights) per block and buffer
  constexpr int NBUF = 3;
  constexpr int TMEM_COLS = 512;
  constexpr uint32_t IDESC_S = idesc_f16(128, kAttnBK, 0, 0);  // Q (K-major) x K^T (K-major)
  constexpr uint32_t IDESC_O = idesc_f16(128, D, 0, 1);        // P (K-major) x V (head_dim contiguous)
  constexpr float kLazy = 8.0f;  // rescale O only when the row maximum grows by more than 2^8

  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* sm_q = smem;                        // [2] query blocks
  uint8_t* sm_k = sm_q + 2 * Q_BYTES;          // [NBUF]
  uint8_t* sm_v = sm_k + NBUF * KV_BYTES;      // [NBUF]
  uint64_t* bar_q = reinterpret_cast<uint64_t*>(sm_v + NBUF * KV_BYTES);
  uint64_t* bar_kv = bar_q + 1;          // [NBUF]     tile loaded (transaction bytes)
  uint64_t* bar_free = bar_kv + NBUF;    // [2][NBUF]  block t has finished with the tile in this ring slot
  uint64_t* bar_s = bar_free + 2 * NBUF; // [2]        scores of block t complete in tensor memory
  uint64_t* bar_sf = bar_s + 2;          // [2]        group t holds its score row in registers
  uint64_t* bar_p = bar_sf + 2;          // [2][2]     weights written to P buffer (tensor memory)
  uint64_t* bar_o = bar_p + 4;           // [2][2]     the P V product that read P buffer is complete
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bar_o + 4);
  if ((smem_u32(smem) & 1023u) != 0u) {  // the swizzled tiles need 1024-byte alignment
    if (threadIdx.x == 0 && a.status != nullptr) *reinterpret_cast<volatile int*>(a.status) = -5;
    return;
  }

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_qt = (a.seq_len + kAttnBQ - 1) / kAttnBQ;
  const int n_pairs = (n_qt + 1) / 2;
  // CTAs are handed out in the order of their index.  Inside a chunk of (request, head) pairs whose K and V fit
  // in L2 together, all pairs of query blocks with the most key tiles come first, then the next shorter ones: the
  // SMs that finish early pick up short work, and every K/V tile is still fetched from memory once.
  const int per_chunk = a.chunk_items * n_pairs;
  const int chunk = blockIdx.x / per_chunk, in_chunk = blockIdx.x - chunk * per_chunk;
  const int first_item = chunk * a.chunk_items, cnt = min(a.chunk_items, a.n_items - first_item);
  const int pair = n_pairs - 1 - in_chunk / cnt;  // longest rows first
  const int item = first_item + in_chunk % cnt;
  const int h = item % a.n_q_heads, b = item / a.n_q_heads;
  const int hk = h / (a.n_q_heads / a.n_kv_heads);
  // causal: block t attends keys 0 .. q0_t + 127 (clipped to the sequence); a block past the sequence has no tiles
  int q0[2], n_kt[2];
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    q0[t] = (2 * pair + t) * kAttnBQ;
    n_kt[t] = q0[t] < a.seq_len ? (min(q0[t] + kAttnBQ, a.seq_len) - 1) / kAttnBK + 1 : 0;
  }
  const int n_all = max(n_kt[0], n_kt[1]);

  auto load_kv = [&](int j) {
    const int buf = j % NBUF;
    mbar_expect_tx(&bar_kv[buf], 2 * KV_BYTES);
#pragma unroll
    for (int sb = 0; sb < SUB; ++sb) {
      tma_load_3d(sm_k + buf * KV_BYTES + sb * KV_SUB, &tm_k, &bar_kv[buf], sb * 64, j * kAttnBK, b * a.n_kv_heads + hk);
      tma_load_3d(sm_v + buf * KV_BYTES + sb * KV_SUB, &tm_v, &bar_kv[buf], sb * 64, j * kAttnBK, b * a.n_kv_heads + hk);
    }
  };

  // The loading thread initialises the barriers and has the first tiles in flight while tensor memory is allocated.
  if (warp == 10 && lane == 0) {
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    mbar_init(bar_q, 1);
    for (int i = 0; i < NBUF; ++i) mbar_init(&bar_kv[i], 1);
    for (int i = 0; i < 2 * NBUF; ++i) mbar_init(&bar_free[i], 1);
    for (int t = 0; t < 2; ++t) {
      mbar_init(&bar_s[t], 1);
      mbar_init(&bar_sf[t], 128);
    }
    for (int i = 0; i < 4; ++i) {
      mbar_init(&bar_p[i], 128);
      mbar_init(&bar_o[i], 1);
    }
    fence_barrier_init();
    pdl_wait();  // Q, K and V are written by the projection in front of this kernel
    mbar_expect_tx(bar_q, 2 * Q_BYTES);
#pragma unroll
    for (int t = 0; t < 2; ++t)
#pragma unroll
      for (int sb = 0; sb < SUB; ++sb)
        tma_load_3d(sm_q + t * Q_BYTES + sb * 16384, &tm_q, bar_q, sb * 64, q0[t], b * a.n_q_heads + h);
    for (int j = 0; j < NBUF && j < n_all; ++j) load_kv(j);
  }
  if (warp == 8) tmem_alloc(tmem_holder, TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_holder);
  // tensor-memory columns: S0 0..63, S1 64..127, O0 128..255, O1 256..383, P[block][buffer] 384 + 64 block + 32 buffer

  if (warp == 10) {
    if (lane == 0) {
      // ring slot of tile j held tile j - NBUF: both blocks' P V products of that tile must have completed
      bool ok = true;
      for (int j = NBUF; j < n_all && ok; ++j) {
#pragma unroll
        for (int t = 0; t < 2; ++t)
          if (ok && j - NBUF < n_kt[t]) ok = mbar_wait(&bar_free[t * NBUF + j % NBUF], (j / NBUF - 1) & 1, a.status);
        if (ok) load_kv(j);
      }
    }
  } else if (warp >= 8) {
    const int t = warp - 8;  // the block this warp issues for
    if (lane == 0 && (t ? n_kt[1] : n_kt[0]) > 0) {
      // Descriptors differ only in the start-address field (bits 0..13, bytes >> 4): one base each, offsets added.
      const uint64_t dq0 = smem_desc_sw128(smem_u32(sm_q + t * Q_BYTES), 16, 1024);
      const uint64_t dk0 = smem_desc_sw128(smem_u32(sm_k), 16, 1024);
      const uint32_t tm_p = tmem_base + TM_P + t * 64;
      const uint64_t dv0 = smem_desc_sw128(smem_u32(sm_v), KV_SUB, 1024);
      const uint32_t tm_s = tmem_base + t * 64, tm_o = tmem_base + 128 + t * 128;
      const int n_t = t ? n_kt[1] : n_kt[0];
      auto wait_kv = [&](int j) { return mbar_wait(&bar_kv[j % NBUF], (j / NBUF) & 1, a.status); };
      auto issue_s = [&](int j) {  // Stage 1: S_t = Q_t K_j^T
        const uint64_t dk = dk0 + static_cast<uint64_t>((j % NBUF) * (KV_BYTES >> 4));
#pragma unroll
        for (int sb = 0; sb < SUB; ++sb)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            tc_mma_f16(tm_s, dq0 + (sb * (16384 >> 4) + 2 * k), dk + (sb * (KV_SUB >> 4) + 2 * k), IDESC_S, (sb | k) != 0);
        tc_commit(&bar_s[t]);
      };
      auto issue_pv = [&](int j) {  // Stage 3: O_t += P_t V_j
        // P: 8 tensor-memory columns per K=16 step.  V: rows are keys (128 B each = 64 head elements), 16 keys
        // per step; the next 64 head elements are one sub-tile further (leading offset)
        const uint32_t ap = tm_p + (j & 1) * 32;
        const uint64_t dv = dv0 + static_cast<uint64_t>((j % NBUF) * (KV_BYTES >> 4));
#pragma unroll
        for (int ks = 0; ks < kAttnBK / 16; ++ks)
          tc_mma_f16_ts(tm_o, ap + ks * 8, dv + ks * (2048 >> 4), IDESC_O, (j | ks) != 0);
        tc_commit(&bar_o[t * 2 + (j & 1)]);
        tc_commit(&bar_free[t * NBUF + j % NBUF]);
      };
      bool ok = mbar_wait(bar_q, 0, a.status) && wait_kv(0);
      if (ok) {
        tc_fence_after();
        issue_s(0);
      }
      for (int j = 0; j < n_t && ok; ++j) {
        if (j + 1 < n_t) {  // the group has read S(j): the columns are free for S(j+1)
          ok = mbar_wait(&bar_sf[t], j & 1, a.status) && wait_kv(j + 1);
          if (!ok) break;
          tc_fence_after();
          issue_s(j + 1);
        }
        ok = mbar_wait(&bar_p[t * 2 + (j & 1)], (j >> 1) & 1, a.status);
        if (!ok) break;
        tc_fence_after();
        issue_pv(j);
      }
    }
  } else {
    const int t = warp >> 2;                    // which query block this group owns
    const int row = (warp & 3) * 32 + lane;     // query row inside the block = TMEM lane
    const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const uint32_t tm_s = lane_addr + t * 64, tm_o = lane_addr + 128 + t * 128;
    const int n_t = t ? n_kt[1] : n_kt[0], q0_t = t ? q0[1] : q0[0];
    float m = -INFINITY, l = 0.f;  // m: the reference maximum baked into O and l
    bool ok = true;
    for (int j = 0; j < n_t && ok; ++j) {
      if (!mbar_wait(&bar_s[t], j & 1, a.status)) { ok = false; break; }
      tc_fence_after();
      // Stage 2: the whole score row of this tile in registers (one pass over tensor memory)
      uint32_t r0[32], r1[32];
      tmem_ld32(tm_s, r0);
      tmem_ld32(tm_s + 32, r1);
      tmem_ld_wait();
      tc_fence_before();
      mbar_arrive(&bar_sf[t]);  // the score columns may be overwritten by S(j+1)
      const int kbase = j * kAttnBK - q0_t;        // key index relative to this block's first row
      const bool masked = kbase + kAttnBK - 1 > 0;  // some key of the tile lies above the diagonal for some row
      // row maximum: four independent chains (a single chain of 64 dependent max operations is all latency),
      // three-input maxima
      float mx;
      {
        float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        if (!masked) {
#pragma unroll
          for (int c = 0; c < 32; ++c) m4[c & 3] = fmax3(m4[c & 3], __uint_as_float(r0[c]), __uint_as_float(r1[c]));
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
      const bool grow = mx > m + kLazy;  // first tile: m = -inf -> true
      const float alpha = grow ? ex2_approx(m - mx) : 1.0f;
      if (grow) m = mx;
      if (j > 0 && __any_sync(0xffffffffu, grow)) {  // tensor-memory accesses are warp-wide
        // O must be complete (P(j-1) V_{j-1} has finished) before it is rescaled
        if (!mbar_wait(&bar_o[t * 2 + ((j - 1) & 1)], ((j - 1) >> 1) & 1, a.status)) { ok = false; break; }
        tc_fence_after();
#pragma unroll 1
        for (int c0 = 0; c0 < D; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(tm_o + c0, r);
          tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 32; ++c) r[c] = __float_as_uint(__uint_as_float(r[c]) * alpha);
          tmem_st32(tm_o + c0, r);
        }
        tmem_st_wait();
      }
      // This tile's P buffer was read by P(j-2) V_{j-2}.  That product was issued before S(j) by the same thread,
      // and the arrival on bar_s that let this tile start follows every MMA issued before it: nothing to wait for.
      // weights, their row sum (FP32, two lanes per instruction), P as packed FP16 for the tensor core -> tensor
      // memory (lane = row, two weights per column)
      uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};
      uint32_t pk[32];
      const uint64_t scale2 = f32x2(a.scale_log2, a.scale_log2), neg_m2 = f32x2(-m, -m);
#pragma unroll
      for (int half = 0; half < 2; ++half) {
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          const uint32_t s0 = half == 0 ? r0[c] : r1[c];
          const uint32_t s1 = half == 0 ? r0[c + 1] : r1[c + 1];
          const float2 x = f32x2_unpack(fma_f32x2(f32x2(__uint_as_float(s0), __uint_as_float(s1)), scale2, neg_m2));
          float p0 = ex2_approx(x.x);
          float p1 = ex2_approx(x.y);
          if (masked) {
            if (kbase + half * 32 + c > row) p0 = 0.f;
            if (kbase + half * 32 + c + 1 > row) p1 = 0.f;
          }
          sum2[(c >> 1) & 3] = add_f32x2(sum2[(c >> 1) & 3], f32x2(p0, p1));
          const half2_t hp = f2_to_h2(p0, p1);
          pk[half * 16 + (c >> 1)] = *reinterpret_cast<const uint32_t*>(&hp);
        }
      }
      tmem_st32(lane_addr + TM_P + t * 64 + (j & 1) * 32, pk);
      tmem_st_wait();
      const float2 sum = f32x2_unpack(add_f32x2(add_f32x2(sum2[0], sum2[1]), add_f32x2(sum2[2], sum2[3])));
      l = l * alpha + (sum.x + sum.y);
      tc_fence_before();
      mbar_arrive(&bar_p[t * 2 + (j & 1)]);
    }
    const int last = n_t - 1;
    if (ok && n_t > 0 && mbar_wait(&bar_o[t * 2 + (last & 1)], (last >> 1) & 1, a.status)) {
      tc_fence_after();
      const float inv = 1.0f / l;
      const int qrow = q0_t + row;
#pragma unroll 1
      for (int c0 = 0; c0 < D; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tm_o + c0, r);
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

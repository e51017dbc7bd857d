// Decode attention for grouped-query models on warp-level tensor cores (Eq. 6,
// the M = 1 case of Section 3.3.2, for G = 4 or 8 query heads that share one KV
// head).  With plain FMA every streamed key costs G dot products and G output
// updates per lane; at G = 8 the instruction issue, not the memory system, is
// then the limit.  Here the G query heads of a pair are the rows of an MMA tile
// (padded to 16), so a block of 16 keys costs 2 * D/16 MMAs for the scores and
// 2 * D/16 for the output, whatever G is:
//
//   S[head, key]  = Q[head, :] . K[key, :]      A = Q (registers, loaded once per segment)
//                                               B = K rows   (shared memory, ldmatrix)
//   softmax over keys, online across blocks     (score fragments: 4 values per lane)
//   O[head, :]   += P[head, key] V[key, :]      A = P (the score fragment, packed to FP16)
//                                               B = V rows   (shared memory, ldmatrix.trans)
//
// K and V rows travel global -> shared memory with 16-byte asynchronous copies
// into a two-stage ring per warp (row r, 16-byte piece c at piece c ^ (r & 7):
// the 8 x 8 matrices ldmatrix reads are free of bank conflicts).  Rows past the
// end of a segment are zero-filled (a weight of exactly 0 times an undefined V
// would not be 0).  The schedule (equal runs of key units over a grid that fills
// the device once) and the merging of warps and segments are those of
// decode_attn.cuh.
#pragma once
#include "decode_attn.cuh"
#include "decode_mma.cuh"

namespace thinfer {

constexpr int kGqaChunk = 16;                              // keys per MMA block of a warp
constexpr int kGqaUnit = kAttnDecWarps * kGqaChunk;        // keys of one CTA-wide iteration
constexpr int kGqaStages = 2;
constexpr int kGqaMaxCluster = 4;   // CTAs of one pair that merge through distributed shared memory

template <int D>
__host__ __device__ constexpr int gqa_ring_bytes() {
  return kAttnDecWarps * kGqaStages * 2 * kGqaChunk * D * 2;  // warps x stages x (K, V) x 16 rows x D halves
}
// dynamic shared memory: the K/V ring, then the buffer the segments of a cluster are merged in
template <int D, int G>
__host__ __device__ constexpr int gqa_smem_bytes() {
  return gqa_ring_bytes<D>() + kGqaMaxCluster * G * (D + 2) * 4;
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t smem_addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t smem_addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_addr));
}

template <int D, int G>
__global__ void __launch_bounds__(kAttnDecWarps * 32) attn_decode_gqa_kernel(const AttnDecArgs a) {
  static_assert(G <= 8 && (D == 64 || D == 128), "one MMA tile of 16 rows holds the query heads of a pair");
  pdl_launch_dependents();
  if (a.dbg != nullptr && threadIdx.x == 0) {
    atomicMin(a.dbg + 10, static_cast<unsigned long long>(global_ns()));  // earliest CTA start
    atomicMax(a.dbg + 12, static_cast<unsigned long long>(global_ns()));  // latest CTA start
  }
  pdl_wait();
  if (a.dbg != nullptr && threadIdx.x == 0) atomicMin(a.dbg + 11, static_cast<unsigned long long>(global_ns()));
  constexpr int KS = D / 16;                // MMA steps along the head dimension (scores)
  constexpr int NT = D / 8;                 // 8-column tiles of the output
  constexpr int ROW_BYTES = D * 2;
  constexpr int PIECES = ROW_BYTES / 16;    // 16-byte pieces per row
  constexpr int TILE_BYTES = kGqaChunk * ROW_BYTES;
  extern __shared__ __align__(128) uint8_t gqa_ring[];
  __shared__ AttnMergeSmem<D, G> sm;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int groups = a.n_q_heads / G;
  const long long n_units = static_cast<long long>(a.n_pairs) * a.units_per_pair;
  const long long grid = gridDim.x;
  const long long u_beg = static_cast<long long>(blockIdx.x) * n_units / grid;
  const long long u_end = (static_cast<long long>(blockIdx.x) + 1) * n_units / grid;
  auto cta_of = [&](long long x) { return static_cast<int>(((x + 1) * grid - 1) / n_units); };

  uint8_t* ring = gqa_ring + warp * (kGqaStages * 2 * TILE_BYTES);  // [stage][K | V][16 rows][ROW_BYTES]
  float* cl_buf = reinterpret_cast<float*>(gqa_ring + gqa_ring_bytes<D>());
  const uint32_t ring_u32 = smem_u32(ring);

  for (long long u = u_beg; u < u_end;) {
    const int pair = static_cast<int>(u / a.units_per_pair);
    const long long pair_u0 = static_cast<long long>(pair) * a.units_per_pair;
    const long long seg_end = min(u_end, pair_u0 + a.units_per_pair);
    const int b = pair / groups, h0 = (pair - b * groups) * G;
    const int hk = h0 / (a.n_q_heads / a.n_kv_heads);
    const int t_len = a.t_len + (a.len_arr != nullptr ? a.len_arr[b] : 0);
    const int t0 = static_cast<int>(u - pair_u0) * kGqaUnit;
    const int t1 = min(t_len, static_cast<int>(seg_end - pair_u0) * kGqaUnit);
    const int first_cta = cta_of(pair_u0), n_seg = cta_of(pair_u0 + a.units_per_pair - 1) - first_cta + 1;
    const int seg = static_cast<int>(blockIdx.x) - first_cta;
    u = seg_end;

    // Q fragments (A operand, rows = heads; rows >= G are zero): step ks holds head g, elements
    // 16 ks + 2t, +1 and 16 ks + 8 + 2t, +1
    uint32_t qa[KS][2];
    {
      const half_t* qrow = a.q + (static_cast<size_t>(b) * a.n_q_heads + h0 + g) * D;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        qa[ks][0] = g < G ? __ldg(reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 2 * t)) : 0u;
        qa[ks][1] = g < G ? __ldg(reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8 + 2 * t)) : 0u;
      }
    }
    const half_t* kb = a.k_cache + (static_cast<size_t>(b) * a.n_kv_heads + hk) * a.t_max * D;
    const half_t* vb = a.v_cache + (static_cast<size_t>(b) * a.n_kv_heads + hk) * a.t_max * D;

    // blocks of 16 keys: this warp takes blocks warp, warp + 4, ... of the segment
    const int n_blocks = (t1 - t0 + kGqaChunk - 1) / kGqaChunk;          // <= 0 for an empty segment
    const int n_mine = n_blocks > warp ? (n_blocks - warp + kAttnDecWarps - 1) / kAttnDecWarps : 0;
    auto request = [&](int i, int stage) {  // copies block i of this warp into a ring stage
      const int key0 = t0 + (warp + i * kAttnDecWarps) * kGqaChunk;
      const uint32_t dst = ring_u32 + stage * (2 * TILE_BYTES);
#pragma unroll
      for (int j = 0; j < kGqaChunk * PIECES / 32; ++j) {
        const int idx = j * 32 + lane, r = idx / PIECES, c = idx - r * PIECES;
        const int key = key0 + r;
        const uint32_t bytes = key < t1 ? 16u : 0u;
        const size_t src = static_cast<size_t>(key < t1 ? key : 0) * D + c * 8;
        const uint32_t off = r * ROW_BYTES + ((c ^ (r & 7)) << 4);
        cp_async_16(dst + off, kb + src, bytes);
        cp_async_16(dst + TILE_BYTES + off, vb + src, bytes);
      }
    };

    float o[NT][4];
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int i = 0; i < 4; ++i) o[j][i] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;  // of head g; l_run: this lane's keys only until the end

    if (n_mine > 0) request(0, 0);
    cp_async_commit();
    for (int i = 0; i < n_mine; ++i) {
      if (i + 1 < n_mine) request(i + 1, (i + 1) & 1);
      cp_async_commit();
      cp_async_wait_group<1>();   // all but the newest group: block i has arrived
      __syncwarp();
      const uint32_t kt = ring_u32 + (i & 1) * (2 * TILE_BYTES), vt = kt + TILE_BYTES;
      // ---- scores of 16 keys: two 8-key tiles
      float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
      {
        // lane -> matrix lane / 8 of an x4 load: key row (matrix / 2) * 8 + lane % 8, piece 2 ks + matrix % 2
        const int mi = lane >> 3, r = (mi >> 1) * 8 + (lane & 7);
        const uint32_t row_addr = kt + r * ROW_BYTES;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
          uint32_t kf[4];
          ldmatrix_x4(kf, row_addr + (((2 * ks + (mi & 1)) ^ (r & 7)) << 4));
          mma_16816(s[0], qa[ks][0], 0u, qa[ks][1], 0u, kf[0], kf[1]);
          mma_16816(s[1], qa[ks][0], 0u, qa[ks][1], 0u, kf[2], kf[3]);
        }
      }
      // ---- online softmax for head g: this lane holds keys 2t, 2t+1 of both tiles
      const int key_base = t0 + (warp + i * kAttnDecWarps) * kGqaChunk;
      float x[4];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e)
          x[nt * 2 + e] = key_base + nt * 8 + 2 * t + e < t1 ? s[nt][e] * a.scale_log2 : -INFINITY;
      float mx = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_new = fmaxf(m_run, mx);           // finite: key key_base is inside the segment
      const float alpha = exp2f(m_run - m_new);       // first block: 2^(-inf) = 0
      m_run = m_new;
      uint32_t pa[2];
      float psum = 0.f;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        const half2_t hp = f2_to_h2(exp2f(x[nt * 2] - m_new), exp2f(x[nt * 2 + 1] - m_new));
        const float2 back = h2_to_f2(hp);       // the sum is taken over the rounded weights
        psum += back.x + back.y;
        pa[nt] = *reinterpret_cast<const uint32_t*>(&hp);
      }
      l_run = l_run * alpha + psum;
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        o[j][0] *= alpha;
        o[j][1] *= alpha;
      }
      // ---- output: O += P V; the V fragments come transposed out of shared memory
      {
        const int mi = lane >> 3, r = (mi & 1) * 8 + (lane & 7);
        const uint32_t row_addr = vt + r * ROW_BYTES;
#pragma unroll
        for (int jj = 0; jj < NT / 2; ++jj) {
          uint32_t vf[4];
          ldmatrix_x4_trans(vf, row_addr + (((2 * jj + (mi >> 1)) ^ (r & 7)) << 4));
          mma_16816(o[2 * jj], pa[0], 0u, pa[1], 0u, vf[0], vf[1]);
          mma_16816(o[2 * jj + 1], pa[0], 0u, pa[1], 0u, vf[2], vf[3]);
        }
      }
      __syncwarp();  // the stage is overwritten by the request of the next iteration
    }
    cp_async_wait_all();
    if (a.dbg != nullptr && lane == 0) {
      atomicMax(a.dbg + 13, static_cast<unsigned long long>(global_ns()));  // latest stream end of a warp
      atomicMin(a.dbg + 9, static_cast<unsigned long long>(global_ns()));   // earliest
    }
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    if (g < G) {
      if (t == 0) {
        sm.m[warp][g] = m_run;
        sm.l[warp][g] = l_run;
      }
#pragma unroll
      for (int j = 0; j < NT; ++j)
        *reinterpret_cast<float2*>(&sm.o[warp][g][8 * j + 2 * t]) = make_float2(o[j][0], o[j][1]);
    }
    __syncthreads();
    attn_finish_segment<D, G>(a, sm, cl_buf, b, h0, pair, seg, n_seg);
    __syncthreads();  // the shared arrays are reused by the next segment
  }
  if (a.dbg != nullptr && threadIdx.x == 0) atomicMax(a.dbg + 15, static_cast<unsigned long long>(global_ns()));
}

}  // namespace thinfer

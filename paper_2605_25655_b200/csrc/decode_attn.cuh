// Decode attention over the FP16 KV cache: Eq. 6 for one query row per
// (request, head), the M = 1 case of the staged attention of Section 3.3.2.
// Per request (selective batching, Section 3.4.1) and bandwidth-bound: K and V
// rows are streamed once with 128-bit loads; the query heads that share a KV
// head are processed in the same pass.  The KV range is split across CTAs
// (split-KV); every lane group keeps a running (max, sum, output) triple that
// is merged by the online-softmax rule first inside the warp, then across the
// CTA's warps, then across splits by whichever CTA of a (request, head group)
// finishes last (a ticket counter; the partials are added in split order, so the
// result does not depend on who that is).
#pragma once
#include "common.cuh"

namespace thinfer {

constexpr int kAttnDecWarps = 4;
constexpr int kAttnDecUnroll = 4;
constexpr int kAttnMaxSplits = 32;

struct AttnDecArgs {
  const __half* q;        // [batch][n_q_heads][D], already rotated
  const __half* k_cache;  // [max_batch][n_kv_heads][t_max][D]
  const __half* v_cache;
  __half* out;            // [batch][n_q_heads * D]
  float* part_o;          // [batch][n_q_heads][splits][D]   un-normalised partial outputs
  float* part_ml;         // [batch][n_q_heads][splits][2]   (max in log2 units, sum)
  int* tickets;           // [batch][n_q_heads / G] arrival counters, zero between launches (splits > 1)
  int n_q_heads, n_kv_heads;
  int t_len;              // keys to attend: positions 0 .. t_len-1
  const int* len_arr;     // ragged: request b attends len_arr[b] + t_len keys (nullptr: t_len for everybody)
  int t_max;
  int splits, chunk;      // chunk = keys per split
  float scale_log2;       // log2(e) / sqrt(D)
  unsigned long long* dbg;  // tracing aid (16 slots) or nullptr
};

// Streams keys t_first, t_first + t_step, ... (< t_end) in groups of UN*KPL and folds them into the
// running (max, sum, output) of this lane group.  kb / vb already point at this lane's 8 head elements.
template <int D, int G, int UN = kAttnDecUnroll, bool PIPELINED = true>
__device__ __forceinline__ void attn_stream_keys(const __half* kb, const __half* vb, const float (&q)[G][8], int t_first,
                                                 int t_end, int t_step, int sub, float (&m)[G], float (&l)[G],
                                                 float (&o)[G][8]) {
  constexpr int LPK = D / 8;
  constexpr int KPL = 32 / LPK;
  // software pipeline: the K/V rows of the next group are requested before the current group is
  // consumed, so loads are in flight during the arithmetic
  uint4 kv[UN], vv[UN];
  auto fetch = [&](int tb, uint4 (&k)[UN], uint4 (&v)[UN]) {
#pragma unroll
    for (int u = 0; u < UN; ++u) {
      const int t = tb + u * KPL + sub;
      if (t < t_end) {
        k[u] = ld_stream(kb + static_cast<size_t>(t) * D);
        v[u] = ld_stream(vb + static_cast<size_t>(t) * D);
      } else {
        k[u] = make_uint4(0, 0, 0, 0);
        v[u] = make_uint4(0, 0, 0, 0);
      }
    }
  };
  if (t_first < t_end) fetch(t_first, kv, vv);
  for (int tb = t_first; tb < t_end; tb += t_step) {
    uint4 kn[UN], vn[UN];
    if (PIPELINED && tb + t_step < t_end) fetch(tb + t_step, kn, vn);
    float s[G][UN];
#pragma unroll
    for (int u = 0; u < UN; ++u) {
      float fk[8];
      unpack8(kv[u], fk);
      const bool valid = (tb + u * KPL + sub) < t_end;
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float d = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) d = fmaf(q[g][i], fk[i], d);
#pragma unroll
        for (int off = LPK / 2; off > 0; off >>= 1) d += __shfl_xor_sync(0xffffffffu, d, off);
        s[g][u] = valid ? d : -INFINITY;
      }
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float mx = m[g];
#pragma unroll
      for (int u = 0; u < UN; ++u) mx = fmaxf(mx, s[g][u]);
      const float ms = (mx == -INFINITY) ? 0.f : mx;
      const float alpha = exp2f(m[g] - ms);  // m = -inf -> 0
      m[g] = mx;
      l[g] *= alpha;
#pragma unroll
      for (int i = 0; i < 8; ++i) o[g][i] *= alpha;
#pragma unroll
      for (int u = 0; u < UN; ++u) {
        const float p = exp2f(s[g][u] - ms);
        l[g] += p;
        float fv[8];
        unpack8(vv[u], fv);
#pragma unroll
        for (int i = 0; i < 8; ++i) o[g][i] = fmaf(p, fv[i], o[g][i]);
      }
    }
    if (PIPELINED) {
#pragma unroll
      for (int u = 0; u < UN; ++u) {
        kv[u] = kn[u];
        vv[u] = vn[u];
      }
    } else if (tb + t_step < t_end) {
      fetch(tb + t_step, kv, vv);
    }
  }
}

// Merges the KPL lane groups of a warp by the online-softmax rule; afterwards every lane holds the
// warp's state for its 8 head elements.
template <int D, int G>
__device__ __forceinline__ void attn_merge_lane_groups(float (&m)[G], float (&l)[G], float (&o)[G][8]) {
  constexpr int LPK = D / 8;
#pragma unroll
  for (int off = LPK; off < 32; off <<= 1) {
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const float m2 = __shfl_xor_sync(0xffffffffu, m[g], off);
      const float l2 = __shfl_xor_sync(0xffffffffu, l[g], off);
      const float mx = fmaxf(m[g], m2);
      const float ms = (mx == -INFINITY) ? 0.f : mx;
      const float a1 = exp2f(m[g] - ms), a2 = exp2f(m2 - ms);
      l[g] = l[g] * a1 + l2 * a2;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float o2 = __shfl_xor_sync(0xffffffffu, o[g][i], off);
        o[g][i] = o[g][i] * a1 + o2 * a2;
      }
      m[g] = mx;
    }
  }
}

template <int D, int G>
__global__ void __launch_bounds__(kAttnDecWarps * 32) attn_decode_kernel(const AttnDecArgs a) {
  pdl_launch_dependents();
  if (a.dbg != nullptr && threadIdx.x == 0) {
    atomicMin(a.dbg + 10, static_cast<unsigned long long>(global_ns()));  // earliest CTA start
    atomicMax(a.dbg + 12, static_cast<unsigned long long>(global_ns()));  // latest CTA start
  }
  pdl_wait();
  if (a.dbg != nullptr && threadIdx.x == 0) atomicMin(a.dbg + 11, static_cast<unsigned long long>(global_ns()));
  constexpr int LPK = D / 8;     // lanes that cover one key row
  constexpr int KPL = 32 / LPK;  // keys per warp-wide load
  constexpr int UN = kAttnDecUnroll;
  __shared__ float sm_m[kAttnDecWarps][G], sm_l[kAttnDecWarps][G];
  __shared__ float sm_o[kAttnDecWarps][G][D];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane / LPK, dl = lane % LPK;
  const int split = blockIdx.x, b = blockIdx.z;
  const int h0 = blockIdx.y * G;                                   // first query head of this CTA
  const int hk = h0 / (a.n_q_heads / a.n_kv_heads);
  const int t_len = a.t_len + (a.len_arr != nullptr ? a.len_arr[b] : 0);
  const int t0 = split * a.chunk;
  const int t1 = min(t_len, t0 + a.chunk);

  float q[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    unpack8(ldg_cached(a.q + (static_cast<size_t>(b) * a.n_q_heads + h0 + g) * D + dl * 8), q[g]);
#pragma unroll
    for (int i = 0; i < 8; ++i) q[g][i] *= a.scale_log2;
  }
  const __half* kb = a.k_cache + (static_cast<size_t>(b) * a.n_kv_heads + hk) * a.t_max * D + dl * 8;
  const __half* vb = a.v_cache + (static_cast<size_t>(b) * a.n_kv_heads + hk) * a.t_max * D + dl * 8;

  float m[G], l[G], o[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    m[g] = -INFINITY;
    l[g] = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) o[g][i] = 0.f;
  }

  attn_stream_keys<D, G>(kb, vb, q, t0 + warp * (UN * KPL), t1, kAttnDecWarps * UN * KPL, sub, m, l, o);
  if (a.dbg != nullptr && lane == 0) {
    atomicMax(a.dbg + 13, static_cast<unsigned long long>(global_ns()));  // latest stream end of a warp
    atomicMin(a.dbg + 9, static_cast<unsigned long long>(global_ns()));   // earliest
  }
  attn_merge_lane_groups<D, G>(m, l, o);
  if (sub == 0) {
#pragma unroll
    for (int g = 0; g < G; ++g) {
      if (dl == 0) {
        sm_m[warp][g] = m[g];
        sm_l[warp][g] = l[g];
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) sm_o[warp][g][dl * 8 + i] = o[g][i];
    }
  }
  __syncthreads();

  for (int idx = threadIdx.x; idx < G * D; idx += kAttnDecWarps * 32) {
    const int g = idx / D, i = idx - g * D;
    float mx = sm_m[0][g];
#pragma unroll
    for (int w = 1; w < kAttnDecWarps; ++w) mx = fmaxf(mx, sm_m[w][g]);
    const float ms = (mx == -INFINITY) ? 0.f : mx;
    float L = 0.f, O = 0.f;
#pragma unroll
    for (int w = 0; w < kAttnDecWarps; ++w) {
      const float al = exp2f(sm_m[w][g] - ms);
      L += sm_l[w][g] * al;
      O += sm_o[w][g][i] * al;
    }
    const int h = h0 + g;
    if (a.splits == 1) {
      a.out[(static_cast<size_t>(b) * a.n_q_heads + h) * D + i] = __float2half_rn(O / L);
    } else {
      const size_t p = (static_cast<size_t>(b) * a.n_q_heads + h) * a.splits + split;
      a.part_o[p * D + i] = O;
      if (i == 0) {
        a.part_ml[p * 2] = mx;
        a.part_ml[p * 2 + 1] = L;
      }
    }
  }
  if (a.dbg != nullptr && threadIdx.x == 0) atomicMax(a.dbg + 14, static_cast<unsigned long long>(global_ns()));
  if (a.splits == 1) return;

  // split-KV: the CTA that arrives last merges the partials of its G heads,
  // out = sum_s o_s 2^(m_s - M) / sum_s l_s 2^(m_s - M), s in split order
  __shared__ int is_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    int* ctr = a.tickets + b * gridDim.y + blockIdx.y;
    const int ticket = atomicAdd(ctr, 1);
    is_last = ticket == a.splits - 1;
    if (is_last) *ctr = 0;  // ready for the next launch
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  // The partials come from L2.  First the (max, sum) pairs of all splits of the G heads in one parallel round
  // trip, from them the weight 2^(m_s - M) / L of every split; then every thread adds its output elements over
  // the splits, in split order, with several independent 16-byte loads in flight.
  __shared__ float sm_pm[G][kAttnMaxSplits], sm_pl[G][kAttnMaxSplits];
  const size_t bh0 = static_cast<size_t>(b) * a.n_q_heads + h0;
  for (int idx = threadIdx.x; idx < G * a.splits; idx += kAttnDecWarps * 32) {
    const int g = idx / a.splits, s = idx - g * a.splits;
    const float2 ml = __ldcg(reinterpret_cast<const float2*>(a.part_ml + ((bh0 + g) * a.splits + s) * 2));
    sm_pm[g][s] = ml.x;
    sm_pl[g][s] = ml.y;
  }
  __syncthreads();
  if (threadIdx.x < G) {
    const int g = threadIdx.x;
    float mx = -INFINITY;
    for (int s = 0; s < a.splits; ++s) mx = fmaxf(mx, sm_pm[g][s]);
    float L = 0.f;
    for (int s = 0; s < a.splits; ++s) {
      const float al = exp2f(sm_pm[g][s] - mx);
      L += sm_pl[g][s] * al;
      sm_pm[g][s] = al;
    }
    sm_pl[g][0] = 1.f / L;
  }
  __syncthreads();
  constexpr int V4 = G * D / 4;  // 16-byte pieces of the G output rows
  for (int idx = threadIdx.x; idx < V4; idx += kAttnDecWarps * 32) {
    const int g = idx / (D / 4), i4 = idx - g * (D / 4);
    const float4* src = reinterpret_cast<const float4*>(a.part_o + (bh0 + g) * a.splits * D) + i4;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int s = 0; s < a.splits; ++s) {
      const float4 v = __ldcg(src + static_cast<size_t>(s) * (D / 4));
      const float al = sm_pm[g][s];
      acc.x = fmaf(v.x, al, acc.x);
      acc.y = fmaf(v.y, al, acc.y);
      acc.z = fmaf(v.z, al, acc.z);
      acc.w = fmaf(v.w, al, acc.w);
    }
    const float inv = sm_pl[g][0];
    uint2 o;
    o.x = pack2(acc.x * inv, acc.y * inv);
    o.y = pack2(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(a.out + (bh0 + g) * D + i4 * 4) = o;
  }
  if (a.dbg != nullptr && threadIdx.x == 0) atomicMax(a.dbg + 15, static_cast<unsigned long long>(global_ns()));
}

}  // namespace thinfer

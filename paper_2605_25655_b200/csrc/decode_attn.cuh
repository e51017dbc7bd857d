// Decode attention over the FP16 KV cache: Eq. 6 for one query row per
// (request, head), the M = 1 case of the staged attention of Section 3.3.2.
// Per request (selective batching, Section 3.4.1) and bandwidth-bound: K and V
// rows are streamed once with 128-bit loads; the query heads that share a KV
// head are processed in the same pass.  The KV ranges are split across CTAs
// (split-KV, in equal runs over a grid that fills the device once); every lane
// group keeps a running (max, sum, output) triple that is merged by the
// online-softmax rule first inside the warp, then across the CTA's warps, then
// across the segments of a (request, head group) by whichever of its CTAs
// finishes last (a ticket counter; the partials are added in segment order, so
// the result does not depend on who that is).
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"

namespace thinfer {

constexpr int kAttnDecWarps = 4;
constexpr int kAttnDecUnroll = 4;
constexpr int kAttnMaxSplits = 32;
constexpr int kAttnMaxCluster = 8;   // CTAs of one pair that merge through distributed shared memory

struct AttnDecArgs {
  const half_t* q;        // [batch][n_q_heads][D], already rotated
  const half_t* k_cache;  // [max_batch][n_kv_heads][t_max][D]
  const half_t* v_cache;
  half_t* out;            // [batch][n_q_heads * D]
  float* part_o;          // [batch][n_q_heads][kAttnMaxSplits][D]   un-normalised partial outputs of the segments
  float* part_ml;         // [batch][n_q_heads][kAttnMaxSplits][2]   (max in log2 units, sum)
  int* tickets;           // [batch][n_q_heads / G] arrival counters, zero between launches
  int n_q_heads, n_kv_heads;
  int t_len;              // keys to attend: positions 0 .. t_len-1
  const int* len_arr;     // ragged: request b attends len_arr[b] + t_len keys (nullptr: t_len for everybody)
  int t_max;
  int n_pairs;            // batch * n_q_heads / G
  int units_per_pair;     // ceil(longest key count / keys per CTA-wide iteration)
  int cluster;            // > 1: the launch uses thread-block clusters of this many CTAs, one cluster per pair; the
                          // segments of a pair are then merged in the shared memory of the cluster's first CTA
  float scale_log2;       // log2(e) / sqrt(D)
  unsigned long long* dbg;  // tracing aid (16 slots) or nullptr
};

// Streams keys t_first, t_first + t_step, ... (< t_end) in groups of UN*KPL and folds them into the
// running (max, sum, output) of this lane group.  kb / vb already point at this lane's 8 head elements.
template <int D, int G, int UN = kAttnDecUnroll, bool PIPELINED = true>
__device__ __forceinline__ void attn_stream_keys(const half_t* kb, const half_t* vb, const float (&q)[G][8], int t_first,
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

// Shared-memory state of one CTA for merging: per warp the running (max, sum, output) of its keys, and the
// weights of a pair's segments during the final merge.
template <int D, int G>
struct AttnMergeSmem {
  float m[kAttnDecWarps][G], l[kAttnDecWarps][G];
  float o[kAttnDecWarps][G][D];
  float pm[G][kAttnMaxSplits], pl[G][kAttnMaxSplits];
  int is_last;
};

// Second half of a segment, after every warp has left its state in `sm` and the CTA has synchronised: merges the
// warps; a pair with one segment is finished here, otherwise the segment's partial goes to global memory and the
// CTA of the pair that arrives last merges all of them, in segment order.
template <int D, int G>
__device__ __forceinline__ void attn_finish_segment(const AttnDecArgs& a, AttnMergeSmem<D, G>& sm, float* cl_buf, int b,
                                                    int h0, int pair, int seg, int n_seg) {
  namespace cg = cooperative_groups;
  const size_t bh0 = static_cast<size_t>(b) * a.n_q_heads + h0;
  const bool clustered = a.cluster > 1;  // then n_seg == a.cluster and seg == the CTA's rank in its cluster
  // cluster path: segment s leaves [G][D + 2] floats (output row, then max and sum) in the first CTA's buffer
  float* lead = clustered ? cg::this_cluster().map_shared_rank(cl_buf, 0) : nullptr;
  for (int idx = threadIdx.x; idx < G * D; idx += kAttnDecWarps * 32) {
    const int g = idx / D, i = idx - g * D;
    float mx = sm.m[0][g];
#pragma unroll
    for (int w = 1; w < kAttnDecWarps; ++w) mx = fmaxf(mx, sm.m[w][g]);
    const float ms = (mx == -INFINITY) ? 0.f : mx;
    float L = 0.f, O = 0.f;
#pragma unroll
    for (int w = 0; w < kAttnDecWarps; ++w) {
      const float al = exp2f(sm.m[w][g] - ms);
      L += sm.l[w][g] * al;
      O += sm.o[w][g][i] * al;
    }
    if (n_seg == 1) {
      a.out[(bh0 + g) * D + i] = f_to_h(O / L);
    } else if (clustered) {
      float* dst = lead + (seg * G + g) * (D + 2);
      dst[i] = O;
      if (i == 0) {
        dst[D] = mx;
        dst[D + 1] = L;
      }
    } else {
      const size_t p = (bh0 + g) * kAttnMaxSplits + seg;
      a.part_o[p * D + i] = O;
      if (i == 0) {
        a.part_ml[p * 2] = mx;
        a.part_ml[p * 2 + 1] = L;
      }
    }
  }
  if (n_seg > 1 && clustered) {
    // every CTA of the pair has stored its segment in the first CTA's shared memory: one cluster barrier, then
    // that CTA merges them in segment order (no round trip through L2, no ticket)
    cg::this_cluster().sync();
    if (seg == 0) {
      if (threadIdx.x < G) {
        const int g = threadIdx.x;
        float mx = -INFINITY;
        for (int sg = 0; sg < n_seg; ++sg) mx = fmaxf(mx, cl_buf[(sg * G + g) * (D + 2) + D]);
        float L = 0.f;
        for (int sg = 0; sg < n_seg; ++sg) {
          float* ml = cl_buf + (sg * G + g) * (D + 2) + D;
          const float al = exp2f(ml[0] - mx);  // an empty segment has max -inf: weight 0
          L += ml[1] * al;
          ml[0] = al;
        }
        cl_buf[g * (D + 2) + D + 1] = 1.f / L;
      }
      __syncthreads();
      for (int idx = threadIdx.x; idx < G * D; idx += kAttnDecWarps * 32) {
        const int g = idx / D, i = idx - g * D;
        float acc = 0.f;
        for (int sg = 0; sg < n_seg; ++sg) {
          const float* row = cl_buf + (sg * G + g) * (D + 2);
          acc = fmaf(row[i], row[D], acc);
        }
        a.out[(bh0 + g) * D + i] = f_to_h(acc * cl_buf[g * (D + 2) + D + 1]);
      }
    }
  } else if (n_seg > 1) {
    // the CTA that arrives last merges the segments of its G heads,
    // out = sum_s o_s 2^(m_s - M) / sum_s l_s 2^(m_s - M), s in segment order
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
      int* ctr = a.tickets + pair;
      const int ticket = atomicAdd(ctr, 1);
      sm.is_last = ticket == n_seg - 1;
      if (sm.is_last) *ctr = 0;  // ready for the next launch
    }
    __syncthreads();
    if (sm.is_last) {
      __threadfence();
      // The partials come from L2.  First the (max, sum) pairs of all segments of the G heads in one parallel
      // round trip, from them the weight 2^(m_s - M) of every segment and 1 / L; then every thread adds its
      // output elements over the segments, in segment order, with several 16-byte loads in flight.
      for (int idx = threadIdx.x; idx < G * n_seg; idx += kAttnDecWarps * 32) {
        const int g = idx / n_seg, sg = idx - g * n_seg;
        const float2 ml = __ldcg(reinterpret_cast<const float2*>(a.part_ml + ((bh0 + g) * kAttnMaxSplits + sg) * 2));
        sm.pm[g][sg] = ml.x;
        sm.pl[g][sg] = ml.y;
      }
      __syncthreads();
      if (threadIdx.x < G) {
        const int g = threadIdx.x;
        float mx = -INFINITY;
        for (int sg = 0; sg < n_seg; ++sg) mx = fmaxf(mx, sm.pm[g][sg]);
        float L = 0.f;
        for (int sg = 0; sg < n_seg; ++sg) {
          const float al = exp2f(sm.pm[g][sg] - mx);  // an empty segment has max -inf: weight 0
          L += sm.pl[g][sg] * al;
          sm.pm[g][sg] = al;
        }
        sm.pl[g][0] = 1.f / L;
      }
      __syncthreads();
      constexpr int V4 = G * D / 4;  // 16-byte pieces of the G output rows
      for (int idx = threadIdx.x; idx < V4; idx += kAttnDecWarps * 32) {
        const int g = idx / (D / 4), i4 = idx - g * (D / 4);
        const float4* src = reinterpret_cast<const float4*>(a.part_o + (bh0 + g) * kAttnMaxSplits * D) + i4;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
        for (int sg = 0; sg < n_seg; ++sg) {
          const float4 v = __ldcg(src + static_cast<size_t>(sg) * (D / 4));
          const float al = sm.pm[g][sg];
          acc.x = fmaf(v.x, al, acc.x);
          acc.y = fmaf(v.y, al, acc.y);
          acc.z = fmaf(v.z, al, acc.z);
          acc.w = fmaf(v.w, al, acc.w);
        }
        const float inv = sm.pl[g][0];
        uint2 ov;
        ov.x = pack2(acc.x * inv, acc.y * inv);
        ov.y = pack2(acc.z * inv, acc.w * inv);
        *reinterpret_cast<uint2*>(a.out + (bh0 + g) * D + i4 * 4) = ov;
      }
    }
  }
}

// Balanced split-KV schedule.  A "pair" is one request and one group of G query heads that share a KV head;
// its keys are cut into units of one CTA-wide iteration (kAttnDecWarps x UN x KPL keys).  The units of all pairs,
// laid end to end, are dealt out in equal contiguous runs to a grid that fills the resident CTA slots of the
// device exactly once: every CTA streams the same number of keys (+- one unit) whatever the batch, head count
// and sequence length are, so there is neither a partly filled last wave nor an idle SM.  A run may end inside
// a pair and continue into the next one: a CTA then works on up to a few (pair, key range) segments in turn.
// The segments of a pair are merged by whichever of its CTAs finishes last (ticket counter), in segment order.
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
  constexpr int UNIT = kAttnDecWarps * UN * KPL;  // keys of one CTA-wide iteration
  __shared__ AttnMergeSmem<D, G> sm;
  __shared__ float cl_buf[kAttnMaxCluster * G * (D + 2)];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane / LPK, dl = lane % LPK;
  const int groups = a.n_q_heads / G;                // pairs per request
  const long long n_units = static_cast<long long>(a.n_pairs) * a.units_per_pair;
  const long long grid = gridDim.x;
  const long long u_beg = static_cast<long long>(blockIdx.x) * n_units / grid;
  const long long u_end = (static_cast<long long>(blockIdx.x) + 1) * n_units / grid;
  // the CTA that holds unit x: the largest i with floor(i * n_units / grid) <= x
  auto cta_of = [&](long long x) { return static_cast<int>(((x + 1) * grid - 1) / n_units); };

  for (long long u = u_beg; u < u_end;) {
    const int pair = static_cast<int>(u / a.units_per_pair);
    const long long pair_u0 = static_cast<long long>(pair) * a.units_per_pair;
    const long long seg_end = min(u_end, pair_u0 + a.units_per_pair);
    const int b = pair / groups, h0 = (pair - b * groups) * G;
    const int hk = h0 / (a.n_q_heads / a.n_kv_heads);
    const int t_len = a.t_len + (a.len_arr != nullptr ? a.len_arr[b] : 0);
    const int t0 = static_cast<int>(u - pair_u0) * UNIT;
    const int t1 = min(t_len, static_cast<int>(seg_end - pair_u0) * UNIT);
    const int first_cta = cta_of(pair_u0), n_seg = cta_of(pair_u0 + a.units_per_pair - 1) - first_cta + 1;
    const int seg = static_cast<int>(blockIdx.x) - first_cta;
    u = seg_end;

    float q[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      unpack8(ldg_cached(a.q + (static_cast<size_t>(b) * a.n_q_heads + h0 + g) * D + dl * 8), q[g]);
#pragma unroll
      for (int i = 0; i < 8; ++i) q[g][i] *= a.scale_log2;
    }
    const half_t* kb = a.k_cache + (static_cast<size_t>(b) * a.n_kv_heads + hk) * a.t_max * D + dl * 8;
    const half_t* vb = a.v_cache + (static_cast<size_t>(b) * a.n_kv_heads + hk) * a.t_max * D + dl * 8;

    float m[G], l[G], o[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      m[g] = -INFINITY;
      l[g] = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) o[g][i] = 0.f;
    }

    attn_stream_keys<D, G>(kb, vb, q, t0 + warp * (UN * KPL), t1, UNIT, sub, m, l, o);
    if (a.dbg != nullptr && lane == 0) {
      atomicMax(a.dbg + 13, static_cast<unsigned long long>(global_ns()));  // latest stream end of a warp
      atomicMin(a.dbg + 9, static_cast<unsigned long long>(global_ns()));   // earliest
    }
    attn_merge_lane_groups<D, G>(m, l, o);
    if (sub == 0) {
#pragma unroll
      for (int g = 0; g < G; ++g) {
        if (dl == 0) {
          sm.m[warp][g] = m[g];
          sm.l[warp][g] = l[g];
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) sm.o[warp][g][dl * 8 + i] = o[g][i];
      }
    }
    __syncthreads();
    attn_finish_segment<D, G>(a, sm, cl_buf, b, h0, pair, seg, n_seg);
    __syncthreads();  // the shared arrays are reused by the next segment
  }
  if (a.dbg != nullptr && threadIdx.x == 0) atomicMax(a.dbg + 15, static_cast<unsigned long long>(global_ns()));
}

}  // namespace thinfer

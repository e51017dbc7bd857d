// Weight-streaming GEMV for decode (the small-M path of Section 3.2.2: the
// activations are shared by everybody, the output features are spread over the
// processors).  Bandwidth-bound: every weight is read once with 128-bit
// streaming loads, the few activation rows stay in L1/L2.
//
// One warp owns a pair of output features (two weight rows) and a slice of K;
// lanes stride over K in 8-element chunks, the 32 partial sums are combined
// with warp shuffles and the K slices of a pair are combined through shared
// memory (split-K inside the CTA).  RMSNorm is fused as a prologue: the gain
// is applied to the activations as they are read, the sum of squares is
// accumulated beside the dot products, and 1/rms scales the finished sums.
#pragma once
#include "epilogue.cuh"

namespace thinfer {

constexpr int kGemvWarps = 8;
constexpr int kGemvUnroll = 4;

struct GemvArgs {
  const half_t* w[3];  // QKV: wq, wk, wv.  SWIGLU: gate, up.  Others: one matrix.
  int n[3];            // rows of each matrix (0 for unused); every count is even
  int k;               // contraction length, multiple of 8
  int rows;            // tokens
  const half_t* x;     // [rows][ldx]
  int ldx;
  const half_t* gamma;  // RMSNorm gain [k] when NORM
  float eps;
  int kslices;          // 1, 2, 4 or 8 warps share one feature pair
  EpiArgs e;
};

template <int NB, int EPI, bool NORM>
__global__ void __launch_bounds__(kGemvWarps * 32) gemv_stream_kernel(const GemvArgs a) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ float red[kGemvWarps][3 * NB];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ks = warp % a.kslices;
  const int pair = blockIdx.x * (kGemvWarps / a.kslices) + warp / a.kslices;
  const int tok0 = blockIdx.y * NB;

  const int n_pairs = (EPI == EPI_SWIGLU) ? a.n[0] : (a.n[0] + a.n[1] + a.n[2]) / 2;
  const bool active = pair < n_pairs;

  const half_t* wa = nullptr;
  const half_t* wb = nullptr;
  if (active) {
    if (EPI == EPI_SWIGLU) {
      wa = a.w[0] + static_cast<size_t>(pair) * a.k;
      wb = a.w[1] + static_cast<size_t>(pair) * a.k;
    } else {
      int n = 2 * pair;
      int m = 0;
      if (n >= a.n[0]) {
        n -= a.n[0];
        m = 1;
        if (n >= a.n[1]) {
          n -= a.n[1];
          m = 2;
        }
      }
      wa = a.w[m] + static_cast<size_t>(n) * a.k;
      wb = wa + a.k;
    }
  }

  float acc0[NB], acc1[NB], ss[NB];
#pragma unroll
  for (int t = 0; t < NB; ++t) acc0[t] = acc1[t] = ss[t] = 0.f;

  if (active) {
    const int chunks = a.k >> 3;
    const int per = (chunks + a.kslices - 1) / a.kslices;
    const int cbeg = ks * per;
    const int cend = min(chunks, cbeg + per);
    for (int c0 = cbeg + lane; c0 < cend; c0 += 32 * kGemvUnroll) {
      uint4 va[kGemvUnroll], vb[kGemvUnroll];
#pragma unroll
      for (int u = 0; u < kGemvUnroll; ++u) {
        const int c = c0 + 32 * u;
        if (c < cend) {
          va[u] = ldg_stream(wa + (static_cast<size_t>(c) << 3));
          vb[u] = ldg_stream(wb + (static_cast<size_t>(c) << 3));
        } else {
          va[u] = make_uint4(0, 0, 0, 0);
          vb[u] = make_uint4(0, 0, 0, 0);
        }
      }
#pragma unroll
      for (int u = 0; u < kGemvUnroll; ++u) {
        const int c = c0 + 32 * u;
        if (c < cend) {
          float fa[8], fb[8], fg[8];
          unpack8(va[u], fa);
          unpack8(vb[u], fb);
          if (NORM) unpack8(ldg_cached(a.gamma + (c << 3)), fg);
#pragma unroll
          for (int t = 0; t < NB; ++t) {
            if (tok0 + t < a.rows) {
              float fx[8];
              unpack8(ldg_cached(a.x + static_cast<size_t>(tok0 + t) * a.ldx + (c << 3)), fx);
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                if (NORM) {
                  ss[t] = fmaf(fx[i], fx[i], ss[t]);
                  fx[i] *= fg[i];
                }
                acc0[t] = fmaf(fa[i], fx[i], acc0[t]);
                acc1[t] = fmaf(fb[i], fx[i], acc1[t]);
              }
            }
          }
        }
      }
    }
  }

#pragma unroll
  for (int t = 0; t < NB; ++t) {
    acc0[t] = warp_sum(acc0[t]);
    acc1[t] = warp_sum(acc1[t]);
    if (NORM) ss[t] = warp_sum(ss[t]);
  }
  if (lane == 0) {
#pragma unroll
    for (int t = 0; t < NB; ++t) {
      red[warp][t] = acc0[t];
      red[warp][NB + t] = acc1[t];
      red[warp][2 * NB + t] = ss[t];
    }
  }
  __syncthreads();
  if (!active || ks != 0 || lane >= NB) return;
  const int r = tok0 + lane;
  if (r >= a.rows) return;

  float s0 = 0.f, s1 = 0.f, sq = 0.f;
  for (int j = 0; j < a.kslices; ++j) {
    s0 += red[warp + j][lane];
    s1 += red[warp + j][NB + lane];
    sq += red[warp + j][2 * NB + lane];
  }
  if (NORM) {
    const float rstd = rsqrtf(sq / static_cast<float>(a.k) + a.eps);
    s0 *= rstd;
    s1 *= rstd;
  }

  const EpiArgs& e = a.e;
  if (EPI == EPI_SWIGLU) {
    reinterpret_cast<half_t*>(e.out)[static_cast<size_t>(r) * e.ld_out + pair] = f_to_h(silu_f(s0) * s1);
  } else if (EPI == EPI_RESID) {
    const size_t o = static_cast<size_t>(r) * e.ld_out + 2 * pair;
    const float2 x = h2_to_f2(*reinterpret_cast<const half2_t*>(e.resid + o));
    *reinterpret_cast<uint32_t*>(reinterpret_cast<half_t*>(e.out) + o) = pack2(x.x + s0, x.y + s1);
  } else if (EPI == EPI_PLAIN_F16) {
    *reinterpret_cast<uint32_t*>(reinterpret_cast<half_t*>(e.out) + static_cast<size_t>(r) * e.ld_out + 2 * pair) =
        pack2(s0, s1);
  } else if (EPI == EPI_PLAIN_F32) {
    *reinterpret_cast<float2*>(reinterpret_cast<float*>(e.out) + static_cast<size_t>(r) * e.ld_out + 2 * pair) =
        make_float2(s0, s1);
  } else {  // EPI_QKV_ROPE: the pair (2j, 2j+1) of one head is exactly this warp's two features
    int kind, i, pos;
    const size_t o = qkv_offset(e, r, 2 * pair, kind, i, pos);
    if (kind != 2) {
      const float c = e.rope_cos[static_cast<size_t>(pos) * (e.head_dim >> 1) + (i >> 1)];
      const float s = e.rope_sin[static_cast<size_t>(pos) * (e.head_dim >> 1) + (i >> 1)];
      const float y0 = s0 * c - s1 * s;
      const float y1 = s1 * c + s0 * s;
      s0 = y0;
      s1 = y1;
    }
    half_t* dst = (kind == 0) ? e.q_out : (kind == 1 ? e.k_cache : e.v_cache);
    *reinterpret_cast<uint32_t*>(dst + o) = pack2(s0, s1);
  }
}

}  // namespace thinfer

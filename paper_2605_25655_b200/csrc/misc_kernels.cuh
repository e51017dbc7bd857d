// Low-density operators that stand alone (Section 3.2: I/O-bound, one pass
// over their data): row RMSNorm in front of the TMA-fed prefill GEMMs,
// embedding gather, last-row gather, greedy argmax, RoPE table.
#pragma once
#include "common.cuh"

namespace thinfer {

// y[r][:] = x[r][:] * gain / sqrt(mean(x[r]^2) + eps); FP32 inside (Section 3.2.4).
// One warp per row, 128-bit accesses; n is a multiple of 8.
__global__ void __launch_bounds__(256) rmsnorm_rows_kernel(const half_t* __restrict__ x, const half_t* __restrict__ gain,
                                                           half_t* __restrict__ y, int rows, int n, float eps) {
  pdl_launch_dependents();
  pdl_wait();
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const half_t* xr = x + static_cast<size_t>(row) * n;
  half_t* yr = y + static_cast<size_t>(row) * n;
  const int chunks = n >> 3;
  float ss = 0.f;
  for (int c = lane; c < chunks; c += 32) {
    float f[8];
    unpack8(ldg_cached(xr + (c << 3)), f);
#pragma unroll
    for (int i = 0; i < 8; ++i) ss = fmaf(f[i], f[i], ss);
  }
  ss = warp_sum(ss);
  const float rstd = rsqrtf(ss / static_cast<float>(n) + eps);
  for (int c = lane; c < chunks; c += 32) {
    float f[8], g[8];
    unpack8(ldg_cached(xr + (c << 3)), f);
    unpack8(ldg_cached(gain + (c << 3)), g);
    uint4 o;
    o.x = pack2(f[0] * rstd * g[0], f[1] * rstd * g[1]);
    o.y = pack2(f[2] * rstd * g[2], f[3] * rstd * g[3]);
    o.z = pack2(f[4] * rstd * g[4], f[5] * rstd * g[5]);
    o.w = pack2(f[6] * rstd * g[6], f[7] * rstd * g[7]);
    *reinterpret_cast<uint4*>(yr + (c << 3)) = o;
  }
}

// The same operator for few rows (decode): one CTA per row, the row is read once into registers.
// n <= 8 * 256 * kRmsSmallChunks.
constexpr int kRmsSmallChunks = 8;
__global__ void __launch_bounds__(256) rmsnorm_few_rows_kernel(const half_t* __restrict__ x,
                                                               const half_t* __restrict__ gain, half_t* __restrict__ y,
                                                               int n, float eps) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ float red[8];
  const half_t* xr = x + static_cast<size_t>(blockIdx.x) * n;
  half_t* yr = y + static_cast<size_t>(blockIdx.x) * n;
  const int chunks = n >> 3;
  uint4 xv[kRmsSmallChunks], gv[kRmsSmallChunks];
#pragma unroll
  for (int j = 0; j < kRmsSmallChunks; ++j) {
    const int c = threadIdx.x + j * 256;
    if (c < chunks) {
      xv[j] = ldg_cached(xr + (c << 3));
      gv[j] = ldg_cached(gain + (c << 3));
    }
  }
  float ss = 0.f;
#pragma unroll
  for (int j = 0; j < kRmsSmallChunks; ++j) {
    if (threadIdx.x + j * 256 < chunks) {
      float f[8];
      unpack8(xv[j], f);
#pragma unroll
      for (int i = 0; i < 8; ++i) ss = fmaf(f[i], f[i], ss);
    }
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];
  const float rstd = rsqrtf(tot / static_cast<float>(n) + eps);
#pragma unroll
  for (int j = 0; j < kRmsSmallChunks; ++j) {
    const int c = threadIdx.x + j * 256;
    if (c < chunks) {
      float f[8], g[8];
      unpack8(xv[j], f);
      unpack8(gv[j], g);
      uint4 o;
      o.x = pack2(f[0] * rstd * g[0], f[1] * rstd * g[1]);
      o.y = pack2(f[2] * rstd * g[2], f[3] * rstd * g[3]);
      o.z = pack2(f[4] * rstd * g[4], f[5] * rstd * g[5]);
      o.w = pack2(f[6] * rstd * g[6], f[7] * rstd * g[7]);
      *reinterpret_cast<uint4*>(yr + (c << 3)) = o;
    }
  }
}

// dst[r][:] = table[ids[r]][:]  (embedding).  One warp per row.
__global__ void __launch_bounds__(256) embed_gather_kernel(const int32_t* __restrict__ ids,
                                                           const half_t* __restrict__ table, half_t* __restrict__ dst,
                                                           int rows, int n, int vocab) {
  pdl_launch_dependents();
  pdl_wait();
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  int id = ids[row];
  id = min(max(id, 0), vocab - 1);
  const uint4* src = reinterpret_cast<const uint4*>(table + static_cast<size_t>(id) * n);
  uint4* d = reinterpret_cast<uint4*>(dst + static_cast<size_t>(row) * n);
  for (int c = lane; c < (n >> 3); c += 32) d[c] = __ldg(src + c);
}

// dst[b][:] = src[b][seq_len-1][:]  (the last prompt position feeds the LM head).
__global__ void __launch_bounds__(256) gather_last_rows_kernel(const half_t* __restrict__ src, half_t* __restrict__ dst,
                                                               int batch, int seq_len, int n,
                                                               const int* __restrict__ lens) {
  pdl_launch_dependents();
  pdl_wait();
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= batch) return;
  const int last = (lens != nullptr ? lens[row] : seq_len) - 1;  // ragged prompts end at their own length
  const uint4* s = reinterpret_cast<const uint4*>(src + (static_cast<size_t>(row) * seq_len + last) * n);
  uint4* d = reinterpret_cast<uint4*>(dst + static_cast<size_t>(row) * n);
  for (int c = lane; c < (n >> 3); c += 32) d[c] = __ldg(s + c);
}

// ids[r] = argmax_n logits[r][n], exact ties to the lowest index.  One CTA per row.
__global__ void __launch_bounds__(1024) argmax_rows_kernel(const float* __restrict__ logits, int32_t* __restrict__ ids,
                                                           int n) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ float sv[32];
  __shared__ int si[32];
  const float* row = logits + static_cast<size_t>(blockIdx.x) * n;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  // eight independent loads in flight per thread: the row comes out of L2 and a dependent chain of single
  // loads would be all latency.
  constexpr int kU = 8;
  int i = threadIdx.x;
  for (; i + (kU - 1) * static_cast<int>(blockDim.x) < n; i += kU * blockDim.x) {
    float v[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) v[u] = __ldcs(row + i + u * blockDim.x);
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int idx = i + u * blockDim.x;
      if (v[u] > best || (v[u] == best && idx < bi)) {
        best = v[u];
        bi = idx;
      }
    }
  }
  for (; i < n; i += blockDim.x) {
    const float v = row[i];
    if (v > best || (v == best && i < bi)) {
      best = v;
      bi = i;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float v2 = __shfl_xor_sync(0xffffffffu, best, o);
    const int i2 = __shfl_xor_sync(0xffffffffu, bi, o);
    if (v2 > best || (v2 == best && i2 < bi)) {
      best = v2;
      bi = i2;
    }
  }
  if ((threadIdx.x & 31) == 0) {
    sv[threadIdx.x >> 5] = best;
    si[threadIdx.x >> 5] = bi;
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    const int nw = blockDim.x >> 5;
    best = threadIdx.x < nw ? sv[threadIdx.x] : -INFINITY;
    bi = threadIdx.x < nw ? si[threadIdx.x] : 0x7fffffff;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float v2 = __shfl_xor_sync(0xffffffffu, best, o);
      const int i2 = __shfl_xor_sync(0xffffffffu, bi, o);
      if (v2 > best || (v2 == best && i2 < bi)) {
        best = v2;
        bi = i2;
      }
    }
    if (threadIdx.x == 0) ids[blockIdx.x] = bi;
  }
}

// cos/sin of pos * base^(-2j/head_dim) in FP32 from double-precision arguments
// (positions reach thousands of radians: fast intrinsics are not accurate there).
__global__ void rope_table_kernel(float* __restrict__ cos_t, float* __restrict__ sin_t, int max_seq, int half_dim,
                                  double base) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= max_seq * half_dim) return;
  const int pos = idx / half_dim, j = idx - pos * half_dim;
  const double theta = pow(base, -static_cast<double>(j) / static_cast<double>(half_dim));
  double s, c;
  sincos(static_cast<double>(pos) * theta, &s, &c);
  cos_t[idx] = static_cast<float>(c);
  sin_t[idx] = static_cast<float>(s);
}

// Tracing aid: resets the 16 slots of every kernel id before a traced step (slots 9 .. 11 collect minima,
// 12 .. 15 maxima), so that no memset sits between the kernels of the step.
__global__ void trace_reset_kernel(unsigned long long* timeline, int kernels) {
  pdl_launch_dependents();
  pdl_wait();  // the kernels behind it in the chain only wait for THIS kernel: it must itself be ordered
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= kernels * 16) return;
  const int slot = i & 15;
  if (slot >= 9 && slot <= 11) timeline[i] = ~0ull;
  else if (slot >= 12) timeline[i] = 0ull;
}

// Self-test of the bounded wait every pipeline of this library relies on: one thread initialises an mbarrier
// that expects an arrival nobody makes, all threads wait on it with the given limit, the wait gives up,
// THINFER_ETIMEOUT lands in the status word and the kernel returns normally (nothing traps or hangs).
__global__ void bounded_wait_selftest_kernel(int* status, unsigned long long limit_ns, unsigned long long* waited_ns) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    fence_barrier_init();
  }
  __syncthreads();
  const uint64_t t0 = global_ns();
  const bool ok = mbar_wait_for(&bar, 0, status, limit_ns);
  if (threadIdx.x == 0 && waited_ns != nullptr) *waited_ns = ok ? 0ull : global_ns() - t0;
}

}  // namespace thinfer

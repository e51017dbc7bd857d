// Weight-streaming skinny GEMM for decode with up to 16 tokens (the small-M
// path of Section 3.2.2 with the fusion units of Section 3.3.1).  The work is
// bandwidth-bound: every weight is read from HBM exactly once and is consumed by
// a warp-level tensor-core instruction (mma.sync m16n8k16, FP16 in, FP32
// accumulate), so that 16 tokens cost no more issue slots than one.
//
// Decomposition.  The output features are cut into one contiguous share per
// CTA, balanced to within one feature pair over a grid that is a multiple of
// the SM count: no wave quantisation and no partial sums that cross CTAs.  A
// share is at most TM tiles of 16 weight rows.  The 8 warps of a CTA take the
// 64-element blocks of K in turn (block b belongs to warp b mod 8), every CTA
// starting at a different block; for its block a warp loads the token fragment
// once and walks all tiles of the share with it, one FP32 fragment per tile in
// registers.  After the stream the 8 fragments of a tile are added in warp
// order through shared memory (a fixed order: results do not depend on timing)
// and the fused epilogue runs.
//
// Weights travel global -> shared memory by 16-byte asynchronous copies
// (cp.async, no registers held) into a ring of ST stages per warp.  The warp
// copies a stage cooperatively, 4 rows x 128 contiguous bytes per instruction,
// into a swizzled layout from which the MMA fragments are read without bank
// conflicts; cp.async.wait_group plus a warp barrier on both sides of the reads
// is all the synchronisation the ring needs.  The ring is filled before the
// wait on the previous kernel.  The kernel uses no tensor memory, so under
// programmatic dependent launch the CTAs of the next projection move in as the
// CTAs of this one leave.
#pragma once
#include "epilogue.cuh"

namespace thinfer {

constexpr int kSkWarps = 8;
constexpr int kSkTokMax = 16;
// ring depth per warp is the template parameter ST; one stage = 16 rows x 64 elements = 2 KB

struct SkinnyArgs {
  const half_t* w[3];  // QKV: wq, wk, wv.  SWIGLU: gate, up.  Others: one matrix.
  int n[3];            // rows of each matrix (0 for unused); every count is even
  int cta0[4];         // CTAs cta0[m] .. cta0[m+1]-1 share matrix m (SWIGLU: everything is "matrix" 0)
  int k;               // contraction length, multiple of 64
  int rows;            // tokens, <= 8 * NT
  const half_t* x;     // [rows][ldx]
  int ldx;
  // folded RMSNorm of the token operand: sums of squares per (part, token), [sumsq_parts][16], as the
  // RESID epilogue of this kernel leaves them (one part per CTA)
  const float* sumsq_in;
  int sumsq_parts;
  int norm_dim;
  float norm_eps;
  // NORM kernels instead take the raw rows in x and the gain here: RMSNorm as a prologue.  Every CTA reads
  // all of x anyway, so the sums of squares come from the token fragments it already holds, the gain is
  // multiplied in (FP16, the rounding of a stored normalised operand) and 1/rms scales the finished sums.
  const half_t* gamma;
  int tiles_max;       // row tiles of the largest CTA share (<= TM)
  EpiArgs e;           // RESID with outg: e.sumsq receives [gridDim.x][16]
  unsigned long long* dbg;  // tracing aid (16 slots) or nullptr
  unsigned long long* cta_log;  // tracing aid: per CTA {SM id, past the dependency wait, last warp's stream end, end} or nullptr
};

__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32." THINFER_MMA_SYNC_TYPES ".f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// 16 bytes global -> shared, bypassing L1; src_bytes = 0 writes zeros and reads nothing
__device__ __forceinline__ void cp_async_16(uint32_t smem_dst, const void* gsrc, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(smem_dst), "l"(gsrc), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_group() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}
// element-wise FP16 product of two groups of 8 halves
__device__ __forceinline__ uint4 hmul2x4(const uint4& a, const uint4& b) {
  uint4 r;
  const half2_t* pa = reinterpret_cast<const half2_t*>(&a);
  const half2_t* pb = reinterpret_cast<const half2_t*>(&b);
  half2_t* pr = reinterpret_cast<half2_t*>(&r);
#pragma unroll
  for (int i = 0; i < 4; ++i) pr[i] = __hmul2(pa[i], pb[i]);
  return r;
}
__device__ __forceinline__ void cp_async_4(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;\n" ::: "memory"); }

// The ring doubles as the parking area of the finished fragments (TM * NT * 128 floats per warp).
__host__ __device__ constexpr int sk_smem_floats(int tm, int stages, int parts) {
  return kSkWarps * stages * 512 + parts * 16 + tm * 16 + 16 * 16 + 16;
}

// A "unit" of the partition is a pair of adjacent features (rows 2u, 2u+1 of the concatenated space), or
// for SWIGLU one feature (its gate row and its up row).  A tile is the 16 rows of one MMA:
//   plain:  MMA row j <-> row (tile start) + j
//   SWIGLU: MMA row j < 8 <-> gate row (tile start) + j, MMA row j + 8 <-> up row (tile start) + j
// In the m16n8k16 fragment layout lane (g = lane / 4, t = lane % 4) holds rows g and g + 8 of A, token g of
// B and the outputs (rows g, g + 8) x (tokens 2t, 2t + 1).  Which k index a register slot stands for is
// irrelevant as long as A and B agree, so every lane simply takes 16 contiguous bytes: of a 64-element
// block, lane t holds elements 8t..8t+7 and 32+8t..32+8t+7 of its rows and of its token.
template <int NT, int TM, int ST, int EPI, bool NORM = false>
__global__ void __launch_bounds__(kSkWarps * 32, 2) skinny_mma_kernel(const SkinnyArgs a) {
  static_assert(ST * 4 >= TM * NT, "the fragments of a warp are parked in its own ring");
  pdl_launch_dependents();
  extern __shared__ __align__(16) float sk_smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  if (a.dbg != nullptr && threadIdx.x == 0) {
    atomicMin(a.dbg + 10, static_cast<unsigned long long>(global_ns()));  // earliest CTA start
    atomicMax(a.dbg + 12, static_cast<unsigned long long>(global_ns()));  // latest CTA start
  }
  // The CTAs are dealt out to the matrices in proportion to their rows, so a share never lies across two
  // matrices; inside its matrix a CTA takes a contiguous run of units, balanced to within one unit.
  const int m = (static_cast<int>(blockIdx.x) >= a.cta0[2]) ? 2 : (static_cast<int>(blockIdx.x) >= a.cta0[1] ? 1 : 0);
  const int m_ctas = a.cta0[m + 1] - a.cta0[m], m_cta = blockIdx.x - a.cta0[m];
  const int units = (EPI == EPI_SWIGLU) ? a.n[0] : a.n[m] >> 1;
  const int u_beg = static_cast<int>(static_cast<long long>(m_cta) * units / m_ctas);
  const int u_end = static_cast<int>(static_cast<long long>(m_cta + 1) * units / m_ctas);
  // Rows of the share, numbered inside the matrix.  SWIGLU: "row" = feature, a tile holds 8 features (8 gate
  // rows and 8 up rows); otherwise a tile holds 16 rows.  Tiles start at the share; the last one may be
  // partial.  Rows outside [r_lo, r_hi) cost no traffic.
  constexpr int TR = (EPI == EPI_SWIGLU) ? 8 : 16;  // share rows per tile
  const int r_lo = (EPI == EPI_SWIGLU) ? u_beg : 2 * u_beg;
  const int r_hi = (EPI == EPI_SWIGLU) ? u_end : 2 * u_end;
  const int row00 = r_lo;                                    // first row of tile 0
  const int r_cat = (m == 0) ? 0 : (m == 1 ? a.n[0] : a.n[0] + a.n[1]);  // row of the concatenated space = r_cat + row
  const int n_tiles = (r_hi - r_lo + TR - 1) / TR;           // <= TM; the walk always takes TM tiles
  const int nkb = a.k >> 6;                                  // k is a multiple of 64 (checked on the host)
  const int nkw = (nkb - warp + kSkWarps - 1) / kSkWarps;    // blocks warp, warp + 8, ...

  // Every CTA starts its walk along K at a different block, so that the CTAs do not all read the same
  // columns of their rows at the same time (the order of the sum is fixed per CTA all the same).
  const int rot = nkw > 0 ? static_cast<int>(blockIdx.x) % nkw : 0;
  auto rotated = [&](int blk) { return blk + rot < nkw ? blk + rot : blk + rot - nkw; };

  uint4* ring = reinterpret_cast<uint4*>(sk_smem) + warp * (ST * 128);  // [stage][16 rows][8 chunks]
  float* part = sk_smem;                                                // after the stream: [warp][TM][nt][4][32]
  float* ssq_in = sk_smem + kSkWarps * ST * 512;                        // [parts][16]
  float* ssq_tile = ssq_in + a.sumsq_parts * 16;                        // [tile][16]
  float* red = ssq_tile + TM * 16;                                      // [16][16]
  float* rstd = red + 256;                                              // [16]

  // The warp copies a (tile, block) pair cooperatively, 4 rows x 128 contiguous bytes per instruction: lane
  // l takes 16-byte chunk l % 8 of tile row l / 8 + 4 j in instruction j.  A stage is row-major
  // [16][128 B] with chunk c of row r at position c ^ 4 (r & 1): the copies and the fragment reads (row g,
  // chunks t and 4 + t) are both free of bank conflicts.  A row outside the share keeps a computable
  // address and a copy size of zero: the copy then writes zeros and reads nothing.
  const int crow = lane >> 3, cchunk = lane & 7;
  const uint32_t coop_dst = smem_u32(ring) + crow * 128 + ((cchunk ^ ((crow & 1) << 2)) << 4);
  const size_t coop_off = static_cast<size_t>(warp) * 64 + cchunk * 8;
  const int lim_hi = r_hi - r_lo - crow;  // tile row TR * tile + 4 j (+ crow) is in the share iff TR * tile + 4 j < lim_hi
  const half_t* tb[TM];  // plain: row crow of the tile, at this lane's chunk of block `warp`
  if (EPI != EPI_SWIGLU) {
#pragma unroll
    for (int tile = 0; tile < TM; ++tile)
      tb[tile] = a.w[m] + static_cast<size_t>(min(row00 + tile * 16 + crow, a.n[m] - 1)) * a.k + coop_off;
  }
  auto request = [&](int tile, int blk, int stage) {
    const size_t off = static_cast<size_t>(rotated(blk)) * (kSkWarps * 64);
    const uint32_t dst = coop_dst + stage * 2048;
    if (EPI == EPI_SWIGLU) {
      const size_t row0 = static_cast<size_t>(r_lo + tile * 8 + crow) * a.k + coop_off + off;
      const uint32_t s0 = tile * 8 < lim_hi ? 16u : 0u, s1 = tile * 8 + 4 < lim_hi ? 16u : 0u;
      const size_t o0 = s0 ? row0 : 0, o1 = s1 ? row0 + static_cast<size_t>(4) * a.k : 0;
      cp_async_16(dst, a.w[0] + o0, s0);
      cp_async_16(dst + 512, a.w[0] + o1, s1);
      cp_async_16(dst + 1024, a.w[1] + o0, s0);
      cp_async_16(dst + 1536, a.w[1] + o1, s1);
    } else {
      const half_t* src = tb[tile] + off;
      const size_t k4 = static_cast<size_t>(4) * a.k;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const bool ok = tile * 16 + 4 * j < lim_hi;
        cp_async_16(dst + 512 * j, ok ? src + j * k4 : a.w[0], ok ? 16u : 0u);
      }
    }
  };

  // Pair number j = blk * TM + tile lives in stage j mod ST and is requested ST pairs ahead of its use.
  // The weights do not depend on the previous kernel: the ring is filled before the wait.
#pragma unroll
  for (int j = 0; j < ST; ++j) {
    if (j / TM < nkw) request(j % TM, j / TM, j);
    cp_async_commit();
  }
  pdl_wait();
  if (a.dbg != nullptr && threadIdx.x == 0) atomicMin(a.dbg + 11, static_cast<unsigned long long>(global_ns()));
  if (a.cta_log != nullptr && threadIdx.x == 0) {
    unsigned int smid;
    asm volatile("mov.u32 %0, %smid;" : "=r"(smid));
    a.cta_log[blockIdx.x * 4] = smid;
    a.cta_log[blockIdx.x * 4 + 1] = global_ns();
    a.cta_log[blockIdx.x * 4 + 2] = 0;
  }

  if (a.sumsq_in != nullptr) {
    // asynchronous copies straight into shared memory: no registers held, consumed after the stream
    // (they join whichever group is committed next; the final wait covers them)
    for (int i = threadIdx.x; i < a.sumsq_parts * 16; i += kSkWarps * 32)
      cp_async_4(ssq_in + i, a.sumsq_in + i);
  }

  // token fragments: XB buffers, requested XB - 1 blocks ahead (the fewer tiles a block has, the further)
  constexpr int XB = TM == 1 ? 4 : (TM <= 3 ? 3 : 2);
  const uint4 zero = make_uint4(0, 0, 0, 0);
  const half_t* xrow[NT];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
    xrow[nt] = (nt * 8 + g < a.rows) ? a.x + static_cast<size_t>(nt * 8 + g) * a.ldx + static_cast<size_t>(warp) * 64 + t * 8
                                     : nullptr;
  uint4 xq[XB][NT][2];
  auto load_x = [&](int blk, uint4 (&x)[NT][2]) {
    const size_t off = static_cast<size_t>(rotated(blk)) * (kSkWarps * 64);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      x[nt][0] = xrow[nt] != nullptr ? ldg_cached(xrow[nt] + off) : zero;
      x[nt][1] = xrow[nt] != nullptr ? ldg_cached(xrow[nt] + off + 32) : zero;
    }
  };
#pragma unroll
  for (int b = 0; b < XB - 1; ++b)
    if (b < nkw) load_x(b, xq[b]);

  float acc[TM][NT][4];
#pragma unroll
  for (int tile = 0; tile < TM; ++tile)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[tile][nt][i] = 0.f;

  float ssx[NT];  // NORM: this lane's share of the sum of squares of token nt * 8 + g
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) ssx[nt] = 0.f;
  const half_t* grow = NORM ? a.gamma + static_cast<size_t>(warp) * 64 + t * 8 : nullptr;

  int stage = 0;
  const int frag0 = g * 8 + (t ^ ((g & 1) << 2));  // row g, chunk t (chunk 4 + t: position ^ 4; row g + 8: + 64)
  for (int i0 = 0; i0 < nkw; i0 += XB) {
#pragma unroll
    for (int b = 0; b < XB; ++b) {
      const int i = i0 + b;
      if (i < nkw) {
        if (i + XB - 1 < nkw) load_x(i + XB - 1, xq[(b + XB - 1) % XB]);
        if (NORM) {
          const size_t off = static_cast<size_t>(rotated(i)) * (kSkWarps * 64);
          const uint4 g0 = ldg_cached(grow + off), g1 = ldg_cached(grow + off + 32);  // 8 KB in all: stays in L1
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            float f[8];
            unpack8(xq[b][nt][0], f);
#pragma unroll
            for (int j = 0; j < 8; ++j) ssx[nt] = fmaf(f[j], f[j], ssx[nt]);
            unpack8(xq[b][nt][1], f);
#pragma unroll
            for (int j = 0; j < 8; ++j) ssx[nt] = fmaf(f[j], f[j], ssx[nt]);
            xq[b][nt][0] = hmul2x4(xq[b][nt][0], g0);
            xq[b][nt][1] = hmul2x4(xq[b][nt][1], g1);
          }
        }
#pragma unroll
        for (int tile = 0; tile < TM; ++tile) {
          // one group per pair, ST pairs ahead: all but the newest ST - 1 groups are complete.  Lanes read
          // what other lanes copied: a warp barrier on both sides of the reads.
          cp_async_wait_group<ST - 1>();
          __syncwarp();
          const uint4* src = ring + stage * 128;
          const uint4 a0 = src[frag0], a1 = src[frag0 ^ 4], b0 = src[64 + frag0], b1 = src[64 + (frag0 ^ 4)];
          __syncwarp();
          // the stage is free again; it receives the pair ST ahead
          const int t2 = (tile + ST) % TM, db = (tile + ST) / TM;  // constants once unrolled
          if (i + db < nkw) request(t2, i + db, stage);
          cp_async_commit();
          if (++stage == ST) stage = 0;
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            mma_16816(acc[tile][nt], a0.x, b0.x, a0.y, b0.y, xq[b][nt][0].x, xq[b][nt][0].y);
            mma_16816(acc[tile][nt], a0.z, b0.z, a0.w, b0.w, xq[b][nt][0].z, xq[b][nt][0].w);
            mma_16816(acc[tile][nt], a1.x, b1.x, a1.y, b1.y, xq[b][nt][1].x, xq[b][nt][1].y);
            mma_16816(acc[tile][nt], a1.z, b1.z, a1.w, b1.w, xq[b][nt][1].z, xq[b][nt][1].w);
          }
        }
      }
    }
  }
  cp_async_wait_all();
  __syncwarp();
  if (a.dbg != nullptr && lane == 0) {
    atomicMax(a.dbg + 13, static_cast<unsigned long long>(global_ns()));  // latest stream end of a warp
    atomicMin(a.dbg + 9, static_cast<unsigned long long>(global_ns()));   // earliest
  }
  if (a.cta_log != nullptr && lane == 0) atomicMax(a.cta_log + blockIdx.x * 4 + 2, static_cast<unsigned long long>(global_ns()));
  // park the fragments in this warp's own ring
  {
    float* dst = part + static_cast<size_t>(warp) * (ST * 512) + lane;
#pragma unroll
    for (int tile = 0; tile < TM; ++tile)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) dst[(tile * NT + nt) * 128 + i * 32] = acc[tile][nt][i];
  }
  if (NORM) {
    // lanes t = 0..3 of a token hold disjoint parts of K; warps hold disjoint blocks
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      ssx[nt] += __shfl_xor_sync(0xffffffffu, ssx[nt], 1);
      ssx[nt] += __shfl_xor_sync(0xffffffffu, ssx[nt], 2);
      if (t == 0) red[warp * 16 + nt * 8 + g] = ssx[nt];
    }
  }
  __syncthreads();
  if (a.dbg != nullptr && threadIdx.x == 0) atomicMax(a.dbg + 14, static_cast<unsigned long long>(global_ns()));
  if (NORM) {
    if (threadIdx.x < 16) {
      float tot = 0.f;
      if (threadIdx.x < NT * 8) {
#pragma unroll
        for (int w = 0; w < kSkWarps; ++w) tot += red[w * 16 + threadIdx.x];
      }
      rstd[threadIdx.x] = rsqrtf(tot / static_cast<float>(a.k) + a.norm_eps);
    }
    __syncthreads();
  }

  // ---- 1/rms per token from the producer's per-part sums (fixed order)
  if (a.sumsq_in != nullptr) {
    const int tok = threadIdx.x & 15, sl = threadIdx.x >> 4;  // 16 slices of parts
    float s = 0.f;
    for (int p = sl; p < a.sumsq_parts; p += 16) s += ssq_in[p * 16 + tok];
    red[sl * 16 + tok] = s;
    __syncthreads();
    if (threadIdx.x < 16) {
      float tot = 0.f;
#pragma unroll
      for (int j = 0; j < 16; ++j) tot += red[j * 16 + threadIdx.x];
      rstd[threadIdx.x] = rsqrtf(tot / static_cast<float>(a.norm_dim) + a.norm_eps);
    }
    __syncthreads();
  }

  // ---- K slices added in warp order, then the fused epilogue; one (tile, token tile) per warp at a time
  const EpiArgs& e = a.e;
  for (int item = warp; item < n_tiles * NT; item += kSkWarps) {
    const int tile = item / NT, nt = item - tile * NT;
    float c[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      c[i] = 0.f;
    }
#pragma unroll
    for (int w = 0; w < kSkWarps; ++w) {
      const float* src = part + static_cast<size_t>(w) * (ST * 512) + (tile * NT + nt) * 128 + lane;
#pragma unroll
      for (int i = 0; i < 4; ++i) c[i] += src[i * 32];
    }
    const int row0 = row00 + tile * TR;  // first share row of the tile (numbered inside the matrix)
    const int ta = nt * 8 + 2 * t, tb = ta + 1;
    if (NORM || a.sumsq_in != nullptr) {
      const float sa = rstd[ta], sb = rstd[tb];
      c[0] *= sa;
      c[1] *= sb;
      c[2] *= sa;
      c[3] *= sb;
    }
    if (EPI == EPI_SWIGLU) {
      const int f = row0 + g;
      if (f < r_hi) {
        half_t* o = reinterpret_cast<half_t*>(e.out);
        if (ta < a.rows) o[static_cast<size_t>(ta) * e.ld_out + f] = f_to_h(silu_f(c[0]) * c[2]);
        if (tb < a.rows) o[static_cast<size_t>(tb) * e.ld_out + f] = f_to_h(silu_f(c[1]) * c[3]);
      }
    } else if (EPI == EPI_QKV_ROPE) {
      // rows g and g + 8 have the parity of g; the other half of a rotation pair sits in lane ^ 4
      const float sgn = (g & 1) ? 1.f : -1.f;
#pragma unroll
      for (int hr = 0; hr < 2; ++hr) {
        const int row = row0 + g + 8 * hr;
        const bool row_ok = row < r_hi;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int tok = ta + j;
          const float val = c[hr * 2 + j];
          const float partner = __shfl_xor_sync(0xffffffffu, val, 4);
          float y = val;
          int kind = 0, i = 0, pos = 0;
          size_t off = 0;
          const bool ok = row_ok && tok < a.rows;
          if (ok) {
            off = qkv_offset(e, tok, r_cat + row, kind, i, pos);
            if (kind != 2) {
              const size_t o = static_cast<size_t>(pos) * (e.head_dim >> 1) + (i >> 1);
              y = fmaf(sgn * partner, __ldg(e.rope_sin + o), val * __ldg(e.rope_cos + o));
            }
          }
          const float y_odd = __shfl_xor_sync(0xffffffffu, y, 4);
          if (ok && !(g & 1)) {
            half_t* dst = (kind == 0) ? e.q_out : (kind == 1 ? e.k_cache : e.v_cache);
            *reinterpret_cast<uint32_t*>(dst + off) = pack2(y, y_odd);
          }
        }
      }
    } else {
      // rows g and g + 1 (g even) are neighbours in memory: the even lane takes both, 4 bytes at a time
      float sq[2] = {0.f, 0.f};
#pragma unroll
      for (int hr = 0; hr < 2; ++hr) {
        const int row = row0 + g + 8 * hr;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int tok = ta + j;
          const float v0 = c[hr * 2 + j];
          const float v1 = __shfl_xor_sync(0xffffffffu, v0, 4);
          if ((g & 1) || row >= r_hi || tok >= a.rows) continue;
          const size_t off = static_cast<size_t>(tok) * e.ld_out + r_cat + row;
          if (EPI == EPI_PLAIN_F32) {
            *reinterpret_cast<float2*>(reinterpret_cast<float*>(e.out) + off) = make_float2(v0, v1);
          } else if (EPI == EPI_PLAIN_F16) {
            *reinterpret_cast<uint32_t*>(reinterpret_cast<half_t*>(e.out) + off) = pack2(v0, v1);
          } else {  // EPI_RESID
            const float2 x = h2_to_f2(*reinterpret_cast<const half2_t*>(e.resid + off));
            const uint32_t yh = pack2(x.x + v0, x.y + v1);
            *reinterpret_cast<uint32_t*>(reinterpret_cast<half_t*>(e.out) + off) = yh;
            if (e.outg != nullptr) {  // folded RMSNorm of the next sub-layer (gain here, 1/rms there)
              const float2 y = h2_to_f2(*reinterpret_cast<const half2_t*>(&yh));
              const float2 gn = h2_to_f2(*reinterpret_cast<const half2_t*>(e.gain_next + r_cat + row));
              *reinterpret_cast<uint32_t*>(e.outg + off) = pack2(y.x * gn.x, y.y * gn.y);
              sq[j] = fmaf(y.x, y.x, fmaf(y.y, y.y, sq[j]));
            }
          }
        }
      }
      if (EPI == EPI_RESID && e.outg != nullptr) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          sq[j] += __shfl_xor_sync(0xffffffffu, sq[j], 4);
          sq[j] += __shfl_xor_sync(0xffffffffu, sq[j], 8);
          sq[j] += __shfl_xor_sync(0xffffffffu, sq[j], 16);
        }
        if (g == 0) {
          ssq_tile[tile * 16 + ta] = sq[0];
          ssq_tile[tile * 16 + tb] = sq[1];
        }
      }
    }
  }
  if (EPI == EPI_RESID && e.outg != nullptr) {
    __syncthreads();
    if (threadIdx.x < 16) {
      float s = 0.f;
      if (NT * 8 > threadIdx.x)
        for (int tile = 0; tile < n_tiles; ++tile) s += ssq_tile[tile * 16 + threadIdx.x];
      e.sumsq[blockIdx.x * 16 + threadIdx.x] = s;
    }
  }
  if (a.dbg != nullptr && lane == 0) atomicMax(a.dbg + 15, static_cast<unsigned long long>(global_ns()));
  if (a.cta_log != nullptr && threadIdx.x == 0) a.cta_log[blockIdx.x * 4 + 3] = global_ns();
}

}  // namespace thinfer

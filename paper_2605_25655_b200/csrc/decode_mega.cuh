// Unified decode kernel (Section 3.3.3: one creation + launch for the whole
// operator graph instead of one per operator).  One persistent, cooperatively
// launched CTA per SM runs every fusion unit of every layer of a decode step:
//
//   prep      x * gain_1 and sum(x^2) of the step's input (first layer only)
//   QKV       stream-K tcgen05 projection, 1/rms applied to the sums, RoPE,
//             KV-cache append (Algorithm 1)
//   attention split over all SMs by cached keys (equal KV bytes per SM)
//   O         projection + residual; the epilogue also emits x1 * gain_2 and
//             the per-tile sums of x1^2 (the next RMSNorm, folded)
//   gate/up   projection, 1/rms, SwiGLU
//   down      projection + residual (+ the folded norm of the next layer)
//
// with a grid-wide barrier between units.  The point of keeping it one kernel is
// the weight stream: the TMA producer never stops at a unit boundary.  While the
// other warps finish a unit's epilogue and meet at the barrier it already pulls
// the next unit's weight tiles into the shared-memory ring (they depend on
// nothing), and only the small token tiles wait for the barrier.
//
// Warps: 0 TMA producer, 1 MMA issuer + TMEM owner, 2..5 epilogue (TMEM lane
// quarters), 2..11 attention / prep workers.  Every wait is bounded: a barrier
// or pipeline that stops making progress records THINFER_ETIMEOUT and all roles
// drain.
#pragma once
#include "decode_attn.cuh"
#include "tc_gemm.cuh"

namespace thinfer {

constexpr int kMegaThreads = 384;
constexpr int kMegaWorkerWarps = 10;  // warps 2..11 (384 threads: 168 registers per thread)
constexpr int kMegaWorkers = kMegaWorkerWarps * 32;
constexpr int kMegaSlots = 10;  // ring of (one 128 x 64 weight tile + one token tile) slots
constexpr int kMegaABytes = kTcBM * 128;

struct alignas(64) MegaLayer {
  CUtensorMap wq, wk, wv, wo, wg, wu, wd;
  const half_t* attn_norm;  // gain of the first RMSNorm (used by the prep unit of the first layer)
  const half_t* ffn_norm;   // gain folded into the O-projection epilogue
  const half_t* next_norm;  // gain folded into the down-projection epilogue (next layer's, or nullptr)
};
struct alignas(64) MegaCommon {
  CUtensorMap x_qkv, x_o, x_gu, x_down;  // token-side operands: xg, attn, x1g, act  (boxes of BN rows)
};

struct MegaArgs {
  const MegaCommon* common;  // device
  const MegaLayer* layers;   // device [n_layers]
  int n_layers, batch, pos;
  int hidden, ffn, n_q_heads, n_kv_heads, t_max;
  float eps;
  const half_t* x_in;  // [batch][hidden] input of the first layer
  half_t* x_out;       // output of the last layer
  half_t *xa, *xb;     // residual stream between layers (ping-pong)
  half_t *xg, *x1, *x1g, *qbuf, *attn, *act;
  float *sumsq0, *sumsq1;  // [feature tiles][64]: sums of squares feeding the first / second RMSNorm
  uint8_t* kv_base;        // K of layer l: kv_base + ((slot * n_layers + l) * 2) * kv_layer_bytes, V one further
  size_t kv_layer_bytes;
  int slot;
  const float *rope_cos, *rope_sin;
  float* gemm_partial;     // stream-K partial accumulators
  int* gemm_counters;      // zero between launches
  float* attn_partial;     // [(items + grid)][G][D + 2]
  int* attn_counters;      // [items], zero between launches
  unsigned int* grid_bar;  // arrival counter of the grid barriers; holds bar_base at launch
  unsigned int bar_base;
  int* status;
  unsigned long long* timeline;  // optional trace: CTA 0 stores %globaltimer at every unit boundary
};

template <int D, int G>
struct MegaAttnSmem {
  float m[kMegaWorkerWarps][G], l[kMegaWorkerWarps][G];
  float o[kMegaWorkerWarps][G][D];
};

template <int BN, int D, int G>
__host__ __device__ constexpr int mega_smem_bytes() {
  return kMegaSlots * (kMegaABytes + BN * 128) + tc_stage_out_bytes(BN) + static_cast<int>(sizeof(MegaAttnSmem<D, G>)) +
         1024 /*alignment slack*/ + 512 /*barriers, flags, 1/rms*/;
}

__device__ __forceinline__ void worker_bar() { asm volatile("bar.sync 2, %0;" ::"n"(kMegaWorkers) : "memory"); }

struct MegaShared {
  uint8_t* ring;
  uint8_t* stage_out;
  uint64_t *full_bar, *empty_bar, *tfull_bar, *tempty_bar;
  int* flag;               // scratch flag of the epilogue / attention finishers
  volatile int* sync_count;  // grid barriers completed, as seen by this CTA
  volatile int* abort;
  float* rstd;             // [BN]
};

struct MegaGemm {
  const CUtensorMap *w0, *w1, *w2, *x;
  TcGemmArgs g;
  int n_tiles, nkb;
};

// Descriptor of projection `phase` (0 QKV, 1 O, 2 gate/up, 3 down) of `layer`.  Every role builds the same one.
template <int BN, int D>
__device__ __forceinline__ void mega_gemm_desc(const MegaArgs& a, int layer, int phase, MegaGemm& m) {
  const MegaLayer& L = a.layers[layer];
  const int qd = a.n_q_heads * D, kvd = a.n_kv_heads * D;
  const half_t* in_l = layer == 0 ? a.x_in : ((layer & 1) ? a.xb : a.xa);
  half_t* out_l = layer == a.n_layers - 1 ? a.x_out : ((layer & 1) ? a.xa : a.xb);
  TcGemmArgs& g = m.g;
  g = TcGemmArgs{};
  g.rows = a.batch;
  g.mode = 1;
  g.static_finisher = 1;  // cooperative launch: all CTAs are resident
  g.dbg = (a.timeline != nullptr && layer == 0) ? a.timeline + 140 + 8 * phase : nullptr;
  g.partial_ws = a.gemm_partial;
  g.tile_counters = a.gemm_counters;
  g.status = a.status;
  EpiArgs& e = g.e;
  if (phase == 0) {
    m.w0 = &L.wq; m.w1 = &L.wk; m.w2 = &L.wv; m.x = &a.common->x_qkv;
    g.n_feat[0] = qd; g.n_feat[1] = kvd; g.n_feat[2] = kvd;
    g.k = a.hidden;
    uint8_t* kc = a.kv_base + (static_cast<size_t>(a.slot) * a.n_layers + layer) * 2 * a.kv_layer_bytes;
    e.q_out = a.qbuf;
    e.k_cache = reinterpret_cast<half_t*>(kc);
    e.v_cache = reinterpret_cast<half_t*>(kc + a.kv_layer_bytes);
    e.rope_cos = a.rope_cos; e.rope_sin = a.rope_sin;
    e.n_q = qd; e.n_kv = kvd; e.head_dim = D; e.n_q_heads = a.n_q_heads; e.n_kv_heads = a.n_kv_heads;
    e.seq_len = 1; e.pos0 = a.pos; e.t_max = a.t_max;
  } else if (phase == 1) {
    m.w0 = m.w1 = m.w2 = &L.wo; m.x = &a.common->x_o;
    g.n_feat[0] = a.hidden; g.k = qd;
    e.out = a.x1; e.resid = in_l; e.ld_out = a.hidden;
    e.outg = a.x1g; e.gain_next = L.ffn_norm; e.sumsq = a.sumsq1;
  } else if (phase == 2) {
    m.w0 = &L.wg; m.w1 = m.w2 = &L.wu; m.x = &a.common->x_gu;
    g.n_feat[0] = a.ffn; g.n_feat[1] = a.ffn; g.k = a.hidden;
    e.out = a.act; e.ld_out = a.ffn;
  } else {
    m.w0 = m.w1 = m.w2 = &L.wd; m.x = &a.common->x_down;
    g.n_feat[0] = a.hidden; g.k = a.ffn;
    e.out = out_l; e.resid = a.x1; e.ld_out = a.hidden;
    if (L.next_norm != nullptr) { e.outg = a.xg; e.gain_next = L.next_norm; e.sumsq = a.sumsq0; }
  }
  for (int i = 0; i < 3; ++i) g.tiles[i] = (g.n_feat[i] + kTcBM - 1) / kTcBM;
  if (phase == 2) g.tiles[1] = 0;
  m.n_tiles = g.tiles[0] + g.tiles[1] + g.tiles[2];  // one token tile
  m.nkb = (g.k + kTcBK - 1) / kTcBK;
  const long long units = static_cast<long long>(m.n_tiles) * m.nkb;
  g.units_per_cta = static_cast<int>((units + gridDim.x - 1) / gridDim.x);
}

// Grid barriers that must have completed before projection `phase` of `layer` may read its token operand:
// prep S1 QKV S2 attention S3 O S4 gate/up S5 down S6 QKV(next layer) ...
__device__ __forceinline__ int mega_need_sync(int layer, int phase) {
  return 1 + 5 * layer + (phase == 0 ? 0 : phase + 1);
}

// Bounded spin on a CTA-local counter that the barrier leader advances.
__device__ __forceinline__ bool mega_wait_sync(const MegaShared& sh, int need, int* status) {
  const uint64_t t0 = global_ns();
  uint32_t polls = 0;
  while (*sh.sync_count < need) {
    if (*sh.abort) return false;
    if ((++polls & 0x3ffu) == 0u && global_ns() - t0 > kWaitLimitNs) {
      if (status != nullptr) *reinterpret_cast<volatile int*>(status) = kErrTimeout;
      *sh.abort = 1;
      return false;
    }
  }
  __threadfence_block();
  fence_proxy_async_all();  // the token tiles about to be fetched by TMA were written with ordinary stores
  return true;
}

// Grid-wide barrier of the worker threads (warps 2..11 of every CTA).  `epoch` counts the barriers so far.
__device__ __forceinline__ bool mega_grid_sync(const MegaArgs& a, const MegaShared& sh, int& epoch, int wtid) {
  ++epoch;
  fence_proxy_async_all();
  __threadfence();
  worker_bar();
  if (wtid == 0) {
    const unsigned int target = a.bar_base + static_cast<unsigned int>(epoch) * gridDim.x;
    atomicAdd(a.grid_bar, 1u);
    const uint64_t t0 = global_ns();
    uint32_t polls = 0;
    for (;;) {
      unsigned int v;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(a.grid_bar) : "memory");
      if (static_cast<int>(v - target) >= 0) break;
      if ((++polls & 0xffu) == 0u) {
        if (*reinterpret_cast<volatile int*>(a.status) != 0 || global_ns() - t0 > kWaitLimitNs) {
          *reinterpret_cast<volatile int*>(a.status) = kErrTimeout;
          *sh.abort = 1;
          break;
        }
      }
    }
    __threadfence();
    *sh.sync_count = epoch;
  }
  worker_bar();
  return *sh.abort == 0;
}

// ------------------------------------------------------------------ producer of one projection
template <int BN, int D, int EPI>
__device__ __forceinline__ bool mega_produce(const MegaArgs& a, const MegaShared& sh, int layer, int phase, uint32_t& n) {
  constexpr int NA = tc_num_a(EPI);
  constexpr int SLOT = kMegaABytes + BN * 128;
  constexpr uint32_t TX = SLOT;
  MegaGemm m;
  mega_gemm_desc<BN, D>(a, layer, phase, m);
  // A ring slot holds one weight tile and the token tile it is multiplied with; the gate and the up tile
  // of a k-block are two consecutive slots.  Pass 1: the weight tiles of the first ring-full of slots are
  // requested as slots come free, before the previous unit has finished (weights depend on nothing).
  uint32_t pre = 0;
  {
    TcSegIter it(m.g, m.n_tiles, m.nkb);
    TcSeg sg;
    while (pre < kMegaSlots && it.next(sg)) {
      const TcTile t = tc_tile_coords<BN, EPI>(m.g, sg.tile, m.n_tiles, 1);
      const CUtensorMap* tmw = (EPI == EPI_QKV_ROPE) ? (t.mat == 0 ? m.w0 : (t.mat == 1 ? m.w1 : m.w2)) : m.w0;
      for (int u = sg.kb0 * NA; u < sg.kb1 * NA && pre < kMegaSlots; ++u, ++pre) {
        const uint32_t q = n + pre;
        const int s = q % kMegaSlots;
        if (!mbar_wait(&sh.empty_bar[s], ((q / kMegaSlots) & 1) ^ 1u, a.status)) return false;
        mbar_expect_tx(&sh.full_bar[s], TX);
        tma_load_2d(sh.ring + s * SLOT, (NA == 2 && (u & 1)) ? m.w1 : tmw, &sh.full_bar[s], (u / NA) * kTcBK, t.feat0);
      }
    }
  }
  // the token operand is written by the unit before the preceding grid barrier
  if (!mega_wait_sync(sh, mega_need_sync(layer, phase), a.status)) return false;
  if (a.timeline != nullptr && blockIdx.x == 0 && layer == 0) a.timeline[110 + phase] = global_ns();
  // pass 2
  TcSegIter it(m.g, m.n_tiles, m.nkb);
  TcSeg sg;
  uint32_t i = 0;
  while (it.next(sg)) {
    const TcTile t = tc_tile_coords<BN, EPI>(m.g, sg.tile, m.n_tiles, 1);
    const CUtensorMap* tmw = (EPI == EPI_QKV_ROPE) ? (t.mat == 0 ? m.w0 : (t.mat == 1 ? m.w1 : m.w2)) : m.w0;
    for (int u = sg.kb0 * NA; u < sg.kb1 * NA; ++u, ++i) {
      const uint32_t q = n + i;
      const int s = q % kMegaSlots;
      uint8_t* st = sh.ring + s * SLOT;
      if (i >= pre) {
        if (!mbar_wait(&sh.empty_bar[s], ((q / kMegaSlots) & 1) ^ 1u, a.status)) return false;
        mbar_expect_tx(&sh.full_bar[s], TX);
        tma_load_2d(st, (NA == 2 && (u & 1)) ? m.w1 : tmw, &sh.full_bar[s], (u / NA) * kTcBK, t.feat0);
      }
      tma_load_2d(st + kMegaABytes, m.x, &sh.full_bar[s], (u / NA) * kTcBK, t.tok0);
    }
  }
  n += i;
  if (a.timeline != nullptr && blockIdx.x == 0 && layer == 0) a.timeline[120 + phase] = global_ns();
  return true;
}

// ------------------------------------------------------------------ MMA issue of one projection
template <int BN, int D, int EPI>
__device__ __forceinline__ bool mega_mma(const MegaArgs& a, const MegaShared& sh, int layer, int phase, uint32_t tmem_base,
                                         uint32_t& n, uint32_t& j) {
  constexpr int NA = tc_num_a(EPI);
  constexpr int SLOT = kMegaABytes + BN * 128;
  constexpr uint32_t IDESC = idesc_f16(kTcBM, BN, 0, 0);
  MegaGemm m;
  mega_gemm_desc<BN, D>(a, layer, phase, m);
  TcSegIter it(m.g, m.n_tiles, m.nkb);
  TcSeg sg;
  while (it.next(sg)) {
    const uint32_t buf = j & 1, use = j >> 1;
    if (!mbar_wait(&sh.tempty_bar[buf], (use & 1) ^ 1u, a.status)) return false;
    tc_fence_after();
    const uint32_t acc = tmem_base + buf * (2 * BN);
    for (int u = sg.kb0 * NA; u < sg.kb1 * NA; ++u, ++n) {
      const int s = n % kMegaSlots;
      if (!mbar_wait(&sh.full_bar[s], (n / kMegaSlots) & 1, a.status)) return false;
      tc_fence_after();
      const uint32_t sa = smem_u32(sh.ring + s * SLOT);
      const uint64_t da = smem_desc_sw128(sa, 16, 1024);
      const uint64_t db = smem_desc_sw128(sa + kMegaABytes, 16, 1024);
      const uint32_t dst = acc + ((NA == 2 && (u & 1)) ? BN : 0);  // gate -> first accumulator, up -> second
      const bool first_kb = (u / NA) == sg.kb0;
#pragma unroll
      for (int k = 0; k < kTcBK / 16; ++k) tc_mma_f16(dst, da + 2 * k, db + 2 * k, IDESC, (!first_kb || k != 0) ? 1u : 0u);
      tc_commit(&sh.empty_bar[s]);
    }
    tc_commit(&sh.tfull_bar[buf]);
    ++j;
  }
  return true;
}

// ------------------------------------------------------------------ epilogue of one projection (warps 2..5)
template <int BN, int D, int EPI>
__device__ __forceinline__ bool mega_epilogue(const MegaArgs& a, const MegaShared& sh, int layer, int phase,
                                              uint32_t tmem_base, uint32_t& j, int warp, int lane, const float* col_scale) {
  MegaGemm m;
  mega_gemm_desc<BN, D>(a, layer, phase, m);
  const int q = warp & 3;
  const int row = q * 32 + lane;
  const int ethread = (warp - 2) * 32 + lane;
  const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
  TcSegIter it(m.g, m.n_tiles, m.nkb);
  TcSeg sg;
  while (it.next(sg)) {
    const uint32_t buf = j & 1, use = j >> 1;
    ++j;
    if (!mbar_wait(&sh.tfull_bar[buf], use & 1, a.status)) return false;
    tc_fence_after();
    if (a.timeline != nullptr && blockIdx.x == 0 && ethread == 0 && layer == 0) a.timeline[100 + phase] = global_ns();
    const TcTile t = tc_tile_coords<BN, EPI>(m.g, sg.tile, m.n_tiles, 1);
    tc_epilogue_segment<BN, EPI>(m.g, sg, t, lane_base + buf * (2 * BN), &sh.tempty_bar[buf], sh.stage_out, sh.flag, row,
                                 ethread, lane, m.nkb, col_scale);
  }
  return true;
}

// 1/rms per token from the per-tile sums of squares (epilogue threads; followed by their barrier).
template <int BN>
__device__ __forceinline__ void mega_rstd(const MegaArgs& a, const MegaShared& sh, const float* sumsq, int ethread) {
  if (ethread < BN) {
    float r = 0.f;
    if (ethread < a.batch) {
      const int parts = (a.hidden + kTcBM - 1) / kTcBM;
      float s = 0.f;
      for (int p = 0; p < parts; ++p) s += __ldcg(sumsq + p * 64 + ethread);
      r = rsqrtf(s / static_cast<float>(a.hidden) + a.eps);
    }
    sh.rstd[ethread] = r;
  }
  epi_bar();
}

// ------------------------------------------------------------------ prep unit (first layer's RMSNorm input)
__device__ __forceinline__ void mega_prep(const MegaArgs& a, float* red, int wtid) {
  const half_t* gain = a.layers[0].attn_norm;
  const int chunks = a.hidden >> 3;
  const int parts = (a.hidden + kTcBM - 1) / kTcBM;
  for (int b = blockIdx.x; b < a.batch; b += gridDim.x) {
    const half_t* xr = a.x_in + static_cast<size_t>(b) * a.hidden;
    half_t* gr = a.xg + static_cast<size_t>(b) * a.hidden;
    float ss = 0.f;
    for (int c = wtid; c < chunks; c += kMegaWorkers) {
      float f[8], g[8];
      unpack8(ldg_cached(xr + (c << 3)), f);
      unpack8(ldg_cached(gain + (c << 3)), g);
#pragma unroll
      for (int i = 0; i < 8; ++i) ss = fmaf(f[i], f[i], ss);
      uint4 o;
      o.x = pack2(f[0] * g[0], f[1] * g[1]);
      o.y = pack2(f[2] * g[2], f[3] * g[3]);
      o.z = pack2(f[4] * g[4], f[5] * g[5]);
      o.w = pack2(f[6] * g[6], f[7] * g[7]);
      *reinterpret_cast<uint4*>(gr + (c << 3)) = o;
    }
    ss = warp_sum(ss);
    if ((wtid & 31) == 0) red[wtid >> 5] = ss;
    worker_bar();
    if (wtid < parts) {
      float tot = 0.f;
      if (wtid == 0)
        for (int w = 0; w < kMegaWorkerWarps; ++w) tot += red[w];
      a.sumsq0[wtid * 64 + b] = tot;  // the whole row's sum in part 0, zeros in the others
    }
    worker_bar();
  }
}

// ------------------------------------------------------------------ attention unit (warps 2..11)
// The cached keys of all (request, head group) pairs form one long sequence; every CTA takes an equal
// share of it, so all SMs stream the same number of KV bytes.  A pair that spans several CTAs is
// finished by the last one to arrive (partials merged in CTA order).
template <int D, int G>
__device__ __forceinline__ void mega_attention(const MegaArgs& a, const MegaShared& sh, MegaAttnSmem<D, G>& sm,
                                               uint8_t* kc_bytes, int wtid) {
  constexpr int LPK = D / 8, KPL = 32 / LPK, UN = 4;
  const int wwarp = wtid >> 5, lane = wtid & 31;
  const int sub = lane / LPK, dl = lane % LPK;
  const int T = a.pos + 1;
  const int groups = a.n_q_heads / G;
  const int ratio = a.n_q_heads / a.n_kv_heads;
  const int items = a.batch * groups;
  const long long total = static_cast<long long>(items) * T;
  const long long per = (total + gridDim.x - 1) / gridDim.x;
  long long cur = per * blockIdx.x;
  const long long end = (cur + per < total) ? cur + per : total;
  const half_t* kcache = reinterpret_cast<const half_t*>(kc_bytes);
  const half_t* vcache = reinterpret_cast<const half_t*>(kc_bytes + a.kv_layer_bytes);
  const float scale_log2 = 1.4426950408889634f * rsqrtf(static_cast<float>(D));
  while (cur < end) {
    const int item = static_cast<int>(cur / T);
    const int t0 = static_cast<int>(cur - static_cast<long long>(item) * T);
    const int t1 = (T - t0 < end - cur) ? T : t0 + static_cast<int>(end - cur);
    cur += t1 - t0;
    const int b = item / groups, h0 = (item - b * groups) * G, hk = h0 / ratio;
    float q[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const uint4 qv = __ldcg(reinterpret_cast<const uint4*>(a.qbuf + (static_cast<size_t>(b) * a.n_q_heads + h0 + g) * D + dl * 8));
      unpack8(qv, q[g]);
#pragma unroll
      for (int i = 0; i < 8; ++i) q[g][i] *= scale_log2;
    }
    const size_t head_off = (static_cast<size_t>(b) * a.n_kv_heads + hk) * a.t_max * D + dl * 8;
    float m[G], l[G], o[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      m[g] = -INFINITY;
      l[g] = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) o[g][i] = 0.f;
    }
    attn_stream_keys<D, G, UN, false>(kcache + head_off,  // not pipelined: 168 registers per thread here
                                      vcache + head_off, q, t0 + wwarp * (UN * KPL), t1,
                           kMegaWorkerWarps * UN * KPL, sub, m, l, o);
    attn_merge_lane_groups<D, G>(m, l, o);
    if (sub == 0) {
#pragma unroll
      for (int g = 0; g < G; ++g) {
        if (dl == 0) {
          sm.m[wwarp][g] = m[g];
          sm.l[wwarp][g] = l[g];
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) sm.o[wwarp][g][dl * 8 + i] = o[g][i];
      }
    }
    worker_bar();
    const long long first_key = static_cast<long long>(item) * T;
    const int first_cta = static_cast<int>(first_key / per);
    const int last_cta = static_cast<int>((first_key + T - 1) / per);
    const int n_seg = last_cta - first_cta + 1;
    float* slot = a.attn_partial + static_cast<size_t>(item + blockIdx.x) * (G * (D + 2));
    for (int idx = wtid; idx < G * D; idx += kMegaWorkers) {
      const int g = idx / D, i = idx - g * D;
      float mx = sm.m[0][g];
#pragma unroll
      for (int w = 1; w < kMegaWorkerWarps; ++w) mx = fmaxf(mx, sm.m[w][g]);
      const float ms = (mx == -INFINITY) ? 0.f : mx;
      float L = 0.f, O = 0.f;
#pragma unroll
      for (int w = 0; w < kMegaWorkerWarps; ++w) {
        const float al = exp2f(sm.m[w][g] - ms);
        L += sm.l[w][g] * al;
        O += sm.o[w][g][i] * al;
      }
      if (n_seg == 1) {
        a.attn[(static_cast<size_t>(b) * a.n_q_heads + h0 + g) * D + i] = f_to_h(O / L);
      } else {
        slot[g * (D + 2) + i] = O;
        if (i == 0) {
          slot[g * (D + 2) + D] = mx;
          slot[g * (D + 2) + D + 1] = L;
        }
      }
    }
    if (n_seg > 1) {
      // The head keys of a split item are the LAST share its CTA works on; every other share of the item is
      // the FIRST one of a later CTA and was parked long ago.  The head CTA merges, the others only park.
      if (t0 != 0) {
        __threadfence();
        worker_bar();
        if (wtid == 0) atomicAdd(a.attn_counters + item, 1);
      } else {
        worker_bar();  // this CTA's own partial is complete in global memory for its own threads
        if (wtid == 0) {
          const uint64_t ts = global_ns();
          uint32_t polls = 0;
          int ok = 1;
          for (;;) {
            int seen;
            asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(a.attn_counters + item) : "memory");
            if (seen >= n_seg - 1) break;
            if ((++polls & 0xffu) == 0u && global_ns() - ts > kWaitLimitNs) {
              *reinterpret_cast<volatile int*>(a.status) = kErrTimeout;
              ok = 0;
              break;
            }
          }
          *sh.flag = ok;
        }
        worker_bar();
        if (*reinterpret_cast<volatile int*>(sh.flag) != 0) {
          for (int idx = wtid; idx < G * D; idx += kMegaWorkers) {
            const int g = idx / D, i = idx - g * D;
            float mx = -INFINITY;
            for (int s = 0; s < n_seg; ++s)
              mx = fmaxf(mx, __ldcg(a.attn_partial + static_cast<size_t>(item + first_cta + s) * (G * (D + 2)) + g * (D + 2) + D));
            float L = 0.f, O = 0.f;
            for (int s = 0; s < n_seg; ++s) {
              const float* p = a.attn_partial + static_cast<size_t>(item + first_cta + s) * (G * (D + 2)) + g * (D + 2);
              const float al = exp2f(__ldcg(p + D) - mx);
              L += __ldcg(p + D + 1) * al;
              O += __ldcg(p + i) * al;
            }
            a.attn[(static_cast<size_t>(b) * a.n_q_heads + h0 + g) * D + i] = f_to_h(O / L);
          }
          if (wtid == 0) a.attn_counters[item] = 0;
        } else {
          *sh.abort = 1;
        }
      }
    }
    worker_bar();  // the merge area is reused by the next share
  }
}

// ==================================================================== the kernel
template <int BN, int D, int G>
__global__ void __launch_bounds__(kMegaThreads, 1) decode_mega_kernel(const MegaArgs a) {
  constexpr int SLOT = kMegaABytes + BN * 128;
  constexpr int TMEM_COLS = (4 * BN) < 32 ? 32 : (4 * BN);  // two buffers of up to two accumulators
  static_assert((TMEM_COLS & (TMEM_COLS - 1)) == 0 && TMEM_COLS <= 512, "tensor memory columns");

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  MegaShared sh;
  sh.ring = smem;
  sh.stage_out = smem + kMegaSlots * SLOT;
  MegaAttnSmem<D, G>& attn_sm = *reinterpret_cast<MegaAttnSmem<D, G>*>(sh.stage_out + tc_stage_out_bytes(BN));
  uint8_t* tail = sh.stage_out + tc_stage_out_bytes(BN) + sizeof(MegaAttnSmem<D, G>);
  sh.full_bar = reinterpret_cast<uint64_t*>(tail);
  sh.empty_bar = sh.full_bar + kMegaSlots;
  sh.tfull_bar = sh.empty_bar + kMegaSlots;
  sh.tempty_bar = sh.tfull_bar + 2;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(sh.tempty_bar + 2);
  sh.flag = reinterpret_cast<int*>(tmem_holder + 1);
  sh.sync_count = sh.flag + 1;
  sh.abort = sh.flag + 2;
  float* red = reinterpret_cast<float*>(sh.flag + 4);  // [worker warps]
  sh.rstd = red + 12;                                   // [BN]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kMegaSlots; ++s) {
      mbar_init(&sh.full_bar[s], 1);
      mbar_init(&sh.empty_bar[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sh.tfull_bar[i], 1);
      mbar_init(&sh.tempty_bar[i], 4);
    }
    *sh.sync_count = 0;
    *sh.abort = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(tmem_holder, TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_holder);

  if (warp == 0) {
    if (lane == 0) {
      uint32_t n = 0;
      bool ok = true;
      for (int l = 0; l < a.n_layers && ok; ++l) {
        ok = mega_produce<BN, D, EPI_QKV_ROPE>(a, sh, l, 0, n);
        ok = ok && mega_produce<BN, D, EPI_RESID>(a, sh, l, 1, n);
        ok = ok && mega_produce<BN, D, EPI_SWIGLU>(a, sh, l, 2, n);
        ok = ok && mega_produce<BN, D, EPI_RESID>(a, sh, l, 3, n);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      uint32_t n = 0, j = 0;
      bool ok = true;
      for (int l = 0; l < a.n_layers && ok; ++l) {
        ok = mega_mma<BN, D, EPI_QKV_ROPE>(a, sh, l, 0, tmem_base, n, j);
        ok = ok && mega_mma<BN, D, EPI_RESID>(a, sh, l, 1, tmem_base, n, j);
        ok = ok && mega_mma<BN, D, EPI_SWIGLU>(a, sh, l, 2, tmem_base, n, j);
        ok = ok && mega_mma<BN, D, EPI_RESID>(a, sh, l, 3, tmem_base, n, j);
      }
    }
  } else {
    const int wtid = threadIdx.x - 64;
    const bool epi = warp < 6;
    int ts_n = 0;
    auto stamp = [&]() {
      if (a.timeline != nullptr && blockIdx.x == 0 && wtid == 0 && ts_n < 250) a.timeline[1 + ts_n++] = global_ns();
    };
    stamp();
    const int ethread = wtid;  // epilogue warps are the first four worker warps
    int epoch = 0;
    uint32_t j = 0;
    bool ok = true;
    mega_prep(a, red, wtid);
    stamp();
    ok = mega_grid_sync(a, sh, epoch, wtid);                                   // S1
    stamp();
    for (int l = 0; l < a.n_layers && ok; ++l) {
      if (epi) {
        mega_rstd<BN>(a, sh, a.sumsq0, ethread);
        if (!mega_epilogue<BN, D, EPI_QKV_ROPE>(a, sh, l, 0, tmem_base, j, warp, lane, sh.rstd)) *sh.abort = 1;
      }
      stamp();
      ok = mega_grid_sync(a, sh, epoch, wtid);                                 // S2: q, K, V written
      stamp();
      if (!ok) break;
      mega_attention<D, G>(a, sh, attn_sm,
                           a.kv_base + (static_cast<size_t>(a.slot) * a.n_layers + l) * 2 * a.kv_layer_bytes, wtid);
      stamp();
      ok = mega_grid_sync(a, sh, epoch, wtid);                                 // S3: attention output written
      stamp();
      if (!ok) break;
      if (epi && !mega_epilogue<BN, D, EPI_RESID>(a, sh, l, 1, tmem_base, j, warp, lane, nullptr)) *sh.abort = 1;
      stamp();
      ok = mega_grid_sync(a, sh, epoch, wtid);                                 // S4: x1, x1g, sums written
      stamp();
      if (!ok) break;
      if (epi) {
        mega_rstd<BN>(a, sh, a.sumsq1, ethread);
        if (!mega_epilogue<BN, D, EPI_SWIGLU>(a, sh, l, 2, tmem_base, j, warp, lane, sh.rstd)) *sh.abort = 1;
      }
      stamp();
      ok = mega_grid_sync(a, sh, epoch, wtid);                                 // S5: act written
      stamp();
      if (!ok) break;
      if (epi && !mega_epilogue<BN, D, EPI_RESID>(a, sh, l, 3, tmem_base, j, warp, lane, nullptr)) *sh.abort = 1;
      stamp();
      if (l + 1 < a.n_layers) ok = mega_grid_sync(a, sh, epoch, wtid);         // S6 = S1 of the next layer
      stamp();
    }
  }

  tc_fence_before();
  __syncthreads();
  if (a.timeline != nullptr && blockIdx.x == 0 && threadIdx.x == 0) a.timeline[0] = global_ns();  // kernel end
  if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
}

}  // namespace thinfer

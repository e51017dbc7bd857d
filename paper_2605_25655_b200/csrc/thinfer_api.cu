// C ABI of the library (include/thinfer.h): context, argument validation, the
// per-layer launch sequences of prefill and decode, the bounded KV slot ring of
// the Prefill-Buffer-Decode pipeline (Section 3.4.2), and the single-operator
// entry points.  Host code only launches kernels; every step of the path runs
// in the kernels of this directory.
#include "../../include/thinfer.h"

#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <string>
#include <vector>

#include "decode_attn.cuh"
#include "decode_attn_gqa.cuh"
#include "decode_gemv.cuh"
#include "decode_mega.cuh"
#include "decode_mma.cuh"
#include "misc_kernels.cuh"
#include "prefill_attn.cuh"
#include "tc_gemm.cuh"

using namespace thinfer;

namespace {

// ----------------------------------------------------------------------------
// driver entry point for tensor-map encoding (no link-time dependency on libcuda)
// ----------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// 16-bit tensor [d2][d1][d0] (d0 contiguous), box [1][box1][64], 128-byte swizzle, zero fill outside.
// stride1 / stride2 in elements.
bool make_map(CUtensorMap* m, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t stride1,
              uint64_t stride2, uint32_t box1, int rank) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[3] = {d0, d1, d2};
  cuuint64_t strides[2] = {stride1 * 2, stride2 * 2};
  cuuint32_t box[3] = {64, box1, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, kStorageType == 1 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, static_cast<cuuint32_t>(rank), const_cast<void*>(base), dims,
                  strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}
bool make_map_2d(CUtensorMap* m, const void* base, uint64_t k, uint64_t rows, uint32_t box_rows) {
  return make_map(m, base, k, rows, 1, k, 0, box_rows, 2);
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct LayerMaps {
  CUtensorMap wq, wk, wv, wo, wg, wu, wd;
  CUtensorMap wg64, wu64;  // 64-row boxes: gate and up rows share one 128-row tile in prefill
};

struct Slot {
  int batch = 0, cur_len = 0;
  bool busy = false;
  // hand-off between the stages: `ready` is recorded behind the prefill that filled the slot (decode on another
  // stream waits for it), `freed` behind the release (a later prefill on another stream waits for it)
  cudaEvent_t ready = nullptr, freed = nullptr;
  cudaStream_t ready_stream = nullptr, freed_stream = nullptr;
  bool ready_valid = false, freed_valid = false;
  // ragged prompts: request b holds lens[b] + steps positions (cur_len is then the longest request's count)
  bool ragged = false;
  int steps = 0;
  std::vector<int> lens;
};

struct ProfEvent {
  cudaEvent_t beg, end;
};

}  // namespace

struct thinfer_ctx {
  thinfer_config cfg{};
  std::vector<thinfer_layer_weights> layers;
  const half_t *embed = nullptr, *final_norm = nullptr, *lm_head = nullptr;
  std::vector<LayerMaps> maps;
  CUtensorMap map_head{};
  uint8_t* kv = nullptr;
  size_t kv_layer_bytes = 0;  // one of K or V for one layer of one slot
  std::vector<Slot> slots;
  // scratch carve-up
  float *rope_cos = nullptr, *rope_sin = nullptr;
  half_t *h = nullptr, *qbuf = nullptr, *attn = nullptr, *x1 = nullptr, *act = nullptr, *xa = nullptr, *xb = nullptr;
  half_t* last = nullptr;
  float* logits = nullptr;
  int32_t* ids_out = nullptr;
  // the decode path has its own (small) activation buffers, so that a prefill of one slot and decode steps of
  // another may run on different streams at the same time (the two stages of the pipeline, Section 3.4.2)
  half_t *d_h = nullptr, *d_qbuf = nullptr, *d_attn = nullptr, *d_x1 = nullptr, *d_act = nullptr, *d_xa = nullptr,
         *d_xb = nullptr;
  float* d_logits = nullptr;
  uint8_t *d_stage_in = nullptr, *d_stage_out = nullptr;
  float *part_o = nullptr, *part_ml = nullptr;
  float* splitk_ws = nullptr;   // stream-K partial accumulators (decode stage)
  int* splitk_counters = nullptr;
  float* pf_splitk_ws = nullptr;  // the same for the prefill stage (its vocabulary projection), so that the two
  int* pf_splitk_counters = nullptr;  // stages may overlap on two streams
  // inspection: copies of the hidden state behind chosen layers (thinfer_capture_hidden)
  std::vector<std::pair<int, void*>> captures;
  // unified decode kernel
  half_t *xg = nullptr, *x1g = nullptr;
  float *sumsq0 = nullptr, *sumsq1 = nullptr, *attn_partial = nullptr;
  int sumsq0_parts = 0, sumsq1_parts = 0;  // parts the last skinny down / O projection left in sumsq0 / sumsq1
  bool skinny_ok = true;    // hidden, ffn and the head widths suit the skinny decode projections
  int* attn_counters = nullptr;
  unsigned int* grid_bar = nullptr;
  unsigned int bar_base = 0;
  unsigned long long* timeline = nullptr;
  bool trace_unified = false;
  int* slot_lens = nullptr;  // [buf_slots][max_batch] prompt lengths of ragged slots (device)
  MegaCommon* mega_common = nullptr;
  MegaLayer* mega_layers = nullptr;
  uint8_t *stage_in = nullptr, *stage_out = nullptr;
  int max_splits = 1;
  int attn_waves = 1, attn_min_units = 2;  // split-KV schedule of decode attention (tuning aids)
  int attn_cluster = 1;                    // merge the segments of a pair inside a thread-block cluster when they fit
  int sk_whole_tiles = 1;                  // tuning aid: shrink the grid to shares of whole tiles when shares are ragged
  int sk_max_tiles = 0;                    // tuning aid: cap on the tiles of a skinny share (0: the built-in limits)
  int trace_cta_kid = -1;                  // kernel id whose CTAs log their own times while tracing is on
  // status word (pinned, mapped)
  int* status_host = nullptr;
  int* status_dev = nullptr;
  int launch_mode = 1;
  int64_t launches = 0;
  int prof_kernel = -1;
  std::vector<ProfEvent> prof_events;
  size_t prof_used = 0;
  std::string err;
  int sm_count = 148;
};

namespace {

int fail(thinfer_ctx* c, int code, const char* fmt, ...) {
  if (c != nullptr) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    c->err = buf;
  }
  return code;
}

thread_local std::string g_global_err;

int validate_config(const thinfer_config* c, std::string* why) {
  auto bad = [&](int code, const char* s) {
    if (why) *why = s;
    return code;
  };
  if (c == nullptr) return bad(THINFER_EINVAL, "config is NULL");
  if (c->hidden <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->head_dim <= 0 || c->ffn <= 0 ||
      c->n_layers <= 0 || c->vocab < 0 || c->max_batch <= 0 || c->max_seq <= 0 || c->buf_slots <= 0)
    return bad(THINFER_EINVAL, "config has a non-positive size");
  if (!(c->rms_eps >= 0.f) || !(c->rope_base > 0.f)) return bad(THINFER_EINVAL, "rms_eps or rope_base out of range");
  if (c->head_dim != 64 && c->head_dim != 128) return bad(THINFER_EUNSUPPORTED, "head_dim must be 64 or 128");
  if (c->n_q_heads % c->n_kv_heads != 0) return bad(THINFER_EUNSUPPORTED, "n_q_heads must be a multiple of n_kv_heads");
  if (c->hidden % 8 != 0 || c->ffn % 8 != 0) return bad(THINFER_EUNSUPPORTED, "hidden and ffn must be multiples of 8");
  if (c->max_batch > 64) return bad(THINFER_EUNSUPPORTED, "max_batch must be <= 64");
  if (c->vocab % 2 != 0) return bad(THINFER_EUNSUPPORTED, "vocab must be even");
  return THINFER_OK;
}

struct ScratchPlan {
  size_t rope_cos, rope_sin, h, qbuf, attn, x1, act, xa, xb, last, logits, ids_out, part_o, part_ml, splitk_ws,
      splitk_counters, pf_splitk_ws, pf_splitk_counters, xg, x1g, sumsq0, sumsq1, attn_partial, attn_counters, grid_bar, timeline, mega_common, mega_layers,
      stage_in, stage_out, slot_lens, d_h, d_qbuf, d_attn, d_x1, d_act, d_xa, d_xb, d_logits, d_stage_in, d_stage_out, total;
  int max_splits, max_tiles, pf_tiles;
};

constexpr int kTcMaxCtas = 160;      // persistent grid bound (a B200 has 148 SMs)
constexpr int kTcDecodeMaxBN = 64;   // token tile of the stream-K decode path
constexpr int kSkMaxCtas = 2 * kTcMaxCtas;  // grid bound of the skinny decode projections that produce sums of squares

ScratchPlan plan_scratch(const thinfer_config& c) {
  ScratchPlan p{};
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 1024);
    return o;
  };
  const size_t M = static_cast<size_t>(c.max_batch) * c.max_seq;
  const size_t qd = static_cast<size_t>(c.n_q_heads) * c.head_dim;
  p.max_splits = kAttnMaxSplits;
  p.rope_cos = take(static_cast<size_t>(c.max_seq) * (c.head_dim / 2) * 4);
  p.rope_sin = take(static_cast<size_t>(c.max_seq) * (c.head_dim / 2) * 4);
  p.h = take(M * c.hidden * 2);
  p.qbuf = take(M * qd * 2);
  p.attn = take(M * qd * 2);
  p.x1 = take(M * c.hidden * 2);
  p.act = take(M * c.ffn * 2);
  p.xa = take(M * c.hidden * 2);
  p.xb = take(M * c.hidden * 2);
  p.last = take(static_cast<size_t>(c.max_batch) * c.hidden * 2);
  p.logits = take(static_cast<size_t>(c.max_batch) * (c.vocab > 0 ? c.vocab : 1) * 4);
  p.ids_out = take(static_cast<size_t>(c.max_batch) * 4);
  p.part_o = take(static_cast<size_t>(c.max_batch) * c.n_q_heads * p.max_splits * c.head_dim * 4);
  p.part_ml = take(static_cast<size_t>(c.max_batch) * c.n_q_heads * p.max_splits * 2 * 4);
  {
    auto t128 = [](size_t n) { return (n + 127) / 128; };
    size_t tiles = t128(qd) + 2 * t128(static_cast<size_t>(c.n_kv_heads) * c.head_dim);
    if (t128(c.ffn) > tiles) tiles = t128(c.ffn);
    if (t128(c.hidden) > tiles) tiles = t128(c.hidden);
    if (c.vocab > 0 && t128(c.vocab) > tiles) tiles = t128(c.vocab);
    p.max_tiles = static_cast<int>(tiles);
    // one slot per (tile, CTA) pair that can occur: tiles + CTAs; a slot holds 128 rows x (2 x 64) FP32 columns
    p.splitk_ws = take((tiles + kTcMaxCtas) * static_cast<size_t>(2 * kTcDecodeMaxBN) * 128 * 4);
    p.splitk_counters = take(tiles * 8);
    // prefill stage: only its vocabulary projection is ever split along K
    const size_t head_tiles = c.vocab > 0 ? t128(c.vocab) : 0;
    p.pf_splitk_ws = take(head_tiles > 0 ? (head_tiles + kTcMaxCtas) * static_cast<size_t>(2 * kTcDecodeMaxBN) * 128 * 4 : 0);
    p.pf_splitk_counters = take(head_tiles * 8);
    p.pf_tiles = static_cast<int>(head_tiles);
  }
  {
    const size_t parts = (static_cast<size_t>(c.hidden) + 127) / 128;
    p.xg = take(static_cast<size_t>(c.max_batch) * c.hidden * 2);
    p.x1g = take(static_cast<size_t>(c.max_batch) * c.hidden * 2);
    // [128-feature tile][64 tokens] (tcgen05 producers) or [CTA][16 tokens] (skinny producers, <= 2 CTAs per SM)
    const size_t ssq = std::max<size_t>(parts * 64 * 4, static_cast<size_t>(kSkMaxCtas) * 16 * 4);
    p.sumsq0 = take(ssq);
    p.sumsq1 = take(ssq);
    p.attn_partial = take((static_cast<size_t>(c.max_batch) * c.n_q_heads + kTcMaxCtas * 4) * (c.head_dim + 2) * 4);
    p.attn_counters = take(static_cast<size_t>(c.max_batch) * c.n_q_heads * 4);
    p.grid_bar = take(64);
    p.timeline = take((256 + 4 * 1024) * 8);  // 16 slots per kernel id, then 4 per CTA of one traced kernel
    p.mega_common = take(sizeof(MegaCommon));
    p.mega_layers = take(sizeof(MegaLayer) * c.n_layers);
  }
  const size_t in_bytes = c.vocab > 0 ? M * 4 : M * c.hidden * 2;
  const size_t out_bytes = c.vocab > 0 ? static_cast<size_t>(c.max_batch) * (4 + static_cast<size_t>(c.vocab) * 4)
                                       : M * c.hidden * 2;
  p.stage_in = take(in_bytes);
  p.stage_out = take(out_bytes);
  {
    const size_t Bm = c.max_batch;
    p.slot_lens = take(static_cast<size_t>(c.buf_slots) * Bm * 4);
    p.d_h = take(Bm * c.hidden * 2);
    p.d_qbuf = take(Bm * qd * 2);
    p.d_attn = take(Bm * qd * 2);
    p.d_x1 = take(Bm * c.hidden * 2);
    p.d_act = take(Bm * c.ffn * 2);
    p.d_xa = take(Bm * c.hidden * 2);
    p.d_xb = take(Bm * c.hidden * 2);
    p.d_logits = take(Bm * (c.vocab > 0 ? c.vocab : 1) * 4);
    p.d_stage_in = take(c.vocab > 0 ? Bm * 4 : Bm * c.hidden * 2);
    p.d_stage_out = take(c.vocab > 0 ? Bm * (4 + static_cast<size_t>(c.vocab) * 4) : Bm * c.hidden * 2);
  }
  p.total = off;
  return p;
}

size_t kv_layer_bytes_of(const thinfer_config& c) {
  return align_up(static_cast<size_t>(c.max_batch) * c.n_kv_heads * c.max_seq * c.head_dim * 2, 1024);
}

// ----------------------------------------------------------------------------
// launch helper: counts, optional event bracketing, error check
// ----------------------------------------------------------------------------
struct Launcher {
  thinfer_ctx* c;
  cudaStream_t st;
  int rc = THINFER_OK;
  bool cooperative = false;  // next launch only: all CTAs must be co-resident (grid-wide barriers inside)
  bool prefill_stage = false;  // stream-K scratch of the prefill stage instead of the decode stage's
  int cluster = 0;             // next launch only: thread-block clusters of this many CTAs along x

  template <typename... KArgs, typename... Args>
  void go(int kid, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, Args&&... args) {
    if (rc != THINFER_OK) return;
    const bool prof = c != nullptr && c->prof_kernel == kid;
    ProfEvent ev{};
    if (prof) {
      if (c->prof_used == c->prof_events.size()) {
        ProfEvent n{};
        if (cudaEventCreate(&n.beg) != cudaSuccess || cudaEventCreate(&n.end) != cudaSuccess) {
          rc = fail(c, THINFER_ECUDA, "cudaEventCreate failed");
          return;
        }
        c->prof_events.push_back(n);
      }
      ev = c->prof_events[c->prof_used++];
      cudaEventRecord(ev.beg, st);
    }
    cudaLaunchConfig_t lc{};
    lc.gridDim = grid;
    lc.blockDim = block;
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute attr[2];
    lc.attrs = attr;
    lc.numAttrs = 0;
    if (cooperative) {
      attr[0].id = cudaLaunchAttributeCooperative;
      attr[0].val.cooperative = 1;
      lc.numAttrs = 1;
      cooperative = false;
    } else if (c != nullptr && c->launch_mode >= 1 && !prof) {
      attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[0].val.programmaticStreamSerializationAllowed = 1;
      lc.numAttrs = 1;
    }
    if (cluster > 1) {
      attr[lc.numAttrs].id = cudaLaunchAttributeClusterDimension;
      attr[lc.numAttrs].val.clusterDim.x = static_cast<unsigned>(cluster);
      attr[lc.numAttrs].val.clusterDim.y = 1;
      attr[lc.numAttrs].val.clusterDim.z = 1;
      ++lc.numAttrs;
    }
    cluster = 0;
    cudaError_t e = cudaLaunchKernelEx(&lc, kernel, static_cast<KArgs>(args)...);
    if (prof) cudaEventRecord(ev.end, st);
    if (e != cudaSuccess) {
      rc = fail(c, THINFER_ECUDA, "kernel launch failed: %s", cudaGetErrorString(e));
      if (c == nullptr) g_global_err = cudaGetErrorString(e);
      return;
    }
    if (c != nullptr) ++c->launches;
  }
};

template <typename K>
bool opt_in_smem(K kernel, int bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
}

// The opt-in above is a per-device property of a kernel.  One of these (a function-local static per kernel
// instantiation) remembers what has been reserved on which device, so that a process that drives several GPUs
// opts in on each of them and a launch pays one cudaGetDevice instead of a driver call.
struct SmemOptIn {
  static constexpr int kMaxDevices = 64;
  int reserved[kMaxDevices] = {};
  template <typename K>
  bool ensure(K kernel, int bytes) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return opt_in_smem(kernel, bytes);
    if (bytes <= reserved[dev]) return true;
    if (!opt_in_smem(kernel, bytes)) return false;
    reserved[dev] = bytes;
    return true;
  }
};

// SM count of the current device for the context-free operator entry points (asked once per device)
int current_sm_count() {
  static int cached[SmemOptIn::kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= SmemOptIn::kMaxDevices) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

// ----------------------------------------------------------------------------
// tcgen05 GEMM dispatch
// ----------------------------------------------------------------------------
template <int BN, int EPI>
void launch_tc(Launcher& L, int kid, const CUtensorMap& w0, const CUtensorMap& w1, const CUtensorMap& w2,
               const CUtensorMap& x, const TcGemmArgs& a) {
  static SmemOptIn opt;
  constexpr int smem = tc_smem_bytes(BN, EPI);
  if (!opt.ensure(tc_gemm_kernel<BN, EPI>, smem)) {
    L.rc = fail(L.c, THINFER_ECUDA, "cannot reserve %d bytes of shared memory", smem);
    return;
  }
  const int n_ft = a.tiles[0] + a.tiles[1] + a.tiles[2];
  const int n_tt = (a.rows + BN - 1) / BN;
  const int n_tiles = n_ft * n_tt;
  int sms = L.c ? L.c->sm_count : current_sm_count();
  if (sms > kTcMaxCtas) sms = kTcMaxCtas;
  TcGemmArgs b = a;
  int grid = n_tiles < sms ? n_tiles : sms;
  if (b.mode == 1) {
    const long long units = static_cast<long long>(n_tiles) * ((a.k + kTcBK - 1) / kTcBK);
    grid = units < sms ? static_cast<int>(units) : sms;
    b.units_per_cta = static_cast<int>((units + grid - 1) / grid);
  }
  L.go(kid, tc_gemm_kernel<BN, EPI>, dim3(grid), dim3(kTcThreads), smem, w0, w1, w2, x, b);
}

int pick_bn(int rows, int epi) {
  if (rows <= 16) return 16;
  if (rows <= 32) return 32;
  if (rows <= 64) return 64;
  if (rows <= 128 || epi == EPI_SWIGLU) return 128;  // gate + up need two accumulators per buffer
  return 256;
}

template <int EPI>
void launch_tc_bn(Launcher& L, int kid, int bn, const CUtensorMap& w0, const CUtensorMap& w1, const CUtensorMap& w2,
                  const CUtensorMap& x, const TcGemmArgs& a) {
  switch (bn) {
    case 16: launch_tc<16, EPI>(L, kid, w0, w1, w2, x, a); break;
    case 32: launch_tc<32, EPI>(L, kid, w0, w1, w2, x, a); break;
    case 64: launch_tc<64, EPI>(L, kid, w0, w1, w2, x, a); break;
    case 128: launch_tc<128, EPI>(L, kid, w0, w1, w2, x, a); break;
    default:
      if constexpr (EPI != EPI_SWIGLU) launch_tc<256, EPI>(L, kid, w0, w1, w2, x, a);
      break;
  }
}

// x: activations [rows][k]; the token-side tensor map is encoded per call (host only, no device work)
template <int EPI>
void tc_linear(Launcher& L, int kid, const CUtensorMap& w0, const CUtensorMap& w1, const CUtensorMap& w2,
               const half_t* x, int rows, int k, const int (&n_feat)[3], const EpiArgs& e, bool stream_k = false,
               const float* sumsq_in = nullptr, float norm_eps = 0.f) {
  if (L.rc != THINFER_OK) return;
  const int bn = pick_bn(rows, EPI);
  CUtensorMap mx;
  if (!make_map_2d(&mx, x, k, rows, bn)) {
    L.rc = fail(L.c, THINFER_ECUDA, "cuTensorMapEncodeTiled failed for an activation operand");
    return;
  }
  TcGemmArgs a{};
  for (int i = 0; i < 3; ++i) {
    a.n_feat[i] = n_feat[i];
    a.tiles[i] = (n_feat[i] + tc_tile_feats(EPI) - 1) / tc_tile_feats(EPI);
  }
  if (EPI == EPI_SWIGLU || EPI == EPI_SWIGLU_IL) a.tiles[1] = 0;  // gate and up rows are processed together
  a.rows = rows;
  a.k = k;
  a.status = L.c ? L.c->status_dev : nullptr;
  a.e = e;
  a.sumsq_in = sumsq_in;
  if (L.c != nullptr && L.c->trace_unified && kid >= 0 && kid < 12) {
    a.dbg = L.c->timeline + 16 * kid;  // tracing aid: 16 slots per kernel id, reset at the start of the step
  }
  a.norm_dim = k;
  a.norm_eps = norm_eps;
  if (stream_k && L.c != nullptr && rows <= kTcDecodeMaxBN) {
    a.mode = 1;
    a.partial_ws = L.prefill_stage ? L.c->pf_splitk_ws : L.c->splitk_ws;
    a.tile_counters = L.prefill_stage ? L.c->pf_splitk_counters : L.c->splitk_counters;
  }
  launch_tc_bn<EPI>(L, kid, bn, w0, w1, w2, mx, a);
}

// ----------------------------------------------------------------------------
// streaming GEMV dispatch (decode)
// ----------------------------------------------------------------------------
int pick_kslices(int n_pairs, int k, int sm_count) {
  // enough independent warps to cover the machine several times; never slice below 512 elements
  int ks = 1;
  while (ks < 8 && static_cast<long long>(n_pairs) * ks < 32LL * sm_count && k / (ks * 2) >= 512) ks *= 2;
  return ks;
}

template <int EPI, bool NORM>
void gemv(Launcher& L, int kid, const half_t* w0, const half_t* w1, const half_t* w2, const int (&n)[3], int k,
          const half_t* x, int ldx, int rows, const half_t* gamma, float eps, const EpiArgs& e) {
  if (L.rc != THINFER_OK) return;
  GemvArgs a{};
  a.w[0] = w0;
  a.w[1] = w1;
  a.w[2] = w2;
  for (int i = 0; i < 3; ++i) a.n[i] = n[i];
  a.k = k;
  a.rows = rows;
  a.x = x;
  a.ldx = ldx;
  a.gamma = gamma;
  a.eps = eps;
  a.e = e;
  const int n_pairs = (EPI == EPI_SWIGLU) ? n[0] : (n[0] + n[1] + n[2]) / 2;
  a.kslices = pick_kslices(n_pairs, k, L.c ? L.c->sm_count : current_sm_count());
  const int pairs_per_cta = kGemvWarps / a.kslices;
  const int gx = (n_pairs + pairs_per_cta - 1) / pairs_per_cta;
  const dim3 block(kGemvWarps * 32);
  if (rows == 1) {
    L.go(kid, gemv_stream_kernel<1, EPI, NORM>, dim3(gx, 1), block, 0, a);
  } else if (rows == 2) {
    L.go(kid, gemv_stream_kernel<2, EPI, NORM>, dim3(gx, 1), block, 0, a);
  } else {
    L.go(kid, gemv_stream_kernel<4, EPI, NORM>, dim3(gx, (rows + 3) / 4), block, 0, a);
  }
}

// ----------------------------------------------------------------------------
// skinny tensor-core streaming dispatch (decode, <= 16 tokens)
// ----------------------------------------------------------------------------
// 16-row tiles per CTA share the kernels are instantiated for: 1 .. 7 with one token tile (up to 8 requests),
// 1 .. 6 with two (the accumulators of a share live in registers; beyond this they spill)
constexpr int kSkMaxTiles1 = 7, kSkMaxTiles2 = 6;

// Deals `grid` CTAs out to the matrices in proportion to their rows (every matrix with rows gets at least
// one) and returns the largest number of tiles a CTA share has (mirrors the kernel's partition).
int skinny_partition(const int (&n)[3], bool swiglu, int grid, int (&cta0)[4]) {
  const int mats = swiglu ? 1 : 3;
  long long total = 0;
  int used = 0;
  for (int m = 0; m < mats; ++m) {
    total += n[m];
    used += n[m] > 0;
  }
  int given = 0, worst = 0;
  long long rows_before = 0;
  cta0[0] = 0;
  for (int m = 0; m < 3; ++m) {
    int ctas = 0;
    if (m < mats && n[m] > 0) {
      --used;
      rows_before += n[m];
      // cumulative rounding keeps the total exact; leave one CTA for every matrix still to come
      ctas = static_cast<int>((rows_before * grid + total / 2) / total) - given;
      if (ctas < 1) ctas = 1;
      if (ctas > grid - given - used) ctas = grid - given - used;
      const int units = swiglu ? n[m] : n[m] / 2, tr = 8;  // 8 units per tile either way
      worst = std::max(worst, ((units + ctas - 1) / ctas + tr - 1) / tr);
    }
    given += ctas;
    cta0[m + 1] = given;
  }
  return worst;
}

template <int NT, int TM, int ST, int EPI, bool NORM>
void launch_skinny_tm(Launcher& L, int kid, int grid, const SkinnyArgs& a) {
  static SmemOptIn opt;
  const int smem = sk_smem_floats(TM, ST, a.sumsq_parts) * 4;
  if (smem > 220 * 1024 || !opt.ensure(skinny_mma_kernel<NT, TM, ST, EPI, NORM>, smem)) {
    L.rc = fail(L.c, THINFER_EUNSUPPORTED, "skinny projection needs %d bytes of shared memory", smem);
    return;
  }
  L.go(kid, skinny_mma_kernel<NT, TM, ST, EPI, NORM>, dim3(grid), dim3(kSkWarps * 32), smem, a);
}

template <int NT, int EPI, bool NORM>
void launch_skinny(Launcher& L, int kid, int grid, const SkinnyArgs& a) {
  switch (a.tiles_max) {
    case 1: launch_skinny_tm<NT, 1, 4, EPI, NORM>(L, kid, grid, a); break;
    case 2: launch_skinny_tm<NT, 2, 4, EPI, NORM>(L, kid, grid, a); break;
    case 3: launch_skinny_tm<NT, 3, 4, EPI, NORM>(L, kid, grid, a); break;
    case 4: launch_skinny_tm<NT, 4, 4, EPI, NORM>(L, kid, grid, a); break;
    case 5: launch_skinny_tm<NT, 5, 4, EPI, NORM>(L, kid, grid, a); break;
    case 6: launch_skinny_tm<NT, 6, 4, EPI, NORM>(L, kid, grid, a); break;
    default:
      if constexpr (NT == 1) launch_skinny_tm<NT, 7, 4, EPI, NORM>(L, kid, grid, a);
      else L.rc = fail(L.c, THINFER_EUNSUPPORTED, "skinny projection: %d tiles per share", a.tiles_max);
      break;
  }
}

// Returns the grid size: a RESID producer leaves one sum-of-squares part per CTA.
template <int EPI, bool NORM = false>
int skinny(Launcher& L, int kid, const half_t* w0, const half_t* w1, const half_t* w2, const int (&n)[3], int k,
           const half_t* x, int ldx, int rows, const float* sumsq_in, int sumsq_parts, float eps, const EpiArgs& e,
           const half_t* gamma = nullptr) {
  if (L.rc != THINFER_OK) return 0;
  SkinnyArgs a{};
  a.w[0] = w0;
  a.w[1] = w1;
  a.w[2] = w2;
  for (int i = 0; i < 3; ++i) a.n[i] = n[i];
  a.k = k;
  a.rows = rows;
  a.x = x;
  a.ldx = ldx;
  a.sumsq_in = sumsq_in;
  a.sumsq_parts = sumsq_in != nullptr ? sumsq_parts : 0;
  a.gamma = gamma;
  a.norm_dim = k;
  a.norm_eps = eps;
  a.e = e;
  if (L.c != nullptr && L.c->trace_unified && kid >= 0 && kid < 12) {
    a.dbg = L.c->timeline + 16 * kid;  // tracing aid: 16 slots per kernel id, reset at the start of the step
    if (kid == L.c->trace_cta_kid) a.cta_log = L.c->timeline + 256;  // per-CTA times of this kernel (grid <= 1024)
  }
  const int units = (EPI == EPI_SWIGLU) ? n[0] : (n[0] + n[1] + n[2]) / 2;
  const bool swiglu = EPI == EPI_SWIGLU;
  const int sms = L.c ? L.c->sm_count : current_sm_count();
  // Two CTAs per SM with a 4-stage ring per warp (a one-CTA variant with an 8-stage ring, tried for the two
  // projections with few features per SM, was slower); more CTAs when a share would exceed kSkMaxTiles tiles.
  const int mats = swiglu ? 1 : (n[0] > 0) + (n[1] > 0) + (n[2] > 0);
  int grid = 2 * sms;
  // never less than one full tile per CTA: for the 7B O and down projections 256 CTAs with full tiles beat
  // 296 CTAs with 14-row tiles (measured), although 40 SMs then run one CTA instead of two
  const int by_work = std::max(units / 8, mats);
  if (grid > by_work) grid = by_work;
  a.tiles_max = skinny_partition(n, swiglu, grid, a.cta0);
  // A grid of two CTAs per SM is one wave of equal shares; more CTAs than that are dealt out as slots free up
  // and some SMs end up with twice the work of others.  So the share grows before the grid does.
  int max_tiles = rows <= 8 ? kSkMaxTiles1 : kSkMaxTiles2;
  if (L.c != nullptr && L.c->sk_max_tiles > 0 && L.c->sk_max_tiles < max_tiles) max_tiles = L.c->sk_max_tiles;
  while (a.tiles_max > max_tiles && grid < 64 * sms) {
    grid += sms;
    a.tiles_max = skinny_partition(n, swiglu, grid, a.cta0);
  }
  // A share that walks tiles_max tiles but holds far fewer real rows (13B-shaped O and down projections: 17.3 rows
  // in shares of 2 tiles) leaves half of every ring stage empty.  With a single matrix the grid may shrink instead,
  // to shares of whole tiles: fewer CTAs, every stage full.
  if (mats == 1 && !swiglu && a.tiles_max >= 2 && L.c != nullptr && L.c->sk_whole_tiles &&
      static_cast<long long>(units) * 4 < 3LL * 8 * a.tiles_max * grid) {
    const int tiles = (units + 7) / 8;
    const int g2 = (tiles + a.tiles_max - 1) / a.tiles_max;
    if (g2 >= sms) {  // at least one CTA per SM
      grid = g2;
      a.tiles_max = skinny_partition(n, swiglu, grid, a.cta0);
    }
  }
  if (a.tiles_max > max_tiles) {
    L.rc = fail(L.c, THINFER_EUNSUPPORTED, "skinny projection: %d tiles per share", a.tiles_max);
    return 0;
  }
  if (grid > 1024) a.cta_log = nullptr;
  if (rows <= 8) launch_skinny<1, EPI, NORM>(L, kid, grid, a);
  else launch_skinny<2, EPI, NORM>(L, kid, grid, a);
  return grid;
}

// ----------------------------------------------------------------------------
// attention dispatch
// ----------------------------------------------------------------------------
// One decode-attention launch on the balanced split-KV schedule.  `unit`: keys of one CTA-wide iteration of the
// kernel; `smem`: its dynamic shared memory.  The number of CTAs that fit on the device at once is asked of the
// runtime once per kernel and device.
template <void (*kernel)(const AttnDecArgs)>
void launch_attn_decode(Launcher& L, thinfer_ctx* c, int unit, int smem, int max_cluster, int pairs_per_request,
                        AttnDecArgs a, int batch, int t_len) {
  static SmemOptIn opt;
  static int per_sm[SmemOptIn::kMaxDevices] = {};
  if (smem > 0 && !opt.ensure(kernel, smem)) {
    L.rc = fail(c, THINFER_ECUDA, "cannot reserve %d bytes of shared memory", smem);
    return;
  }
  int dev = 0, ctas_per_sm = 2;
  if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < SmemOptIn::kMaxDevices) {
    if (per_sm[dev] == 0) {
      int n = 0;
      if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, kAttnDecWarps * 32, smem) != cudaSuccess || n < 1) n = 2;
      per_sm[dev] = n;
    }
    ctas_per_sm = per_sm[dev];
  }
  a.n_pairs = batch * pairs_per_request;
  a.units_per_pair = (t_len + unit - 1) / unit;
  const long long n_units = static_cast<long long>(a.n_pairs) * a.units_per_pair;
  // One CTA per resident slot (times attn_waves, a tuning aid), every CTA the same number of units; not more
  // CTAs than pairs of units, and few enough that no pair is cut into more than kAttnMaxSplits segments.
  const long long slots = static_cast<long long>(ctas_per_sm) * c->sm_count * c->attn_waves;
  long long grid = slots;
  grid = std::min(grid, std::max<long long>(1, n_units / c->attn_min_units));
  grid = std::min(grid, static_cast<long long>(kAttnMaxSplits - 2) * a.n_pairs);
  // Every segment costs a query load, a merge and a ticket.  When a whole number of equal segments per pair
  // fills at least 80 % of the slots, that grid (every CTA exactly one segment) beats the exactly balanced one.
  long long per_pair = grid / a.n_pairs;
  bool aligned = per_pair >= 1 && per_pair * a.n_pairs * 10 >= slots * 8;
  // A pair whose segments fit one thread-block cluster merges them in shared memory of the cluster instead of
  // through L2 and a ticket.  Small problems (a few units per CTA: all latency) take that route even when it
  // leaves slots empty.
  if (c->attn_cluster && per_pair >= 2 &&
      ((aligned && per_pair <= max_cluster) || a.units_per_pair <= 4LL * max_cluster)) {
    per_pair = std::min<long long>(per_pair, max_cluster);
    aligned = true;
    a.cluster = static_cast<int>(per_pair);
    L.cluster = a.cluster;
  }
  if (aligned) grid = per_pair * a.n_pairs;
  L.go(THINFER_K_ATTN, kernel, dim3(static_cast<unsigned>(grid)), dim3(kAttnDecWarps * 32), smem, a);
}

template <int D, int G>
void attn_decode_dg(Launcher& L, thinfer_ctx* c, const AttnDecArgs& a, int batch, int t_len) {
  if constexpr (G >= 4) {
    // grouped-query models: the G heads of a pair are the rows of a tensor-core tile
    launch_attn_decode<attn_decode_gqa_kernel<D, G>>(L, c, kGqaUnit, gqa_smem_bytes<D, G>(), kGqaMaxCluster, a.n_q_heads / G, a,
                                                     batch, t_len);
  } else {
    constexpr int kUnit = kAttnDecWarps * kAttnDecUnroll * (32 / (D / 8));
    launch_attn_decode<attn_decode_kernel<D, G>>(L, c, kUnit, 0, kAttnMaxCluster, a.n_q_heads / G, a, batch, t_len);
  }
}

template <int D>
void attn_decode_d(Launcher& L, thinfer_ctx* c, const AttnDecArgs& a, int batch, int t_len, int ratio) {
  if (ratio % 8 == 0) attn_decode_dg<D, 8>(L, c, a, batch, t_len);
  else if (ratio % 4 == 0) attn_decode_dg<D, 4>(L, c, a, batch, t_len);
  else if (ratio % 2 == 0) attn_decode_dg<D, 2>(L, c, a, batch, t_len);
  else attn_decode_dg<D, 1>(L, c, a, batch, t_len);
}

// t_len: keys the longest request attends (the unit count of the schedule); with `len_arr` (ragged slots) request b
// attends len_arr[b] + len_add keys
void attn_decode(Launcher& L, thinfer_ctx* c, const half_t* q, const half_t* kc, const half_t* vc, half_t* out,
                 int batch, int t_len, const int* len_arr = nullptr, int len_add = 0) {
  if (L.rc != THINFER_OK) return;
  const thinfer_config& cf = c->cfg;
  AttnDecArgs a{};
  a.q = q;
  a.k_cache = kc;
  a.v_cache = vc;
  a.out = out;
  a.part_o = c->part_o;
  a.part_ml = c->part_ml;
  a.tickets = c->attn_counters;
  a.n_q_heads = cf.n_q_heads;
  a.n_kv_heads = cf.n_kv_heads;
  a.t_len = len_arr != nullptr ? len_add : t_len;  // ragged: per-request count = len_arr[b] + len_add
  a.len_arr = len_arr;
  a.t_max = cf.max_seq;
  a.scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(cf.head_dim));
  if (c->trace_unified) a.dbg = c->timeline + 16 * THINFER_K_ATTN;
  const int ratio = cf.n_q_heads / cf.n_kv_heads;
  if (cf.head_dim == 128) attn_decode_d<128>(L, c, a, batch, t_len, ratio);
  else attn_decode_d<64>(L, c, a, batch, t_len, ratio);
}

template <int D>
void attn_prefill_d(Launcher& L, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                    const AttnPreArgs& a, int batch) {
  static SmemOptIn opt;
  constexpr int smem = attn_pre_smem_bytes(D);
  if (!opt.ensure(attn_prefill_kernel<D>, smem)) {
    L.rc = fail(L.c, THINFER_ECUDA, "cannot reserve %d bytes of shared memory", smem);
    return;
  }
  const int n_qt = (a.seq_len + kAttnBQ - 1) / kAttnBQ;
  AttnPreArgs b = a;
  b.n_items = batch * a.n_q_heads;
  // K and V of one (request, query head) pair: 2 x seq x D 16-bit values, shared by the query heads of a KV head.
  // Up to eight rounds of CTAs are walked longest first in chunks whose K and V (32 MB) stay in L2; with more rounds
  // than that the tail is short anyway and the query blocks of one pair stay next to each other (measured:
  // 13B-shaped, 2560 CTAs: 524 TFLOP/s next to each other, 515 in chunks, 452 longest first throughout).
  const long long kv_bytes = 4LL * a.seq_len * D * a.n_kv_heads / a.n_q_heads;
  const int sms = L.c ? L.c->sm_count : current_sm_count();
  const long long n_ctas = static_cast<long long>((n_qt + 1) / 2) * b.n_items;
  b.chunk_items = n_ctas > 8LL * sms
                      ? 1
                      : static_cast<int>(std::max<long long>(1, std::min<long long>(b.n_items, (32LL << 20) / std::max<long long>(kv_bytes, 1))));
  L.go(THINFER_K_ATTN, attn_prefill_kernel<D>, dim3(((n_qt + 1) / 2) * b.n_items), dim3(kAttnThreads), smem, mq, mk, mv, b);
}

void attn_prefill(Launcher& L, const half_t* q, const half_t* k, const half_t* v, half_t* out, int batch, int n_q_heads,
                  int n_kv_heads, int seq, int kv_stride, int head_dim, int* status) {
  if (L.rc != THINFER_OK) return;
  CUtensorMap mq, mk, mv;
  const uint64_t d = head_dim;
  bool ok = make_map(&mq, q, d, seq, static_cast<uint64_t>(batch) * n_q_heads, d, static_cast<uint64_t>(seq) * d,
                     kAttnBQ, 3);
  ok = ok && make_map(&mk, k, d, seq, static_cast<uint64_t>(batch) * n_kv_heads, d, static_cast<uint64_t>(kv_stride) * d,
                      kAttnBK, 3);
  ok = ok && make_map(&mv, v, d, seq, static_cast<uint64_t>(batch) * n_kv_heads, d, static_cast<uint64_t>(kv_stride) * d,
                      kAttnBK, 3);
  if (!ok) {
    L.rc = fail(L.c, THINFER_ECUDA, "cuTensorMapEncodeTiled failed for an attention operand");
    return;
  }
  AttnPreArgs a{};
  a.out = out;
  a.n_q_heads = n_q_heads;
  a.n_kv_heads = n_kv_heads;
  a.seq_len = seq;
  a.scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(head_dim));
  a.status = status;
  if (head_dim == 128) attn_prefill_d<128>(L, mq, mk, mv, a, batch);
  else attn_prefill_d<64>(L, mq, mk, mv, a, batch);
}

void rmsnorm_rows(Launcher& L, const half_t* x, const half_t* g, half_t* y, int rows, int n, float eps) {
  if (rows <= 256 && n <= 8 * 256 * kRmsSmallChunks) {
    L.go(THINFER_K_RMSNORM, rmsnorm_few_rows_kernel, dim3(rows), dim3(256), 0, x, g, y, n, eps);
    return;
  }
  L.go(THINFER_K_RMSNORM, rmsnorm_rows_kernel, dim3((rows + 7) / 8), dim3(256), 0, x, g, y, rows, n, eps);
}

// ----------------------------------------------------------------------------
// the layer sequences
// ----------------------------------------------------------------------------
EpiArgs qkv_epi(thinfer_ctx* c, half_t* qbuf, half_t* kc, half_t* vc, int seq_len, int pos0,
                const int* pos_arr = nullptr) {
  const thinfer_config& cf = c->cfg;
  EpiArgs e{};
  e.q_out = qbuf;
  e.k_cache = kc;
  e.v_cache = vc;
  e.rope_cos = c->rope_cos;
  e.rope_sin = c->rope_sin;
  e.n_q = cf.n_q_heads * cf.head_dim;
  e.n_kv = cf.n_kv_heads * cf.head_dim;
  e.head_dim = cf.head_dim;
  e.n_q_heads = cf.n_q_heads;
  e.n_kv_heads = cf.n_kv_heads;
  e.seq_len = seq_len;
  e.pos0 = pos0;
  e.pos_arr = pos_arr;
  e.t_max = cf.max_seq;
  return e;
}

half_t* kv_ptr(thinfer_ctx* c, int slot, int layer, int which) {
  const size_t idx = (static_cast<size_t>(slot) * c->cfg.n_layers + layer) * 2 + which;
  return reinterpret_cast<half_t*>(c->kv + idx * c->kv_layer_bytes);
}

void layer_prefill(Launcher& L, thinfer_ctx* c, int slot, int layer, const half_t* x_in, half_t* x_out, int batch,
                   int seq) {
  const thinfer_config& cf = c->cfg;
  const thinfer_layer_weights& w = c->layers[layer];
  const LayerMaps& m = c->maps[layer];
  const int rows = batch * seq;
  const int qd = cf.n_q_heads * cf.head_dim, kvd = cf.n_kv_heads * cf.head_dim;
  half_t* kc = kv_ptr(c, slot, layer, 0);
  half_t* vc = kv_ptr(c, slot, layer, 1);

  rmsnorm_rows(L, x_in, static_cast<const half_t*>(w.attn_norm), c->h, rows, cf.hidden, cf.rms_eps);
  {
    const int nf[3] = {qd, kvd, kvd};
    tc_linear<EPI_QKV_ROPE>(L, THINFER_K_QKV, m.wq, m.wk, m.wv, c->h, rows, cf.hidden, nf, qkv_epi(c, c->qbuf, kc, vc, seq, 0));
  }
  attn_prefill(L, c->qbuf, kc, vc, c->attn, batch, cf.n_q_heads, cf.n_kv_heads, seq, cf.max_seq, cf.head_dim,
               c->status_dev);
  {
    EpiArgs e{};
    e.out = c->x1;
    e.resid = x_in;
    e.ld_out = cf.hidden;
    const int nf[3] = {cf.hidden, 0, 0};
    tc_linear<EPI_RESID>(L, THINFER_K_OPROJ, m.wo, m.wo, m.wo, c->attn, rows, qd, nf, e);
  }
  rmsnorm_rows(L, c->x1, static_cast<const half_t*>(w.ffn_norm), c->h, rows, cf.hidden, cf.rms_eps);
  {
    EpiArgs e{};
    e.out = c->act;
    e.ld_out = cf.ffn;
    const int nf[3] = {cf.ffn, cf.ffn, 0};
    if (rows > 64) tc_linear<EPI_SWIGLU_IL>(L, THINFER_K_GATEUP, m.wg64, m.wu64, m.wu64, c->h, rows, cf.hidden, nf, e);
    else tc_linear<EPI_SWIGLU>(L, THINFER_K_GATEUP, m.wg, m.wu, m.wu, c->h, rows, cf.hidden, nf, e);
  }
  {
    EpiArgs e{};
    e.out = x_out;
    e.resid = c->x1;
    e.ld_out = cf.hidden;
    const int nf[3] = {cf.hidden, 0, 0};
    tc_linear<EPI_RESID>(L, THINFER_K_DOWN, m.wd, m.wd, m.wd, c->act, rows, cf.ffn, nf, e);
  }
}

// pos: position of the new token (uniform slots), or the number of decode steps so far when `lens` (device,
// per-request prompt lengths of a ragged slot) is given; max_t: keys the longest request attends.
void layer_decode(Launcher& L, thinfer_ctx* c, int slot, int layer, const half_t* x_in, half_t* x_out, int batch,
                  int pos, const int* lens, int max_t) {
  const thinfer_config& cf = c->cfg;
  const thinfer_layer_weights& w = c->layers[layer];
  const int qd = cf.n_q_heads * cf.head_dim, kvd = cf.n_kv_heads * cf.head_dim;
  half_t* kc = kv_ptr(c, slot, layer, 0);
  half_t* vc = kv_ptr(c, slot, layer, 1);
  auto H = [](const void* p) { return static_cast<const half_t*>(p); };
  if (batch <= kSkTokMax && c->skinny_ok) {
    // Up to 16 tokens: every projection is a balanced weight stream into warp-level tensor-core fragments
    // (no partial sums across CTAs, no tensor memory, so the CTAs of the next projection move in as this
    // one's leave and fill their rings before the dependency wait).  The RMSNorm in front of a projection
    // is folded into the projection before it (gain there, 1/rms here); the first norm of a step has no
    // projection in front of it and runs as a prologue of the QKV projection.
    const bool first_norm_folded = layer > 0;
    const half_t* next_gain = layer + 1 < cf.n_layers ? H(c->layers[layer + 1].attn_norm) : nullptr;
    {
      const int n[3] = {qd, kvd, kvd};
      if (first_norm_folded)
        skinny<EPI_QKV_ROPE>(L, THINFER_K_QKV, H(w.wq), H(w.wk), H(w.wv), n, cf.hidden, c->xg, cf.hidden, batch, c->sumsq0,
                             c->sumsq0_parts, cf.rms_eps, qkv_epi(c, c->d_qbuf, kc, vc, 1, pos, lens));
      else
        skinny<EPI_QKV_ROPE, true>(L, THINFER_K_QKV, H(w.wq), H(w.wk), H(w.wv), n, cf.hidden, x_in, cf.hidden, batch, nullptr,
                                   0, cf.rms_eps, qkv_epi(c, c->d_qbuf, kc, vc, 1, pos, lens), H(w.attn_norm));
    }
    attn_decode(L, c, c->d_qbuf, kc, vc, c->d_attn, batch, max_t, lens, pos + 1);
    {
      EpiArgs e{};
      e.out = c->d_x1;
      e.resid = x_in;
      e.ld_out = cf.hidden;
      e.outg = c->x1g;
      e.gain_next = H(w.ffn_norm);
      e.sumsq = c->sumsq1;
      const int n[3] = {cf.hidden, 0, 0};
      c->sumsq1_parts = skinny<EPI_RESID>(L, THINFER_K_OPROJ, H(w.wo), nullptr, nullptr, n, qd, c->d_attn, qd, batch,
                                          nullptr, 0, 0.f, e);
    }
    {
      EpiArgs e{};
      e.out = c->d_act;
      e.ld_out = cf.ffn;
      const int n[3] = {cf.ffn, cf.ffn, 0};
      skinny<EPI_SWIGLU>(L, THINFER_K_GATEUP, H(w.w_gate), H(w.w_up), nullptr, n, cf.hidden, c->x1g, cf.hidden, batch,
                         c->sumsq1, c->sumsq1_parts, cf.rms_eps, e);
    }
    {
      EpiArgs e{};
      e.out = x_out;
      e.resid = c->d_x1;
      e.ld_out = cf.hidden;
      if (next_gain != nullptr) {
        e.outg = c->xg;
        e.gain_next = next_gain;
        e.sumsq = c->sumsq0;
      }
      const int n[3] = {cf.hidden, 0, 0};
      c->sumsq0_parts = skinny<EPI_RESID>(L, THINFER_K_DOWN, H(w.w_down), nullptr, nullptr, n, cf.ffn, c->d_act, cf.ffn,
                                          batch, nullptr, 0, 0.f, e);
    }
    return;
  }
  if (batch >= 2) {
    // batched decode: the weight stream feeds the tensor cores (stream-K over all SMs); plain FMA
    // cannot keep up with HBM beyond a couple of tokens per weight
    const LayerMaps& m = c->maps[layer];
    // The RMSNorm in front of a projection is folded into the projection before it: that one's residual
    // epilogue also writes (output x next gain) and the per-tile sums of squares; the consumer multiplies
    // its sums by 1/rms.  Only the first norm of a step still needs its own small kernel.
    const bool first_norm_folded = layer > 0;
    const half_t* next_gain = layer + 1 < cf.n_layers ? H(c->layers[layer + 1].attn_norm) : nullptr;
    if (!first_norm_folded) rmsnorm_rows(L, x_in, H(w.attn_norm), c->d_h, batch, cf.hidden, cf.rms_eps);
    {
      const int nf[3] = {qd, kvd, kvd};
      tc_linear<EPI_QKV_ROPE>(L, THINFER_K_QKV, m.wq, m.wk, m.wv, first_norm_folded ? c->xg : c->d_h, batch, cf.hidden, nf,
                              qkv_epi(c, c->d_qbuf, kc, vc, 1, pos, lens), true, first_norm_folded ? c->sumsq0 : nullptr, cf.rms_eps);
    }
    attn_decode(L, c, c->d_qbuf, kc, vc, c->d_attn, batch, max_t, lens, pos + 1);
    {
      EpiArgs e{};
      e.out = c->d_x1;
      e.resid = x_in;
      e.ld_out = cf.hidden;
      e.outg = c->x1g;
      e.gain_next = H(w.ffn_norm);
      e.sumsq = c->sumsq1;
      const int nf[3] = {cf.hidden, 0, 0};
      tc_linear<EPI_RESID>(L, THINFER_K_OPROJ, m.wo, m.wo, m.wo, c->d_attn, batch, qd, nf, e, true);
    }
    {
      EpiArgs e{};
      e.out = c->d_act;
      e.ld_out = cf.ffn;
      const int nf[3] = {cf.ffn, cf.ffn, 0};
      tc_linear<EPI_SWIGLU>(L, THINFER_K_GATEUP, m.wg, m.wu, m.wu, c->x1g, batch, cf.hidden, nf, e, true, c->sumsq1,
                            cf.rms_eps);
    }
    {
      EpiArgs e{};
      e.out = x_out;
      e.resid = c->d_x1;
      e.ld_out = cf.hidden;
      if (next_gain != nullptr) {
        e.outg = c->xg;
        e.gain_next = next_gain;
        e.sumsq = c->sumsq0;
      }
      const int nf[3] = {cf.hidden, 0, 0};
      tc_linear<EPI_RESID>(L, THINFER_K_DOWN, m.wd, m.wd, m.wd, c->d_act, batch, cf.ffn, nf, e, true);
    }
    return;
  }
  {
    const int n[3] = {qd, kvd, kvd};
    gemv<EPI_QKV_ROPE, true>(L, THINFER_K_QKV, H(w.wq), H(w.wk), H(w.wv), n, cf.hidden, x_in, cf.hidden, batch,
                             H(w.attn_norm), cf.rms_eps, qkv_epi(c, c->d_qbuf, kc, vc, 1, pos, lens));
  }
  attn_decode(L, c, c->d_qbuf, kc, vc, c->d_attn, batch, max_t, lens, pos + 1);
  {
    EpiArgs e{};
    e.out = c->d_x1;
    e.resid = x_in;
    e.ld_out = cf.hidden;
    const int n[3] = {cf.hidden, 0, 0};
    gemv<EPI_RESID, false>(L, THINFER_K_OPROJ, H(w.wo), nullptr, nullptr, n, qd, c->d_attn, qd, batch, nullptr, 0.f, e);
  }
  {
    EpiArgs e{};
    e.out = c->d_act;
    e.ld_out = cf.ffn;
    const int n[3] = {cf.ffn, cf.ffn, 0};
    gemv<EPI_SWIGLU, true>(L, THINFER_K_GATEUP, H(w.w_gate), H(w.w_up), nullptr, n, cf.hidden, c->d_x1, cf.hidden, batch,
                           H(w.ffn_norm), cf.rms_eps, e);
  }
  {
    EpiArgs e{};
    e.out = x_out;
    e.resid = c->d_x1;
    e.ld_out = cf.hidden;
    const int n[3] = {cf.hidden, 0, 0};
    gemv<EPI_RESID, false>(L, THINFER_K_DOWN, H(w.w_down), nullptr, nullptr, n, cf.ffn, c->d_act, cf.ffn, batch, nullptr,
                           0.f, e);
  }
}

// ----------------------------------------------------------------------------
// unified decode kernel: all layers of a step in one cooperative launch
// ----------------------------------------------------------------------------
template <int D, int G>
void launch_mega(Launcher& L, thinfer_ctx* c, const MegaArgs& a) {
  static SmemOptIn opt;
  constexpr int smem = mega_smem_bytes<16, D, G>();
  if (!opt.ensure(decode_mega_kernel<16, D, G>, smem)) {
    L.rc = fail(c, THINFER_ECUDA, "cannot reserve %d bytes of shared memory", smem);
    return;
  }
  L.cooperative = true;
  L.go(THINFER_K_DECODE_UNIFIED, decode_mega_kernel<16, D, G>, dim3(c->sm_count < kTcMaxCtas ? c->sm_count : kTcMaxCtas),
       dim3(kMegaThreads), smem, a);
}

bool mega_supported(const thinfer_ctx* c, int batch) { return batch <= 16; }

void layers_decode_unified(Launcher& L, thinfer_ctx* c, int slot, const half_t* x_in, half_t* x_out, int batch, int pos) {
  const thinfer_config& cf = c->cfg;
  MegaArgs a{};
  a.common = c->mega_common;
  a.layers = c->mega_layers;
  a.n_layers = cf.n_layers;
  a.batch = batch;
  a.pos = pos;
  a.hidden = cf.hidden;
  a.ffn = cf.ffn;
  a.n_q_heads = cf.n_q_heads;
  a.n_kv_heads = cf.n_kv_heads;
  a.t_max = cf.max_seq;
  a.eps = cf.rms_eps;
  a.x_in = x_in;
  a.x_out = x_out;
  a.xa = c->d_xa;
  a.xb = c->d_xb;
  a.xg = c->xg;
  a.x1 = c->d_x1;
  a.x1g = c->x1g;
  a.qbuf = c->d_qbuf;
  a.attn = c->d_attn;
  a.act = c->d_act;
  a.sumsq0 = c->sumsq0;
  a.sumsq1 = c->sumsq1;
  a.kv_base = c->kv;
  a.kv_layer_bytes = c->kv_layer_bytes;
  a.slot = slot;
  a.rope_cos = c->rope_cos;
  a.rope_sin = c->rope_sin;
  a.gemm_partial = c->splitk_ws;
  a.gemm_counters = c->splitk_counters;
  a.attn_partial = c->attn_partial;
  a.attn_counters = c->attn_counters;
  a.grid_bar = c->grid_bar;
  a.bar_base = c->bar_base;
  a.status = c->status_dev;
  a.timeline = c->trace_unified ? c->timeline : nullptr;
  const int ratio = cf.n_q_heads / cf.n_kv_heads;
  const int g = (ratio % 4 == 0) ? 4 : (ratio % 2 == 0) ? 2 : 1;
  if (cf.head_dim == 128) {
    if (g == 4) launch_mega<128, 4>(L, c, a);
    else if (g == 2) launch_mega<128, 2>(L, c, a);
    else launch_mega<128, 1>(L, c, a);
  } else {
    if (g == 4) launch_mega<64, 4>(L, c, a);
    else if (g == 2) launch_mega<64, 2>(L, c, a);
    else launch_mega<64, 1>(L, c, a);
  }
  // every CTA arrives once per grid barrier: 5 per layer
  // (a launch that failed enqueued nothing: the device counter did not move either)
  const unsigned int grid = c->sm_count < kTcMaxCtas ? c->sm_count : kTcMaxCtas;
  if (L.rc == THINFER_OK) c->bar_base += 5u * cf.n_layers * grid;
}

// final RMSNorm + LM head + greedy argmax on `batch` rows of x [batch][hidden]
void head_and_argmax(Launcher& L, thinfer_ctx* c, const half_t* x, int batch, int32_t* ids_out, float* logits_out,
                     bool decode) {
  const thinfer_config& cf = c->cfg;
  float* lg = logits_out != nullptr ? logits_out : (decode ? c->d_logits : c->logits);
  half_t* hbuf = decode ? c->d_h : c->h;
  EpiArgs e{};
  e.out = lg;
  e.ld_out = cf.vocab;
  const int n[3] = {cf.vocab, 0, 0};
  if (batch <= kSkTokMax && c->skinny_ok && cf.vocab % 2 == 0) {
    // final RMSNorm as the prologue of the vocabulary projection, one balanced weight stream
    skinny<EPI_PLAIN_F32, true>(L, THINFER_K_HEAD, c->lm_head, nullptr, nullptr, n, cf.hidden, x, cf.hidden, batch, nullptr, 0,
                                cf.rms_eps, e, c->final_norm);
  } else if (batch >= 2) {
    rmsnorm_rows(L, x, c->final_norm, hbuf, batch, cf.hidden, cf.rms_eps);
    tc_linear<EPI_PLAIN_F32>(L, THINFER_K_HEAD, c->map_head, c->map_head, c->map_head, hbuf, batch, cf.hidden, n, e, true);
  } else {
    gemv<EPI_PLAIN_F32, true>(L, THINFER_K_HEAD, c->lm_head, nullptr, nullptr, n, cf.hidden, x, cf.hidden, batch,
                              c->final_norm, cf.rms_eps, e);
  }
  if (ids_out != nullptr)
    L.go(THINFER_K_ARGMAX, argmax_rows_kernel, dim3(batch), dim3(1024), 0, static_cast<const float*>(lg), ids_out,
         cf.vocab);
}

// inspection hook: a copy of the hidden state behind `layer` (-1: the input of layer 0), enqueued on the stream
void capture_hidden(Launcher& L, thinfer_ctx* c, int layer, const half_t* x, size_t rows) {
  if (L.rc != THINFER_OK) return;
  for (const auto& cap : c->captures) {
    if (cap.first != layer) continue;
    if (cudaMemcpyAsync(cap.second, x, rows * c->cfg.hidden * 2, cudaMemcpyDeviceToDevice, L.st) != cudaSuccess)
      L.rc = fail(c, THINFER_ECUDA, "copying a captured hidden state failed");
  }
}

int run_prefill(thinfer_ctx* c, int slot, const void* input, int batch, int seq, void* out_primary, void* out_logits,
                cudaStream_t st, const int* lens_dev = nullptr) {
  const thinfer_config& cf = c->cfg;
  Launcher L{c, st};
  L.prefill_stage = true;
  if (c->trace_unified) L.go(-3, trace_reset_kernel, dim3(1), dim3(256), 0, c->timeline, 12);
  const int rows = batch * seq;
  const half_t* x = nullptr;
  if (cf.vocab > 0) {
    L.go(THINFER_K_EMBED, embed_gather_kernel, dim3((rows + 7) / 8), dim3(256), 0, static_cast<const int32_t*>(input),
         c->embed, c->xa, rows, cf.hidden, cf.vocab);
    x = c->xa;
  } else {
    x = static_cast<const half_t*>(input);
  }
  half_t* pong[2] = {c->xb, c->xa};
  if (!c->captures.empty()) capture_hidden(L, c, -1, x, rows);
  for (int l = 0; l < cf.n_layers; ++l) {
    half_t* dst = (cf.vocab == 0 && l == cf.n_layers - 1) ? static_cast<half_t*>(out_primary) : pong[l & 1];
    layer_prefill(L, c, slot, l, x, dst, batch, seq);
    x = dst;
    if (!c->captures.empty()) capture_hidden(L, c, l, x, rows);
  }
  if (cf.vocab > 0) {
    L.go(THINFER_K_EMBED, gather_last_rows_kernel, dim3((batch + 7) / 8), dim3(256), 0, x, c->last, batch, seq,
         cf.hidden, lens_dev);
    head_and_argmax(L, c, c->last, batch, static_cast<int32_t*>(out_primary), static_cast<float*>(out_logits), false);
  }
  return L.rc;
}

int run_decode(thinfer_ctx* c, int slot, const void* input, int batch, int pos, void* out_primary, void* out_logits,
               cudaStream_t st) {
  const thinfer_config& cf = c->cfg;
  Launcher L{c, st};
  if (c->trace_unified) L.go(-3, trace_reset_kernel, dim3(1), dim3(256), 0, c->timeline, 12);
  const half_t* x = nullptr;
  if (cf.vocab > 0) {
    L.go(THINFER_K_EMBED, embed_gather_kernel, dim3((batch + 7) / 8), dim3(256), 0, static_cast<const int32_t*>(input),
         c->embed, c->d_xa, batch, cf.hidden, cf.vocab);
    x = c->d_xa;
  } else {
    x = static_cast<const half_t*>(input);
  }
  half_t* pong[2] = {c->d_xb, c->d_xa};
  const Slot& sl = c->slots[slot];
  const int* lens = sl.ragged ? c->slot_lens + static_cast<size_t>(slot) * cf.max_batch : nullptr;
  const int step_pos = sl.ragged ? sl.steps : pos;  // ragged: every request adds its own prompt length on the device
  if (!c->captures.empty()) capture_hidden(L, c, -1, x, batch);
  if (c->launch_mode == 2 && mega_supported(c, batch) && !sl.ragged) {
    for (const auto& cap : c->captures)
      if (cap.first >= 0 && cap.first != cf.n_layers - 1)
        return fail(c, THINFER_EUNSUPPORTED, "launch mode 2 runs all layers in one kernel: only the last layer's "
                                             "hidden state can be captured");
    half_t* dst = cf.vocab == 0 ? static_cast<half_t*>(out_primary) : pong[(cf.n_layers - 1) & 1];
    layers_decode_unified(L, c, slot, x, dst, batch, pos);
    x = dst;
    if (!c->captures.empty()) capture_hidden(L, c, cf.n_layers - 1, x, batch);
  } else {
    for (int l = 0; l < cf.n_layers; ++l) {
      half_t* dst = (cf.vocab == 0 && l == cf.n_layers - 1) ? static_cast<half_t*>(out_primary) : pong[l & 1];
      layer_decode(L, c, slot, l, x, dst, batch, step_pos, lens, pos + 1);
      x = dst;
      if (!c->captures.empty()) capture_hidden(L, c, l, x, batch);
    }
  }
  if (cf.vocab > 0)
    head_and_argmax(L, c, x, batch, static_cast<int32_t*>(out_primary), static_cast<float*>(out_logits), true);
  return L.rc;
}

// Stage hand-off on the device (Section 3.4.2): a prefill waits until the slot's previous tenant has been
// released on whatever stream that happened; the first decode step of a slot waits for the prefill that filled it.
bool before_prefill(thinfer_ctx* c, Slot& s, cudaStream_t st) {
  if (s.freed_valid && s.freed_stream != st && cudaStreamWaitEvent(st, s.freed, 0) != cudaSuccess) return false;
  (void)c;
  return true;
}
bool after_prefill(Slot& s, cudaStream_t st, int batch, int seq_len) {
  s.busy = true;
  s.batch = batch;
  s.cur_len = seq_len;
  s.steps = 0;
  s.ready_stream = st;
  s.ready_valid = cudaEventRecord(s.ready, st) == cudaSuccess;
  return s.ready_valid;
}
bool before_decode(Slot& s, cudaStream_t st) {
  if (s.ready_valid && s.ready_stream != st) {
    if (cudaStreamWaitEvent(st, s.ready, 0) != cudaSuccess) return false;
    s.ready_stream = st;  // later steps on this stream are ordered by the stream itself
  }
  return true;
}

int check_prefill_args(thinfer_ctx* c, int slot, const void* input, int batch, int seq, void* out_primary,
                       void* out_logits) {
  if (c == nullptr) return THINFER_EINVAL;
  const thinfer_config& cf = c->cfg;
  if (slot < 0 || slot >= cf.buf_slots) return fail(c, THINFER_EINVAL, "slot %d outside [0, %d)", slot, cf.buf_slots);
  if (input == nullptr) return fail(c, THINFER_EINVAL, "input is NULL");
  if (batch <= 0 || seq <= 0) return fail(c, THINFER_EINVAL, "batch and seq_len must be positive");
  if (batch > cf.max_batch) return fail(c, THINFER_ECAPACITY, "batch %d > max_batch %d", batch, cf.max_batch);
  if (seq > cf.max_seq) return fail(c, THINFER_ECAPACITY, "seq_len %d > max_seq %d", seq, cf.max_seq);
  if (cf.vocab == 0) {
    if (out_primary == nullptr) return fail(c, THINFER_EINVAL, "out_primary is NULL");
    if (out_logits != nullptr) return fail(c, THINFER_EINVAL, "out_logits must be NULL in layer-only mode");
  } else if (out_primary == nullptr && out_logits == nullptr) {
    return fail(c, THINFER_EINVAL, "both outputs are NULL");
  }
  if (c->slots[slot].busy) return fail(c, THINFER_EBUSY, "slot %d holds an unreleased sequence", slot);
  return THINFER_OK;
}

int check_decode_args(thinfer_ctx* c, int slot, const void* input, void* out_primary, void* out_logits) {
  if (c == nullptr) return THINFER_EINVAL;
  const thinfer_config& cf = c->cfg;
  if (slot < 0 || slot >= cf.buf_slots) return fail(c, THINFER_EINVAL, "slot %d outside [0, %d)", slot, cf.buf_slots);
  if (input == nullptr) return fail(c, THINFER_EINVAL, "input is NULL");
  if (!c->slots[slot].busy) return fail(c, THINFER_EINVAL, "slot %d is empty: prefill first", slot);
  if (c->slots[slot].cur_len >= cf.max_seq)
    return fail(c, THINFER_ECAPACITY, "slot %d is full (%d positions)", slot, cf.max_seq);
  if (cf.vocab == 0) {
    if (out_primary == nullptr) return fail(c, THINFER_EINVAL, "out_primary is NULL");
    if (out_logits != nullptr) return fail(c, THINFER_EINVAL, "out_logits must be NULL in layer-only mode");
  } else if (out_primary == nullptr && out_logits == nullptr) {
    return fail(c, THINFER_EINVAL, "both outputs are NULL");
  }
  return THINFER_OK;
}

}  // namespace

// ============================================================================
// exported functions
// ============================================================================
extern "C" {

int thinfer_storage_type(void) { return kStorageType; }

int thinfer_workspace_bytes(const thinfer_config* cfg, size_t* kv_bytes, size_t* scratch_bytes) {
  int rc = validate_config(cfg, &g_global_err);
  if (rc != THINFER_OK) return rc;
  if (kv_bytes == nullptr || scratch_bytes == nullptr) return THINFER_EINVAL;
  *kv_bytes = kv_layer_bytes_of(*cfg) * 2 * static_cast<size_t>(cfg->n_layers) * cfg->buf_slots;
  *scratch_bytes = plan_scratch(*cfg).total;
  return THINFER_OK;
}

int thinfer_create(const thinfer_config* cfg, const thinfer_weights* weights, void* kv_workspace, size_t kv_bytes,
                   void* scratch, size_t scratch_bytes, thinfer_ctx** out) {
  int rc = validate_config(cfg, &g_global_err);
  if (rc != THINFER_OK) return rc;
  if (weights == nullptr || weights->layers == nullptr || kv_workspace == nullptr || scratch == nullptr ||
      out == nullptr)
    return THINFER_EINVAL;
  if ((reinterpret_cast<uintptr_t>(kv_workspace) & 255) != 0 || (reinterpret_cast<uintptr_t>(scratch) & 255) != 0)
    return THINFER_EINVAL;
  for (int l = 0; l < cfg->n_layers; ++l) {
    const thinfer_layer_weights& w = weights->layers[l];
    const void* ps[9] = {w.attn_norm, w.wq, w.wk, w.wv, w.wo, w.ffn_norm, w.w_gate, w.w_up, w.w_down};
    for (const void* p : ps)
      if (p == nullptr || (reinterpret_cast<uintptr_t>(p) & 15) != 0) return THINFER_EINVAL;
  }
  if (cfg->vocab > 0 && (weights->embed == nullptr || weights->final_norm == nullptr || weights->lm_head == nullptr))
    return THINFER_EINVAL;
  size_t need_kv = 0, need_scratch = 0;
  thinfer_workspace_bytes(cfg, &need_kv, &need_scratch);
  if (kv_bytes < need_kv || scratch_bytes < need_scratch) return THINFER_ECAPACITY;

  int dev = 0;
  cudaDeviceProp prop{};
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return THINFER_ECUDA;
  if (prop.major != 10) {
    g_global_err = "this library runs on sm_100 devices only";
    return THINFER_EUNSUPPORTED;
  }
  if (encode_tiled_fn() == nullptr) return THINFER_ECUDA;

  thinfer_ctx* c = new thinfer_ctx();
  c->cfg = *cfg;
  c->sm_count = prop.multiProcessorCount;
  c->skinny_ok = cfg->hidden % 64 == 0 && cfg->ffn % 64 == 0 && (cfg->n_q_heads * cfg->head_dim) % 64 == 0;
  c->layers.assign(weights->layers, weights->layers + cfg->n_layers);
  c->embed = static_cast<const half_t*>(weights->embed);
  c->final_norm = static_cast<const half_t*>(weights->final_norm);
  c->lm_head = static_cast<const half_t*>(weights->lm_head);
  c->kv = static_cast<uint8_t*>(kv_workspace);
  c->kv_layer_bytes = kv_layer_bytes_of(*cfg);
  c->slots.assign(cfg->buf_slots, Slot{});
  for (Slot& sl : c->slots) {
    if (cudaEventCreateWithFlags(&sl.ready, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&sl.freed, cudaEventDisableTiming) != cudaSuccess) {
      for (Slot& s2 : c->slots) {
        if (s2.ready) cudaEventDestroy(s2.ready);
        if (s2.freed) cudaEventDestroy(s2.freed);
      }
      delete c;
      return THINFER_ECUDA;
    }
  }

  const ScratchPlan p = plan_scratch(*cfg);
  uint8_t* s = static_cast<uint8_t*>(scratch);
  c->rope_cos = reinterpret_cast<float*>(s + p.rope_cos);
  c->rope_sin = reinterpret_cast<float*>(s + p.rope_sin);
  c->h = reinterpret_cast<half_t*>(s + p.h);
  c->qbuf = reinterpret_cast<half_t*>(s + p.qbuf);
  c->attn = reinterpret_cast<half_t*>(s + p.attn);
  c->x1 = reinterpret_cast<half_t*>(s + p.x1);
  c->act = reinterpret_cast<half_t*>(s + p.act);
  c->xa = reinterpret_cast<half_t*>(s + p.xa);
  c->xb = reinterpret_cast<half_t*>(s + p.xb);
  c->last = reinterpret_cast<half_t*>(s + p.last);
  c->logits = reinterpret_cast<float*>(s + p.logits);
  c->ids_out = reinterpret_cast<int32_t*>(s + p.ids_out);
  c->part_o = reinterpret_cast<float*>(s + p.part_o);
  c->part_ml = reinterpret_cast<float*>(s + p.part_ml);
  c->splitk_ws = reinterpret_cast<float*>(s + p.splitk_ws);
  c->splitk_counters = reinterpret_cast<int*>(s + p.splitk_counters);
  c->pf_splitk_ws = reinterpret_cast<float*>(s + p.pf_splitk_ws);
  c->pf_splitk_counters = reinterpret_cast<int*>(s + p.pf_splitk_counters);
  c->xg = reinterpret_cast<half_t*>(s + p.xg);
  c->x1g = reinterpret_cast<half_t*>(s + p.x1g);
  c->sumsq0 = reinterpret_cast<float*>(s + p.sumsq0);
  c->sumsq1 = reinterpret_cast<float*>(s + p.sumsq1);
  c->attn_partial = reinterpret_cast<float*>(s + p.attn_partial);
  c->attn_counters = reinterpret_cast<int*>(s + p.attn_counters);
  c->grid_bar = reinterpret_cast<unsigned int*>(s + p.grid_bar);
  c->timeline = reinterpret_cast<unsigned long long*>(s + p.timeline);
  c->mega_common = reinterpret_cast<MegaCommon*>(s + p.mega_common);
  c->mega_layers = reinterpret_cast<MegaLayer*>(s + p.mega_layers);
  c->stage_in = s + p.stage_in;
  c->stage_out = s + p.stage_out;
  c->slot_lens = reinterpret_cast<int*>(s + p.slot_lens);
  c->d_h = reinterpret_cast<half_t*>(s + p.d_h);
  c->d_qbuf = reinterpret_cast<half_t*>(s + p.d_qbuf);
  c->d_attn = reinterpret_cast<half_t*>(s + p.d_attn);
  c->d_x1 = reinterpret_cast<half_t*>(s + p.d_x1);
  c->d_act = reinterpret_cast<half_t*>(s + p.d_act);
  c->d_xa = reinterpret_cast<half_t*>(s + p.d_xa);
  c->d_xb = reinterpret_cast<half_t*>(s + p.d_xb);
  c->d_logits = reinterpret_cast<float*>(s + p.d_logits);
  c->d_stage_in = s + p.d_stage_in;
  c->d_stage_out = s + p.d_stage_out;
  c->max_splits = p.max_splits;
  {
    // tuning aids for experiments; the defaults are what the library is measured with
    auto env_int = [](const char* name, int lo, int hi, int dflt) {
      const char* v = std::getenv(name);
      if (v == nullptr || *v == 0) return dflt;
      const long x = std::strtol(v, nullptr, 10);
      return x < lo || x > hi ? dflt : static_cast<int>(x);
    };
    c->attn_waves = env_int("THINFER_ATTN_WAVES", 1, 8, c->attn_waves);
    c->attn_min_units = env_int("THINFER_ATTN_MIN_UNITS", 1, 64, c->attn_min_units);
    c->attn_cluster = env_int("THINFER_ATTN_CLUSTER", 0, 1, c->attn_cluster);
    c->sk_max_tiles = env_int("THINFER_SK_MAX_TILES", 1, 7, 0);
    c->sk_whole_tiles = env_int("THINFER_SK_WHOLE_TILES", 0, 1, c->sk_whole_tiles);
    c->trace_cta_kid = env_int("THINFER_TRACE_CTA_KID", 0, THINFER_K_COUNT - 1, -1);
  }

  auto cleanup = [&](int code) {
    for (Slot& sl : c->slots) {
      if (sl.ready) cudaEventDestroy(sl.ready);
      if (sl.freed) cudaEventDestroy(sl.freed);
    }
    if (c->status_host) cudaFreeHost(c->status_host);
    delete c;
    return code;
  };
  if (cudaHostAlloc(reinterpret_cast<void**>(&c->status_host), 64, cudaHostAllocMapped) != cudaSuccess)
    return cleanup(THINFER_ECUDA);
  *c->status_host = 0;
  if (cudaHostGetDevicePointer(reinterpret_cast<void**>(&c->status_dev), c->status_host, 0) != cudaSuccess)
    return cleanup(THINFER_ECUDA);

  // tensor maps of the weights: [n_out][k], 128-row x 64-column boxes
  c->maps.resize(cfg->n_layers);
  const uint64_t D = cfg->hidden, qd = static_cast<uint64_t>(cfg->n_q_heads) * cfg->head_dim,
                 kvd = static_cast<uint64_t>(cfg->n_kv_heads) * cfg->head_dim, F = cfg->ffn;
  bool ok = true;
  for (int l = 0; l < cfg->n_layers && ok; ++l) {
    const thinfer_layer_weights& w = c->layers[l];
    LayerMaps& m = c->maps[l];
    ok = ok && make_map_2d(&m.wq, w.wq, D, qd, 128) && make_map_2d(&m.wk, w.wk, D, kvd, 128) &&
         make_map_2d(&m.wv, w.wv, D, kvd, 128) && make_map_2d(&m.wo, w.wo, qd, D, 128) &&
         make_map_2d(&m.wg, w.w_gate, D, F, 128) && make_map_2d(&m.wu, w.w_up, D, F, 128) &&
         make_map_2d(&m.wd, w.w_down, F, D, 128) && make_map_2d(&m.wg64, w.w_gate, D, F, 64) &&
         make_map_2d(&m.wu64, w.w_up, D, F, 64);
  }
  if (ok && cfg->vocab > 0) ok = make_map_2d(&c->map_head, c->lm_head, D, cfg->vocab, 128);
  if (!ok) {
    g_global_err = "cuTensorMapEncodeTiled failed for a weight matrix";
    return cleanup(THINFER_ECUDA);
  }

  const int n_tab = cfg->max_seq * (cfg->head_dim / 2);
  rope_table_kernel<<<(n_tab + 255) / 256, 256>>>(c->rope_cos, c->rope_sin, cfg->max_seq, cfg->head_dim / 2,
                                                  static_cast<double>(cfg->rope_base));
  if (cudaMemsetAsync(c->splitk_counters, 0, static_cast<size_t>(p.max_tiles) * 8, 0) != cudaSuccess ||
      (p.pf_tiles > 0 && cudaMemsetAsync(c->pf_splitk_counters, 0, static_cast<size_t>(p.pf_tiles) * 8, 0) != cudaSuccess))
    return cleanup(THINFER_ECUDA);
  {
    // parameter blocks of the unified decode kernel: weight tensor maps per layer, token-operand maps
    // over the fixed scratch buffers (boxes of 16 token rows; rows beyond the batch are never stored)
    std::vector<MegaLayer> ml(cfg->n_layers);
    for (int l = 0; l < cfg->n_layers; ++l) {
      const LayerMaps& m = c->maps[l];
      ml[l].wq = m.wq; ml[l].wk = m.wk; ml[l].wv = m.wv; ml[l].wo = m.wo; ml[l].wg = m.wg; ml[l].wu = m.wu; ml[l].wd = m.wd;
      ml[l].attn_norm = static_cast<const half_t*>(c->layers[l].attn_norm);
      ml[l].ffn_norm = static_cast<const half_t*>(c->layers[l].ffn_norm);
      ml[l].next_norm = l + 1 < cfg->n_layers ? static_cast<const half_t*>(c->layers[l + 1].attn_norm) : nullptr;
    }
    MegaCommon mc;
    const uint64_t rows = cfg->max_batch;
    bool mok = make_map_2d(&mc.x_qkv, c->xg, D, rows, 16) && make_map_2d(&mc.x_o, c->d_attn, qd, rows, 16) &&
               make_map_2d(&mc.x_gu, c->x1g, D, rows, 16) && make_map_2d(&mc.x_down, c->d_act, F, rows, 16);
    if (!mok) return cleanup(THINFER_ECUDA);
    if (cudaMemcpy(c->mega_layers, ml.data(), sizeof(MegaLayer) * ml.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(c->mega_common, &mc, sizeof(mc), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemset(c->attn_counters, 0, static_cast<size_t>(cfg->max_batch) * cfg->n_q_heads * 4) != cudaSuccess ||
        cudaMemset(c->grid_bar, 0, 64) != cudaSuccess)
      return cleanup(THINFER_ECUDA);
  }
  if (cudaDeviceSynchronize() != cudaSuccess) return cleanup(THINFER_ECUDA);
  *out = c;
  return THINFER_OK;
}

int thinfer_prefill(thinfer_ctx* c, int32_t slot, const void* input, int32_t batch, int32_t seq_len, void* out_primary,
                    void* out_logits, void* cuda_stream) {
  int rc = check_prefill_args(c, slot, input, batch, seq_len, out_primary, out_logits);
  if (rc != THINFER_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (!before_prefill(c, c->slots[slot], st)) return fail(c, THINFER_ECUDA, "waiting for the slot's release failed");
  rc = run_prefill(c, slot, input, batch, seq_len, out_primary, out_logits, st);
  if (rc != THINFER_OK) return rc;
  c->slots[slot].ragged = false;
  if (!after_prefill(c->slots[slot], st, batch, seq_len)) return fail(c, THINFER_ECUDA, "recording the hand-off event failed");
  return THINFER_OK;
}

int thinfer_prefill_ragged(thinfer_ctx* c, int32_t slot, const void* input, int32_t batch, int32_t seq_len,
                           const int32_t* seq_lens, void* out_primary, void* out_logits, void* cuda_stream) {
  int rc = check_prefill_args(c, slot, input, batch, seq_len, out_primary, out_logits);
  if (rc != THINFER_OK) return rc;
  if (seq_lens == nullptr) return fail(c, THINFER_EINVAL, "seq_lens is NULL");
  int longest = 0;
  for (int b = 0; b < batch; ++b) {
    if (seq_lens[b] < 1 || seq_lens[b] > seq_len)
      return fail(c, THINFER_EINVAL, "seq_lens[%d] = %d outside [1, %d]", b, seq_lens[b], seq_len);
    if (seq_lens[b] > longest) longest = seq_lens[b];
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  Slot& s = c->slots[slot];
  if (!before_prefill(c, s, st)) return fail(c, THINFER_ECUDA, "waiting for the slot's release failed");
  s.lens.assign(seq_lens, seq_lens + batch);
  int* lens_dev = c->slot_lens + static_cast<size_t>(slot) * c->cfg.max_batch;
  if (cudaMemcpyAsync(lens_dev, s.lens.data(), static_cast<size_t>(batch) * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return fail(c, THINFER_ECUDA, "copying the prompt lengths failed");
  rc = run_prefill(c, slot, input, batch, seq_len, out_primary, out_logits, st, lens_dev);
  if (rc != THINFER_OK) return rc;
  s.ragged = true;
  if (!after_prefill(s, st, batch, longest)) return fail(c, THINFER_ECUDA, "recording the hand-off event failed");
  return THINFER_OK;
}

int thinfer_slot_lengths(const thinfer_ctx* c, int32_t slot, int32_t* lens_out) {
  if (c == nullptr || lens_out == nullptr || slot < 0 || slot >= c->cfg.buf_slots) return THINFER_EINVAL;
  const Slot& s = c->slots[slot];
  for (int b = 0; b < s.batch; ++b) lens_out[b] = s.ragged ? s.lens[b] + s.steps : s.cur_len;
  return THINFER_OK;
}

int thinfer_decode_step(thinfer_ctx* c, int32_t slot, const void* input, void* out_primary, void* out_logits,
                        void* cuda_stream) {
  int rc = check_decode_args(c, slot, input, out_primary, out_logits);
  if (rc != THINFER_OK) return rc;
  Slot& s = c->slots[slot];
  if (!before_decode(s, static_cast<cudaStream_t>(cuda_stream))) return fail(c, THINFER_ECUDA, "waiting for the prefill failed");
  rc = run_decode(c, slot, input, s.batch, s.cur_len, out_primary, out_logits, static_cast<cudaStream_t>(cuda_stream));
  if (rc != THINFER_OK) return rc;
  ++s.cur_len;
  ++s.steps;
  return THINFER_OK;
}

int thinfer_prefill_host(thinfer_ctx* c, int32_t slot, const void* host_input, int32_t batch, int32_t seq_len,
                         void* host_out_primary, void* host_out_logits, void* cuda_stream) {
  int rc = check_prefill_args(c, slot, host_input, batch, seq_len, host_out_primary, host_out_logits);
  if (rc != THINFER_OK) return rc;
  const thinfer_config& cf = c->cfg;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t rows = static_cast<size_t>(batch) * seq_len;
  const size_t in_bytes = cf.vocab > 0 ? rows * 4 : rows * cf.hidden * 2;
  if (!before_prefill(c, c->slots[slot], st)) return fail(c, THINFER_ECUDA, "waiting for the slot's release failed");
  if (cudaMemcpyAsync(c->stage_in, host_input, in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return fail(c, THINFER_ECUDA, "host-to-device copy failed");
  void* d_primary = c->stage_out;
  float* d_logits = reinterpret_cast<float*>(c->stage_out + static_cast<size_t>(cf.max_batch) * 4);
  rc = run_prefill(c, slot, c->stage_in, batch, seq_len, (cf.vocab == 0 || host_out_primary) ? d_primary : nullptr,
                   (cf.vocab > 0 && host_out_logits) ? d_logits : nullptr, st);
  if (rc != THINFER_OK) return rc;
  cudaError_t e = cudaSuccess;
  if (cf.vocab == 0) {
    e = cudaMemcpyAsync(host_out_primary, d_primary, rows * cf.hidden * 2, cudaMemcpyDeviceToHost, st);
  } else {
    if (host_out_primary) e = cudaMemcpyAsync(host_out_primary, d_primary, static_cast<size_t>(batch) * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && host_out_logits)
      e = cudaMemcpyAsync(host_out_logits, d_logits, static_cast<size_t>(batch) * cf.vocab * 4, cudaMemcpyDeviceToHost, st);
  }
  if (e != cudaSuccess) return fail(c, THINFER_ECUDA, "device-to-host copy failed");
  c->slots[slot].ragged = false;
  if (!after_prefill(c->slots[slot], st, batch, seq_len)) return fail(c, THINFER_ECUDA, "recording the hand-off event failed");
  return THINFER_OK;
}

int thinfer_decode_step_host(thinfer_ctx* c, int32_t slot, const void* host_input, void* host_out_primary,
                             void* host_out_logits, void* cuda_stream) {
  int rc = check_decode_args(c, slot, host_input, host_out_primary, host_out_logits);
  if (rc != THINFER_OK) return rc;
  const thinfer_config& cf = c->cfg;
  Slot& s = c->slots[slot];
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t in_bytes = cf.vocab > 0 ? static_cast<size_t>(s.batch) * 4 : static_cast<size_t>(s.batch) * cf.hidden * 2;
  if (!before_decode(s, st)) return fail(c, THINFER_ECUDA, "waiting for the prefill failed");
  if (cudaMemcpyAsync(c->d_stage_in, host_input, in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return fail(c, THINFER_ECUDA, "host-to-device copy failed");
  void* d_primary = c->d_stage_out;
  float* d_logits = reinterpret_cast<float*>(c->d_stage_out + static_cast<size_t>(cf.max_batch) * 4);
  rc = run_decode(c, slot, c->d_stage_in, s.batch, s.cur_len, (cf.vocab == 0 || host_out_primary) ? d_primary : nullptr,
                  (cf.vocab > 0 && host_out_logits) ? d_logits : nullptr, st);
  if (rc != THINFER_OK) return rc;
  cudaError_t e = cudaSuccess;
  if (cf.vocab == 0) {
    e = cudaMemcpyAsync(host_out_primary, d_primary, static_cast<size_t>(s.batch) * cf.hidden * 2, cudaMemcpyDeviceToHost, st);
  } else {
    if (host_out_primary) e = cudaMemcpyAsync(host_out_primary, d_primary, static_cast<size_t>(s.batch) * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && host_out_logits)
      e = cudaMemcpyAsync(host_out_logits, d_logits, static_cast<size_t>(s.batch) * cf.vocab * 4, cudaMemcpyDeviceToHost, st);
  }
  if (e != cudaSuccess) return fail(c, THINFER_ECUDA, "device-to-host copy failed");
  ++s.cur_len;
  ++s.steps;
  return THINFER_OK;
}

int thinfer_release_slot(thinfer_ctx* c, int32_t slot, void* cuda_stream) {
  if (c == nullptr) return THINFER_EINVAL;
  if (slot < 0 || slot >= c->cfg.buf_slots) return fail(c, THINFER_EINVAL, "slot %d outside [0, %d)", slot, c->cfg.buf_slots);
  Slot& s = c->slots[slot];
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  s.busy = false;
  s.batch = 0;
  s.cur_len = 0;
  s.ragged = false;
  s.steps = 0;
  s.ready_valid = false;
  s.freed_stream = st;
  s.freed_valid = cudaEventRecord(s.freed, st) == cudaSuccess;  // a later prefill on another stream waits for this
  return s.freed_valid ? THINFER_OK : fail(c, THINFER_ECUDA, "recording the release event failed");
}

int thinfer_slot_state(const thinfer_ctx* c, int32_t slot, int32_t* batch, int32_t* cur_len) {
  if (c == nullptr || slot < 0 || slot >= c->cfg.buf_slots) return THINFER_EINVAL;
  if (batch) *batch = c->slots[slot].batch;
  if (cur_len) *cur_len = c->slots[slot].cur_len;
  return THINFER_OK;
}

int thinfer_kv_pointer(const thinfer_ctx* c, int32_t slot, int32_t layer, int32_t which, void** device_ptr) {
  if (c == nullptr || device_ptr == nullptr || slot < 0 || slot >= c->cfg.buf_slots || layer < 0 ||
      layer >= c->cfg.n_layers || which < 0 || which > 1)
    return THINFER_EINVAL;
  *device_ptr = kv_ptr(const_cast<thinfer_ctx*>(c), slot, layer, which);
  return THINFER_OK;
}

int thinfer_status(thinfer_ctx* c, int32_t* device_status) {
  if (c == nullptr || device_status == nullptr) return THINFER_EINVAL;
  *device_status = *reinterpret_cast<volatile int*>(c->status_host);
  return THINFER_OK;
}

int thinfer_clear_status(thinfer_ctx* c) {
  if (c == nullptr) return THINFER_EINVAL;
  // the caller has synchronised: nothing of this context is running.  A kernel that gave up may have left
  // arrival counters and the grid barrier half-way: put all of them back to their initial state.
  const ScratchPlan p = plan_scratch(c->cfg);
  if (cudaDeviceSynchronize() != cudaSuccess) return fail(c, THINFER_ECUDA, "device synchronisation failed");
  if (cudaMemset(c->splitk_counters, 0, static_cast<size_t>(p.max_tiles) * 8) != cudaSuccess ||
      (p.pf_tiles > 0 && cudaMemset(c->pf_splitk_counters, 0, static_cast<size_t>(p.pf_tiles) * 8) != cudaSuccess) ||
      cudaMemset(c->attn_counters, 0, static_cast<size_t>(c->cfg.max_batch) * c->cfg.n_q_heads * 4) != cudaSuccess ||
      cudaMemset(c->grid_bar, 0, 64) != cudaSuccess)
    return fail(c, THINFER_ECUDA, "resetting the device counters failed");
  c->bar_base = 0;
  *reinterpret_cast<volatile int*>(c->status_host) = 0;
  return THINFER_OK;
}

int thinfer_selftest_bounded_wait(thinfer_ctx* c, int64_t limit_ns, void* cuda_stream) {
  if (c == nullptr) return THINFER_EINVAL;
  if (limit_ns < 1000 || limit_ns > 100000000) return fail(c, THINFER_EINVAL, "limit_ns outside [1 us, 100 ms]");
  Launcher L{c, static_cast<cudaStream_t>(cuda_stream)};
  L.go(-4, bounded_wait_selftest_kernel, dim3(1), dim3(64), 0, c->status_dev, static_cast<unsigned long long>(limit_ns),
       c->timeline + 255);
  return L.rc;
}

int thinfer_capture_hidden(thinfer_ctx* c, int32_t n, const int32_t* layers, void* const* device_bufs) {
  if (c == nullptr || n < 0) return THINFER_EINVAL;
  if (n > 0 && (layers == nullptr || device_bufs == nullptr)) return fail(c, THINFER_EINVAL, "layers or device_bufs is NULL");
  for (int i = 0; i < n; ++i)
    if (layers[i] < -1 || layers[i] >= c->cfg.n_layers || device_bufs[i] == nullptr)
      return fail(c, THINFER_EINVAL, "capture %d: layer %d outside [-1, %d) or NULL buffer", i, layers[i], c->cfg.n_layers);
  c->captures.clear();
  for (int i = 0; i < n; ++i) c->captures.emplace_back(layers[i], device_bufs[i]);
  return THINFER_OK;
}

int thinfer_set_launch_mode(thinfer_ctx* c, int32_t mode) {
  if (c == nullptr) return THINFER_EINVAL;
  if (mode < 0 || mode > 2) return fail(c, THINFER_EUNSUPPORTED, "launch mode %d is not available in this build", mode);
  c->launch_mode = mode;
  return THINFER_OK;
}

int thinfer_profile_select(thinfer_ctx* c, int32_t kernel_id) {
  if (c == nullptr || kernel_id < -1 || kernel_id >= THINFER_K_COUNT) return THINFER_EINVAL;
  c->prof_kernel = kernel_id;
  c->prof_used = 0;
  return THINFER_OK;
}

int thinfer_profile_read(thinfer_ctx* c, int32_t* launches, float* total_ms) {
  if (c == nullptr || launches == nullptr || total_ms == nullptr) return THINFER_EINVAL;
  float sum = 0.f;
  for (size_t i = 0; i < c->prof_used; ++i) {
    float ms = 0.f;
    if (cudaEventSynchronize(c->prof_events[i].end) != cudaSuccess ||
        cudaEventElapsedTime(&ms, c->prof_events[i].beg, c->prof_events[i].end) != cudaSuccess)
      return fail(c, THINFER_ECUDA, "reading profile events failed");
    sum += ms;
  }
  *launches = static_cast<int32_t>(c->prof_used);
  *total_ms = sum;
  c->prof_used = 0;
  return THINFER_OK;
}

int thinfer_trace_unified(thinfer_ctx* c, int32_t enable, uint64_t* host_out, int32_t max_entries) {
  if (c == nullptr) return THINFER_EINVAL;
  c->trace_unified = enable != 0;
  if (host_out != nullptr && max_entries > 0) {
    const int n = max_entries < 256 + 4 * 1024 ? max_entries : 256 + 4 * 1024;
    if (cudaMemcpy(host_out, c->timeline, static_cast<size_t>(n) * 8, cudaMemcpyDeviceToHost) != cudaSuccess)
      return fail(c, THINFER_ECUDA, "reading the timeline failed");
  }
  return THINFER_OK;
}

int64_t thinfer_launch_count(const thinfer_ctx* c) { return c ? c->launches : 0; }

const char* thinfer_last_error(const thinfer_ctx* c) { return c ? c->err.c_str() : g_global_err.c_str(); }

void thinfer_destroy(thinfer_ctx* c) {
  if (c == nullptr) return;
  for (ProfEvent& e : c->prof_events) {
    cudaEventDestroy(e.beg);
    cudaEventDestroy(e.end);
  }
  for (Slot& sl : c->slots) {
    if (sl.ready) cudaEventDestroy(sl.ready);
    if (sl.freed) cudaEventDestroy(sl.freed);
  }
  if (c->status_host) cudaFreeHost(c->status_host);
  delete c;
}

// ---------------------------------------------------------------- operators
int thinfer_op_linear(const void* x, const void* w, void* y, int32_t rows, int32_t n_out, int32_t k, int32_t out_fp32,
                      int32_t path, void* cuda_stream) {
  if (x == nullptr || w == nullptr || y == nullptr || rows <= 0 || n_out <= 0 || k <= 0) return THINFER_EINVAL;
  if (k % 8 != 0 || n_out % 2 != 0) return THINFER_EUNSUPPORTED;
  Launcher L{nullptr, static_cast<cudaStream_t>(cuda_stream)};
  EpiArgs e{};
  e.out = y;
  e.ld_out = n_out;
  const int n[3] = {n_out, 0, 0};
  if (path == 1) {
    if (rows > 16) return THINFER_EUNSUPPORTED;
    if (out_fp32)
      gemv<EPI_PLAIN_F32, false>(L, -2, static_cast<const half_t*>(w), nullptr, nullptr, n, k,
                                 static_cast<const half_t*>(x), k, rows, nullptr, 0.f, e);
    else
      gemv<EPI_PLAIN_F16, false>(L, -2, static_cast<const half_t*>(w), nullptr, nullptr, n, k,
                                 static_cast<const half_t*>(x), k, rows, nullptr, 0.f, e);
  } else if (path == 2) {
    if (rows > kSkTokMax || k % 64 != 0) return THINFER_EUNSUPPORTED;
    if (out_fp32)
      skinny<EPI_PLAIN_F32>(L, -2, static_cast<const half_t*>(w), nullptr, nullptr, n, k, static_cast<const half_t*>(x), k,
                            rows, nullptr, 0, 0.f, e);
    else
      skinny<EPI_PLAIN_F16>(L, -2, static_cast<const half_t*>(w), nullptr, nullptr, n, k, static_cast<const half_t*>(x), k,
                            rows, nullptr, 0, 0.f, e);
  } else if (path == 0) {
    CUtensorMap mw;
    if (!make_map_2d(&mw, w, k, n_out, 128)) return THINFER_ECUDA;
    if (out_fp32) tc_linear<EPI_PLAIN_F32>(L, -2, mw, mw, mw, static_cast<const half_t*>(x), rows, k, n, e);
    else tc_linear<EPI_PLAIN_F16>(L, -2, mw, mw, mw, static_cast<const half_t*>(x), rows, k, n, e);
  } else {
    return THINFER_EINVAL;
  }
  return L.rc;
}

// ---------------------------------------------------------------------------
// Allocation-free linear.  The stream-K scratch (arrival counters, then one FP32
// partial-accumulator slot per (tile, CTA) pair) is a fixed array in the library
// image.  In host code the array's name is only a handle: the kernel needs the
// device address, which cudaGetSymbolAddress returns for the current device.
// ---------------------------------------------------------------------------
namespace {
constexpr int kNoAllocMaxRows = 16;
constexpr int kNoAllocMaxNOut = 16384;
constexpr size_t kNoAllocCounterBytes = 1024;             // 128 tiles x 2 counters x 4 bytes
constexpr size_t kNoAllocSlotBytes = 16 * kTcBM * 4;      // 16 token columns x 128 features, FP32
constexpr size_t kNoAllocBytes = kNoAllocCounterBytes + (kNoAllocMaxNOut / kTcBM + kTcMaxCtas) * kNoAllocSlotBytes;
constexpr int kNoAllocMaxDevices = 64;
std::mutex g_noalloc_mutex;
unsigned char* g_noalloc_ptr[kNoAllocMaxDevices] = {};
}  // namespace
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

int thinfer_op_linear_noalloc(const void* x, const void* w, void* y, int32_t rows, int32_t n_out, int32_t k,
                              int32_t out_fp32, void* cuda_stream) {
  if (x == nullptr || w == nullptr || y == nullptr || rows <= 0 || n_out <= 0 || k <= 0) return THINFER_EINVAL;
  if (k % 8 != 0 || n_out % 2 != 0) return THINFER_EUNSUPPORTED;
  if (rows > kNoAllocMaxRows || n_out > kNoAllocMaxNOut) {
    g_global_err = "thinfer_op_linear_noalloc: rows <= 16 and n_out <= 16384 is the limit of the built-in scratch";
    return THINFER_ECAPACITY;
  }
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNoAllocMaxDevices) return THINFER_ECUDA;
  unsigned char* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (g_noalloc_ptr[dev] == nullptr) {  // set-up, once per device, with that device current
      void* p = nullptr;
      const cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
      if (e != cudaSuccess || p == nullptr) {
        g_global_err = std::string("cudaGetSymbolAddress failed: ") + cudaGetErrorString(e);
        return THINFER_ECUDA;
      }
      g_noalloc_ptr[dev] = static_cast<unsigned char*>(p);
    }
    scratch = g_noalloc_ptr[dev];
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // the counters must start at zero whatever an earlier (possibly failed) call left behind
  if (cudaMemsetAsync(scratch, 0, kNoAllocCounterBytes, st) != cudaSuccess) return THINFER_ECUDA;
  CUtensorMap mw, mx;
  if (!make_map_2d(&mw, w, k, n_out, 128) || !make_map_2d(&mx, x, k, rows, 16)) return THINFER_ECUDA;
  Launcher L{nullptr, st};
  TcGemmArgs a{};
  a.n_feat[0] = n_out;
  a.tiles[0] = (n_out + kTcBM - 1) / kTcBM;
  a.rows = rows;
  a.k = k;
  a.mode = 1;
  a.tile_counters = reinterpret_cast<int*>(scratch);
  a.partial_ws = reinterpret_cast<float*>(scratch + kNoAllocCounterBytes);
  a.status = nullptr;
  a.e.out = y;
  a.e.ld_out = n_out;
  if (out_fp32) launch_tc<16, EPI_PLAIN_F32>(L, -2, mw, mw, mw, mx, a);
  else launch_tc<16, EPI_PLAIN_F16>(L, -2, mw, mw, mw, mx, a);
  return L.rc;
}

int thinfer_op_attention_prefill(const void* q, const void* k, const void* v, void* out, int32_t batch,
                                 int32_t n_q_heads, int32_t n_kv_heads, int32_t seq, int32_t kv_stride,
                                 int32_t head_dim, void* cuda_stream) {
  if (q == nullptr || k == nullptr || v == nullptr || out == nullptr || batch <= 0 || n_q_heads <= 0 ||
      n_kv_heads <= 0 || seq <= 0 || kv_stride < seq)
    return THINFER_EINVAL;
  if ((head_dim != 64 && head_dim != 128) || n_q_heads % n_kv_heads != 0) return THINFER_EUNSUPPORTED;
  Launcher L{nullptr, static_cast<cudaStream_t>(cuda_stream)};
  attn_prefill(L, static_cast<const half_t*>(q), static_cast<const half_t*>(k), static_cast<const half_t*>(v),
               static_cast<half_t*>(out), batch, n_q_heads, n_kv_heads, seq, kv_stride, head_dim, nullptr);
  return L.rc;
}

int thinfer_op_attention_decode(thinfer_ctx* c, int32_t slot, int32_t layer, const void* q, void* out, int32_t batch,
                                int32_t t_len, const int32_t* seq_lens, void* cuda_stream) {
  if (c == nullptr) return THINFER_EINVAL;
  const thinfer_config& cf = c->cfg;
  if (q == nullptr || out == nullptr || slot < 0 || slot >= cf.buf_slots || layer < 0 || layer >= cf.n_layers)
    return fail(c, THINFER_EINVAL, "NULL pointer, or slot / layer out of range");
  if (batch < 1 || batch > cf.max_batch) return fail(c, THINFER_ECAPACITY, "batch %d outside [1, %d]", batch, cf.max_batch);
  int longest = t_len;
  if (seq_lens != nullptr) {
    longest = 0;
    for (int b = 0; b < batch; ++b) {
      if (seq_lens[b] < 1 || seq_lens[b] > cf.max_seq) return fail(c, THINFER_ECAPACITY, "seq_lens[%d] = %d", b, seq_lens[b]);
      longest = std::max(longest, seq_lens[b]);
    }
  }
  if (longest < 1 || longest > cf.max_seq) return fail(c, THINFER_ECAPACITY, "%d keys outside [1, %d]", longest, cf.max_seq);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int* lens_dev = nullptr;
  if (seq_lens != nullptr) {
    int* dst = c->slot_lens + static_cast<size_t>(slot) * cf.max_batch;
    if (cudaMemcpyAsync(dst, seq_lens, static_cast<size_t>(batch) * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return fail(c, THINFER_ECUDA, "copying the key counts failed");
    lens_dev = dst;
  }
  Launcher L{c, st};
  attn_decode(L, c, static_cast<const half_t*>(q), kv_ptr(c, slot, layer, 0), kv_ptr(c, slot, layer, 1),
              static_cast<half_t*>(out), batch, longest, lens_dev, 0);
  return L.rc;
}

int thinfer_op_argmax(const void* logits, void* ids, int32_t rows, int32_t n, void* cuda_stream) {
  if (logits == nullptr || ids == nullptr || rows <= 0 || n <= 0) return THINFER_EINVAL;
  Launcher L{nullptr, static_cast<cudaStream_t>(cuda_stream)};
  L.go(-2, argmax_rows_kernel, dim3(rows), dim3(1024), 0, static_cast<const float*>(logits), static_cast<int32_t*>(ids), n);
  return L.rc;
}

int thinfer_op_rmsnorm(const void* x, const void* gain, void* y, int32_t rows, int32_t n, float eps, void* cuda_stream) {
  if (x == nullptr || gain == nullptr || y == nullptr || rows <= 0 || n <= 0) return THINFER_EINVAL;
  if (n % 8 != 0) return THINFER_EUNSUPPORTED;
  Launcher L{nullptr, static_cast<cudaStream_t>(cuda_stream)};
  rmsnorm_rows(L, static_cast<const half_t*>(x), static_cast<const half_t*>(gain), static_cast<half_t*>(y), rows, n, eps);
  return L.rc;
}

}  // extern "C"

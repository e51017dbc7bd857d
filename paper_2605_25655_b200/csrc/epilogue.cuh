// Epilogue arguments shared by the weight-streaming GEMV and the tcgen05 GEMM:
// the "[low-density] - high-density - [low-density]" fusion units of
// Section 3.3.1 differ only in what happens to an accumulator element
// (feature n, token r) once the contraction is complete.
#pragma once
#include "common.cuh"

namespace thinfer {

enum Epi : int {
  EPI_PLAIN_F16 = 0,  // y[r][n] = acc                         (FP16 store)
  EPI_PLAIN_F32 = 1,  // y[r][n] = acc                         (FP32 store: logits)
  EPI_QKV_ROPE = 2,   // RoPE on q and k rows, q -> q buffer, k/v -> KV cache (Algorithm 1)
  EPI_RESID = 3,      // y[r][n] = resid[r][n] + acc           (O and down projections)
  EPI_SWIGLU = 4,     // a[r][f] = silu(acc_gate) * acc_up     (gate/up projection; two accumulators per tile)
  EPI_SWIGLU_IL = 5   // the same with 64 gate rows and 64 up rows interleaved in ONE 128-row tile (prefill)
};

struct EpiArgs {
  void* out;            // PLAIN / RESID / SWIGLU destination, row-major [rows][ld_out]
  const half_t* resid;  // RESID: residual stream, same layout as out
  int ld_out;
  // QKV + RoPE + cache append
  half_t* q_out;        // [batch][n_q_heads][seq_len][head_dim]
  half_t* k_cache;      // [max_batch][n_kv_heads][t_max][head_dim], K after rotation
  half_t* v_cache;
  const float* rope_cos;  // [max_seq][head_dim/2]
  const float* rope_sin;
  int n_q;              // n_q_heads * head_dim   (rows of wq)
  int n_kv;             // n_kv_heads * head_dim  (rows of wk and of wv)
  int head_dim, n_q_heads, n_kv_heads;
  int seq_len;          // tokens per request in this call (1 in decode)
  int pos0;             // position of the first token of each request
  const int* pos_arr;   // ragged decode: request b sits at position pos_arr[b] + pos0 (nullptr: pos0 for everybody)
  int t_max;            // KV positions per request in the cache
  // RESID only, optional (outg != nullptr): the next RMSNorm is folded into this epilogue.  Beside
  // y = resid + acc the kernel writes outg = y * gain_next (the operand the next projection reads)
  // and, per 128-feature tile and token, the sum of y^2 (sumsq[feature_tile][64 tokens]); the next
  // projection multiplies its result by rsqrt(sum over tiles / n + eps) per token.
  half_t* outg;
  const half_t* gain_next;
  float* sumsq;
};

// Destination of element (token r, feature n of the concatenated q|k|v space).
// kind: 0 = q, 1 = k, 2 = v.  Returns the element offset inside the matching buffer.
__device__ __forceinline__ size_t qkv_offset(const EpiArgs& e, int r, int n, int& kind, int& i_in_head, int& pos) {
  const int b = r / e.seq_len;
  const int s = r - b * e.seq_len;
  pos = e.pos0 + s + (e.pos_arr != nullptr ? e.pos_arr[b] : 0);
  if (n < e.n_q) {
    kind = 0;
    const int h = n / e.head_dim;
    i_in_head = n - h * e.head_dim;
    return ((static_cast<size_t>(b) * e.n_q_heads + h) * e.seq_len + s) * e.head_dim + i_in_head;
  }
  n -= e.n_q;
  kind = 1;
  if (n >= e.n_kv) {
    n -= e.n_kv;
    kind = 2;
  }
  const int h = n / e.head_dim;
  i_in_head = n - h * e.head_dim;
  return ((static_cast<size_t>(b) * e.n_kv_heads + h) * e.t_max + pos) * e.head_dim + i_in_head;
}

}  // namespace thinfer

// The C ABI (include/critiprefill.h): argument validation and kernel dispatch.
#include "cp_common.cuh"

#include <vector>

namespace {

using namespace cp;

int validate(const cp_params* p, Dims* out) {
  if (p == nullptr) return CP_ERR_NULL;
  if (p->batch <= 0 || p->n_q_heads <= 0 || p->n_kv_heads <= 0 || p->seq_len <= 0 || p->head_dim <= 0 ||
      p->segment_size <= 0 || p->block_size <= 0 || p->budget_blocks <= 0)
    return CP_ERR_SHAPE;
  if (p->dtype != CP_BF16 && p->dtype != CP_F32 && p->dtype != CP_F16) return CP_ERR_UNSUPPORTED;
  if (p->n_q_heads % p->n_kv_heads) return CP_ERR_SHAPE;
  if (p->segment_size % p->block_size) return CP_ERR_SHAPE;
  Dims m = make_dims(*p);
  if (m.k < m.r) return CP_ERR_SHAPE;
  if (p->forced_blocks < 0 || (p->forced_blocks & 0xffff) + ((p->forced_blocks >> 16) & 0xffff) > m.k - m.r) return CP_ERR_SHAPE;
  if (m.d != 64 && m.d != 128) return CP_ERR_UNSUPPORTED;
  const int64_t align = 16 / m.es;
  const int64_t* strides[4] = {p->q_stride, p->k_stride, p->v_stride, p->o_stride};
  for (auto s : strides)
    for (int i = 0; i < 3; ++i)
      if (s[i] < 0 || s[i] % align) return CP_ERR_SHAPE;
  for (auto s : strides)
    if (s[2] < m.d) return CP_ERR_SHAPE;
  *out = m;
  return CP_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_ws(const Dims& m, const void* ws, size_t ws_bytes) {
  if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 255u) || ws_bytes < ws_layout(m).total)
    return CP_ERR_WORKSPACE;
  return CP_OK;
}

int attention_common(const cp_params* p, const void* Q, const void* K, const void* V, const int32_t* idx,
                     const int32_t* cnt, void* O, float* lse, void* ws, size_t ws_bytes, void* stream, bool dense) {
  Dims m;
  int rc = validate(p, &m);
  if (rc != CP_OK) return rc;
  if (!Q || !K || !V || !O || (!dense && (!idx || !cnt))) return CP_ERR_NULL;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return CP_ERR_SHAPE;
  if ((rc = check_ws(m, ws, ws_bytes)) != CP_OK) return rc;
  DeviceStatus* st = static_cast<DeviceStatus*>(ws);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (sm100_path_applies(*p, m)) return launch_attention_sm100(*p, m, Q, K, V, idx, cnt, O, lse, st, dense, s);
  return launch_attention_simt(*p, m, Q, K, V, idx, cnt, O, lse, st, dense, s);
}

}  // namespace

extern "C" {

int critiprefill_workspace_bytes(const cp_params* p, size_t* bytes_out) {
  if (bytes_out == nullptr) return CP_ERR_NULL;
  Dims m;
  const int rc = validate(p, &m);
  if (rc != CP_OK) return rc;
  *bytes_out = ws_layout(m).total;
  return CP_OK;
}

int critiprefill_estimate(const cp_params* p, const void* Q, const void* K, const double* S_prev, double* S_out,
                          void* ws, size_t ws_bytes, void* cuda_stream) {
  Dims m;
  int rc = validate(p, &m);
  if (rc != CP_OK) return rc;
  const bool ready = (p->flags & CP_FLAG_SUMMARIES_READY) != 0;   // ws already holds the representatives (critiprefill_project_qk)
  if ((!ready && (!Q || !K)) || !S_out) return CP_ERR_NULL;
  if ((!ready && (!aligned16(Q) || !aligned16(K))) || S_out == S_prev) return CP_ERR_SHAPE;
  if (S_prev != nullptr && !(p->alpha >= 0.0f && p->alpha <= 1.0f)) return CP_ERR_SHAPE;   // line 14 is a convex combination (NaN fails too)
  if (m.n2 > kMaxBlocksN2) return CP_ERR_UNSUPPORTED;
  if ((rc = check_ws(m, ws, ws_bytes)) != CP_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (!ready && (rc = launch_summarize(*p, m, Q, K, static_cast<char*>(ws), s)) != CP_OK) return rc;
  return launch_score(*p, m, static_cast<char*>(ws), S_prev, S_out, s);
}

int critiprefill_select(const cp_params* p, const double* S, int32_t* idx, int32_t* cnt, void* ws, size_t ws_bytes,
                        void* cuda_stream) {
  Dims m;
  int rc = validate(p, &m);
  if (rc != CP_OK) return rc;
  if (!S || !idx || !cnt) return CP_ERR_NULL;
  if ((rc = check_ws(m, ws, ws_bytes)) != CP_OK) return rc;
  return launch_select(*p, m, S, idx, cnt, static_cast<cudaStream_t>(cuda_stream));
}

int critiprefill_project_qkv(const cp_params* p, const void* X, const void* Wq, const void* Wk, const void* Wv,
                             const float* rope_cos, const float* rope_sin, int32_t d_model, void* Q_out, void* K_out,
                             void* V_out, void* ws, size_t ws_bytes, void* cuda_stream) {
  Dims m;
  int rc = validate(p, &m);
  if (rc != CP_OK) return rc;
  if (!X || !Wq || !Wk || !Q_out || !K_out || ((rope_cos == nullptr) != (rope_sin == nullptr)) || ((Wv == nullptr) != (V_out == nullptr)))
    return CP_ERR_NULL;
  if (!aligned16(X) || !aligned16(Wq) || !aligned16(Wk) || !aligned16(Wv) || !aligned16(Q_out) || !aligned16(K_out) ||
      !aligned16(V_out) || !aligned16(rope_cos) || !aligned16(rope_sin) || d_model <= 0)
    return CP_ERR_SHAPE;
  if ((rc = check_ws(m, ws, ws_bytes)) != CP_OK) return rc;
  return launch_project(*p, m, X, Wq, Wk, Wv, rope_cos, rope_sin, d_model, Q_out, K_out, V_out, static_cast<char*>(ws),
                        static_cast<cudaStream_t>(cuda_stream));
}

int critiprefill_project_qk(const cp_params* p, const void* X, const void* Wq, const void* Wk, const float* rope_cos,
                            const float* rope_sin, int32_t d_model, void* Q_out, void* K_out, void* ws, size_t ws_bytes,
                            void* cuda_stream) {
  return critiprefill_project_qkv(p, X, Wq, Wk, nullptr, rope_cos, rope_sin, d_model, Q_out, K_out, nullptr, ws, ws_bytes,
                                  cuda_stream);
}

int critiprefill_decode_estimate(const cp_params* p, const void* q_last, const void* K, double* S_out, void* ws,
                                 size_t ws_bytes, void* cuda_stream) {
  Dims m;
  int rc = validate(p, &m);
  if (rc != CP_OK) return rc;
  if (!q_last || !K || !S_out) return CP_ERR_NULL;
  if (!aligned16(q_last) || !aligned16(K)) return CP_ERR_SHAPE;
  if (m.n2 > kMaxBlocksN2) return CP_ERR_UNSUPPORTED;
  if ((rc = check_ws(m, ws, ws_bytes)) != CP_OK) return rc;
  // Algorithm 1 on one segment that holds the last token alone: one "segment" per head that sees every block
  Dims md = m;
  md.n1 = 1; md.seg = m.n; md.r = 1;
  cp_params pd = *p;
  pd.flags &= ~CP_FLAG_MASK_BEFORE_SOFTMAX;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  char* w = static_cast<char*>(ws);
  if ((rc = launch_summarize(pd, md, nullptr, K, w, s)) != CP_OK) return rc;
  const WsLayout wl = ws_layout(md);
  const size_t q_bytes = size_t(m.B) * m.Hq * m.d * m.es;      // Qmax = Qmin = q
  if (cudaMemcpyAsync(w + wl.qmax, q_last, q_bytes, cudaMemcpyDeviceToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(w + wl.qmin, q_last, q_bytes, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return CP_ERR_CUDA;
  return launch_score(pd, md, w, nullptr, S_out, s);
}

int critiprefill_decode_select(const cp_params* p, const double* S, int32_t* idx, int32_t* cnt, void* ws, size_t ws_bytes,
                               void* cuda_stream) {
  Dims m;
  int rc = validate(p, &m);
  if (rc != CP_OK) return rc;
  if (!S || !idx || !cnt) return CP_ERR_NULL;
  if (m.n2 > kMaxBlocksN2) return CP_ERR_UNSUPPORTED;
  if ((rc = check_ws(m, ws, ws_bytes)) != CP_OK) return rc;
  Dims md = m;
  md.n1 = 1; md.r = 1;                       // one row per head; its only "diagonal" block is the last block
  return launch_select(*p, md, S, idx, cnt, static_cast<cudaStream_t>(cuda_stream), m.n2 - 1);
}

int critiprefill_attention(const cp_params* p, const void* Q, const void* K, const void* V, const int32_t* idx,
                           const int32_t* cnt, void* O, float* lse, void* ws, size_t ws_bytes, void* cuda_stream) {
  return attention_common(p, Q, K, V, idx, cnt, O, lse, ws, ws_bytes, cuda_stream, false);
}

int critiprefill_dense_attention(const cp_params* p, const void* Q, const void* K, const void* V, void* O,
                                 float* lse, void* ws, size_t ws_bytes, void* cuda_stream) {
  return attention_common(p, Q, K, V, nullptr, nullptr, O, lse, ws, ws_bytes, cuda_stream, true);
}

namespace {
// cu_seqlens checked, and the packed offsets of sequence i's S / idx / cnt arrays (in elements)
struct SeqSlot { int64_t s, idx, cnt; int len; };
int varlen_walk(const cp_params* p, const int32_t* cu, int32_t n_seqs, std::vector<SeqSlot>* slots, SeqSlot* total) {
  if (p == nullptr || cu == nullptr) return CP_ERR_NULL;
  if (n_seqs <= 0 || cu[0] != 0 || p->batch != 1 || p->segment_size <= 0 || p->block_size <= 0 || p->budget_blocks <= 0 ||
      p->n_q_heads <= 0)
    return CP_ERR_SHAPE;
  SeqSlot at{0, 0, 0, 0};
  for (int i = 0; i < n_seqs; ++i) {
    const int64_t len = int64_t(cu[i + 1]) - cu[i];
    if (len <= 0 || len > p->seq_len) return CP_ERR_SHAPE;
    const int64_t n1 = (len + p->segment_size - 1) / p->segment_size, n2 = (len + p->block_size - 1) / p->block_size;
    at.len = int(len);
    if (slots != nullptr) slots->push_back(at);
    at.s += int64_t(p->n_q_heads) * n1 * n2;
    at.idx += int64_t(p->n_q_heads) * n1 * p->budget_blocks;
    at.cnt += int64_t(p->n_q_heads) * n1;
  }
  *total = at;
  return CP_OK;
}
}  // namespace

int critiprefill_varlen_sizes(const cp_params* p, const int32_t* cu_seqlens, int32_t n_seqs, int64_t* s_elems,
                              int64_t* idx_elems, int64_t* cnt_elems) {
  if (!s_elems || !idx_elems || !cnt_elems) return CP_ERR_NULL;
  SeqSlot total;
  const int rc = varlen_walk(p, cu_seqlens, n_seqs, nullptr, &total);
  if (rc != CP_OK) return rc;
  *s_elems = total.s; *idx_elems = total.idx; *cnt_elems = total.cnt;
  return CP_OK;
}

int critiprefill_prefill_varlen(const cp_params* p, const int32_t* cu_seqlens, int32_t n_seqs, const void* Q,
                                const void* K, const void* V, const double* S_prev, double* S_out, int32_t* idx,
                                int32_t* cnt, void* O, float* lse, void* ws, size_t ws_bytes, void* cuda_stream) {
  std::vector<SeqSlot> slots;
  SeqSlot total;
  int rc = varlen_walk(p, cu_seqlens, n_seqs, &slots, &total);
  if (rc != CP_OK) return rc;
  Dims m;
  if ((rc = validate(p, &m)) != CP_OK) return rc;   // the longest sequence: strides, dtype, head geometry, budget
  if (!Q || !K || !V || !O || !S_out || !idx || !cnt) return CP_ERR_NULL;
  if (p->flags & CP_FLAG_SUMMARIES_READY) return CP_ERR_UNSUPPORTED;   // the workspace holds one sequence's representatives at a time
  if ((rc = check_ws(m, ws, ws_bytes)) != CP_OK) return rc;
  auto at = [&](const void* base, int64_t token, const int64_t* stride) {
    return static_cast<const char*>(base) + token * stride[2] * m.es;
  };
  for (int i = 0; i < n_seqs; ++i) {
    cp_params q = *p;
    q.seq_len = slots[i].len;
    const int64_t t0 = cu_seqlens[i];
    const void* Qi = at(Q, t0, p->q_stride);
    const void* Ki = at(K, t0, p->k_stride);
    const void* Vi = at(V, t0, p->v_stride);
    void* Oi = const_cast<char*>(at(O, t0, p->o_stride));
    double* Si = S_out + slots[i].s;
    int32_t* idx_i = idx + slots[i].idx;
    int32_t* cnt_i = cnt + slots[i].cnt;
    if ((rc = critiprefill_estimate(&q, Qi, Ki, S_prev ? S_prev + slots[i].s : nullptr, Si, ws, ws_bytes, cuda_stream)) != CP_OK) return rc;
    if ((rc = critiprefill_select(&q, Si, idx_i, cnt_i, ws, ws_bytes, cuda_stream)) != CP_OK) return rc;
    if ((rc = critiprefill_attention(&q, Qi, Ki, Vi, idx_i, cnt_i, Oi, lse ? lse + int64_t(p->n_q_heads) * t0 : nullptr, ws, ws_bytes,
                                     cuda_stream)) != CP_OK)
      return rc;
  }
  return CP_OK;
}

int critiprefill_device_status(const void* ws, int32_t* status_out, void* cuda_stream) {
  if (ws == nullptr || status_out == nullptr) return CP_ERR_NULL;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  int32_t code = 0;
  if (cudaMemcpyAsync(&code, ws, sizeof(code), cudaMemcpyDeviceToHost, s) != cudaSuccess) return CP_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return CP_ERR_CUDA;
  *status_out = code;
  return CP_OK;
}

const char* critiprefill_status_string(int status) {
  switch (status) {
    case CP_OK: return "ok";
    case CP_ERR_NULL: return "a required pointer is NULL";
    case CP_ERR_SHAPE: return "sizes, strides or alignment violate the requirements";
    case CP_ERR_UNSUPPORTED: return "problem outside the implemented envelope";
    case CP_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case CP_ERR_CUDA: return "a CUDA call failed";
    case CP_ERR_TIMEOUT: return "device: a bounded pipeline wait expired";
    case CP_ERR_BOUNDS: return "device: a block list broke its contract";
    case CP_ERR_STATIC_LIMIT: return "problem needs more scratch than the library's built-in static array holds";
    default: return "unknown status";
  }
}

}  // extern "C"

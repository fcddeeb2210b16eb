// Shared host/device declarations of the CUDA path (not used by the CPU oracle).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "critiprefill.h"

namespace cp {

constexpr int kStatusBytes = 256;   // head of the workspace: status word + diagnostics
constexpr int kMaxBlocksN2 = 8192;  // estimate: fp64 logits in the shared memory of up to 8 clustered CTAs; select: 32 keys/thread

// Derived sizes of one problem.
struct Dims {
  int B, Hq, Hkv, g, n, d, seg, blk, k, n1, n2, r, es;  // es = element size in bytes
};

inline Dims make_dims(const cp_params& p) {
  Dims m;
  m.B = p.batch; m.Hq = p.n_q_heads; m.Hkv = p.n_kv_heads; m.g = p.n_q_heads / p.n_kv_heads;
  m.n = p.seq_len; m.d = p.head_dim; m.seg = p.segment_size; m.blk = p.block_size;
  m.k = p.budget_blocks;
  m.n1 = (p.seq_len + p.segment_size - 1) / p.segment_size;   // the last segment / block may be shorter
  m.n2 = (p.seq_len + p.block_size - 1) / p.block_size;
  m.r = p.segment_size / p.block_size; m.es = p.dtype == CP_F32 ? 4 : 2;
  return m;
}

// Workspace layout: [status 256 B][Qmax][Qmin][Kmax][Kmin][stats][kabs]: summaries in the input dtype;
// stats = the four log-sum-exps of every (head, segment) row, [B,Hq,n1,4] fp64; kabs = largest magnitude
// in each key block's summaries, [B,Hkv,n2] fp32.
struct WsLayout {
  size_t qmax, qmin, kmax, kmin, stats, kabs, total;
};
inline WsLayout ws_layout(const Dims& m) {
  auto up = [](size_t x) { return (x + 255) & ~size_t(255); };
  WsLayout w;
  size_t qs = up(size_t(m.B) * m.Hq * m.n1 * m.d * m.es);
  size_t ks = up(size_t(m.B) * m.Hkv * m.n2 * m.d * m.es);
  w.qmax = kStatusBytes; w.qmin = w.qmax + qs; w.kmax = w.qmin + qs; w.kmin = w.kmax + ks;
  w.stats = w.kmin + ks;
  w.kabs = w.stats + up(size_t(m.B) * m.Hq * m.n1 * 4 * sizeof(double));
  w.total = w.kabs + up(size_t(m.B) * m.Hkv * m.n2 * sizeof(float));
  return w;
}

// Device status block.
struct DeviceStatus {
  int32_t code;     // cp_status, first error wins
  int32_t where;    // kernel-specific site id
  int32_t info[6];  // e.g. batch, head, segment, offending value
};

__device__ __forceinline__ void report(DeviceStatus* st, int code, int where, int a = 0, int b = 0,
                                       int c = 0, int d = 0) {
  if (st == nullptr) return;
  if (atomicCAS(&st->code, 0, code) == 0) {
    st->where = where; st->info[0] = a; st->info[1] = b; st->info[2] = c; st->info[3] = d;
  }
}

// Kernel launchers (each returns a cp_status).
int launch_summarize(const cp_params& p, const Dims& m, const void* Q, const void* K, char* ws,
                     cudaStream_t s);
int launch_score(const cp_params& p, const Dims& m, char* ws, const double* S_prev,
                 double* S_out, cudaStream_t s);
int launch_lse(const cp_params& p, const Dims& m, char* ws, cudaStream_t s);   // stats region of ws <- row log-sum-exps
int launch_score_generic(const cp_params& p, const Dims& m, const char* ws, const double* S_prev,
                         double* S_out, double* stats_out, cudaStream_t s);
int launch_select(const cp_params& p, const Dims& m, const double* S, int32_t* idx, int32_t* cnt,
                  cudaStream_t s, int past_fixed = -1);
int launch_attention_simt(const cp_params& p, const Dims& m, const void* Q, const void* K,
                          const void* V, const int32_t* idx, const int32_t* cnt, void* O, float* lse,
                          DeviceStatus* st, bool dense, cudaStream_t s);
int launch_attention_sm100(const cp_params& p, const Dims& m, const void* Q, const void* K,
                           const void* V, const int32_t* idx, const int32_t* cnt, void* O,
                           float* lse, DeviceStatus* st, bool dense, cudaStream_t s);
bool sm100_path_applies(const cp_params& p, const Dims& m);
int launch_project(const cp_params& p, const Dims& m, const void* X, const void* Wq, const void* Wk, const void* Wv,
                   const float* cosT, const float* sinT, int d_model, void* Q, void* K, void* V, char* ws, cudaStream_t st);

inline int check_launch() { return cudaGetLastError() == cudaSuccess ? CP_OK : CP_ERR_CUDA; }

}  // namespace cp

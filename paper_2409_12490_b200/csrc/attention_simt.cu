// Plain SIMT attention over a block list (Algorithm 2, lines 6-13) and dense causal attention
// (Eq. 2): one warp per query row, online softmax, fp32 arithmetic.  This is the path for
// fp32 inputs and for shapes outside the tensor-core envelope; it is not tuned.
#include <math_constants.h>

#include "cp_common.cuh"

namespace cp {
namespace {

constexpr int kWarps = 4;

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <> __device__ __forceinline__ float to_f32<__half>(__half x) { return __half2float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ __half from_f32<__half>(float x) { return __float2half_rn(x); }
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// The list contract: at most k entries, ascending, unique, each a block that segment j can see.
__device__ __forceinline__ bool list_ok(const int32_t* list, int c, int j, int r_full, int n2, int k, int lane) {
  const int vis = min(n2, (j + 1) * r_full);
  bool ok = (c >= 0) && (c <= k);
  if (ok) {
    for (int i = lane; i < c; i += 32) {
      const int v = list[i];
      ok = ok && (v >= 0) && (v < vis) && (i == 0 || list[i - 1] < v);
    }
  }
  return __all_sync(0xffffffffu, ok);
}

template <typename T, int D>
__global__ void __launch_bounds__(kWarps * 32)
attention_simt_kernel(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
                      const int32_t* __restrict__ idx, const int32_t* __restrict__ cnt,
                      T* __restrict__ O, float* __restrict__ lse, DeviceStatus* st, int B, int Hq, int g,
                      int n, int seg, int blk, int k, int r,
                      int64_t qsb, int64_t qsh, int64_t qst, int64_t ksb, int64_t ksh, int64_t kst,
                      int64_t vsb, int64_t vsh, int64_t vst, int64_t osb, int64_t osh, int64_t ost,
                      float sm_scale, int dense) {
  __shared__ float qs[kWarps][D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long rowid = (long long)blockIdx.x * kWarps + warp;   // (b*Hq + h)*n + t
  if (rowid >= (long long)B * Hq * n) return;
  const int t = int(rowid % n);
  const long long bh = rowid / n;
  const int h = int(bh % Hq), b = int(bh / Hq);
  const int j = t / seg, n1 = (n + seg - 1) / seg, n2 = (n + blk - 1) / blk;
  const T* q = Q + b * qsb + h * qsh + int64_t(t) * qst;
  const T* Kh = K + b * ksb + (h / g) * ksh;
  const T* Vh = V + b * vsb + (h / g) * vsh;
  for (int c = lane; c < D; c += 32) qs[warp][c] = to_f32(q[c]);
  __syncwarp();

  const int32_t* list = nullptr;
  int n_ranges = 1;
  if (!dense) {
    const long long u = bh * n1 + j;
    list = idx + u * k;
    n_ranges = cnt[u];
    if (!list_ok(list, n_ranges, j, r, n2, k, lane)) {
      if (lane == 0) report(st, CP_ERR_BOUNDS, 100, b, h, j, n_ranges);
      return;
    }
  }

  constexpr int CPL = D / 32;   // output channels per lane
  float acc[CPL];
#pragma unroll
  for (int i = 0; i < CPL; ++i) acc[i] = 0.f;
  float m_run = -CUDART_INF, l_run = 0.f;

  for (int e = 0; e < n_ranges; ++e) {
    int u0, u1;   // key range [u0, u1)
    if (dense) { u0 = 0; u1 = t + 1; }
    else { u0 = list[e] * blk; u1 = min(u0 + blk, t + 1); }
    for (int base = u0; base < u1; base += 32) {
      const int u = base + lane;
      float s = -CUDART_INF;
      if (u < u1) {
        const T* kr = Kh + int64_t(u) * kst;
        float a = 0.f;
#pragma unroll 8
        for (int c = 0; c < D; ++c) a = fmaf(qs[warp][c], to_f32(kr[c]), a);
        s = a * sm_scale;
      }
      float mx = s;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_new = fmaxf(m_run, mx);
      const float corr = (m_run == -CUDART_INF) ? 0.f : expf(m_run - m_new);
      const float p = (u < u1) ? expf(s - m_new) : 0.f;
      float ps = p;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
      l_run = l_run * corr + ps;
      m_run = m_new;
#pragma unroll
      for (int i = 0; i < CPL; ++i) acc[i] *= corr;
      const int cnt_here = min(32, u1 - base);
      for (int kk = 0; kk < cnt_here; ++kk) {
        const float pk = __shfl_sync(0xffffffffu, p, kk);
        const T* vr = Vh + int64_t(base + kk) * vst;
#pragma unroll
        for (int i = 0; i < CPL; ++i) acc[i] = fmaf(pk, to_f32(vr[lane + 32 * i]), acc[i]);
      }
    }
  }
  T* o = O + b * osb + h * osh + int64_t(t) * ost;
  const float inv = l_run > 0.f ? 1.f / l_run : 0.f;   // a row without any visible key: zeros, lse = ln 0
#pragma unroll
  for (int i = 0; i < CPL; ++i) o[lane + 32 * i] = from_f32<T>(acc[i] * inv);
  if (lse != nullptr && lane == 0) lse[rowid] = m_run + logf(l_run);
}

template <typename T, int D>
int launch_t(const cp_params& p, const Dims& m, const void* Q, const void* K, const void* V,
             const int32_t* idx, const int32_t* cnt, void* O, float* lse, DeviceStatus* st, bool dense,
             cudaStream_t s) {
  const long long rows = (long long)m.B * m.Hq * m.n;
  const long long ctas = (rows + kWarps - 1) / kWarps;
  if (ctas > 0x7fffffffLL) return CP_ERR_UNSUPPORTED;
  attention_simt_kernel<T, D><<<unsigned(ctas), kWarps * 32, 0, s>>>(
      static_cast<const T*>(Q), static_cast<const T*>(K), static_cast<const T*>(V), idx, cnt,
      static_cast<T*>(O), lse, st, m.B, m.Hq, m.g, m.n, m.seg, m.blk, m.k, m.r,
      p.q_stride[0], p.q_stride[1], p.q_stride[2], p.k_stride[0], p.k_stride[1], p.k_stride[2],
      p.v_stride[0], p.v_stride[1], p.v_stride[2], p.o_stride[0], p.o_stride[1], p.o_stride[2],
      p.sm_scale, dense ? 1 : 0);
  return check_launch();
}

}  // namespace

int launch_attention_simt(const cp_params& p, const Dims& m, const void* Q, const void* K,
                          const void* V, const int32_t* idx, const int32_t* cnt, void* O, float* lse,
                          DeviceStatus* st, bool dense, cudaStream_t s) {
  if (p.dtype == CP_BF16) {
    if (m.d == 128) return launch_t<__nv_bfloat16, 128>(p, m, Q, K, V, idx, cnt, O, lse, st, dense, s);
    if (m.d == 64) return launch_t<__nv_bfloat16, 64>(p, m, Q, K, V, idx, cnt, O, lse, st, dense, s);
  } else if (p.dtype == CP_F16) {
    if (m.d == 128) return launch_t<__half, 128>(p, m, Q, K, V, idx, cnt, O, lse, st, dense, s);
    if (m.d == 64) return launch_t<__half, 64>(p, m, Q, K, V, idx, cnt, O, lse, st, dense, s);
  } else {
    if (m.d == 128) return launch_t<float, 128>(p, m, Q, K, V, idx, cnt, O, lse, st, dense, s);
    if (m.d == 64) return launch_t<float, 64>(p, m, Q, K, V, idx, cnt, O, lse, st, dense, s);
  }
  return CP_ERR_UNSUPPORTED;
}

}  // namespace cp

// K2: criticality scores from the representatives (Algorithm 1, lines 9-14), in fp64 and in
// the log domain.  One CTA per (batch, query head, segment): it forms the four logit rows
// l1..l4 against every key block of its KV group, their log-sum-exps, and
//   ln S = max( ln((S1+S3)/2), ln((S2+S4)/2) ),  mask,  ln(alpha S + (1-alpha) S').
// The representatives are exact in the input dtype, every product is exact in fp64, so this
// differs from an fp64 CPU evaluation only by summation order and libm rounding.
#include <math_constants.h>

#include "cp_common.cuh"

namespace cp {
namespace {

constexpr int kThreads = 256;

template <typename T> __device__ __forceinline__ double to_f64(T x);
template <> __device__ __forceinline__ double to_f64<float>(float x) { return double(x); }
template <> __device__ __forceinline__ double to_f64<__nv_bfloat16>(__nv_bfloat16 x) { return double(__bfloat162float(x)); }

__device__ __forceinline__ double logaddexp(double a, double b) {
  const double hi = fmax(a, b), lo = fmin(a, b);
  if (hi == -CUDART_INF) return -CUDART_INF;
  return hi + log1p(exp(lo - hi));
}

// online (max, sum exp) pair
struct MS { double m, s; };
__device__ __forceinline__ void ms_add(MS& a, double x) {
  if (x == -CUDART_INF) return;
  if (x > a.m) { a.s = a.s * exp(a.m - x) + 1.0; a.m = x; } else { a.s += exp(x - a.m); }
}
__device__ __forceinline__ MS ms_merge(MS a, MS b) {
  if (b.m == -CUDART_INF) return a;
  if (a.m == -CUDART_INF) return b;
  MS r;
  r.m = fmax(a.m, b.m);
  r.s = a.s * exp(a.m - r.m) + b.s * exp(b.m - r.m);
  return r;
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
score_kernel(const T* __restrict__ Qmax, const T* __restrict__ Qmin, const T* __restrict__ Kmax,
             const T* __restrict__ Kmin, const double* __restrict__ S_prev, double* __restrict__ S_out,
             int Hq, int g, int n1, int n2, int seg, int blk, double est_scale, double ln_alpha,
             double ln_1m_alpha, int fuse, int mask_first) {
  extern __shared__ double smem[];
  double* qmx = smem;            // [D]
  double* qmn = smem + D;        // [D]
  double* lg = smem + 2 * D;     // [4][n2]
  __shared__ MS red[4][kThreads / 32];
  __shared__ double lse_sh[4];

  const int unit = blockIdx.x;   // (b*Hq + h)*n1 + j
  const int j = unit % n1;
  const int bh = unit / n1;
  const int h = bh % Hq, b = bh / Hq;
  const int kvh = b * (Hq / g) + h / g;
  const int tid = threadIdx.x;

  for (int c = tid; c < D; c += kThreads) {
    qmx[c] = to_f64(Qmax[size_t(unit) * D + c]);
    qmn[c] = to_f64(Qmin[size_t(unit) * D + c]);
  }
  __syncthreads();

  // blocks that start at or after the end of the segment are masked (line 13)
  const int visible = min(n2, ((j + 1) * seg + blk - 1) / blk);
  const T* kmx_base = Kmax + size_t(kvh) * n2 * D;
  const T* kmn_base = Kmin + size_t(kvh) * n2 * D;

  MS acc[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) { acc[i].m = -CUDART_INF; acc[i].s = 0.0; }

  constexpr int VE = 16 / sizeof(T);  // elements per 16-byte load
  for (int bb = tid; bb < n2; bb += kThreads) {
    const uint4* pmx = reinterpret_cast<const uint4*>(kmx_base + size_t(bb) * D);
    const uint4* pmn = reinterpret_cast<const uint4*>(kmn_base + size_t(bb) * D);
    double l1 = 0.0, l2 = 0.0, l3 = 0.0, l4 = 0.0;
#pragma unroll 4
    for (int v = 0; v < D / VE; ++v) {
      uint4 a = __ldg(pmx + v), c = __ldg(pmn + v);
      const T* ka = reinterpret_cast<const T*>(&a);
      const T* kc = reinterpret_cast<const T*>(&c);
#pragma unroll
      for (int e = 0; e < VE; ++e) {
        const double kx = to_f64(ka[e]), kn = to_f64(kc[e]);
        const double qx = qmx[v * VE + e], qn = qmn[v * VE + e];
        l1 = fma(qx, kx, l1); l2 = fma(qx, kn, l2); l3 = fma(qn, kx, l3); l4 = fma(qn, kn, l4);
      }
    }
    l1 *= est_scale; l2 *= est_scale; l3 *= est_scale; l4 *= est_scale;
    if (mask_first && bb >= visible) { l1 = l2 = l3 = l4 = -CUDART_INF; }
    lg[0 * n2 + bb] = l1; lg[1 * n2 + bb] = l2; lg[2 * n2 + bb] = l3; lg[3 * n2 + bb] = l4;
    ms_add(acc[0], l1); ms_add(acc[1], l2); ms_add(acc[2], l3); ms_add(acc[3], l4);
  }
  // log-sum-exp of each of the four rows (softmax over blocks, lines 9-10)
#pragma unroll
  for (int i = 0; i < 4; ++i) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      MS t;
      t.m = __shfl_xor_sync(0xffffffffu, acc[i].m, o);
      t.s = __shfl_xor_sync(0xffffffffu, acc[i].s, o);
      acc[i] = ms_merge(acc[i], t);
    }
    if ((tid & 31) == 0) red[i][tid >> 5] = acc[i];
  }
  __syncthreads();
  if (tid < 4) {
    MS t = red[tid][0];
    for (int w = 1; w < kThreads / 32; ++w) t = ms_merge(t, red[tid][w]);
    lse_sh[tid] = t.m + log(t.s);
  }
  __syncthreads();
  const double e1 = lse_sh[0], e2 = lse_sh[1], e3 = lse_sh[2], e4 = lse_sh[3];
  const double ln2 = 0.693147180559945309417232121458;
  double* out = S_out + size_t(unit) * n2;
  const double* prev = fuse ? S_prev + size_t(unit) * n2 : nullptr;
  for (int bb = tid; bb < n2; bb += kThreads) {
    double v;
    if (bb >= visible) {
      v = -CUDART_INF;
    } else {
      const double L1 = lg[0 * n2 + bb] - e1, L2 = lg[1 * n2 + bb] - e2;
      const double L3 = lg[2 * n2 + bb] - e3, L4 = lg[3 * n2 + bb] - e4;
      const double Lmax = logaddexp(L1, L3) - ln2;   // ln (S1+S3)/2
      const double Lmin = logaddexp(L2, L4) - ln2;   // ln (S2+S4)/2
      v = fmax(Lmax, Lmin);
      if (fuse) v = logaddexp(ln_alpha + v, ln_1m_alpha + prev[bb]);
    }
    out[bb] = v;
  }
}

template <typename T, int D>
int launch_t(const Dims& m, const char* ws, const WsLayout& w, const double* S_prev, double* S_out,
             double est_scale, double alpha, int fuse, int mask_first, cudaStream_t st) {
  const size_t smem = sizeof(double) * (2 * D + 4 * size_t(m.n2));
  auto kern = score_kernel<T, D>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess)
    return CP_ERR_CUDA;
  const long long units = (long long)m.B * m.Hq * m.n1;
  if (units > 0x7fffffffLL) return CP_ERR_UNSUPPORTED;
  kern<<<unsigned(units), kThreads, smem, st>>>(
      reinterpret_cast<const T*>(ws + w.qmax), reinterpret_cast<const T*>(ws + w.qmin),
      reinterpret_cast<const T*>(ws + w.kmax), reinterpret_cast<const T*>(ws + w.kmin), S_prev, S_out,
      m.Hq, m.g, m.n1, m.n2, m.seg, m.blk, est_scale, log(alpha), log1p(-alpha), fuse, mask_first);
  return check_launch();
}

}  // namespace

int launch_score(const cp_params& p, const Dims& m, const char* ws, const double* S_prev,
                 double* S_out, cudaStream_t st) {
  const WsLayout w = ws_layout(m);
  const int fuse = (S_prev != nullptr && p.alpha != 1.0f) ? 1 : 0;
  const int mask_first = (p.flags & CP_FLAG_MASK_BEFORE_SOFTMAX) ? 1 : 0;
  const double es = double(p.est_scale), al = double(p.alpha);
  if (p.dtype == CP_BF16) {
    if (m.d == 128) return launch_t<__nv_bfloat16, 128>(m, ws, w, S_prev, S_out, es, al, fuse, mask_first, st);
    if (m.d == 64) return launch_t<__nv_bfloat16, 64>(m, ws, w, S_prev, S_out, es, al, fuse, mask_first, st);
  } else {
    if (m.d == 128) return launch_t<float, 128>(m, ws, w, S_prev, S_out, es, al, fuse, mask_first, st);
    if (m.d == 64) return launch_t<float, 64>(m, ws, w, S_prev, S_out, es, al, fuse, mask_first, st);
  }
  return CP_ERR_UNSUPPORTED;
}

}  // namespace cp

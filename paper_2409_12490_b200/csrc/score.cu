// K2: criticality scores from the representatives (Algorithm 1, lines 9-14), in fp64 and in
// the log domain.  One CTA handles one segment j for U query heads of the same KV group: the
// key summaries of the group are read and widened to fp64 once and used for all U heads.
// Per head it forms the four logit rows l1..l4 against every key block, their log-sum-exps, and
//   ln S = max( ln((S1+S3)/2), ln((S2+S4)/2) ),  mask,  ln(alpha S + (1-alpha) S').
// The representatives are exact in the input dtype, every product is exact in fp64, so this
// differs from an fp64 CPU evaluation only by summation order and libm rounding.
#include <math_constants.h>

#include "cp_common.cuh"

namespace cp {
namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;

template <typename T> __device__ __forceinline__ double to_f64(T x);
template <> __device__ __forceinline__ double to_f64<float>(float x) { return double(x); }
template <> __device__ __forceinline__ double to_f64<__nv_bfloat16>(__nv_bfloat16 x) { return double(__bfloat162float(x)); }

__device__ __forceinline__ double logaddexp(double a, double b) {
  const double hi = fmax(a, b), lo = fmin(a, b);
  if (hi == -CUDART_INF) return -CUDART_INF;
  return hi + log1p(exp(lo - hi));
}

// Shared memory: q[U][D] as (max, min) pairs, then logits lg[U][4][n2].
template <typename T, int D, int U>
__global__ void __launch_bounds__(kThreads)
score_kernel(const T* __restrict__ Qmax, const T* __restrict__ Qmin, const T* __restrict__ Kmax,
             const T* __restrict__ Kmin, const double* __restrict__ S_prev, double* __restrict__ S_out,
             int Hq, int g, int n1, int n2, int seg, int blk, double est_scale, double ln_alpha,
             double ln_1m_alpha, int fuse, int mask_first) {
  extern __shared__ double smem[];
  double2* q2 = reinterpret_cast<double2*>(smem);   // [U][D]: .x = Qmax, .y = Qmin
  double* lg = smem + 2 * U * D;                    // [U][4][n2]
  __shared__ double red[4 * U][kWarps];
  __shared__ double stat[4 * U];

  // CTA -> (b, kv head, head subgroup, segment)
  const int groups = g / U;
  int x = blockIdx.x;
  const int j = x % n1; x /= n1;
  const int sub = x % groups; x /= groups;
  const int kvh = x;                                 // b*Hkv + kv head
  const int Hkv = Hq / g;
  const int b = kvh / Hkv;
  const int h0 = (kvh % Hkv) * g + sub * U;          // first query head of this CTA
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  auto unit_of = [&](int u) { return (size_t(b) * Hq + h0 + u) * n1 + j; };

  for (int i = tid; i < U * D; i += kThreads) {
    const int u = i / D, c = i % D;
    const size_t off = unit_of(u) * D + c;
    q2[i] = make_double2(to_f64(Qmax[off]), to_f64(Qmin[off]));
  }
  __syncthreads();

  // blocks that start at or after the end of the segment are masked (line 13)
  const int visible = min(n2, ((j + 1) * seg + blk - 1) / blk);
  const T* kmx_base = Kmax + size_t(kvh) * n2 * D;
  const T* kmn_base = Kmin + size_t(kvh) * n2 * D;
  constexpr int VE = 16 / sizeof(T);   // elements per 16-byte load

  for (int bb = tid; bb < n2; bb += kThreads) {
    const uint4* pmx = reinterpret_cast<const uint4*>(kmx_base + size_t(bb) * D);
    const uint4* pmn = reinterpret_cast<const uint4*>(kmn_base + size_t(bb) * D);
    double acc[U][4];
#pragma unroll
    for (int u = 0; u < U; ++u) acc[u][0] = acc[u][1] = acc[u][2] = acc[u][3] = 0.0;
#pragma unroll 4
    for (int v = 0; v < D / VE; ++v) {
      const uint4 a = __ldg(pmx + v), c = __ldg(pmn + v);
      const T* ka = reinterpret_cast<const T*>(&a);
      const T* kc = reinterpret_cast<const T*>(&c);
      double kx[VE], kn[VE];
#pragma unroll
      for (int e = 0; e < VE; ++e) { kx[e] = to_f64(ka[e]); kn[e] = to_f64(kc[e]); }
#pragma unroll
      for (int u = 0; u < U; ++u) {
#pragma unroll
        for (int e = 0; e < VE; ++e) {
          const double2 q = q2[u * D + v * VE + e];
          acc[u][0] = fma(q.x, kx[e], acc[u][0]); acc[u][1] = fma(q.x, kn[e], acc[u][1]);
          acc[u][2] = fma(q.y, kx[e], acc[u][2]); acc[u][3] = fma(q.y, kn[e], acc[u][3]);
        }
      }
    }
    const bool hide = mask_first && bb >= visible;
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int i = 0; i < 4; ++i) lg[(u * 4 + i) * n2 + bb] = hide ? -CUDART_INF : acc[u][i] * est_scale;
  }
  __syncthreads();

  // log-sum-exp of each of the 4U logit rows (softmax over blocks, lines 9-10): max, then sum
  double part[4 * U];
#pragma unroll
  for (int rI = 0; rI < 4 * U; ++rI) {
    double m = -CUDART_INF;
    for (int bb = tid; bb < n2; bb += kThreads) m = fmax(m, lg[rI * n2 + bb]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) red[rI][warp] = m;
  }
  __syncthreads();
  if (tid < 4 * U) {
    double m = red[tid][0];
    for (int w = 1; w < kWarps; ++w) m = fmax(m, red[tid][w]);
    stat[tid] = m;
  }
  __syncthreads();
#pragma unroll
  for (int rI = 0; rI < 4 * U; ++rI) {
    const double m = stat[rI];
    double sum = 0.0;
    for (int bb = tid; bb < n2; bb += kThreads) sum += exp(lg[rI * n2 + bb] - m);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    part[rI] = sum;
  }
  __syncthreads();   // red[] is reused
#pragma unroll
  for (int rI = 0; rI < 4 * U; ++rI)
    if (lane == 0) red[rI][warp] = part[rI];
  __syncthreads();
  if (tid < 4 * U) {
    double sum = 0.0;
    for (int w = 0; w < kWarps; ++w) sum += red[tid][w];
    stat[tid] = stat[tid] + log(sum);
  }
  __syncthreads();

  const double ln2 = 0.693147180559945309417232121458;
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const double e1 = stat[u * 4 + 0], e2 = stat[u * 4 + 1], e3 = stat[u * 4 + 2], e4 = stat[u * 4 + 3];
    double* out = S_out + unit_of(u) * n2;
    const double* prev = fuse ? S_prev + unit_of(u) * n2 : nullptr;
    const double* l = lg + u * 4 * n2;
    for (int bb = tid; bb < n2; bb += kThreads) {
      double v;
      if (bb >= visible) {
        v = -CUDART_INF;
      } else {
        const double L1 = l[bb] - e1, L2 = l[n2 + bb] - e2, L3 = l[2 * n2 + bb] - e3, L4 = l[3 * n2 + bb] - e4;
        const double Lmax = logaddexp(L1, L3) - ln2;   // ln (S1+S3)/2
        const double Lmin = logaddexp(L2, L4) - ln2;   // ln (S2+S4)/2
        v = fmax(Lmax, Lmin);
        if (fuse) v = logaddexp(ln_alpha + v, ln_1m_alpha + prev[bb]);
      }
      out[bb] = v;
    }
  }
}

template <typename T, int D, int U>
int launch_u(const Dims& m, const char* ws, const WsLayout& w, const double* S_prev, double* S_out,
             double est_scale, double alpha, int fuse, int mask_first, cudaStream_t st) {
  const size_t smem = sizeof(double) * (2 * size_t(U) * D + 4 * size_t(U) * m.n2);
  auto kern = score_kernel<T, D, U>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess)
    return CP_ERR_CUDA;
  const long long ctas = (long long)m.B * m.Hkv * (m.g / U) * m.n1;
  if (ctas > 0x7fffffffLL) return CP_ERR_UNSUPPORTED;
  kern<<<unsigned(ctas), kThreads, smem, st>>>(
      reinterpret_cast<const T*>(ws + w.qmax), reinterpret_cast<const T*>(ws + w.qmin),
      reinterpret_cast<const T*>(ws + w.kmax), reinterpret_cast<const T*>(ws + w.kmin), S_prev, S_out,
      m.Hq, m.g, m.n1, m.n2, m.seg, m.blk, est_scale, log(alpha), log1p(-alpha), fuse, mask_first);
  return check_launch();
}

template <typename T, int D>
int launch_t(const Dims& m, const char* ws, const WsLayout& w, const double* S_prev, double* S_out,
             double est_scale, double alpha, int fuse, int mask_first, cudaStream_t st) {
  // as many heads per CTA as divide the group and keep the logits within ~200 KB of shared memory
  const size_t budget = 200 * 1024;
  auto fits = [&](int U) { return m.g % U == 0 && sizeof(double) * (2 * size_t(U) * D + 4 * size_t(U) * m.n2) <= budget; };
  if (fits(4)) return launch_u<T, D, 4>(m, ws, w, S_prev, S_out, est_scale, alpha, fuse, mask_first, st);
  if (fits(2)) return launch_u<T, D, 2>(m, ws, w, S_prev, S_out, est_scale, alpha, fuse, mask_first, st);
  if (fits(1)) return launch_u<T, D, 1>(m, ws, w, S_prev, S_out, est_scale, alpha, fuse, mask_first, st);
  return CP_ERR_UNSUPPORTED;
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

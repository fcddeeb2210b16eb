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

// ln(e^a + e^b).  When the smaller term is more than e^-50 below the larger one it cannot change
// the rounded result (|hi| is at most a few hundred here), so the transcendental pair is skipped.
__device__ __forceinline__ double logaddexp(double a, double b) {
  const double hi = fmax(a, b), lo = fmin(a, b);
  const double d = lo - hi;                 // <= 0, or NaN when both are -inf
  if (!(d > -50.0)) return hi;
  return hi + log1p(exp(d));
}

// Shared memory: logits lg[U][4][n2].
template <typename T, int D, int U>
__global__ void __launch_bounds__(kThreads)
score_kernel(const T* __restrict__ Qmax, const T* __restrict__ Qmin, const T* __restrict__ Kmax,
             const T* __restrict__ Kmin, const double* __restrict__ S_prev, double* __restrict__ S_out,
             int Hq, int g, int n1, int n2, int seg, int blk, double est_scale, double ln_alpha,
             double ln_1m_alpha, int fuse, int mask_first) {
  extern __shared__ double smem[];
  double* lg = smem;                                // [U][4][n2]
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

  // blocks that start at or after the end of the segment are masked (line 13)
  const int visible = min(n2, ((j + 1) * seg + blk - 1) / blk);
  const T* kmx_base = Kmax + size_t(kvh) * n2 * D;
  const T* kmn_base = Kmin + size_t(kvh) * n2 * D;

  // The 8 x n2 x D logit products run on the fp64 tensor-core path (mma.m8n8k4): the 8 rows of
  // A are (head u, representative) = (u0 max, u0 min, u1 max, ...); B columns are key blocks.
  // Lane l supplies A[l/4][l%4] and B[l%4][l/4] per k-step and owns C[l/4][2(l%4)+{0,1}].
  // The channel order inside the dot product is free, so lane-in-quad q takes the D/4
  // contiguous channels [q*D/4, (q+1)*D/4): one contiguous slice of a summary row per lane.
  constexpr int KS = D / 4;                 // k-steps
  constexpr int VE = 16 / sizeof(T);        // elements per 16-byte load
  constexpr int NV = KS / VE;               // 16-byte loads per lane per row
  const int quad = lane & 3, grp = lane >> 2;
  double afrag[KS];
  {
    const int u = grp >> 1, rep = grp & 1;
    const T* src = (rep == 0 ? Qmax : Qmin) + (u < U ? unit_of(u) : unit_of(0)) * D + quad * KS;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) afrag[ks] = u < U ? to_f64(src[ks]) : 0.0;
  }
  const int n_tiles = (n2 + 7) / 8;
  for (int t = warp; t < n_tiles; t += kWarps) {
    const int bblk = min(t * 8 + grp, n2 - 1);          // this lane's B column (clamped in a ragged last tile)
    const uint4* pmx = reinterpret_cast<const uint4*>(kmx_base + size_t(bblk) * D + quad * KS);
    const uint4* pmn = reinterpret_cast<const uint4*>(kmn_base + size_t(bblk) * D + quad * KS);
    uint4 vx[NV], vn[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) { vx[v] = __ldg(pmx + v); vn[v] = __ldg(pmn + v); }
    double cx0 = 0.0, cx1 = 0.0, cn0 = 0.0, cn1 = 0.0;
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const T* ka = reinterpret_cast<const T*>(&vx[v]);
      const T* kc = reinterpret_cast<const T*>(&vn[v]);
#pragma unroll
      for (int e = 0; e < VE; ++e) {
        const double a = afrag[v * VE + e];
        const double bx = to_f64(ka[e]), bn = to_f64(kc[e]);
        asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                     : "+d"(cx0), "+d"(cx1) : "d"(a), "d"(bx));
        asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                     : "+d"(cn0), "+d"(cn1) : "d"(a), "d"(bn));
      }
    }
    // C rows: grp = (u, rep); rep 0 (Qmax): cx = l1, cn = l2; rep 1 (Qmin): cx = l3, cn = l4
    const int u = grp >> 1, rep = grp & 1;
    if (u < U) {
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int bb = t * 8 + quad * 2 + i;
        if (bb < n2) {
          const bool hide = mask_first && bb >= visible;
          lg[(u * 4 + rep * 2 + 0) * n2 + bb] = hide ? -CUDART_INF : (i ? cx1 : cx0) * est_scale;
          lg[(u * 4 + rep * 2 + 1) * n2 + bb] = hide ? -CUDART_INF : (i ? cn1 : cn0) * est_scale;
        }
      }
    }
  }
  __syncthreads();

  // log-sum-exp of each of the 4U logit rows (softmax over blocks, lines 9-10): a warp owns a
  // row, so only shuffles are needed; terms more than e^-50 below the maximum are skipped
#pragma unroll 1
  for (int rI = warp; rI < 4 * U; rI += kWarps) {
    const double* rowp = lg + rI * n2;
    double m = -CUDART_INF;
    for (int bb = lane; bb < n2; bb += 32) m = fmax(m, rowp[bb]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
    double sum = 0.0;
#pragma unroll 4
    for (int bb = lane; bb < n2; bb += 32) {
      const double d = rowp[bb] - m;
      if (d > -50.0) sum += exp(d);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) stat[rI] = m + log(sum);
  }
  __syncthreads();

  // combine (lines 11-12), mask (13), fusion (14) over the U rows of this CTA, flattened
  const double ln2 = 0.693147180559945309417232121458;
#pragma unroll 2
  for (int e = tid; e < U * n2; e += kThreads) {
    const int u = e / n2, bb = e - u * n2;
    double v;
    if (bb >= visible) {
      v = -CUDART_INF;
    } else {
      const double* l = lg + u * 4 * n2;
      const double L1 = l[bb] - stat[u * 4 + 0], L2 = l[n2 + bb] - stat[u * 4 + 1];
      const double L3 = l[2 * n2 + bb] - stat[u * 4 + 2], L4 = l[3 * n2 + bb] - stat[u * 4 + 3];
      const double Lmax = logaddexp(L1, L3) - ln2;   // ln (S1+S3)/2
      const double Lmin = logaddexp(L2, L4) - ln2;   // ln (S2+S4)/2
      v = fmax(Lmax, Lmin);
      if (fuse) v = logaddexp(ln_alpha + v, ln_1m_alpha + S_prev[unit_of(u) * n2 + bb]);
    }
    S_out[unit_of(u) * n2 + bb] = v;
  }
}

template <typename T, int D, int U>
int launch_u(const Dims& m, const char* ws, const WsLayout& w, const double* S_prev, double* S_out,
             double est_scale, double alpha, int fuse, int mask_first, cudaStream_t st) {
  const size_t smem = sizeof(double) * (4 * size_t(U) * m.n2);
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
  auto fits = [&](int U) { return m.g % U == 0 && sizeof(double) * (4 * size_t(U) * m.n2) <= budget; };
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

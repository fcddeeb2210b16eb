// K2: criticality scores from the representatives (Algorithm 1, lines 9-14), in fp64 and in
// the log domain.  One CTA handles one segment j for U query heads of the same KV group: the
// key summaries of the group are read and widened to fp64 once and used for all U heads.
// Per head it forms the four logit rows l1..l4 against every key block, their log-sum-exps, and
//   ln S = max( ln((S1+S3)/2), ln((S2+S4)/2) ),  mask,  ln(alpha S + (1-alpha) S').
// The representatives are exact in the input dtype, every product is exact in fp64, so this
// differs from an fp64 CPU evaluation only by summation order and libm rounding.
#include <cooperative_groups.h>
#include <math_constants.h>

#include "cp_common.cuh"

namespace cp {
namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;

template <typename T> __device__ __forceinline__ double to_f64(T x);
template <> __device__ __forceinline__ double to_f64<float>(float x) { return double(x); }
template <> __device__ __forceinline__ double to_f64<__nv_bfloat16>(__nv_bfloat16 x) { return double(__bfloat162float(x)); }
template <> __device__ __forceinline__ double to_f64<__half>(__half x) { return double(__half2float(x)); }

// ln(e^a + e^b).  When the smaller term is more than e^-50 below the larger one it cannot change
// the rounded result (|hi| is at most a few hundred here), so the transcendental pair is skipped.
__device__ __forceinline__ double logaddexp(double a, double b) {
  const double hi = fmax(a, b), lo = fmin(a, b);
  const double d = lo - hi;                 // <= 0, or NaN when both are -inf
  if (!(d > -50.0)) return hi;
  return hi + log1p(exp(d));
}

// Shared memory: logits lg[U][4][nb] for the nb key blocks this CTA owns.  When the 4*U*n2 logits
// of a row group do not fit one CTA's shared memory, CL CTAs of a thread-block cluster split the
// key blocks and merge their per-row (max, sum) pairs through distributed shared memory.
template <typename T, int D, int U>
__global__ void __launch_bounds__(kThreads)
score_kernel(const T* __restrict__ Qmax, const T* __restrict__ Qmin, const T* __restrict__ Kmax,
             const T* __restrict__ Kmin, const double* __restrict__ S_prev, double* __restrict__ S_out,
             int Hq, int g, int n1, int n2, int seg, int blk, double est_scale, double ln_alpha,
             double ln_1m_alpha, int fuse, int mask_first, int CL, int nb) {
  extern __shared__ double smem[];
  double* lg = smem;                                // [U][4][nb]
  __shared__ double stat[4 * U];
  __shared__ double2 part[4 * U];                   // this CTA's (max, sum exp) per logit row

  // cluster rank -> owned key blocks [b_lo, b_lo + nloc)
  const int rank = CL > 1 ? int(blockIdx.x % CL) : 0;
  const int b_lo = rank * nb;
  const int nloc = max(0, min(n2, b_lo + nb) - b_lo);

  // CTA -> (b, kv head, head subgroup, segment)
  const int groups = g / U;
  int x = blockIdx.x / CL;
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
  const int n_tiles = (nloc + 7) / 8;
  for (int t = warp; t < n_tiles; t += kWarps) {
    const int bblk = b_lo + min(t * 8 + grp, nloc - 1);  // this lane's B column (clamped in a ragged last tile)
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
        const int lb = t * 8 + quad * 2 + i;           // local block index
        if (lb < nloc) {
          const bool hide = mask_first && b_lo + lb >= visible;
          lg[(u * 4 + rep * 2 + 0) * nb + lb] = hide ? -CUDART_INF : (i ? cx1 : cx0) * est_scale;
          lg[(u * 4 + rep * 2 + 1) * nb + lb] = hide ? -CUDART_INF : (i ? cn1 : cn0) * est_scale;
        }
      }
    }
  }
  __syncthreads();

  // log-sum-exp of each of the 4U logit rows (softmax over blocks, lines 9-10): a warp owns a
  // row, so only shuffles are needed; terms more than e^-50 below the maximum are skipped
#pragma unroll 1
  for (int rI = warp; rI < 4 * U; rI += kWarps) {
    const double* rowp = lg + rI * nb;
    double m = -CUDART_INF;
    for (int lb = lane; lb < nloc; lb += 32) m = fmax(m, rowp[lb]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
    double sum = 0.0;
#pragma unroll 4
    for (int lb = lane; lb < nloc; lb += 32) {
      const double d = rowp[lb] - m;
      if (d > -50.0) sum += exp(d);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) part[rI] = make_double2(m, sum);
  }
  __syncthreads();
  if (CL > 1) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    cluster.sync();                                   // every CTA's partials are in place
    if (tid < 4 * U) {
      double M = -CUDART_INF;
      for (int r = 0; r < CL; ++r) M = fmax(M, cluster.map_shared_rank(part, r)[tid].x);
      double Ssum = 0.0;
      for (int r = 0; r < CL; ++r) {
        const double2 pr = cluster.map_shared_rank(part, r)[tid];
        if (pr.y > 0.0) Ssum += pr.y * exp(pr.x - M);
      }
      stat[tid] = M + log(Ssum);
    }
    cluster.sync();                                   // nobody leaves while its partials may still be read
  } else if (tid < 4 * U) {
    stat[tid] = part[tid].x + log(part[tid].y);
  }
  __syncthreads();

  // combine (lines 11-12), mask (13), fusion (14) over this CTA's blocks of the U rows, flattened
  const double ln2 = 0.693147180559945309417232121458;
#pragma unroll 2
  for (int e = tid; e < U * nloc; e += kThreads) {
    const int u = e / nloc, lb = e - u * nloc, bb = b_lo + lb;
    double v;
    if (bb >= visible) {
      v = -CUDART_INF;
    } else {
      const double* l = lg + u * 4 * nb;
      const double L1 = l[lb] - stat[u * 4 + 0], L2 = l[nb + lb] - stat[u * 4 + 1];
      const double L3 = l[2 * nb + lb] - stat[u * 4 + 2], L4 = l[3 * nb + lb] - stat[u * 4 + 3];
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
             double est_scale, double alpha, int fuse, int mask_first, int CL, int nb, cudaStream_t st) {
  const size_t smem = sizeof(double) * (4 * size_t(U) * nb);
  auto kern = score_kernel<T, D, U>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess)
    return CP_ERR_CUDA;
  const long long ctas = (long long)m.B * m.Hkv * (m.g / U) * m.n1 * CL;
  if (ctas > 0x7fffffffLL) return CP_ERR_UNSUPPORTED;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(ctas));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = unsigned(CL); attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = CL > 1 ? 1 : 0;
  const cudaError_t e = cudaLaunchKernelEx(
      &cfg, kern, reinterpret_cast<const T*>(ws + w.qmax), reinterpret_cast<const T*>(ws + w.qmin),
      reinterpret_cast<const T*>(ws + w.kmax), reinterpret_cast<const T*>(ws + w.kmin), S_prev, S_out,
      m.Hq, m.g, m.n1, m.n2, m.seg, m.blk, est_scale, log(alpha), log1p(-alpha), fuse, mask_first, CL, nb);
  return e == cudaSuccess ? check_launch() : CP_ERR_CUDA;
}

template <typename T, int D>
int launch_t(const Dims& m, const char* ws, const WsLayout& w, const double* S_prev, double* S_out,
             double est_scale, double alpha, int fuse, int mask_first, cudaStream_t st) {
  // as many heads per CTA as divide the group (the fp64 MMA has 8 rows = 4 heads x 2 representatives);
  // key blocks are split over a cluster of 1, 2, 4 or 8 CTAs until the logits fit ~200 KB per CTA
  const size_t budget = 200 * 1024;
  const int U = m.g % 4 == 0 ? 4 : (m.g % 2 == 0 ? 2 : 1);
  for (int CL = 1; CL <= 8; CL *= 2) {
    const int nb = (((m.n2 + CL - 1) / CL) + 7) & ~7;
    if (sizeof(double) * 4 * size_t(U) * nb > budget) continue;
    if (U == 4) return launch_u<T, D, 4>(m, ws, w, S_prev, S_out, est_scale, alpha, fuse, mask_first, CL, nb, st);
    if (U == 2) return launch_u<T, D, 2>(m, ws, w, S_prev, S_out, est_scale, alpha, fuse, mask_first, CL, nb, st);
    return launch_u<T, D, 1>(m, ws, w, S_prev, S_out, est_scale, alpha, fuse, mask_first, CL, nb, st);
  }
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
  } else if (p.dtype == CP_F16) {
    if (m.d == 128) return launch_t<__half, 128>(m, ws, w, S_prev, S_out, es, al, fuse, mask_first, st);
    if (m.d == 64) return launch_t<__half, 64>(m, ws, w, S_prev, S_out, es, al, fuse, mask_first, st);
  } else {
    if (m.d == 128) return launch_t<float, 128>(m, ws, w, S_prev, S_out, es, al, fuse, mask_first, st);
    if (m.d == 64) return launch_t<float, 64>(m, ws, w, S_prev, S_out, es, al, fuse, mask_first, st);
  }
  return CP_ERR_UNSUPPORTED;
}

}  // namespace cp

// K1: per-channel max / min over the tokens of each query segment and each key block
// (Algorithm 1, lines 3-8).  Pure HBM scan: 16-byte loads, comparisons only, results exact
// in the input dtype.
//
// One launch covers Q (groups of `seg` rows) and K (groups of `blk` rows).  A row of d
// elements is read by LPR = d*es/16 neighbouring lanes, so a warp covers 32/LPR rows per
// load instruction.  Groups of <= 128 rows are owned by one warp; larger groups by a whole
// CTA whose warps stride over the rows and combine through shared memory.
#include "cp_common.cuh"

namespace cp {
namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;

template <typename T> struct Vec;
template <> struct Vec<__nv_bfloat16> {
  uint4 v;
  static constexpr uint32_t kNegInf = 0xFF80FF80u, kPosInf = 0x7F807F80u;   // packed pairs
  __device__ static Vec load(const void* p) { Vec r; r.v = __ldg(reinterpret_cast<const uint4*>(p)); return r; }
  __device__ void store(void* p) const { *reinterpret_cast<uint4*>(p) = v; }
  __device__ static uint32_t mx(uint32_t a, uint32_t b) {
    __nv_bfloat162 r = __hmax2(*reinterpret_cast<__nv_bfloat162*>(&a), *reinterpret_cast<__nv_bfloat162*>(&b));
    return *reinterpret_cast<uint32_t*>(&r);
  }
  __device__ static uint32_t mn(uint32_t a, uint32_t b) {
    __nv_bfloat162 r = __hmin2(*reinterpret_cast<__nv_bfloat162*>(&a), *reinterpret_cast<__nv_bfloat162*>(&b));
    return *reinterpret_cast<uint32_t*>(&r);
  }
};
template <> struct Vec<__half> {
  uint4 v;
  static constexpr uint32_t kNegInf = 0xFC00FC00u, kPosInf = 0x7C007C00u;
  __device__ static Vec load(const void* p) { Vec r; r.v = __ldg(reinterpret_cast<const uint4*>(p)); return r; }
  __device__ void store(void* p) const { *reinterpret_cast<uint4*>(p) = v; }
  __device__ static uint32_t mx(uint32_t a, uint32_t b) {
    __half2 r = __hmax2(*reinterpret_cast<__half2*>(&a), *reinterpret_cast<__half2*>(&b));
    return *reinterpret_cast<uint32_t*>(&r);
  }
  __device__ static uint32_t mn(uint32_t a, uint32_t b) {
    __half2 r = __hmin2(*reinterpret_cast<__half2*>(&a), *reinterpret_cast<__half2*>(&b));
    return *reinterpret_cast<uint32_t*>(&r);
  }
};
template <> struct Vec<float> {
  uint4 v;
  static constexpr uint32_t kNegInf = 0xFF800000u, kPosInf = 0x7F800000u;
  __device__ static Vec load(const void* p) { Vec r; r.v = __ldg(reinterpret_cast<const uint4*>(p)); return r; }
  __device__ void store(void* p) const { *reinterpret_cast<uint4*>(p) = v; }
  __device__ static uint32_t mx(uint32_t a, uint32_t b) { return __float_as_uint(fmaxf(__uint_as_float(a), __uint_as_float(b))); }
  __device__ static uint32_t mn(uint32_t a, uint32_t b) { return __float_as_uint(fminf(__uint_as_float(a), __uint_as_float(b))); }
};

// largest magnitude among the elements of a 16-byte vector
template <typename T> __device__ __forceinline__ float vec_absmax(const uint4& a);
template <> __device__ __forceinline__ float vec_absmax<float>(const uint4& a) {
  return fmaxf(fmaxf(fabsf(__uint_as_float(a.x)), fabsf(__uint_as_float(a.y))), fmaxf(fabsf(__uint_as_float(a.z)), fabsf(__uint_as_float(a.w))));
}
template <> __device__ __forceinline__ float vec_absmax<__nv_bfloat16>(const uint4& a) {
  const uint32_t w[4] = {a.x, a.y, a.z, a.w};
  float m = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {   // a bf16 is the upper half of a float
    m = fmaxf(m, fabsf(__uint_as_float(w[i] << 16)));
    m = fmaxf(m, fabsf(__uint_as_float(w[i] & 0xffff0000u)));
  }
  return m;
}
template <> __device__ __forceinline__ float vec_absmax<__half>(const uint4& a) {
  const uint32_t w[4] = {a.x, a.y, a.z, a.w};
  float m = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
    m = fmaxf(m, fmaxf(fabsf(f.x), fabsf(f.y)));
  }
  return m;
}
// largest magnitude of a group's summaries: every lane holds the group's (max, min) slice of column slot lane % LPR
template <typename T, int LPR>
__device__ __forceinline__ float group_absmax(const uint4& mx, const uint4& mn) {
  float m = fmaxf(vec_absmax<T>(mx), vec_absmax<T>(mn));
#pragma unroll
  for (int o = 1; o < LPR; o <<= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  return m;
}

template <typename T>
__device__ __forceinline__ void vmax(uint4& a, const uint4& b) {
  a.x = Vec<T>::mx(a.x, b.x); a.y = Vec<T>::mx(a.y, b.y); a.z = Vec<T>::mx(a.z, b.z); a.w = Vec<T>::mx(a.w, b.w);
}
template <typename T>
__device__ __forceinline__ void vmin(uint4& a, const uint4& b) {
  a.x = Vec<T>::mn(a.x, b.x); a.y = Vec<T>::mn(a.y, b.y); a.z = Vec<T>::mn(a.z, b.z); a.w = Vec<T>::mn(a.w, b.w);
}
__device__ __forceinline__ uint4 shfl_xor4(const uint4& a, int m) {
  uint4 r;
  r.x = __shfl_xor_sync(0xffffffffu, a.x, m); r.y = __shfl_xor_sync(0xffffffffu, a.y, m);
  r.z = __shfl_xor_sync(0xffffffffu, a.z, m); r.w = __shfl_xor_sync(0xffffffffu, a.w, m);
  return r;
}

struct Side {            // one tensor (Q or K) and where its summaries go
  const char* base;      // element (b,h,t,0) at base + (b*sb + h*sh + t*st) * es
  int64_t sb, sh, st;    // strides in elements
  int H, groups_per_head, G, n;  // heads, groups per head (ceil(n/G)), rows per group (the last may be shorter), tokens
  char *omax, *omin;     // [B,H,groups,d] contiguous
  float* oabs;           // nullable, [B,H,groups]: largest magnitude in the group's summaries
  long long n_groups;    // B*H*groups_per_head
  long long cta_begin;   // first CTA of this side
  int groups_per_cta;    // kWarps (warp-owned groups) or 1 (CTA-owned group)
};

// Fold rows first+sub, first+sub+step, ... (< first+nrows) of a group into the lane's 16-byte
// slice of (max, min).  The accumulators start at -inf / +inf, so a lane without rows is neutral.
template <typename T, int LPR>
__device__ __forceinline__ void scan_rows(const char* gbase, int64_t st_bytes, int first, int nrows,
                                          int step, int lane, uint4& mx, uint4& mn) {
  const int sub = lane / LPR, col = lane % LPR;
  const char* p0 = gbase + int64_t(first + sub) * st_bytes + col * 16;
  mx = make_uint4(Vec<T>::kNegInf, Vec<T>::kNegInf, Vec<T>::kNegInf, Vec<T>::kNegInf);
  mn = make_uint4(Vec<T>::kPosInf, Vec<T>::kPosInf, Vec<T>::kPosInf, Vec<T>::kPosInf);
  constexpr int UNROLL = 8;
  int i = first + sub;
  const int end = first + nrows;
  for (; i + (UNROLL - 1) * step < end; i += UNROLL * step) {
    uint4 v[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) v[u] = Vec<T>::load(p0 + int64_t(i - first - sub + u * step) * st_bytes).v;
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) { vmax<T>(mx, v[u]); vmin<T>(mn, v[u]); }
  }
  for (; i < end; i += step) {
    const uint4 v = Vec<T>::load(p0 + int64_t(i - first - sub) * st_bytes).v;
    vmax<T>(mx, v); vmin<T>(mn, v);
  }
}

template <typename T, int LPR>
__global__ void __launch_bounds__(kThreads) summarize_kernel(Side q, Side k, int d) {
  __shared__ uint4 red[2][kWarps][LPR];
  const Side& s = (blockIdx.x >= k.cta_begin) ? k : q;
  const long long cta = blockIdx.x - s.cta_begin;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int RPW = 32 / LPR;
  const int es = sizeof(T);
  const int64_t st_bytes = s.st * es;

  if (s.groups_per_cta == 1) {
    // a CTA owns the group; its warps take rows warp*RPW + sub, stride kWarps*RPW
    const long long grp = cta;
    const int gi = int(grp % s.groups_per_head);
    const long long bh = grp / s.groups_per_head;
    const int h = int(bh % s.H), b = int(bh / s.H);
    const char* gbase = s.base + (int64_t(b) * s.sb + int64_t(h) * s.sh + int64_t(gi) * s.G * s.st) * es;
    const int rows = min(s.G, s.n - gi * s.G);
    uint4 mx, mn;
    scan_rows<T, LPR>(gbase, st_bytes, warp * RPW, rows - warp * RPW, kWarps * RPW, lane, mx, mn);
#pragma unroll
    for (int m = LPR; m < 32; m <<= 1) { uint4 o = shfl_xor4(mx, m); vmax<T>(mx, o); o = shfl_xor4(mn, m); vmin<T>(mn, o); }
    if (lane < LPR) { red[0][warp][lane] = mx; red[1][warp][lane] = mn; }
    __syncthreads();
    if (warp == 0) {
      const int col = lane % LPR;
      mx = red[0][0][col]; mn = red[1][0][col];
#pragma unroll
      for (int w = 1; w < kWarps; ++w) { vmax<T>(mx, red[0][w][col]); vmin<T>(mn, red[1][w][col]); }
      if (lane < LPR) {
        const size_t off = (size_t(grp) * d) * es + lane * 16;
        *reinterpret_cast<uint4*>(s.omax + off) = mx;
        *reinterpret_cast<uint4*>(s.omin + off) = mn;
      }
      if (s.oabs != nullptr) {
        const float am = group_absmax<T, LPR>(mx, mn);
        if (lane == 0) s.oabs[grp] = am;
      }
    }
  } else {
    // each warp owns one group of G <= 128 rows
    const long long grp = cta * kWarps + warp;
    if (grp >= s.n_groups) return;
    const int gi = int(grp % s.groups_per_head);
    const long long bh = grp / s.groups_per_head;
    const int h = int(bh % s.H), b = int(bh / s.H);
    const char* gbase = s.base + (int64_t(b) * s.sb + int64_t(h) * s.sh + int64_t(gi) * s.G * s.st) * es;
    const int rows = min(s.G, s.n - gi * s.G);
    uint4 mx, mn;
    scan_rows<T, LPR>(gbase, st_bytes, 0, rows, RPW, lane, mx, mn);
#pragma unroll
    for (int m = LPR; m < 32; m <<= 1) { uint4 o = shfl_xor4(mx, m); vmax<T>(mx, o); o = shfl_xor4(mn, m); vmin<T>(mn, o); }
    if (lane < LPR) {
      const size_t off = (size_t(grp) * d) * es + lane * 16;
      *reinterpret_cast<uint4*>(s.omax + off) = mx;
      *reinterpret_cast<uint4*>(s.omin + off) = mn;
    }
    if (s.oabs != nullptr) {
      const float am = group_absmax<T, LPR>(mx, mn);
      if (lane == 0) s.oabs[grp] = am;
    }
  }
}

template <typename T, int LPR>
int launch_t(const Side& q, const Side& k, long long ctas, int d, cudaStream_t st) {
  summarize_kernel<T, LPR><<<(unsigned)ctas, kThreads, 0, st>>>(q, k, d);
  return check_launch();
}

}  // namespace

int launch_summarize(const cp_params& p, const Dims& m, const void* Q, const void* K, char* ws,
                     cudaStream_t st) {
  const WsLayout w = ws_layout(m);
  auto mk = [&](const void* base, const int64_t* s, int H, int G, char* omax, char* omin) {
    Side x;
    x.base = static_cast<const char*>(base); x.sb = s[0]; x.sh = s[1]; x.st = s[2];
    x.H = H; x.G = G; x.n = m.n; x.groups_per_head = (m.n + G - 1) / G; x.omax = omax; x.omin = omin; x.oabs = nullptr;
    x.n_groups = (long long)m.B * H * x.groups_per_head;
    x.groups_per_cta = G > 128 ? 1 : kWarps;
    x.cta_begin = 0;
    return x;
  };
  Side q = mk(Q, p.q_stride, m.Hq, m.seg, ws + w.qmax, ws + w.qmin);
  Side k = mk(K, p.k_stride, m.Hkv, m.blk, ws + w.kmax, ws + w.kmin);
  if (Q == nullptr) q.n_groups = 0;          // key side only (the caller supplies the query representatives itself)
  k.oabs = reinterpret_cast<float*>(ws + w.kabs);
  const long long q_ctas = (q.n_groups + q.groups_per_cta - 1) / q.groups_per_cta;
  const long long k_ctas = (k.n_groups + k.groups_per_cta - 1) / k.groups_per_cta;
  k.cta_begin = q_ctas;
  const long long ctas = q_ctas + k_ctas;
  if (ctas > 0x7fffffffLL) return CP_ERR_UNSUPPORTED;
  const int lpr = m.d * m.es / 16;
  if (p.dtype == CP_BF16) {
    if (lpr == 16) return launch_t<__nv_bfloat16, 16>(q, k, ctas, m.d, st);
    if (lpr == 8) return launch_t<__nv_bfloat16, 8>(q, k, ctas, m.d, st);
  } else if (p.dtype == CP_F16) {
    if (lpr == 16) return launch_t<__half, 16>(q, k, ctas, m.d, st);
    if (lpr == 8) return launch_t<__half, 8>(q, k, ctas, m.d, st);
  } else {
    if (lpr == 32) return launch_t<float, 32>(q, k, ctas, m.d, st);
    if (lpr == 16) return launch_t<float, 16>(q, k, ctas, m.d, st);
  }
  return CP_ERR_UNSUPPORTED;
}

}  // namespace cp

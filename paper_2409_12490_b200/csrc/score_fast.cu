// K2 for 16-bit inputs with head_dim 128 (Algorithm 1, lines 9-14), split in two kernels:
//   lse (see lse_sm100.cu / the general kernel)  the four log-sum-exps of every (head, segment) row, which need every
//        key block of the row but only to the accuracy with which a term can still change the sum, and
//   score_visible_kernel (this file)  the exact fp64 logits of the blocks a segment can see, combined
//        straight out of the MMA accumulators:  ln S = max( ln((S1+S3)/2), ln((S2+S4)/2) ), fusion with S'.
// Blocks that start at or after the end of the segment are masked by line 13 whatever their logits, so the
// exact fp64 products -- the cost of this step -- are spent on the visible half of the map only.
#include "score_common.cuh"

namespace cp {
namespace {

constexpr int kThreads = 256;   // 8 warps x <= 85 registers: three CTAs per SM, so a CTA's set-up and tile epilogues run under the others' MMAs
constexpr int kWarps = kThreads / 32;
#ifndef CP_SCORE_FAST_MIN
#define CP_SCORE_FAST_MIN 3000000
#endif
constexpr long long kFastMinScores = CP_SCORE_FAST_MIN;   // (batch x heads x segments x blocks) from which the two-kernel path is used
constexpr int kG = 4;                       // segments per CTA: one MMA column group = 4 segments x {Qmax, Qmin} of one head

// One CTA: G = 4 consecutive segments x U query heads of one KV group.  The fp64 MMA m16n8k16 runs with 16 key
// blocks on the M side (streamed from the summaries, widened to fp64 once and used for all 4*U segment-head
// pairs) and, on the N side, the 8 columns (segment s, representative) = (s0 max, s0 min, s1 max, ...) of one
// head.  Lane (grp = lane/4, tig = lane%4) then owns, for head u, segment tig and the two blocks grp, grp+8,
// all four logits l1..l4 in its accumulators (Kmax product: cx, Kmin product: cn; even element: Qmax, odd:
// Qmin) and finishes the element without shared memory.
template <typename T, int D, int U>
__global__ void __launch_bounds__(kThreads, 3)
score_visible_kernel(const T* __restrict__ Qmax, const T* __restrict__ Qmin, const T* __restrict__ Kmax,
                     const T* __restrict__ Kmin, const double* __restrict__ stats, const double* __restrict__ S_prev,
                     double* __restrict__ S_out, int Hq, int g, int n1, int n2, int seg, int blk, double est_scale,
                     double ln_alpha, double ln_1m_alpha, int fuse, int n_chunks) {
  constexpr int KS = D / 4;                 // channels per lane slice (lane tig owns channels [tig*KS, (tig+1)*KS))
  constexpr int CE = 16 / sizeof(T);        // elements per 16-byte load
  constexpr int NCH = KS / CE;              // loads per slice
  constexpr int SPC = CE / 4;               // MMA k-steps per load
  constexpr int QS = D + 2;                 // row stride of qs in doubles (odd number of 16-byte units: conflict-free)
  __shared__ __align__(16) double qs[U * 8 * QS];   // B operand: row = (head u, column c = 2*s + rep), [k-step][tig][4 channels]
  __shared__ double st_sh[U * kG * 4];              // log-sum-exps of the (head, segment) rows of this CTA
  __shared__ double sp_tab[kSpIntervals * kSpStride];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tig = lane & 3, grp = lane >> 2;
  // CTA -> (chunk of 4 segments, b, kv head, head subgroup); the chunks with the most visible blocks go first
  const int groups = g / U;
  int x = blockIdx.x;
  const int per_chunk = gridDim.x / n_chunks;
  const int chunk = n_chunks - 1 - x / per_chunk; x %= per_chunk;
  const int sub = x % groups; x /= groups;
  const int kvh = x;                                 // b*Hkv + kv head
  const int Hkv = Hq / g;
  const int b = kvh / Hkv;
  const int h0 = (kvh % Hkv) * g + sub * U;          // first query head of this CTA
  const int j0 = chunk * kG;
  auto unit_of = [&](int u, int s) { return (size_t(b) * Hq + h0 + u) * n1 + j0 + s; };
  auto visible_of = [&](int j) { return min(n2, ((j + 1) * seg + blk - 1) / blk); };   // first masked block of segment j
  const int n_seg = min(kG, n1 - j0);                // segments of this chunk that exist
  const int vis_hi = visible_of(j0 + n_seg - 1);

  for (int e = tid; e < kSpIntervals * kSpCoef; e += kThreads)
    sp_tab[(e / kSpCoef) * kSpStride + e % kSpCoef] = kSoftplusTable[e];
  for (int e = tid; e < U * kG * 4; e += kThreads) {
    const int u = e / (kG * 4), s = (e / 4) % kG;
    st_sh[e] = s < n_seg ? stats[unit_of(u, s) * 4 + (e & 3)] : 0.0;
  }
  for (int e = tid; e < U * 8 * D; e += kThreads) {
    const int row = e / D, ch = e % D;               // row = u*8 + s*2 + rep
    const int u = row >> 3, s = (row >> 1) & 3, rep = row & 1;
    const int tq = ch / KS, within = ch % KS;        // owner lane-in-quad, position in its slice
    const double v = s < n_seg ? to_f64(((rep == 0 ? Qmax : Qmin) + unit_of(u, s) * D)[ch]) : 0.0;
    qs[row * QS + ((within >> 2) * 4 + tq) * 4 + (within & 3)] = v;
  }
  // blocks at or after the end of a segment: -inf (line 13)
  for (int r = warp; r < U * n_seg; r += kWarps) {
    const int u = r / n_seg, s = r % n_seg;
    double* row = S_out + unit_of(u, s) * n2;
    for (int bb = visible_of(j0 + s) + lane; bb < n2; bb += 32) row[bb] = -CUDART_INF;
  }
  __syncthreads();

  const T* kmx_base = Kmax + size_t(kvh) * n2 * D;
  const T* kmn_base = Kmin + size_t(kvh) * n2 * D;
  const int my_vis = tig < n_seg ? visible_of(j0 + tig) : 0;     // this lane's segment
  const double ln2 = 0.693147180559945309417232121458;
  const int n_tiles = (vis_hi + 15) / 16;
  for (int t = warp; t < n_tiles; t += kWarps) {
    const int blk0 = min(t * 16 + grp, n2 - 1), blk1 = min(t * 16 + grp + 8, n2 - 1);   // clamped in a ragged last tile
    const uint4* src[4] = {reinterpret_cast<const uint4*>(kmx_base + size_t(blk0) * D + tig * KS),
                           reinterpret_cast<const uint4*>(kmx_base + size_t(blk1) * D + tig * KS),
                           reinterpret_cast<const uint4*>(kmn_base + size_t(blk0) * D + tig * KS),
                           reinterpret_cast<const uint4*>(kmn_base + size_t(blk1) * D + tig * KS)};
    double cx[U][4], cn[U][4];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int i = 0; i < 4; ++i) { cx[u][i] = 0.0; cn[u][i] = 0.0; }
    uint4 cur[4], nxt[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) cur[i] = __ldg(src[i]);
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) {
      if (ch + 1 < NCH) {
#pragma unroll
        for (int i = 0; i < 4; ++i) nxt[i] = __ldg(src[i] + ch + 1);
      }
#pragma unroll
      for (int sp = 0; sp < SPC; ++sp) {
        const int step = ch * SPC + sp;
        double ax[8], an[8];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          ax[2 * c] = to_f64(reinterpret_cast<const T*>(&cur[0])[sp * 4 + c]);
          ax[2 * c + 1] = to_f64(reinterpret_cast<const T*>(&cur[1])[sp * 4 + c]);
          an[2 * c] = to_f64(reinterpret_cast<const T*>(&cur[2])[sp * 4 + c]);
          an[2 * c + 1] = to_f64(reinterpret_cast<const T*>(&cur[3])[sp * 4 + c]);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const double* qrow = &qs[(u * 8 + grp) * QS + (step * 4 + tig) * 4];
          const double2 b01 = *reinterpret_cast<const double2*>(qrow);
          const double2 b23 = *reinterpret_cast<const double2*>(qrow + 2);
          asm volatile(
              "mma.sync.aligned.m16n8k16.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5,%6,%7,%8,%9,%10,%11}, "
              "{%12,%13,%14,%15}, {%0,%1,%2,%3};"
              : "+d"(cx[u][0]), "+d"(cx[u][1]), "+d"(cx[u][2]), "+d"(cx[u][3])
              : "d"(ax[0]), "d"(ax[1]), "d"(ax[2]), "d"(ax[3]), "d"(ax[4]), "d"(ax[5]), "d"(ax[6]), "d"(ax[7]),
                "d"(b01.x), "d"(b01.y), "d"(b23.x), "d"(b23.y));
          asm volatile(
              "mma.sync.aligned.m16n8k16.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5,%6,%7,%8,%9,%10,%11}, "
              "{%12,%13,%14,%15}, {%0,%1,%2,%3};"
              : "+d"(cn[u][0]), "+d"(cn[u][1]), "+d"(cn[u][2]), "+d"(cn[u][3])
              : "d"(an[0]), "d"(an[1]), "d"(an[2]), "d"(an[3]), "d"(an[4]), "d"(an[5]), "d"(an[6]), "d"(an[7]),
                "d"(b01.x), "d"(b01.y), "d"(b23.x), "d"(b23.y));
        }
      }
      if (ch + 1 < NCH) {
#pragma unroll
        for (int i = 0; i < 4; ++i) cur[i] = nxt[i];
      }
    }
    // C[i]: block grp + 8*(i/2), column 2*tig + (i%2) = (segment tig, representative i%2).
    // Qmax columns: cx = l1, cn = l2; Qmin columns: cx = l3, cn = l4.
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const double* stp = &st_sh[(u * kG + tig) * 4];
      const double st1 = stp[0], st2 = stp[1], st3 = stp[2], st4 = stp[3];
      const size_t out_row = unit_of(u, tig) * n2;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int bb = t * 16 + grp + half * 8;
        if (bb < my_vis) {
          const double L1 = cx[u][2 * half] * est_scale - st1, L2 = cn[u][2 * half] * est_scale - st2;
          const double L3 = cx[u][2 * half + 1] * est_scale - st3, L4 = cn[u][2 * half + 1] * est_scale - st4;
          // max( ln (S1+S3)/2, ln (S2+S4)/2 ).  ln(e^a + e^b) lies in [max(a,b), max(a,b) + ln 2], so the pair with the
          // larger maximum wins outright unless the two maxima are within ln 2 of each other: one evaluation, rarely two.
          const double h13 = fmax(L1, L3), h24 = fmax(L2, L4);
          const bool first = h13 >= h24;
          double v = logaddexp(first ? L1 : L2, first ? L3 : L4, sp_tab);
          if (fabs(h13 - h24) < ln2) v = fmax(v, logaddexp(first ? L2 : L1, first ? L4 : L3, sp_tab));
          v -= ln2;
          if (fuse) v = logaddexp(ln_alpha + v, ln_1m_alpha + S_prev[out_row + bb], sp_tab);
          S_out[out_row + bb] = v;
        }
      }
    }
  }
}

template <typename T, int U>
int launch_visible(const Dims& m, const char* ws, const WsLayout& w, const double* S_prev, double* S_out,
                   double est_scale, double alpha, int fuse, cudaStream_t st) {
  const int n_chunks = (m.n1 + kG - 1) / kG;
  const long long ctas = (long long)m.B * m.Hkv * (m.g / U) * n_chunks;
  if (ctas > 0x7fffffffLL) return CP_ERR_UNSUPPORTED;
  score_visible_kernel<T, 128, U><<<unsigned(ctas), kThreads, 0, st>>>(
      reinterpret_cast<const T*>(ws + w.qmax), reinterpret_cast<const T*>(ws + w.qmin),
      reinterpret_cast<const T*>(ws + w.kmax), reinterpret_cast<const T*>(ws + w.kmin),
      reinterpret_cast<const double*>(ws + w.stats), S_prev, S_out, m.Hq, m.g, m.n1, m.n2, m.seg, m.blk, est_scale,
      log(alpha), log1p(-alpha), fuse, n_chunks);
  return check_launch();
}

template <typename T>
int launch_visible_t(const Dims& m, const char* ws, const WsLayout& w, const double* S_prev, double* S_out,
                     double est_scale, double alpha, int fuse, cudaStream_t st) {
  // One head per CTA: 80 registers, three CTAs of 8 warps per SM.  More heads per CTA amortise the widening of the A operand
  // over more MMAs but leave fewer CTAs to overlap (measured at n2 = 4096: U = 4 with one CTA of 12 warps 0.69 ms, U = 2 with two
  // CTAs 0.65 ms, U = 1 with three 0.62 ms; four CTAs at 64 registers spill and gain nothing).
  return launch_visible<T, 1>(m, ws, w, S_prev, S_out, est_scale, alpha, fuse, st);
}

}  // namespace

// K2 dispatcher.  16-bit inputs with head_dim 128 take the two-kernel path (log-sum-exps, then exact logits of
// the visible blocks); everything else the general kernel.
int launch_score(const cp_params& p, const Dims& m, char* ws, const double* S_prev, double* S_out, cudaStream_t st) {
  // The two-kernel path pays for an extra launch and for the serial sweeps of the log-sum-exp kernel; it wins once the
  // score map is large (measured: 2x at 33 M scores, nothing below a few million), so small maps keep the general kernel.
  const long long scores = (long long)m.B * m.Hq * m.n1 * m.n2;
  const bool fast = (p.dtype == CP_BF16 || p.dtype == CP_F16) && m.d == 128 &&
                    (scores >= kFastMinScores || (p.flags & CP_FLAG_FORCE_SPLIT_SCORE));
  if (!fast) return launch_score_generic(p, m, ws, S_prev, S_out, nullptr, st);
  const WsLayout w = ws_layout(m);
  int rc = launch_lse(p, m, ws, st);
  if (rc != CP_OK) return rc;
  const int fuse = (S_prev != nullptr && p.alpha != 1.0f) ? 1 : 0;
  const double es = double(p.est_scale), al = double(p.alpha);
  if (p.dtype == CP_BF16) return launch_visible_t<__nv_bfloat16>(m, ws, w, S_prev, S_out, es, al, fuse, st);
  return launch_visible_t<__half>(m, ws, w, S_prev, S_out, es, al, fuse, st);
}

}  // namespace cp

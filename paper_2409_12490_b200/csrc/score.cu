// K2: criticality scores from the representatives (Algorithm 1, lines 9-14), in fp64 and in
// the log domain.  One CTA handles one segment j for U query heads of the same KV group: the
// key summaries of the group are read and widened to fp64 once and used for all U heads.
// Per head it forms the four logit rows l1..l4 against every key block, their log-sum-exps, and
//   ln S = max( ln((S1+S3)/2), ln((S2+S4)/2) ),  mask,  ln(alpha S + (1-alpha) S').
// The representatives are exact in the input dtype and every product is exact in fp64, so this differs
// from an fp64 CPU evaluation only by summation order, libm rounding and the 1e-15 of the ln(1 + e^-x) table.
#include <cooperative_groups.h>
#include <math_constants.h>

#include "score_common.cuh"

namespace cp {
namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;

// Shared memory: logits lg[U][4][nb] (fp64) for the nb key blocks this CTA owns, plus an fp32 copy that
// the log-sum-exp uses as a filter.  When the 4*U*n2 logits of a row group do not fit one CTA's shared
// memory, CL CTAs of a thread-block cluster split the key blocks and merge their per-row (max, sum)
// pairs through distributed shared memory.
template <typename T, int D, int U>
__global__ void __launch_bounds__(kThreads)
score_kernel(const T* __restrict__ Qmax, const T* __restrict__ Qmin, const T* __restrict__ Kmax,
             const T* __restrict__ Kmin, const double* __restrict__ S_prev, double* __restrict__ S_out,
             int Hq, int g, int n1, int n2, int seg, int blk, double est_scale, double ln_alpha,
             double ln_1m_alpha, int fuse, int mask_first, int CL, int nb, double* __restrict__ stats_out) {
  extern __shared__ double smem[];
  double* lg = smem;                                // [U][4][nb]
  float* lf = reinterpret_cast<float*>(smem + 4 * U * nb);   // the same logits rounded to fp32: a cheap filter for the log-sum-exp
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

  // The 8 x n2 x D logit products run on the fp64 tensor cores as mma.m16n8k16 with the key blocks on the
  // M side: per warp tile, A = 16 key blocks x 16 channels (streamed from the summaries, widened to fp64),
  // B = 16 channels x 8 columns, the columns being (head u, representative) = (u0 max, u0 min, u1 max, ...),
  // C = 16 blocks x 8 columns.  Lane (grp = lane/4, tig = lane%4) supplies A[grp | grp+8][c*4+tig],
  // B[i*4+tig][grp] and owns C[grp | grp+8][2*tig + {0,1}].  The channel order inside a dot product is
  // free, so lane tig takes the D/4 contiguous channels [tig*D/4, (tig+1)*D/4) of a summary row, four of
  // them per MMA: 16-byte loads, and each key value is converted once per CTA.
  constexpr int KS = D / 4;                 // channels per lane slice
  constexpr int CE = 16 / sizeof(T);        // elements per 16-byte load
  constexpr int NCH = KS / CE;              // loads per slice
  constexpr int SPC = CE / 4;               // MMA k-steps per load
  constexpr int QS = D + 2;                 // row stride of qs in doubles (odd number of 16-byte units: conflict-free)
  __shared__ __align__(16) double qs[8 * QS];   // B operand, row = column index n, laid out [k-step][tig][4 channels]
  __shared__ double sp_tab[kSpIntervals * kSpStride];
  for (int e = threadIdx.x; e < kSpIntervals * kSpCoef; e += kThreads)
    sp_tab[(e / kSpCoef) * kSpStride + e % kSpCoef] = kSoftplusTable[e];
  const int tig = lane & 3, grp = lane >> 2;
  if (fuse && (lane & 15) == 0) {
    // the previous layer's scores of this CTA's elements are read once, at the very end: start them towards L2 now
    for (int u = 0; u < U; ++u)
      for (int lb = tid; lb < nloc && b_lo + lb < visible; lb += kThreads)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(S_prev + unit_of(u) * n2 + b_lo + lb));
  }
  for (int e = tid; e < 8 * D; e += kThreads) {
    const int n = e / D, ch = e % D;        // column n = (head n/2, representative n%2); channel ch
    const int u = n >> 1, rep = n & 1;
    const int tq = ch / KS, within = ch % KS;                         // owner lane-in-quad, position in its slice
    const double v = u < U ? to_f64(((rep == 0 ? Qmax : Qmin) + unit_of(u) * D)[ch]) : 0.0;
    qs[n * QS + ((within >> 2) * 4 + tq) * 4 + (within & 3)] = v;
  }
  __syncthreads();
  const int n_tiles = (nloc + 15) / 16;
  for (int t = warp; t < n_tiles; t += kWarps) {
    if (mask_first && b_lo + t * 16 >= visible) {
      // normalising over the visible blocks only: a tile of future blocks needs no products at all
      for (int e = lane; e < 4 * U * 16; e += 32) {
        const int lb = t * 16 + (e & 15);
        if (lb < nloc) { lg[(e >> 4) * nb + lb] = -CUDART_INF; lf[(e >> 4) * nb + lb] = -CUDART_INF_F; }
      }
      continue;
    }
    // this lane's two A rows (clamped in a ragged last tile), for the max and the min summaries
    const int blk0 = b_lo + min(t * 16 + grp, nloc - 1), blk1 = b_lo + min(t * 16 + grp + 8, nloc - 1);
    const uint4* src[4] = {reinterpret_cast<const uint4*>(kmx_base + size_t(blk0) * D + tig * KS),
                           reinterpret_cast<const uint4*>(kmx_base + size_t(blk1) * D + tig * KS),
                           reinterpret_cast<const uint4*>(kmn_base + size_t(blk0) * D + tig * KS),
                           reinterpret_cast<const uint4*>(kmn_base + size_t(blk1) * D + tig * KS)};
    double cx[4] = {0.0, 0.0, 0.0, 0.0}, cn[4] = {0.0, 0.0, 0.0, 0.0};
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
        const double2 b01 = *reinterpret_cast<const double2*>(&qs[grp * QS + (step * 4 + tig) * 4]);
        const double2 b23 = *reinterpret_cast<const double2*>(&qs[grp * QS + (step * 4 + tig) * 4 + 2]);
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5,%6,%7,%8,%9,%10,%11}, "
            "{%12,%13,%14,%15}, {%0,%1,%2,%3};"
            : "+d"(cx[0]), "+d"(cx[1]), "+d"(cx[2]), "+d"(cx[3])
            : "d"(ax[0]), "d"(ax[1]), "d"(ax[2]), "d"(ax[3]), "d"(ax[4]), "d"(ax[5]), "d"(ax[6]), "d"(ax[7]),
              "d"(b01.x), "d"(b01.y), "d"(b23.x), "d"(b23.y));
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5,%6,%7,%8,%9,%10,%11}, "
            "{%12,%13,%14,%15}, {%0,%1,%2,%3};"
            : "+d"(cn[0]), "+d"(cn[1]), "+d"(cn[2]), "+d"(cn[3])
            : "d"(an[0]), "d"(an[1]), "d"(an[2]), "d"(an[3]), "d"(an[4]), "d"(an[5]), "d"(an[6]), "d"(an[7]),
              "d"(b01.x), "d"(b01.y), "d"(b23.x), "d"(b23.y));
      }
      if (ch + 1 < NCH) {
#pragma unroll
        for (int i = 0; i < 4; ++i) cur[i] = nxt[i];
      }
    }
    // C[i]: block grp + 8*(i/2), column 2*tig + (i%2) = (head tig, representative i%2);
    // representative 0 (Qmax): cx = l1, cn = l2; representative 1 (Qmin): cx = l3, cn = l4
    if (tig < U) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int lb = t * 16 + grp + (i >> 1) * 8;      // local block index
        const int rep = i & 1;
        if (lb < nloc) {
          const bool hide = mask_first && b_lo + lb >= visible;
          const double vx = hide ? -CUDART_INF : cx[i] * est_scale, vn = hide ? -CUDART_INF : cn[i] * est_scale;
          lg[(tig * 4 + rep * 2 + 0) * nb + lb] = vx;
          lg[(tig * 4 + rep * 2 + 1) * nb + lb] = vn;
          lf[(tig * 4 + rep * 2 + 0) * nb + lb] = float(vx);
          lf[(tig * 4 + rep * 2 + 1) * nb + lb] = float(vn);
        }
      }
    }
  }
  __syncthreads();

  // log-sum-exp of each of the 4U logit rows (softmax over blocks, lines 9-10): a warp owns a row, so only
  // shuffles are needed.  Terms more than e^-50 below the row maximum cannot change the rounded sum and
  // are skipped.  Only a few percent of a row survive that test, scattered over the lanes, so the row is
  // first scanned in fp32 and the candidates -- fp32 value within 50 + a rounding margin of the fp32
  // maximum, which always includes the true maximum and every term that counts -- are compacted into a
  // dense index list (in place, over the fp32 row); the fp64 maximum and the exponentials then run on full warps.
#pragma unroll 1
  for (int rI = warp; rI < 4 * U; rI += kWarps) {
    const double* rowp = lg + rI * nb;
    float* rowf = lf + rI * nb;
    float mf = -CUDART_INF_F;
#pragma unroll 4
    for (int lb = lane; lb < nloc; lb += 32) mf = fmaxf(mf, rowf[lb]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mf = fmaxf(mf, __shfl_xor_sync(0xffffffffu, mf, o));
    const float thr = mf - (51.0f + fabsf(mf) * 1e-6f);     // -inf when the whole (local) row is masked: no candidates
    int* cand = reinterpret_cast<int*>(rowf);                // entry i is written after element i has been read
    int ncand = 0;
    for (int base = 0; base < nloc; base += 32) {
      const int lb = base + lane;
      const bool c = lb < nloc && rowf[lb] > thr;
      const unsigned ballot = __ballot_sync(0xffffffffu, c);
      if (c) cand[ncand + __popc(ballot & ((1u << lane) - 1u))] = lb;
      ncand += __popc(ballot);
    }
    __syncwarp();
    double m = -CUDART_INF;
    for (int i = lane; i < ncand; i += 32) m = fmax(m, rowp[cand[i]]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
    double sum = 0.0;
    for (int i = lane; i < ncand; i += 32) {
      const double d = rowp[cand[i]] - m;
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
    // thread (row, r) fetches rank r's pair of that row; the CL lanes of a row are adjacent, so the merge is shuffles
    if (warp * 32 < 4 * U * CL) {                     // whole warps take part in the shuffles
      const bool act = tid < 4 * U * CL;
      const int row = act ? tid / CL : 0, r = tid % CL;
      const double2 pr = cluster.map_shared_rank(part, r)[row];
      double M = pr.x;
      for (int o = CL >> 1; o > 0; o >>= 1) M = fmax(M, __shfl_xor_sync(0xffffffffu, M, o));
      double Ssum = pr.y > 0.0 ? pr.y * exp(pr.x - M) : 0.0;
      for (int o = CL >> 1; o > 0; o >>= 1) Ssum += __shfl_xor_sync(0xffffffffu, Ssum, o);
      if (act && r == 0) stat[row] = M + log(Ssum);
    }
    // no CTA may exit while a peer can still read its partials: arrive now, wait at the end of the kernel
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  } else if (tid < 4 * U) {
    stat[tid] = part[tid].x + log(part[tid].y);
  }
  __syncthreads();

  // stats_out given: this launch only produces the four log-sum-exps of every (head, segment) row
  if (stats_out != nullptr && rank == 0 && tid < 4 * U) stats_out[unit_of(tid >> 2) * 4 + (tid & 3)] = stat[tid];

  // combine (lines 11-12), mask (13), fusion (14) over this CTA's blocks of the U rows
  const double ln2 = 0.693147180559945309417232121458;
#pragma unroll 1
  for (int u = 0; u < (stats_out != nullptr ? 0 : U); ++u) {
    const double* l = lg + u * 4 * nb;
    const double st1 = stat[u * 4 + 0], st2 = stat[u * 4 + 1], st3 = stat[u * 4 + 2], st4 = stat[u * 4 + 3];
    const size_t out_row = unit_of(u) * n2 + b_lo;
#pragma unroll 2
    for (int lb = tid; lb < nloc; lb += kThreads) {
      double v;
      if (b_lo + lb >= visible) {
        v = -CUDART_INF;
      } else {
        const double L1 = l[lb] - st1, L2 = l[nb + lb] - st2, L3 = l[2 * nb + lb] - st3, L4 = l[3 * nb + lb] - st4;
        // max( ln (S1+S3)/2, ln (S2+S4)/2 ).  ln(e^a + e^b) lies in [max(a,b), max(a,b) + ln 2], so the pair with the
        // larger maximum wins outright unless the two maxima are within ln 2 of each other: one evaluation, rarely two.
        const double h13 = fmax(L1, L3), h24 = fmax(L2, L4);
        const bool first = h13 >= h24;
        v = logaddexp(first ? L1 : L2, first ? L3 : L4, sp_tab);
        if (fabs(h13 - h24) < ln2) v = fmax(v, logaddexp(first ? L2 : L1, first ? L4 : L3, sp_tab));
        v -= ln2;
        if (fuse) v = logaddexp(ln_alpha + v, ln_1m_alpha + S_prev[out_row + lb], sp_tab);
      }
      S_out[out_row + lb] = v;
    }
  }
  if (CL > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <typename T, int D, int U>
int launch_u(const Dims& m, const char* ws, const WsLayout& w, const double* S_prev, double* S_out,
             double est_scale, double alpha, int fuse, int mask_first, int CL, int nb, double* stats_out, cudaStream_t st) {
  const size_t smem = (sizeof(double) + sizeof(float)) * (4 * size_t(U) * nb);   // fp64 logits + their fp32 copies
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
      m.Hq, m.g, m.n1, m.n2, m.seg, m.blk, est_scale, log(alpha), log1p(-alpha), fuse, mask_first, CL, nb, stats_out);
  return e == cudaSuccess ? check_launch() : CP_ERR_CUDA;
}

template <typename T, int D>
int launch_t(const Dims& m, const char* ws, const WsLayout& w, const double* S_prev, double* S_out,
             double est_scale, double alpha, int fuse, int mask_first, double* stats_out, cudaStream_t st) {
  // as many heads per CTA as divide the group (the fp64 MMA has 8 rows = 4 heads x 2 representatives);
  // key blocks are split over a cluster of 1, 2, 4 or 8 CTAs until the logits fit ~200 KB per CTA
  const size_t budget = 200 * 1024;
  const int U = m.g % 4 == 0 ? 4 : (m.g % 2 == 0 ? 2 : 1);
  for (int CL = 1; CL <= 8; CL *= 2) {
    const int nb = (((m.n2 + CL - 1) / CL) + 7) & ~7;
    if ((sizeof(double) + sizeof(float)) * 4 * size_t(U) * nb > budget) continue;
    if (U == 4) return launch_u<T, D, 4>(m, ws, w, S_prev, S_out, est_scale, alpha, fuse, mask_first, CL, nb, stats_out, st);
    if (U == 2) return launch_u<T, D, 2>(m, ws, w, S_prev, S_out, est_scale, alpha, fuse, mask_first, CL, nb, stats_out, st);
    return launch_u<T, D, 1>(m, ws, w, S_prev, S_out, est_scale, alpha, fuse, mask_first, CL, nb, stats_out, st);
  }
  return CP_ERR_UNSUPPORTED;
}

}  // namespace

// The general kernel: any dtype, head_dim 64 or 128.  With stats_out it only writes the four log-sum-exps
// of every (head, segment) row, [B,Hq,n1,4], and leaves S_out alone.
int launch_score_generic(const cp_params& p, const Dims& m, const char* ws, const double* S_prev,
                         double* S_out, double* stats_out, cudaStream_t st) {
  const WsLayout w = ws_layout(m);
  const int fuse = (S_prev != nullptr && p.alpha != 1.0f) ? 1 : 0;
  const int mask_first = (p.flags & CP_FLAG_MASK_BEFORE_SOFTMAX) ? 1 : 0;
  const double es = double(p.est_scale), al = double(p.alpha);
  if (p.dtype == CP_BF16) {
    if (m.d == 128) return launch_t<__nv_bfloat16, 128>(m, ws, w, S_prev, S_out, es, al, fuse, mask_first, stats_out, st);
    if (m.d == 64) return launch_t<__nv_bfloat16, 64>(m, ws, w, S_prev, S_out, es, al, fuse, mask_first, stats_out, st);
  } else if (p.dtype == CP_F16) {
    if (m.d == 128) return launch_t<__half, 128>(m, ws, w, S_prev, S_out, es, al, fuse, mask_first, stats_out, st);
    if (m.d == 64) return launch_t<__half, 64>(m, ws, w, S_prev, S_out, es, al, fuse, mask_first, stats_out, st);
  } else {
    if (m.d == 128) return launch_t<float, 128>(m, ws, w, S_prev, S_out, es, al, fuse, mask_first, stats_out, st);
    if (m.d == 64) return launch_t<float, 64>(m, ws, w, S_prev, S_out, es, al, fuse, mask_first, stats_out, st);
  }
  return CP_ERR_UNSUPPORTED;
}

}  // namespace cp

// K3: critical block selection (Algorithm 2, line 8).  One CTA per (batch, query head,
// segment j).  The r diagonal blocks are always taken; the other m = k - r slots go to the
// strictly-past blocks with the largest score, ties to the larger block index.  Exact:
// an 8-pass MSB-first radix select on order-preserving 64-bit keys (held in registers) finds
// the m-th largest score, equal keys are resolved towards larger indices by counting, and an
// ordered block-wide compaction writes the list ascending.
#include "cp_common.cuh"

namespace cp {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

__device__ __forceinline__ unsigned long long ordered_key(double x) {
  if (x == 0.0) x = 0.0;   // -0.0 and +0.0 compare equal and must map to one key
  unsigned long long u = (unsigned long long)__double_as_longlong(x);
  return (u & 0x8000000000000000ull) ? ~u : (u | 0x8000000000000000ull);
}

// KPT = keys per thread; block b of the row lives in thread b % 256, slot b / 256.
template <int KPT>
__global__ void __launch_bounds__(kThreads)
select_kernel(const double* __restrict__ S, int32_t* __restrict__ idx, int32_t* __restrict__ cnt,
              int n1, int n2, int r, int k) {
  __shared__ unsigned int hist[256];
  __shared__ int warp_sum[kWarps];
  __shared__ unsigned long long prefix_sh;
  __shared__ int remaining_sh;
  __shared__ int warp_tot[2][kWarps];
  __shared__ int base_sh[2];

  const int unit = blockIdx.x;
  const int j = unit % n1;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const double* row = S + size_t(unit) * n2;
  int32_t* out = idx + size_t(unit) * k;
  const int past = j * r;
  const int rj = min(n2, past + r) - past;   // diagonal blocks of this segment (fewer in a short last segment)
  const int m = k - rj;

  if (past <= m) {
    // every visible block fits in the budget
    const int c = past + rj;
    for (int i = tid; i < k; i += kThreads) out[i] = i < c ? i : -1;
    if (tid == 0) cnt[unit] = c;
    return;
  }

  if (m == 0) {
    // the budget holds the diagonal blocks only
    for (int i = tid; i < k; i += kThreads) out[i] = i < rj ? past + i : -1;
    if (tid == 0) cnt[unit] = rj;
    return;
  }

  unsigned long long key[KPT];
#pragma unroll
  for (int s = 0; s < KPT; ++s) {
    const int b = s * kThreads + tid;
    key[s] = b < past ? ordered_key(row[b]) : 0ull;
  }

  // ---- radix select: key of the m-th largest past score --------------------------------
  unsigned long long prefix = 0;   // bits decided so far (high bits)
  int remaining = m;               // how many still to take among keys matching the prefix
  for (int pass = 0; pass < 8; ++pass) {
    const int shift = 56 - 8 * pass;
    hist[tid] = 0;
    __syncthreads();
    const unsigned long long himask = pass == 0 ? 0ull : (~0ull << (shift + 8));
#pragma unroll
    for (int s = 0; s < KPT; ++s) {
      const int b = s * kThreads + tid;
      if (b < past && (key[s] & himask) == prefix) atomicAdd(&hist[(key[s] >> shift) & 0xff], 1u);
    }
    __syncthreads();
    // suffix sums over the 256 bins: thread t owns bin t; above(t) = keys with a larger digit
    const int mine = int(hist[tid]);
    int incl = mine;   // inclusive suffix sum within the warp (towards higher lanes)
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_down_sync(0xffffffffu, incl, o);
      if (lane + o < 32) incl += v;
    }
    if (lane == 0) warp_sum[warp] = incl;
    __syncthreads();
    int above = incl - mine;
    for (int w = warp + 1; w < kWarps; ++w) above += warp_sum[w];
    if (above < remaining && remaining <= above + mine) {   // exactly one bin satisfies this
      prefix_sh = prefix | ((unsigned long long)tid << shift);
      remaining_sh = remaining - above;
    }
    __syncthreads();
    prefix = prefix_sh;
    remaining = remaining_sh;
  }
  const unsigned long long thr = prefix;   // the m-th largest key
  const int need_eq = remaining;           // of the keys equal to thr, take this many (largest indices)

  // total number of keys equal to the threshold
  if (tid == 0) base_sh[0] = 0;
  __syncthreads();
  int eq_local = 0;
#pragma unroll
  for (int s = 0; s < KPT; ++s) eq_local += (s * kThreads + tid < past) && key[s] == thr;
  for (int o = 16; o > 0; o >>= 1) eq_local += __shfl_xor_sync(0xffffffffu, eq_local, o);
  if (lane == 0 && eq_local) atomicAdd(&base_sh[0], eq_local);
  __syncthreads();
  const int eq_skip = base_sh[0] - need_eq;   // equal keys with the smallest indices are dropped
  __syncthreads();

  // ---- ordered compaction -----------------------------------------------------------------
  if (tid == 0) { base_sh[0] = 0; base_sh[1] = 0; }   // [0]: written so far, [1]: equals seen so far
  __syncthreads();
#pragma unroll
  for (int s = 0; s < KPT; ++s) {
    const int b0 = s * kThreads;
    if (b0 >= past) break;
    const int b = b0 + tid;
    const bool in = b < past;
    const bool gt = in && key[s] > thr, eq = in && key[s] == thr;
    const unsigned eq_ballot = __ballot_sync(0xffffffffu, eq);
    const int eq_before_warp = __popc(eq_ballot & ((1u << lane) - 1));
    if (lane == 0) warp_tot[1][warp] = __popc(eq_ballot);
    __syncthreads();
    int eq_before = base_sh[1] + eq_before_warp;
    for (int w = 0; w < warp; ++w) eq_before += warp_tot[1][w];
    const bool take = gt || (eq && eq_before >= eq_skip);
    const unsigned tk_ballot = __ballot_sync(0xffffffffu, take);
    if (lane == 0) warp_tot[0][warp] = __popc(tk_ballot);
    __syncthreads();
    int pos = base_sh[0] + __popc(tk_ballot & ((1u << lane) - 1));
    for (int w = 0; w < warp; ++w) pos += warp_tot[0][w];
    if (take && pos < m) out[pos] = b;
    __syncthreads();
    if (tid == 0) {
      int a = 0, e = 0;
      for (int w = 0; w < kWarps; ++w) { a += warp_tot[0][w]; e += warp_tot[1][w]; }
      base_sh[0] += a; base_sh[1] += e;
    }
    __syncthreads();
  }
  for (int i = tid; i < rj; i += kThreads) out[m + i] = past + i;   // diagonal blocks
  if (tid == 0) cnt[unit] = k;
}

}  // namespace

int launch_select(const cp_params& p, const Dims& m, const double* S, int32_t* idx, int32_t* cnt,
                  cudaStream_t st) {
  (void)p;
  const long long units = (long long)m.B * m.Hq * m.n1;
  if (units > 0x7fffffffLL) return CP_ERR_UNSUPPORTED;
  const int kpt = (m.n2 + kThreads - 1) / kThreads;
  const unsigned grid = unsigned(units);
  if (kpt <= 4) select_kernel<4><<<grid, kThreads, 0, st>>>(S, idx, cnt, m.n1, m.n2, m.r, m.k);
  else if (kpt <= 8) select_kernel<8><<<grid, kThreads, 0, st>>>(S, idx, cnt, m.n1, m.n2, m.r, m.k);
  else if (kpt <= 16) select_kernel<16><<<grid, kThreads, 0, st>>>(S, idx, cnt, m.n1, m.n2, m.r, m.k);
  else if (kpt <= 32) select_kernel<32><<<grid, kThreads, 0, st>>>(S, idx, cnt, m.n1, m.n2, m.r, m.k);
  else return CP_ERR_UNSUPPORTED;
  return check_launch();
}

}  // namespace cp

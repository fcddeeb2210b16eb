// K3: critical block selection (Algorithm 2, line 8).  One CTA per (batch, query head,
// segment j).  The r diagonal blocks are always taken; the other m = k - r slots go to the
// strictly-past blocks with the largest score, ties to the larger block index.  Exact:
// an 8-pass MSB-first radix select on order-preserving 64-bit keys finds the m-th largest
// score, a second sweep resolves ties by index, and an ordered block-wide compaction writes
// the list ascending.
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

__global__ void __launch_bounds__(kThreads)
select_kernel(const double* __restrict__ S, int32_t* __restrict__ idx, int32_t* __restrict__ cnt,
              int n1, int n2, int r, int k) {
  __shared__ unsigned int hist[256];
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
  const int m = k - r;

  if (past <= m) {
    // every visible block fits in the budget
    const int c = past + r;
    for (int i = tid; i < k; i += kThreads) out[i] = i < c ? i : -1;
    if (tid == 0) cnt[unit] = c;
    return;
  }

  // ---- radix select: key of the m-th largest past score --------------------------------
  unsigned long long prefix = 0;   // bits decided so far (high bits)
  int remaining = m;               // how many still to take among keys matching the prefix
  for (int pass = 0; pass < 8; ++pass) {
    const int shift = 56 - 8 * pass;
    for (int i = tid; i < 256; i += kThreads) hist[i] = 0;
    __syncthreads();
    const unsigned long long himask = pass == 0 ? 0ull : (~0ull << (shift + 8));
    for (int b = tid; b < past; b += kThreads) {
      const unsigned long long key = ordered_key(row[b]);
      if ((key & himask) == prefix) atomicAdd(&hist[(key >> shift) & 0xff], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      int acc = 0, d = 255;
      for (; d > 0; --d) {
        if (acc + int(hist[d]) >= remaining) break;
        acc += int(hist[d]);
      }
      prefix_sh = prefix | ((unsigned long long)d << shift);
      remaining_sh = remaining - acc;   // to take among keys with this digit
    }
    __syncthreads();
    prefix = prefix_sh;
    remaining = remaining_sh;
    __syncthreads();
  }
  const unsigned long long thr = prefix;   // the m-th largest key
  const int need_eq = remaining;           // of the keys equal to thr, take this many (largest indices)

  // total number of keys equal to the threshold
  if (tid == 0) base_sh[0] = 0;
  __syncthreads();
  int eq_local = 0;
  for (int b = tid; b < past; b += kThreads) eq_local += ordered_key(row[b]) == thr;
  for (int o = 16; o > 0; o >>= 1) eq_local += __shfl_xor_sync(0xffffffffu, eq_local, o);
  if (lane == 0 && eq_local) atomicAdd(&base_sh[0], eq_local);
  __syncthreads();
  const int eq_skip = base_sh[0] - need_eq;   // equal keys with the smallest indices are dropped
  __syncthreads();

  // ---- ordered compaction -----------------------------------------------------------------
  if (tid == 0) { base_sh[0] = 0; base_sh[1] = 0; }   // [0]: written so far, [1]: equals seen so far
  __syncthreads();
  for (int b0 = 0; b0 < past; b0 += kThreads) {
    const int b = b0 + tid;
    unsigned long long key = 0;
    bool gt = false, eq = false;
    if (b < past) { key = ordered_key(row[b]); gt = key > thr; eq = key == thr; }
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
  for (int i = tid; i < r; i += kThreads) out[m + i] = past + i;   // diagonal blocks
  if (tid == 0) cnt[unit] = k;
}

}  // namespace

int launch_select(const cp_params& p, const Dims& m, const double* S, int32_t* idx, int32_t* cnt,
                  cudaStream_t st) {
  (void)p;
  const long long units = (long long)m.B * m.Hq * m.n1;
  if (units > 0x7fffffffLL) return CP_ERR_UNSUPPORTED;
  select_kernel<<<unsigned(units), kThreads, 0, st>>>(S, idx, cnt, m.n1, m.n2, m.r, m.k);
  return check_launch();
}

}  // namespace cp

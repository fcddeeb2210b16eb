// K3: critical block selection (Algorithm 2, line 8).  One CTA per (batch, query head,
// segment j).  The r diagonal blocks are always taken; the other m = k - r slots go to the
// strictly-past blocks with the largest score, ties to the larger block index.  Exact:
// an MSB-first radix select (8 bits per pass, at most 8 passes, usually 3-4) on order-preserving 64-bit
// keys held in registers finds the m-th largest score, equal keys are resolved towards larger indices by
// counting, and an ordered block-wide compaction (two scans) writes the list ascending.
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

// Block-wide exclusive scan of one int per thread (256 threads); *total receives the sum.  Two barriers.
__device__ __forceinline__ int block_exclusive_scan(int v, int lane, int warp, int* warp_tot, int* total) {
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  int before = 0, all = 0;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) {
    const int t = warp_tot[w];
    before += w < warp ? t : 0;
    all += t;
  }
  __syncthreads();                      // warp_tot may be reused by the next scan
  *total = all;
  return before + incl - v;
}

// KPT = keys per thread; thread t owns the KPT consecutive blocks [t*KPT, (t+1)*KPT), so the ordered
// compaction at the end is two block-wide scans instead of a barrier-separated step per key slot.
// `pool` > 1: one CTA per (batch, KV head, segment); the key of a block is the largest of the pool's `pool`
// consecutive query heads' scores, and the one list is written for each of them.  n_sink / n_local: the first
// n_sink blocks and the n_local blocks right before the segment get the largest possible key, so they are taken
// before any scored block (the host has checked that they fit into the k - r free slots).
// Resident CTAs per SM are set by registers: the kernel waits on barriers most of the time, so 16 keys per thread are held to 64
// registers (4 CTAs instead of the 3 that 80 registers allow: 13 % faster at n2 = 4096; 48 registers spill and are slower).
template <int KPT>
__global__ void __launch_bounds__(kThreads, KPT <= 4 ? 5 : (KPT <= 16 ? 4 : 2))
select_kernel(const double* __restrict__ S, int32_t* __restrict__ idx, int32_t* __restrict__ cnt,
              int n1, int n2, int r, int k, int pool, int n_sink, int n_local, int past_fixed) {
  __shared__ unsigned int hist[256];
  __shared__ int warp_sum[kWarps];
  __shared__ unsigned long long prefix_sh;
  __shared__ int remaining_sh, bin_count_sh;
  __shared__ int warp_tot[kWarps];

  // CTA -> (batch * heads / pool + pooled head, segment); its first query head's unit is `unit`
  const int j = blockIdx.x % n1;
  const int unit = (blockIdx.x / n1) * pool * n1 + j;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const double* row = S + size_t(unit) * n2;
  const int past = past_fixed >= 0 ? past_fixed : j * r;   // past_fixed: the caller names the first diagonal block (decoding: the last block)
  const int rj = min(n2, past + r) - past;   // diagonal blocks of this segment (fewer in a short last segment)
  const int m = k - rj;

  if (past <= m) {
    // every visible block fits in the budget
    const int c = past + rj;
    for (int u = 0; u < pool; ++u) {
      int32_t* out = idx + (size_t(unit) + size_t(u) * n1) * k;
      for (int i = tid; i < k; i += kThreads) out[i] = i < c ? i : -1;
      if (tid == 0) cnt[unit + u * n1] = c;
    }
    return;
  }

  if (m == 0) {
    // the budget holds the diagonal blocks only
    for (int u = 0; u < pool; ++u) {
      int32_t* out = idx + (size_t(unit) + size_t(u) * n1) * k;
      for (int i = tid; i < k; i += kThreads) out[i] = i < rj ? past + i : -1;
      if (tid == 0) cnt[unit + u * n1] = rj;
    }
    return;
  }

  const int b0 = tid * KPT;                  // first block owned by this thread
  unsigned long long key[KPT];
#pragma unroll
  for (int s = 0; s < KPT; ++s) {
    const int bb = b0 + s;
    unsigned long long kk = 0ull;
    if (bb < past) {
      if (bb < n_sink || bb >= past - n_local) {
        kk = ~0ull;                          // forced block
      } else {
        kk = ordered_key(__ldg(row + bb));
        for (int u = 1; u < pool; ++u) kk = max(kk, ordered_key(__ldg(row + size_t(u) * n1 * n2 + bb)));
      }
    }
    key[s] = kk;
  }
  hist[tid] = 0;
  __syncthreads();

  // ---- radix select: key of the m-th largest past score --------------------------------
  // MSB-first, 8 bits per pass.  A pass ends the search early when the bin that holds the m-th largest key
  // holds exactly as many keys as are still to be taken: then every key of that bin (and above) is selected
  // and no tie has to be resolved.  With distinct scores this happens after 3-4 of the 8 passes.
  unsigned long long prefix = 0;   // bits decided so far (high bits)
  int remaining = m;               // how many still to take among keys matching the prefix
  bool all_of_bin = false;
  for (int pass = 0; pass < 8; ++pass) {
    const int shift = 56 - 8 * pass;
    const unsigned long long himask = pass == 0 ? 0ull : (~0ull << (shift + 8));
#pragma unroll
    for (int s = 0; s < KPT; ++s)
      if (b0 + s < past && (key[s] & himask) == prefix) atomicAdd(&hist[(key[s] >> shift) & 0xff], 1u);
    __syncthreads();
    // suffix sums over the 256 bins: thread t owns bin t; above(t) = keys with a larger digit
    const int mine = int(hist[tid]);
    hist[tid] = 0;                 // only its owner reads a bin, so it can be cleared for the next pass right away
    int incl = mine;               // inclusive suffix sum within the warp (towards higher lanes)
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
      bin_count_sh = mine;
    }
    __syncthreads();
    prefix = prefix_sh;
    remaining = remaining_sh;
    if (bin_count_sh == remaining) { all_of_bin = true; break; }   // uniform: read from shared memory by all
  }
  // all_of_bin: take every key >= prefix (its undecided low bits are zero).  Otherwise prefix is the m-th
  // largest key itself: take the keys above it and, of the keys equal to it, the `remaining` largest indices.
  const unsigned long long thr = prefix;
  int n_gt = 0, n_eq = 0;
#pragma unroll
  for (int s = 0; s < KPT; ++s) {
    const bool in = b0 + s < past;
    n_gt += in && (all_of_bin ? key[s] >= thr : key[s] > thr);
    n_eq += in && !all_of_bin && key[s] == thr;
  }
  int eq_before = 0, eq_skip = 0;
  if (!all_of_bin) {                         // uniform branch
    int total_eq;
    eq_before = block_exclusive_scan(n_eq, lane, warp, warp_tot, &total_eq);
    eq_skip = total_eq - remaining;          // equal keys with the smallest indices are dropped
  }
  int n_take = n_gt;
  if (!all_of_bin) {
#pragma unroll
    for (int s = 0, e = eq_before; s < KPT; ++s)
      if (b0 + s < past && key[s] == thr) { n_take += e >= eq_skip; ++e; }
  }

  // ---- ordered compaction: blocks are owned in index order, so positions are an exclusive scan ----
  int total_take;
  const int pos0 = block_exclusive_scan(n_take, lane, warp, warp_tot, &total_take);
  for (int u = 0; u < pool; ++u) {           // the same list for every head of the pool
    int32_t* out = idx + (size_t(unit) + size_t(u) * n1) * k;
    int pos = pos0;
#pragma unroll
    for (int s = 0, e = eq_before; s < KPT; ++s) {
      if (b0 + s >= past) break;
      bool take;
      if (all_of_bin) take = key[s] >= thr;
      else if (key[s] == thr) { take = e >= eq_skip; ++e; }
      else take = key[s] > thr;
      if (take) { if (pos < m) out[pos] = b0 + s; ++pos; }
    }
    for (int i = tid; i < rj; i += kThreads) out[m + i] = past + i;   // diagonal blocks
    if (tid == 0) cnt[unit + u * n1] = k;
  }
}

}  // namespace

int launch_select(const cp_params& p, const Dims& m, const double* S, int32_t* idx, int32_t* cnt,
                  cudaStream_t st, int past_fixed) {
  const int pool = (p.flags & CP_FLAG_SHARED_GROUP_LISTS) ? m.g : 1;
  const int n_sink = p.forced_blocks & 0xffff, n_local = (p.forced_blocks >> 16) & 0xffff;
  const long long units = (long long)m.B * (m.Hq / pool) * m.n1;
  if (units > 0x7fffffffLL) return CP_ERR_UNSUPPORTED;
  const int kpt = (m.n2 + kThreads - 1) / kThreads;
  const unsigned grid = unsigned(units);
  if (kpt <= 4) select_kernel<4><<<grid, kThreads, 0, st>>>(S, idx, cnt, m.n1, m.n2, m.r, m.k, pool, n_sink, n_local, past_fixed);
  else if (kpt <= 8) select_kernel<8><<<grid, kThreads, 0, st>>>(S, idx, cnt, m.n1, m.n2, m.r, m.k, pool, n_sink, n_local, past_fixed);
  else if (kpt <= 16) select_kernel<16><<<grid, kThreads, 0, st>>>(S, idx, cnt, m.n1, m.n2, m.r, m.k, pool, n_sink, n_local, past_fixed);
  else if (kpt <= 32) select_kernel<32><<<grid, kThreads, 0, st>>>(S, idx, cnt, m.n1, m.n2, m.r, m.k, pool, n_sink, n_local, past_fixed);
  else return CP_ERR_UNSUPPORTED;
  return check_launch();
}

}  // namespace cp

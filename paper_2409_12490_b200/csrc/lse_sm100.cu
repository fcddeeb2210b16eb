// K2a: the row log-sum-exps of the four logit maps (Algorithm 1, lines 9-10: the normaliser of each softmax
// over ALL key blocks), for 16-bit inputs with head_dim 128.
//
// A row's log-sum-exp needs every one of its n2 logits, but only a few of them to full accuracy: a term that
// lies D below the row maximum contributes e^-D to the sum.  So the logits are first formed approximately on the
// tcgen05 tensor cores (16-bit operands, fp32 accumulation in tensor memory; the error bound is derived below)
// and only the terms that are close enough to the maximum for that error to matter are re-evaluated exactly in
// fp64:
//   sweep A   approximate logits of all blocks -> approximate row maxima M~
//   sweep B   approximate logits again; an element within `window` of M~ flags its key block for the exact
//             pass (per MMA column group of 8 rows); the other elements are summed as exp(x~ - M~) in fp32
//   exact     the flagged blocks, gathered 16 at a time, go through fp64 mma.m16n8k16 against the 8 rows of
//             their group; their exp(x - M~) are summed in fp64
//   lse = M~ + ln(exact sum + approximate sum)
// Error bound.  An approximate logit differs from the exact one by at most eps = 2^-15 * |est_scale| * |q|_1 *
// max|k| (the products of two 16-bit values are exact in fp32; if each of the 8 chained K=16 MMAs aligns its 17
// addends to the largest one and truncates each by up to one unit in the last place, it loses at most 17 * 2^-22
// of the largest magnitude, itself at most |q|_1 * max|k|: 2^-14.9 in total.  Measured on this part with inputs
// spread over 24 binades: 2^-20 of sum |q||k|, i.e. 30 times less) plus the fp32 rounding of M~ and of the difference.  An element not
// flagged lies at least window - 2 eps below the true maximum, so with window = ln(n2 * eps / 1e-11) + 2 eps the
// approximately summed terms change the sum, which is at least e^-eps, by less than 1e-11 in total: ln S keeps
// its 1e-9.  When eps is too large for this reasoning (> 4) every block is flagged and the result is the plain
// fp64 evaluation.
//
// One CTA: 128 logit rows = the (Qmax, Qmin) representatives of 64 / U consecutive segments x U query heads of
// one KV group, as the M = 128 rows of the MMA's A operand; key blocks stream through as N = 128 tiles (TMA, 4-slot
// ring), accumulators rotate through the 4 x 128 columns of tensor memory.  Warps 0-7: one thread per (row, Kmax | Kmin)
// (max / sums need no cross-thread reduction), warp 8: TMA producer, warp 9: MMA issuer; all 12 warps share the
// exact pass.  Every wait is bounded.
#include "score_common.cuh"
#include "sm100_ptx.cuh"

namespace cp {
namespace {

constexpr int kThreads = 384;
constexpr int kWarps = kThreads / 32;
constexpr int kD = 128;
constexpr int kRows = 128;                     // logit rows (MMA M) per CTA
constexpr int kTileN = 128;                    // key blocks per tile (MMA N)
constexpr int kHalfBytes = 128 * 64 * 2;       // [128 rows x 64 channels] 16-bit, 128-byte swizzled
constexpr int kTileBytes = 2 * kHalfBytes;
constexpr int kSlots = 4;                      // K tile ring
constexpr int kStages = 4;                     // accumulator stages in tensor memory (4 x 128 columns)
constexpr int kLists = 32;                     // (column group of 8 rows) x (Kmax | Kmin)
constexpr int kQueue = 1056;                   // per-warp queue of flagged block indices: 15 left over + 32 words x 32 bits
constexpr int kQS = kD + 2;                    // row stride (doubles) of the exact pass's B operand in shared memory
constexpr int kSmemQ = 0;
constexpr int kSmemKV = kTileBytes;
constexpr int kSmemFixed = kSmemKV + kSlots * kTileBytes;   // then: masks | queues | Mref | row l1 norms | exact sums | barriers
static_assert(kWarps * 8 * kQS * 8 <= kSlots * kTileBytes, "the exact pass keeps its B operands in the idle K ring");

struct LseBars {
  unsigned long long kv_full[kSlots], kv_empty[kSlots], acc_full[kStages], acc_empty[kStages];
  uint32_t tmem_base;
  volatile int abort_flag;
  int next_list;                 // exact pass: the lists are handed out to the warps as they become free
  float kabs_red[kWarps];
};

struct LseArgs {
  const void *Qmax, *Qmin, *Kmax, *Kmin;   // summaries in the workspace
  const float* kabs;                        // [B*Hkv, n2]
  double* stats;                            // [B,Hq,n1,4]
  DeviceStatus* st;
  int Hq, g, U, n1, n2, seg, blk, segs_per_cta, n_qchunks, mask_first, box_rows;
  float es;
};

template <bool kF16> struct Elem { using type = __nv_bfloat16; };
template <> struct Elem<true> { using type = __half; };

template <bool kF16>
__device__ __forceinline__ void issue_tile(uint32_t d_tmem, uint32_t q_smem, uint32_t k_smem) {
  const uint64_t base = desc_base(16);
#pragma unroll
  for (int kk = 0; kk < kD / 16; ++kk) {
    const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
    umma_ss(d_tmem, desc_at(base, q_smem + off), desc_at(base, k_smem + off), Idesc<kF16>::qk, kk > 0);
  }
}

// Roles during the sweeps (384 threads): warps 0-3 take the Kmax products (one thread per logit row), warps 4-7 the
// Kmin products of the same rows, warp 8 is the TMA producer, warp 9 the MMA issuer; all 12 warps share the exact pass.
template <bool kF16>
__global__ void __launch_bounds__(kThreads, 1)
lse_sm100_kernel(const __grid_constant__ CUtensorMap tmKmax, const __grid_constant__ CUtensorMap tmKmin, const LseArgs a) {
  using T = typename Elem<kF16>::type;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t smem_base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (smem_base - raw);
  const int n_words = ((a.n2 + kTileN - 1) / kTileN) * 4;              // 32-block words per list
  uint32_t* masks = reinterpret_cast<uint32_t*>(sm + kSmemFixed);       // [kLists][n_words]
  uint16_t* queues = reinterpret_cast<uint16_t*>(masks + kLists * n_words);   // [kWarps][kQueue]
  float* mref = reinterpret_cast<float*>(queues + kWarps * kQueue);     // [kRows][2]
  float* ql1 = mref + kRows * 2;                                        // [kRows]
  double* exact_sum = reinterpret_cast<double*>(ql1 + kRows);           // [kRows][2]
  LseBars* bars = reinterpret_cast<LseBars*>(exact_sum + kRows * 2);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // CTA -> (b*Hkv + kv head, head subgroup, chunk of segs_per_cta segments)
  const int groups = a.g / a.U;
  int x = blockIdx.x;
  const int qchunk = x % a.n_qchunks; x /= a.n_qchunks;
  const int sub = x % groups; x /= groups;
  const int kvh = x;
  const int Hkv = a.Hq / a.g;
  const int b = kvh / Hkv;
  const int h0 = (kvh % Hkv) * a.g + sub * a.U;
  const int j0 = qchunk * a.segs_per_cta;
  // row m of the CTA: column group m/8 = (4-segment chunk c4, head u); within it (segment s, representative)
  auto row_seg = [&](int m) {            // rows beyond the CTA's share of segments (or beyond n1) map past the end: unused
    const int local = ((m >> 3) / a.U) * 4 + ((m >> 1) & 3);
    return local < a.segs_per_cta ? j0 + local : a.n1;
  };
  auto row_unit = [&](int m) { return (size_t(b) * a.Hq + h0 + (m >> 3) % a.U) * a.n1 + row_seg(m); };
  auto row_limit = [&](int m) {          // blocks [0, limit) enter the row's softmax
    const int j = row_seg(m);
    if (j >= a.n1) return 0;
    return a.mask_first ? min(a.n2, ((j + 1) * a.seg + a.blk - 1) / a.blk) : a.n2;
  };
  const int j_last = min(a.n1, j0 + a.segs_per_cta) - 1;
  const int lim_max = a.mask_first ? min(a.n2, ((j_last + 1) * a.seg + a.blk - 1) / a.blk) : a.n2;
  const int n_tiles = (lim_max + kTileN - 1) / kTileN;

#ifdef CP_LSE_DEBUG
  const long long t_start = clock64();
#endif
  // ---------------- set-up
  if (tid == 0) {
    for (int i = 0; i < kSlots; ++i) { mbar_init(&bars->kv_full[i], 1); mbar_init(&bars->kv_empty[i], 1); }
    for (int i = 0; i < kStages; ++i) { mbar_init(&bars->acc_full[i], 1); mbar_init(&bars->acc_empty[i], 128); }
    bars->abort_flag = 0;
    bars->next_list = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8 && lane == 0) { prefetch_tmap(&tmKmax); prefetch_tmap(&tmKmin); }
  if (warp == 9) { tmem_alloc(&bars->tmem_base, 512); tmem_relinquish(); }
  // largest magnitude among this KV head's key summaries
  {
    float m = 0.f;
    const float* ka = a.kabs + size_t(kvh) * a.n2;
    for (int i = tid; i < a.n2; i += kThreads) m = fmaxf(m, ka[i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) bars->kabs_red[warp] = m;
  }
  for (int i = tid; i < kRows * 2; i += kThreads) exact_sum[i] = 0.0;
  // the A operand: row m of the tile = representative m, K-major, 128-byte swizzled (two halves of 64 channels)
  const int my_row = tid & 127;                          // meaningful for warps 0-7
  const int my_kr = (tid >> 7) & 1;                      // warps 0-3: Kmax products, warps 4-7: Kmin products
  const bool my_valid = tid < 2 * kRows && row_seg(my_row) < a.n1;
  const int my_lim = tid < 2 * kRows ? row_limit(my_row) : 0;
  if (tid < kRows) {
    const int m = tid;
    float l1 = 0.f;
    const uint4* src = reinterpret_cast<const uint4*>(static_cast<const T*>((m & 1) ? a.Qmin : a.Qmax) + row_unit(m) * kD);
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (my_valid) v = __ldg(src + c);
      const T* e = reinterpret_cast<const T*>(&v);
#pragma unroll
      for (int i = 0; i < 8; ++i) l1 += fabsf(float(e[i]));
      *reinterpret_cast<uint4*>(sm + kSmemQ + (c >> 3) * kHalfBytes + m * 128 + (((c & 7) ^ (m & 7)) << 4)) = v;
    }
    ql1[m] = l1 * 1.0001f;                               // fp32 summation slack
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the MMAs read the tile through the async proxy
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  float kabs_max = 0.f;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) kabs_max = fmaxf(kabs_max, bars->kabs_red[w]);
  const uint32_t tm = bars->tmem_base;
  const uint32_t n_items = 4u * uint32_t(n_tiles);     // sweep A then sweep B; per tile the Kmax (even) and the Kmin (odd) product

  float Mx = -CUDART_INF_F;                            // approximate row maximum of this thread's (row, Kmax | Kmin) logits
  float asum = 0.f;                                    // its approximately summed terms

  if (warp == 8) {
    // ---------------- TMA producer
    for (uint32_t it = 0; it < n_items; ++it) {
      const uint32_t slot = it % kSlots, use = it / kSlots;
      if (use > 0 && !mbar_wait(&bars->kv_empty[slot], (use - 1) & 1, &bars->abort_flag, a.st, 60)) break;
      if (lane == 0) {
        const int tile = int((it % (2u * n_tiles)) >> 1);
        const CUtensorMap* map = (it & 1) ? &tmKmin : &tmKmax;
        const uint32_t dst = smem_base + kSmemKV + slot * kTileBytes;
        mbar_expect_tx(&bars->kv_full[slot], uint32_t(a.box_rows) * 128u * 2u);
        tma_load_3d(dst, map, &bars->kv_full[slot], 0, tile * kTileN, kvh);
        tma_load_3d(dst + kHalfBytes, map, &bars->kv_full[slot], 64, tile * kTileN, kvh);
      }
      __syncwarp();
    }
  } else if (warp == 9) {
    // ---------------- MMA issuer
    for (uint32_t it = 0; it < n_items; ++it) {
      const uint32_t slot = it % kSlots, stage = it % kStages;
      if (!mbar_wait(&bars->kv_full[slot], (it / kSlots) & 1, &bars->abort_flag, a.st, 61)) break;
      if (it >= kStages && !mbar_wait(&bars->acc_empty[stage], ((it / kStages) - 1) & 1, &bars->abort_flag, a.st, 62)) break;
      tc_fence_after();
      issue_tile<kF16>(tm + stage * kTileN, smem_base + kSmemQ, smem_base + kSmemKV + slot * kTileBytes);
      umma_commit(&bars->acc_full[stage]);
      umma_commit(&bars->kv_empty[slot]);
    }
  } else if (warp < 8) {
    // ---------------- one thread per (logit row, Kmax | Kmin): items of its parity only
    const uint32_t t_row = tm + (uint32_t((warp & 3) * 32) << 16);
    const float es = a.es, l2e = 1.4426950408889634f;
    float flagT = -CUDART_INF_F, mref_l2 = 0.f;
#ifdef CP_LSE_DEBUG
    long long dbg_wait = 0, dbg_a = 0, dbg_b = 0;
#endif
    const float es_l2 = es * l2e;
    for (uint32_t it = uint32_t(my_kr); it < n_items; it += 2) {
      const uint32_t stage = it % kStages;
      const bool sweep_b = it >= 2u * n_tiles;
      const int tile = int((it % (2u * n_tiles)) >> 1);
      if (it == 2u * n_tiles + uint32_t(my_kr)) {
        // between the sweeps: the reference maximum for everyone, and this row's flagging threshold
        mref[my_row * 2 + my_kr] = Mx;
        const float eps = 3.0517578125e-5f * fabsf(es) * ql1[my_row] * kabs_max + 9.5367431640625e-7f * (fabsf(Mx) + 64.f);
        const float window = __logf(float(a.n2)) + __logf(fmaxf(eps, 1e-6f)) + 25.4f + 2.f * eps;
        flagT = (eps < 4.f) ? Mx - window : -CUDART_INF_F;     // eps too large (or NaN): flag everything
        mref_l2 = Mx * l2e;
      }
#ifdef CP_LSE_DEBUG
      const long long tw0 = clock64();
#endif
      if (!mbar_wait(&bars->acc_full[stage], (it / kStages) & 1, &bars->abort_flag, a.st, 63)) break;
#ifdef CP_LSE_DEBUG
      const long long tw1 = clock64();
      dbg_wait += tw1 - tw0;
#endif
      tc_fence_after();
      const uint32_t t_acc = t_row + stage * kTileN;
      uint32_t va[32], vb[32];
      tmem_ld32(t_acc, va);
      auto piece_fn = [&](const uint32_t (&v)[32], int piece) {
        const int b0 = tile * kTileN + piece * 32;
        const int n_in = min(32, my_lim - b0);               // elements of this piece inside the row's softmax (<= 0: none)
        if (!sweep_b) {
          float m0 = Mx, m1 = -CUDART_INF_F;
          if (n_in >= 32) {
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              m0 = fmaxf(m0, __uint_as_float(v[i]) * es);
              m1 = fmaxf(m1, __uint_as_float(v[i + 1]) * es);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) m0 = (i < n_in) ? fmaxf(m0, __uint_as_float(v[i]) * es) : m0;
          }
          Mx = fmaxf(m0, m1);
        } else {
          uint32_t own = 0;
#pragma unroll
          for (int i = 0; i < 32; ++i) own |= ((i < n_in) && (__uint_as_float(v[i]) * es > flagT)) ? (1u << i) : 0u;
          if (!my_valid) own = 0;
          uint32_t gm = own;                                  // OR over the 8 rows of the column group
          gm |= __shfl_xor_sync(0xffffffffu, gm, 1);
          gm |= __shfl_xor_sync(0xffffffffu, gm, 2);
          gm |= __shfl_xor_sync(0xffffffffu, gm, 4);
          const uint32_t add = ~gm & (n_in >= 32 ? 0xffffffffu : (n_in <= 0 ? 0u : ((1u << n_in) - 1u)));
          float s0 = 0.f, s1 = 0.f;
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float t0 = ex2(fmaf(__uint_as_float(v[i]), es_l2, -mref_l2));
            const float t1 = ex2(fmaf(__uint_as_float(v[i + 1]), es_l2, -mref_l2));
            s0 += ((add >> i) & 1u) ? t0 : 0.f;
            s1 += ((add >> (i + 1)) & 1u) ? t1 : 0.f;
          }
          asum += s0 + s1;
          if ((lane & 7) == 0) masks[((my_row >> 3) * 2 + my_kr) * n_words + tile * 4 + piece] = gm;
        }
      };
      // pieces of 32 columns, the next one in flight while the current one is processed
      tmem_wait_ld(); tmem_ld32(t_acc + 32, vb); piece_fn(va, 0);
      tmem_wait_ld(); tmem_ld32(t_acc + 64, va); piece_fn(vb, 1);
      tmem_wait_ld(); tmem_ld32(t_acc + 96, vb); piece_fn(va, 2);
      tmem_wait_ld(); piece_fn(vb, 3);
      tc_fence_before();
      mbar_arrive(&bars->acc_empty[stage]);
#ifdef CP_LSE_DEBUG
      if (sweep_b) dbg_b += clock64() - tw1; else dbg_a += clock64() - tw1;
#endif
    }
#ifdef CP_LSE_DEBUG
    if (blockIdx.x == 0 && tid == 0) {
      long long* dbg = reinterpret_cast<long long*>(reinterpret_cast<char*>(a.st) + 216);
      dbg[0] = dbg_wait; dbg[1] = dbg_a; dbg[2] = dbg_b;
    }
#endif
  }
  tc_fence_before();
  __syncthreads();
  const bool aborted = bars->abort_flag != 0;
#ifdef CP_LSE_DEBUG
  long long t_sweeps = clock64();
#endif

  // ---------------- exact pass over the flagged blocks: list l = (column group, Kmax | Kmin)
  if (!aborted) {
    const int grp = lane >> 2, tig = lane & 3;
    uint16_t* queue = queues + warp * kQueue;
    double* qs = reinterpret_cast<double*>(sm + kSmemKV) + warp * 8 * kQS;   // this warp's B operand, in the idle K ring
    const double es_d = double(a.es);
    for (;;) {
      // lists differ a lot in length (a few rows near their maximum flag most of the blocks), so they are taken first
      // come, first served (a fixed round-robin left the slowest warp 25 % behind; halving the lists for a finer grain
      // costs more in B-operand set-up than it balances)
      int l = 0;
      if (lane == 0) l = atomicAdd(&bars->next_list, 1);
      l = __shfl_sync(0xffffffffu, l, 0);
      if (l >= kLists) break;
      const int cg = l >> 1, kr = l & 1;
      if (row_seg(cg * 8) >= a.n1) continue;              // the group's first segment does not exist: nothing flagged
      // B operand: the 8 rows of the group widened to fp64, [row][k-step][lane-in-quad][4 channels]
      __syncwarp();
      for (int e = lane; e < 8 * 16; e += 32) {
        const int r = e >> 4, c16 = e & 15, mb = cg * 8 + r;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (row_seg(mb) < a.n1)
          v = __ldg(reinterpret_cast<const uint4*>(static_cast<const T*>((mb & 1) ? a.Qmin : a.Qmax) + row_unit(mb) * kD) + c16);
        const T* el = reinterpret_cast<const T*>(&v);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int ch = c16 * 8 + i, tq = ch >> 5, within = ch & 31;
          qs[r * kQS + ((within >> 2) * 4 + tq) * 4 + (within & 3)] = to_f64(el[i]);
        }
      }
      __syncwarp();
      // this lane's two output columns: rows 2*tig, 2*tig+1 of the group
      const int mc = cg * 8 + 2 * tig;
      const double Mc0 = double(mref[mc * 2 + kr]), Mc1 = double(mref[(mc + 1) * 2 + kr]);
      const int lim0 = row_limit(mc), lim1 = row_limit(mc + 1);
      const T* kbase = static_cast<const T*>(kr ? a.Kmin : a.Kmax) + size_t(kvh) * a.n2 * kD + tig * 32;
      double acc0 = 0.0, acc1 = 0.0;

      auto load_rows = [&](const uint16_t* ptr, int cnt, uint4 (&w0)[4], uint4 (&w1)[4], int& r0, int& r1) {
        r0 = ptr[min(grp, cnt - 1)]; r1 = ptr[min(grp + 8, cnt - 1)];
        const uint4* s0 = reinterpret_cast<const uint4*>(kbase + size_t(r0) * kD);
        const uint4* s1 = reinterpret_cast<const uint4*>(kbase + size_t(r1) * kD);
#pragma unroll
        for (int c = 0; c < 4; ++c) { w0[c] = __ldg(s0 + c); w1[c] = __ldg(s1 + c); }
      };
      auto compute = [&](const uint4 (&w0)[4], const uint4 (&w1)[4], int r0, int r1, int cnt) {   // cnt in [1, 16] flagged blocks
        double c2[2][4];                                       // two independent accumulation chains
#pragma unroll
        for (int q = 0; q < 2; ++q)
#pragma unroll
          for (int i = 0; i < 4; ++i) c2[q][i] = 0.0;
#pragma unroll
        for (int step = 0; step < 8; ++step) {
          double ax[8];
          const T* e0 = reinterpret_cast<const T*>(&w0[step >> 1]) + (step & 1) * 4;
          const T* e1 = reinterpret_cast<const T*>(&w1[step >> 1]) + (step & 1) * 4;
#pragma unroll
          for (int c = 0; c < 4; ++c) { ax[2 * c] = to_f64(e0[c]); ax[2 * c + 1] = to_f64(e1[c]); }
          const double* qrow = &qs[grp * kQS + (step * 4 + tig) * 4];
          const double2 b01 = *reinterpret_cast<const double2*>(qrow);
          const double2 b23 = *reinterpret_cast<const double2*>(qrow + 2);
          double* cc = c2[step & 1];
          asm volatile(
              "mma.sync.aligned.m16n8k16.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5,%6,%7,%8,%9,%10,%11}, "
              "{%12,%13,%14,%15}, {%0,%1,%2,%3};"
              : "+d"(cc[0]), "+d"(cc[1]), "+d"(cc[2]), "+d"(cc[3])
              : "d"(ax[0]), "d"(ax[1]), "d"(ax[2]), "d"(ax[3]), "d"(ax[4]), "d"(ax[5]), "d"(ax[6]), "d"(ax[7]),
                "d"(b01.x), "d"(b01.y), "d"(b23.x), "d"(b23.y));
        }
        // C[i]: block row grp + 8*(i/2), column 2*tig + (i%2)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const double xv = (c2[0][i] + c2[1][i]) * es_d;
          const int rowi = grp + 8 * (i >> 1);
          const int blk_i = (i >> 1) ? r1 : r0;
          if (rowi < cnt) {
            if (i & 1) { if (blk_i < lim1) acc1 += exp(xv - Mc1); }
            else       { if (blk_i < lim0) acc0 += exp(xv - Mc0); }
          }
        }
      };

      int qn = 0;
      const uint32_t* lm = masks + l * n_words;
      const int words = n_tiles * 4;
      for (int w0i = 0; w0i < words; w0i += 32) {
        const int wi = w0i + lane;
        const uint32_t word = wi < words ? lm[wi] : 0u;
        const int c = __popc(word);
        int incl = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += t;
        }
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        int pos = qn + incl - c;
        uint32_t wbits = word;
        while (wbits) {
          const int bit = __ffs(wbits) - 1;
          wbits &= wbits - 1;
          queue[pos++] = uint16_t(wi * 32 + bit);
        }
        __syncwarp();
#ifdef CP_LSE_DEBUG
        if (lane == 0) atomicAdd(reinterpret_cast<unsigned long long*>(reinterpret_cast<char*>(a.st) + 192), (unsigned long long)total);
#endif
        qn += total;
        const int n_full = qn >> 4;                            // full tiles of 16 flagged blocks available now
        if (n_full > 0) {
          uint4 cw0[4], cw1[4], nw0[4], nw1[4];
          int cr0, cr1, nr0 = 0, nr1 = 0;
          load_rows(queue, 16, cw0, cw1, cr0, cr1);
          for (int t = 0; t < n_full; ++t) {
            if (t + 1 < n_full) load_rows(queue + 16 * (t + 1), 16, nw0, nw1, nr0, nr1);   // in flight under this tile's MMAs
            compute(cw0, cw1, cr0, cr1, 16);
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) { cw0[c4] = nw0[c4]; cw1[c4] = nw1[c4]; }
            cr0 = nr0; cr1 = nr1;
          }
        }
        const int head = n_full * 16, left = qn - head;        // < 16 left over
        uint16_t keep = 0;
        if (lane < left) keep = queue[head + lane];
        __syncwarp();
        if (lane < left) queue[lane] = keep;
        __syncwarp();
        qn = left;
      }
      if (qn > 0) {
        uint4 cw0[4], cw1[4];
        int cr0, cr1;
        load_rows(queue, qn, cw0, cw1, cr0, cr1);
        compute(cw0, cw1, cr0, cr1, qn);
      }
      // totals of the two columns over the 8 block rows held by lanes with equal tig
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) {
        acc0 += __shfl_xor_sync(0xffffffffu, acc0, o);
        acc1 += __shfl_xor_sync(0xffffffffu, acc1, o);
      }
      if (grp == 0) { exact_sum[mc * 2 + kr] = acc0; exact_sum[(mc + 1) * 2 + kr] = acc1; }
    }
  }
  __syncthreads();
#ifdef CP_LSE_DEBUG
  if (blockIdx.x == 0 && tid == 0) {
    long long* dbg = reinterpret_cast<long long*>(reinterpret_cast<char*>(a.st) + 200);
    dbg[0] = t_sweeps - t_start; dbg[1] = clock64() - t_sweeps;
  }
#endif
  if (!aborted && my_valid) {
    // row my_row = (segment, representative rep = my_row % 2): Qmax rows give l1 (Kmax) and l2 (Kmin), Qmin rows l3 and l4
    const double tot = double(asum) + exact_sum[my_row * 2 + my_kr];
    a.stats[row_unit(my_row) * 4 + (my_row & 1) * 2 + my_kr] = double(Mx) + log(tot);
  }
  if (aborted) {
    for (int i = 0; i < 200; ++i) __nanosleep(1000);       // let copies and MMAs in flight land before the CTA's resources go
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 9) tmem_dealloc(bars->tmem_base, 512);
}

// [B*Hkv, n2, 128] 16-bit summaries; box = 64 channels x `rows` blocks
bool make_kmap(CUtensorMap* map, const void* base, long long heads, int n2, int rows, bool f16) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[3] = {cuuint64_t(kD), cuuint64_t(n2), cuuint64_t(heads)};
  cuuint64_t strides[2] = {cuuint64_t(kD) * 2, cuuint64_t(n2) * kD * 2};
  cuuint32_t box[3] = {64, cuuint32_t(rows), 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides,
            box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

int launch_lse(const cp_params& p, const Dims& m, char* ws, cudaStream_t st) {
  const WsLayout w = ws_layout(m);
  double* stats = reinterpret_cast<double*>(ws + w.stats);
  const bool f16 = p.dtype == CP_F16;
  if (!((p.dtype == CP_BF16 || f16) && m.d == kD)) return launch_score_generic(p, m, ws, nullptr, nullptr, stats, st);
  LseArgs a;
  a.Qmax = ws + w.qmax; a.Qmin = ws + w.qmin; a.Kmax = ws + w.kmax; a.Kmin = ws + w.kmin;
  a.kabs = reinterpret_cast<const float*>(ws + w.kabs);
  a.stats = stats;
  a.st = reinterpret_cast<DeviceStatus*>(ws);
  a.Hq = m.Hq; a.g = m.g; a.U = m.g % 4 == 0 ? 4 : (m.g % 2 == 0 ? 2 : 1);
  a.n1 = m.n1; a.n2 = m.n2; a.seg = m.seg; a.blk = m.blk;
  // a CTA has 128 logit rows = 64 / U segments; on mid-sized problems fewer segments per CTA (rows left unused) put more
  // SMs to work on the sweeps and the exact pass, which run per CTA one after the other
  a.segs_per_cta = 64 / a.U;
  const long long per_chunk = (long long)m.B * m.Hkv * (m.g / a.U);
  while (a.segs_per_cta > 4 && per_chunk * ((m.n1 + a.segs_per_cta - 1) / a.segs_per_cta) < 100) a.segs_per_cta /= 2;
  a.n_qchunks = (m.n1 + a.segs_per_cta - 1) / a.segs_per_cta;
  a.mask_first = (p.flags & CP_FLAG_MASK_BEFORE_SOFTMAX) ? 1 : 0;
  a.box_rows = m.n2 < kTileN ? m.n2 : kTileN;
  a.es = p.est_scale;
  CUtensorMap tmKmax, tmKmin;
  const long long heads = (long long)m.B * m.Hkv;
  if (!make_kmap(&tmKmax, a.Kmax, heads, m.n2, a.box_rows, f16) || !make_kmap(&tmKmin, a.Kmin, heads, m.n2, a.box_rows, f16))
    return CP_ERR_CUDA;
  const int n_words = ((m.n2 + kTileN - 1) / kTileN) * 4;
  const size_t smem = size_t(kSmemFixed) + size_t(kLists) * n_words * 4 + size_t(kWarps) * kQueue * 2 + kRows * 3 * 4 +
                      kRows * 2 * 8 + sizeof(LseBars) + 1024;
  if (smem > 227 * 1024) return launch_score_generic(p, m, ws, nullptr, nullptr, stats, st);
  auto kern = f16 ? lse_sm100_kernel<true> : lse_sm100_kernel<false>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess) return CP_ERR_CUDA;
  const long long ctas = heads * (m.g / a.U) * a.n_qchunks;
  if (ctas > 0x7fffffffLL) return CP_ERR_UNSUPPORTED;
  kern<<<unsigned(ctas), kThreads, smem, st>>>(tmKmax, tmKmin, a);
  return check_launch();
}

}  // namespace cp

// K4 / K5: block-sparse (Algorithm 2, lines 6-13) and dense causal (Eq. 2) attention on the
// sm_100a tensor cores.  bf16 or fp16 operands, fp32 accumulation in tensor memory, online softmax.
//
// Persistent CTAs (one per SM) walk over work units; a unit is 256 consecutive query rows of one
// (batch, query head): two 128-row tiles "A" and "B" that share every K/V tile the producer brings in
// (tile B is absent in the last unit of a segment with an odd number of 128-row tiles).  Roles (384 threads):
//   warps 0-3  softmax for tile A (one thread per query row)
//   warps 4-7  softmax for tile B
//   warp  8    TMA producer: K/V tiles through a 5-slot ring of 32 KB buffers; a gathered
//              tile is assembled from 128/blk boxes addressed by the block list
//   warp  9    MMA issuer (warps 10-11 idle; they complete the third warpgroup): S = Q K^T
//              (operands in shared memory), O += P V (P read from tensor memory, where the
//              softmax warps overwrite S with 16-bit probabilities)
// Tensor memory (512 columns): S_A | S_B | O_A | O_B, 128 fp32 columns each.
// The tile sequence of a unit is: gathered past tiles, contiguous unmasked tiles, then the
// diagonal tiles; tile A stops one tile earlier than B.  Units are handed out by an atomic
// counter (producer warp) and published to the other warps.  Every wait is bounded: on
// expiry the waiter raises a CTA-wide abort flag and CP_ERR_TIMEOUT, and all roles drain.
#include "sm100_ptx.cuh"

namespace cp {
namespace {

constexpr int kD = 128;
constexpr int kTile = 128;
constexpr int kHalfBytes = kTile * 64 * 2;   // [128 rows x 64 cols] of 16-bit elements, 128-byte swizzled
constexpr int kTileBytes = 2 * kHalfBytes;   // both halves of head_dim
constexpr int kSlots = 5;
constexpr int kThreads = 384;   // 3 warpgroups: softmax A, softmax B, {producer, MMA, 2 idle}
constexpr int kSmemQ = 0;
constexpr int kSmemKV = 2 * kTileBytes;
constexpr int kSmemBar = kSmemKV + kSlots * kTileBytes;
constexpr int kBarBytes = 512;
constexpr int kSmemTotal = kSmemBar + kBarBytes + 1024;   // + barrier block + slack to align the tiles to 1024 bytes
constexpr float kRescaleThreshold = 8.0f;           // in log2 units
#ifndef CP_EMUL_EVERY
#define CP_EMUL_EVERY 8
#endif
constexpr int kEmulEvery = CP_EMUL_EVERY;           // 0: all exponentials on the MUFU; n: every n-th pair on the FMA pipes
constexpr int kRegPoolNeeded = 256 * 216 + 128 * 64;   // registers the roles hold after setmaxnreg (softmax 216, producer/MMA 64)

// One work unit, decoded (the producer warp decodes it once and publishes it to the other warps:
// the decoding is a chain of integer divisions that would otherwise sit at the start of every unit).
struct Unit {
  int b, h, kvh;
  int q_tok;        // first query row of tile A
  int n_past;       // listed blocks strictly before the segment
  int n_past_tiles; // gathered tiles
  int last_cols;    // valid key columns of the last gathered tile
  int c_tok, n_cont;// contiguous unmasked tiles: first token, count
  int d_tok;        // first token of diagonal tile d0 (d1 follows)
  int T;            // K/V tiles the unit streams
  int nA, nB;       // tiles query tile A / B consumes (nB = 0: the unit has no tile B)
  const int32_t* list;
  int seg_j;
  int rj;           // diagonal blocks of the segment (r, fewer in a short last segment)
  int cnt;
  int generic;      // the list is not "past blocks, then exactly the diagonal blocks": every listed block is gathered and
                    // every tile is masked element by element (a key counts iff its token is not after the query's)
  int rowsB;        // the unit has a second 128-row query tile
};

struct Bars {
  unsigned long long q_full;
  unsigned long long q_empty;
  unsigned long long kv_full[kSlots];
  unsigned long long kv_empty[kSlots];
  unsigned long long s_full[2];
  unsigned long long p_full[2];
  unsigned long long o_done[2];
  unsigned long long sched_full[2];
  unsigned long long sched_empty[2];
  int sched_unit[2];
  Unit sched_u[2];                   // the published unit, decoded; its cnt carries kBadList / kEmptyUnit
  uint32_t tmem_base;
  volatile int abort_flag;
};

struct Args {
  const int32_t* idx;
  const int32_t* cnt;
  uint16_t* O;                  // bf16 or fp16 elements
  float* lse;
  DeviceStatus* st;
  int B, Hq, Hkv, g, n, seg, blk, k, r, n1, n2;
  int64_t osb, osh, ost;
  float sm_scale;
  int dense;
  int n_units;
  int o_vec32;                  // O rows are 32-byte aligned: the epilogue may use 32-byte stores
  int emul;                     // long units: part of the exponentials on the FMA pipes (see launch_attention_sm100)
  int withhold_v;               // test hook: the producer never issues V tiles, so a bounded wait must expire
  unsigned int* work_counter;   // next unit to hand out (zeroed by the host before the launch)
};

// Optional event trace (compiled only with -DCP_TRACE, never in the product build): in CTA 0 the first softmax warp of
// each query tile, the producer and the MMA warp each append (clock, tag) pairs for units 4..7 to a region of their own
// in the workspace behind the status block (plain stores, a counter in a register: the traced warp never waits).
#ifdef CP_TRACE
__device__ __forceinline__ unsigned long long trace_clock() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%clock64;" : "=l"(t) :: "memory");
  return t;
}
#define CP_EV_DECL unsigned ev_n = 0
#define CP_EV(cond, q, tag) do { if ((cond) && blockIdx.x == 0 && (q) >= 4u && (q) < 8u && ev_n < 1024u) { \
    reinterpret_cast<unsigned long long*>(reinterpret_cast<char*>(a.st) + 4096)[((tag) / 100 - 1 + ((tag) >= 110 && (tag) < 120 ? 3 : 0)) * 1024 + ev_n++] = \
        (trace_clock() << 12) | (unsigned long long)(tag); } } while (0)
#else
#define CP_EV_DECL
#define CP_EV(cond, q, tag) do { } while (0)
#endif

// bounded wait on one of this kernel's barriers (the CTA's abort flag lives in the barrier block)
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity, Bars* bars, DeviceStatus* st, int site) {
  return mbar_wait(bar, parity, &bars->abort_flag, st, site);
}

// ---------------------------------------------------------------- unit geometry

// Units are ordered KV-head-major so that CTAs resident at the same time share K/V tiles in
// L2; within a KV head the dense kernel takes the longest rows first.
// `cnt` is the unit's list length when the caller already has it, kLoadCnt to read it from global memory.
constexpr int kLoadCnt = -2, kBadList = -1, kEmptyUnit = -3, kZeroUnit = -4;   // kEmptyUnit: no query row of the unit lies inside the sequence;
                                                                                // kZeroUnit: an empty list -- the unit's rows are zeros
__device__ __forceinline__ Unit decode_unit(const Args& a, int x, int cnt) {
  Unit u;
  u.list = nullptr;
  u.cnt = 0;
  if (a.dense) {
    const int ntiles = (a.n + kTile - 1) / kTile;
    const int np = (ntiles + 1) / 2;
    const int per_kvh = a.g * np;
    const int bkv = x / per_kvh;
    const int rest = x - bkv * per_kvh;
    const int pair = np - 1 - rest / a.g;
    const int gi = rest % a.g;
    u.b = bkv / a.Hkv; u.kvh = bkv % a.Hkv; u.h = u.kvh * a.g + gi;
    u.q_tok = pair * 256;
    u.n_past = 0; u.n_past_tiles = 0; u.last_cols = kTile;
    u.c_tok = 0; u.n_cont = 2 * pair; u.d_tok = pair * 256;
    u.seg_j = 0; u.rj = 0;
    u.nB = (2 * pair + 1 < ntiles) ? 1 : 0;
  } else {
    const int q_tiles = a.seg / kTile;
    const int pp = (q_tiles + 1) / 2;
    const int gi_p = a.g * pp;
    const int per_kvh = a.n1 * gi_p;
    const int bkv = x / per_kvh;
    const int rest = x - bkv * per_kvh;
    const int j = a.n1 - 1 - rest / gi_p;
    const int gi = (rest % gi_p) / pp;
    const int p = rest % pp;
    u.b = bkv / a.Hkv; u.kvh = bkv % a.Hkv; u.h = u.kvh * a.g + gi;
    u.seg_j = j;
    u.q_tok = j * a.seg + p * 256;
    const long long unit = ((long long)u.b * a.Hq + u.h) * a.n1 + j;
    u.list = a.idx + unit * a.k;
    u.cnt = cnt == kLoadCnt ? a.cnt[unit] : cnt;
    u.rj = min(a.n2, (j + 1) * a.r) - j * a.r;
    u.n_past = min(max(u.cnt - u.rj, 0), a.k);
    u.n_past_tiles = (u.n_past * a.blk + kTile - 1) / kTile;
    u.last_cols = u.n_past * a.blk - (u.n_past_tiles - 1) * kTile;
    u.c_tok = j * a.seg; u.n_cont = 2 * p; u.d_tok = u.q_tok;
    u.nB = (2 * p + 1 < q_tiles && u.q_tok + kTile < a.n) ? 1 : 0;   // tile B exists and starts inside the sequence
  }
  u.generic = 0;
  u.rowsB = u.nB ? 1 : 0;
  u.nA = u.n_past_tiles + u.n_cont + 1;       // up to and including its own diagonal tile
  u.nB = u.nB ? u.nA + 1 : 0;                 // one more diagonal tile; 0 when the segment has an odd tile count
  u.T = u.nB ? u.nB : u.nA;
  return u;
}

// The list contract, checked by the producer warp before it publishes a unit: at most k entries, ascending, unique,
// each a block the segment can see (0 <= b < (j+1)*r).  Returns 0 when the list has the form the selection emits
// (past blocks, then exactly the diagonal blocks of the segment: the fast tile sequence applies), 1 for any other
// valid list (generic tile sequence), -1 for a list that breaks the contract.
__device__ __forceinline__ int classify_unit(const Args& a, const Unit& u, int lane) {
  if (a.dense) return 0;
  const int vis = min(a.n2, (u.seg_j + 1) * a.r);
  bool gen_ok = (u.cnt >= 0) && (u.cnt <= a.k);
  bool std_ok = gen_ok && (u.cnt >= u.rj);
  if (gen_ok) {
    for (int i = lane; i < u.cnt; i += 32) {
      const int v = u.list[i];
      const bool asc = v >= 0 && v < vis && (i == 0 || u.list[i - 1] < v);
      gen_ok = gen_ok && asc;
      if (i >= u.n_past) std_ok = std_ok && (v == u.seg_j * a.r + (i - u.n_past));
      else std_ok = std_ok && asc && v < u.seg_j * a.r;
    }
  }
  gen_ok = __all_sync(0xffffffffu, gen_ok);
  std_ok = __all_sync(0xffffffffu, std_ok);
  return !gen_ok ? -1 : (std_ok ? 0 : 1);
}

__device__ __forceinline__ bool stop_requested(const Args& a, Bars* bars) {
  return bars->abort_flag || (a.st != nullptr && *reinterpret_cast<volatile int32_t*>(&a.st->code) == CP_ERR_TIMEOUT);
}

// ---------------------------------------------------------------- unit scheduler
// Units are handed out dynamically (an atomic counter in global memory) so that SMs that run
// faster take more of them.  The producer warp draws the q-th unit of this CTA, reads and checks
// its block list, and publishes (unit, list length) through a two-entry ring; the MMA warp and
// the eight softmax warps take it from there and touch no global memory at a unit's start.
// A list that breaks its contract is published with length kBadList and skipped by everyone.
__device__ __forceinline__ bool publish_unit(const Args& a, Bars* bars, uint32_t q, int lane, int* x_out, Unit* u_out) {
  const uint32_t slot = q & 1;
  if (q >= 2 && !mbar_wait(&bars->sched_empty[slot], ((q >> 1) - 1) & 1, bars, a.st, 50)) return false;
  int x = 0;
  if (lane == 0) x = int(min(atomicAdd(a.work_counter, 1u), 0x7fffffffu));
  x = __shfl_sync(0xffffffffu, x, 0);
  int cnt = 0;
  if (x < a.n_units) {
    *u_out = decode_unit(a, x, kLoadCnt);
    cnt = u_out->cnt;
    if (u_out->q_tok >= a.n) {
      cnt = kEmptyUnit;                               // a short last segment has fewer units
    } else {
      const int cls = classify_unit(a, *u_out, lane);
      if (cls < 0) {
        if (lane == 0) report(a.st, CP_ERR_BOUNDS, 1, u_out->b, u_out->h, u_out->seg_j, u_out->cnt);
        cnt = kBadList;
      } else if (cls == 1) {
        // any other valid list: all listed blocks are gathered, both query tiles consume every tile
        u_out->generic = 1;
        u_out->n_past = cnt;
        u_out->n_past_tiles = (cnt * a.blk + kTile - 1) / kTile;
        u_out->last_cols = cnt * a.blk - (u_out->n_past_tiles - 1) * kTile;
        u_out->n_cont = 0;
        u_out->nA = u_out->n_past_tiles;
        u_out->nB = u_out->rowsB ? u_out->n_past_tiles : 0;
        u_out->T = u_out->n_past_tiles;
        if (u_out->T == 0) cnt = kZeroUnit;           // nothing listed: the rows are zeros
      }
    }
  }
  u_out->cnt = cnt;
  if (lane == 0) {
    bars->sched_unit[slot] = x;
    if (x < a.n_units) bars->sched_u[slot] = *u_out;
    mbar_arrive(&bars->sched_full[slot]);
  }
  *x_out = x;
  return true;
}
__device__ __forceinline__ bool receive_unit(const Args& a, Bars* bars, uint32_t q, int lane, int* x_out, Unit* u_out) {
  const uint32_t slot = q & 1;
  if (!mbar_wait(&bars->sched_full[slot], (q >> 1) & 1, bars, a.st, 51)) return false;
  *x_out = *reinterpret_cast<volatile int*>(&bars->sched_unit[slot]);
  if (*x_out < a.n_units) *u_out = bars->sched_u[slot];
  else u_out->cnt = kEmptyUnit;
  __syncwarp();
  if (lane == 0) mbar_arrive(&bars->sched_empty[slot]);
  return true;
}

// ---------------------------------------------------------------- softmax role
constexpr int kMaskNone = 0, kMaskCausal = 1, kMaskCols = 2, kMaskGeneric = 3;

template <bool kF16>
__device__ __forceinline__ void softmax_role(const Args& a, Bars* bars, int which, int warp_in_wg, int lane) {
  const uint32_t tm = bars->tmem_base;
  const uint32_t lane_off = uint32_t(warp_in_wg * 32) << 16;
  const uint32_t tS = tm + lane_off + which * 128;
  const uint32_t tO = tm + lane_off + 256 + which * 128;
  const int row = warp_in_wg * 32 + lane;
  const float c = a.sm_scale * 1.4426950408889634f;   // logits -> log2 units
  CP_EV_DECL;
  uint32_t n_tiles = 0;                               // S tiles consumed so far (all units)
  uint32_t n_units = 0;                               // units finished so far

  for (uint32_t q = 0;; ++q) {
    int x;
    Unit u;
    if (!receive_unit(a, bars, q, lane, &x, &u) || x >= a.n_units || bars->abort_flag) return;
    if (u.cnt == kBadList || u.cnt == kEmptyUnit) continue;
    if (u.cnt == kZeroUnit) {
      // an empty list: no key is visible to any row of the unit -- zeros, and lse = ln 0
      const int t = u.q_tok + which * kTile + row;
      if ((which == 0 || u.rowsB) && t < a.n) {
        uint4* dst = reinterpret_cast<uint4*>(a.O + u.b * a.osb + u.h * a.osh + int64_t(t) * a.ost);
#pragma unroll
        for (int i = 0; i < kD * 2 / 16; ++i) dst[i] = make_uint4(0u, 0u, 0u, 0u);
        if (a.lse != nullptr) a.lse[((long long)u.b * a.Hq + u.h) * a.n + t] = -CUDART_INF;
      }
      continue;
    }
    const int my_tiles = which == 0 ? u.nA : u.nB;
    if (my_tiles == 0) continue;                        // this unit has no tile B
    float m_run = -CUDART_INF, l_run = 0.f;

    for (int jt = 0; jt < my_tiles; ++jt, ++n_tiles) {
      CP_EV(warp_in_wg == 0 && lane == 0, q, 100 + which * 10 + 0);          // waiting for S
      if (!mbar_wait(&bars->s_full[which], n_tiles & 1, bars, a.st, 10 + which)) return;
      CP_EV(warp_in_wg == 0 && lane == 0, q, 100 + which * 10 + 1);          // S ready
      tc_fence_after();
      uint32_t sv[128];
      tmem_ld128(tS, sv);
      tmem_wait_ld();
      float* s = reinterpret_cast<float*>(sv);

      int kind = kMaskNone, cols = kTile;
      if (u.generic) kind = kMaskGeneric;
      else if (jt == my_tiles - 1) kind = kMaskCausal;                              // own diagonal tile
      else if (jt == u.n_past_tiles - 1 && u.last_cols < kTile) { kind = kMaskCols; cols = u.last_cols; }
      if (kind == kMaskGeneric) {
        // a gathered tile of a generic list: the tile holds 128/blk listed blocks; key column i belongs to token
        // list[...]*blk + i % blk and counts iff that token is not after this row's token.  lim[q] = last visible
        // offset inside sub-block q (-1: none, also for sub-blocks beyond the list)
        const int t_row = u.q_tok + which * kTile + row;
        const int bpt = kTile / a.blk;
        int lim[4];
#pragma unroll
        for (int qq = 0; qq < 4; ++qq) {
          const int li = jt * bpt + qq;
          lim[qq] = (qq < bpt && li < u.cnt) ? t_row - __ldg(u.list + li) * a.blk : -1;
        }
        if (a.blk == 128) {
#pragma unroll
          for (int i = 0; i < 128; ++i) s[i] = (i > lim[0]) ? -CUDART_INF : s[i];
        } else if (a.blk == 64) {
#pragma unroll
          for (int i = 0; i < 128; ++i) s[i] = ((i & 63) > lim[i >> 6]) ? -CUDART_INF : s[i];
        } else {
#pragma unroll
          for (int i = 0; i < 128; ++i) s[i] = ((i & 31) > lim[i >> 5]) ? -CUDART_INF : s[i];
        }
      } else if (kind == kMaskCausal) {
#pragma unroll
        for (int i = 0; i < 128; ++i) s[i] = (i > row) ? -CUDART_INF : s[i];
      } else if (kind == kMaskCols) {
#pragma unroll
        for (int i = 0; i < 128; ++i) s[i] = (i >= cols) ? -CUDART_INF : s[i];
      }
      float mx0 = s[0], mx1 = s[1], mx2 = s[2], mx3 = s[3];
#pragma unroll
      for (int i = 4; i < 124; i += 8) {
        mx0 = max3(mx0, s[i], s[i + 1]); mx1 = max3(mx1, s[i + 2], s[i + 3]);
        mx2 = max3(mx2, s[i + 4], s[i + 5]); mx3 = max3(mx3, s[i + 6], s[i + 7]);
      }
      mx0 = max3(mx0, s[124], s[125]); mx1 = max3(mx1, s[126], s[127]);
      const float m_tile = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
      const float m_new = fmaxf(m_run, m_tile);
      // lazy rescale: keep the old reference maximum while the new one exceeds it by < 2^8
      const bool need = (m_new - m_run) * c > kRescaleThreshold;   // true on the first tile (m_run = -inf)
      if (jt == 0) {
        m_run = m_new;
      } else if (__any_sync(0xffffffffu, need)) {
        const float f = need ? ex2((m_run - m_new) * c) : 1.f;
        if (need) { m_run = m_new; l_run *= f; }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t ov[32];
          tmem_ld32(tO + q * 32, ov);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * f);
          tmem_st32(tO + q * 32, ov);
        }
      }
      const float neg_mc = (m_run == -CUDART_INF) ? 0.f : -m_run * c;   // a row that has not seen a key yet (generic lists only): exp2(-inf) = 0
      const float2 c2 = make_float2(c, c), nm2 = make_float2(neg_mc, neg_mc);
      float2 sum2 = make_float2(0.f, 0.f);
      uint32_t pk[64];
      if (kind == kMaskNone && a.emul) {
        // unmasked tile of a long unit: every kEmulEvery-th pair takes the polynomial path, the rest the MUFU
#pragma unroll
        for (int i = 0; i < 128; i += 2) {
          const float2 xx = __ffma2_rn(make_float2(s[i], s[i + 1]), c2, nm2);
          float2 p;
          if (kEmulEvery > 0 && (i >> 1) % kEmulEvery == kEmulEvery - 1) { p = exp2_poly2(xx); }
          else { p.x = ex2(xx.x); p.y = ex2(xx.y); }
          sum2 = __fadd2_rn(sum2, p);
          pk[i >> 1] = pack2<kF16>(p.x, p.y);
        }
      } else {
#pragma unroll
        for (int i = 0; i < 128; i += 2) {
          const float2 xx = __ffma2_rn(make_float2(s[i], s[i + 1]), c2, nm2);
          float2 p;
          p.x = ex2(xx.x); p.y = ex2(xx.y);
          sum2 = __fadd2_rn(sum2, p);
          pk[i >> 1] = pack2<kF16>(p.x, p.y);
        }
      }
      l_run += sum2.x + sum2.y;
      tmem_st64(tS, pk);
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bars->p_full[which]);
      CP_EV(warp_in_wg == 0 && lane == 0, q, 100 + which * 10 + 2);          // P handed over
    }

    // epilogue: O / l -> bf16 -> global.  The next unit's first PV cannot start before this
    // thread signals its next P, so O is not overwritten while it is being read.
    if (!mbar_wait(&bars->o_done[which], n_units & 1, bars, a.st, 20 + which)) return;
    CP_EV(warp_in_wg == 0 && lane == 0, q, 100 + which * 10 + 3);            // O complete
    ++n_units;
    tc_fence_after();
    const int t = u.q_tok + which * kTile + row;
    uint16_t* orow = a.O + u.b * a.osb + u.h * a.osh + int64_t(t) * a.ost;
    const float inv = l_run > 0.f ? 1.f / l_run : 0.f;   // a row without any visible key (generic lists only): zeros
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint32_t ov[32];
      tmem_ld32(tO + q * 32, ov);
      tmem_wait_ld();
      uint32_t w[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) w[i] = pack2<kF16>(__uint_as_float(ov[2 * i]) * inv, __uint_as_float(ov[2 * i + 1]) * inv);
      if (t < a.n) {                                 // rows past the end of the sequence (ragged last tile) are dropped
        if (a.o_vec32) {
          // 32-byte stores: every store fills whole 32-byte sectors (a thread owns a row, so the lanes of a
          // store instruction hit 32 different rows; 16-byte stores would touch every sector twice)
          st_global_v8(orow + q * 32, w);
          st_global_v8(orow + q * 32 + 16, w + 8);
        } else {
          uint4* dst = reinterpret_cast<uint4*>(orow + q * 32);
#pragma unroll
          for (int i = 0; i < 4; ++i) dst[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
        }
      }
    }
    if (a.lse != nullptr && t < a.n)
      a.lse[((long long)u.b * a.Hq + u.h) * a.n + t] = m_run * a.sm_scale + __logf(l_run);
    CP_EV(warp_in_wg == 0 && lane == 0, q, 100 + which * 10 + 4);            // epilogue done
  }
}

// ---------------------------------------------------------------- producer role
__device__ __forceinline__ void producer_role(const Args& a, Bars* bars, uint32_t smem_base, const CUtensorMap* tmQ,
                                              const CUtensorMap* tmKb, const CUtensorMap* tmVb,
                                              const CUtensorMap* tmKt, const CUtensorMap* tmVt, int lane) {
  const int bpt = kTile / a.blk;
  CP_EV_DECL;
  uint32_t item = 0;      // K/V tiles issued so far (all units): item i lives in slot i % kSlots
  uint32_t n_units = 0;
  // One unit of look-ahead: unit q+1 is drawn, checked and published before the loads of unit q
  // are issued, so the other warps never wait for the counter or for the list to be read.
  int x;
  Unit u;
  if (!publish_unit(a, bars, 0, lane, &x, &u)) return;
  for (uint32_t q = 0;; ++q) {
    if (x >= a.n_units) return;
    // Only this warp reads the status word in global memory (a round trip the other roles would otherwise
    // pay at every unit); it tells them through the CTA's abort flag, which their waits poll.
    if (stop_requested(a, bars)) { bars->abort_flag = 1; return; }
    const Unit u_cur = u;
    CP_EV(lane == 0, q, 300);                                                // producer starts unit q
    if (!publish_unit(a, bars, q + 1, lane, &x, &u)) return;
    CP_EV(lane == 0, q, 301);                                                // unit q+1 published
    if (u_cur.cnt == kBadList || u_cur.cnt == kEmptyUnit || u_cur.cnt == kZeroUnit) continue;
    // Q tiles: the buffer is free once every QK^T of the previous unit has completed
    if (n_units > 0 && !mbar_wait(&bars->q_empty, (n_units - 1) & 1, bars, a.st, 31)) return;
    CP_EV(lane == 0, q, 302);                                                // Q buffer free: Q loads go out
    if (lane == 0) {
      const int nq = u_cur.nB ? 2 : 1;
      mbar_expect_tx(&bars->q_full, nq * kTileBytes);
      for (int w = 0; w < nq; ++w)
        for (int hf = 0; hf < 2; ++hf)
          tma_load_4d(smem_base + kSmemQ + w * kTileBytes + hf * kHalfBytes, tmQ, &bars->q_full, hf * 64,
                      u_cur.q_tok + w * kTile, u_cur.h, u_cur.b);
    }
    ++n_units;
    for (int it = 0; it < 2 * u_cur.T; ++it, ++item) {   // 2*jt = K tile jt, 2*jt+1 = V tile jt
      const uint32_t slot = item % kSlots, use = item / kSlots;
      if (use > 0 && !mbar_wait(&bars->kv_empty[slot], (use - 1) & 1, bars, a.st, 30)) return;
      CP_EV(lane == 0, q, 310 + (it < 40 ? it : 40));                        // slot free: K/V item `it` goes out
      if (lane == 0 && !(a.withhold_v && (it & 1))) {
        const int jt = it >> 1;
        const bool is_v = it & 1;
        const uint32_t dst = smem_base + kSmemKV + slot * kTileBytes;
        unsigned long long* bar = &bars->kv_full[slot];
        mbar_expect_tx(bar, kTileBytes);
        if (jt < u_cur.n_past_tiles) {
          const CUtensorMap* tm = is_v ? tmVb : tmKb;
          for (int q = 0; q < bpt; ++q) {
            const int li = jt * bpt + q;
            // boxes beyond the list read past the end of the tensor and arrive as zeros
            const int tok = li < u_cur.n_past ? u_cur.list[li] * a.blk : a.n;
            for (int hf = 0; hf < 2; ++hf)
              tma_load_4d(dst + hf * kHalfBytes + q * a.blk * 128, tm, bar, hf * 64, tok, u_cur.kvh, u_cur.b);
          }
        } else {
          const CUtensorMap* tm = is_v ? tmVt : tmKt;
          const int ci = jt - u_cur.n_past_tiles;
          const int tok = ci < u_cur.n_cont ? u_cur.c_tok + ci * kTile : u_cur.d_tok + (ci - u_cur.n_cont) * kTile;
          for (int hf = 0; hf < 2; ++hf) tma_load_4d(dst + hf * kHalfBytes, tm, bar, hf * 64, tok, u_cur.kvh, u_cur.b);
        }
      }
      __syncwarp();
    }
  }
}

// ---------------------------------------------------------------- MMA role
template <bool kF16>
__device__ __forceinline__ void issue_qk(uint32_t d_tmem, uint32_t q_smem, uint32_t k_smem) {
  const uint64_t base = desc_base(16);
#pragma unroll
  for (int kk = 0; kk < kD / 16; ++kk) {
    const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
    umma_ss(d_tmem, desc_at(base, q_smem + off), desc_at(base, k_smem + off), Idesc<kF16>::qk, kk > 0);
  }
}
template <bool kF16>
__device__ __forceinline__ void issue_pv(uint32_t d_tmem, uint32_t p_tmem, uint32_t v_smem, bool acc) {
  const uint64_t base = desc_base(kHalfBytes);   // the two 64-column halves of head_dim are 16 KB apart
#pragma unroll
  for (int kk = 0; kk < kTile / 16; ++kk)
    umma_ts(d_tmem, p_tmem + kk * 8, desc_at(base, v_smem + kk * 16 * 128), Idesc<kF16>::pv, (acc || kk > 0) ? 1u : 0u);
}

template <bool kF16>
__device__ __forceinline__ void mma_role(const Args& a, Bars* bars, uint32_t smem_base, int lane) {
  const uint32_t tm = __shfl_sync(0xffffffffu, bars->tmem_base, 0);
  const uint32_t tS[2] = {tm, tm + 128}, tO[2] = {tm + 256, tm + 384};
  const uint32_t qA = smem_base + kSmemQ, qB = qA + kTileBytes;
  CP_EV_DECL;
  uint32_t item0 = 0;                 // first K/V item of the current unit
  uint32_t nA = 0, nB = 0;            // P tiles consumed so far per query tile (all units)
  uint32_t n_units = 0;
  auto slot_addr = [&](uint32_t item) { return smem_base + kSmemKV + (item % kSlots) * kTileBytes; };
  auto full_wait = [&](uint32_t item) {
    return mbar_wait(&bars->kv_full[item % kSlots], (item / kSlots) & 1, bars, a.st, 40);
  };
  for (uint32_t q = 0;; ++q) {
    int x;
    Unit u;
    CP_EV(lane == 0, q, 205);                                                // asks for the unit
    if (!receive_unit(a, bars, q, lane, &x, &u) || x >= a.n_units || bars->abort_flag) return;
    if (u.cnt == kBadList || u.cnt == kEmptyUnit || u.cnt == kZeroUnit) continue;
    const int T = u.T, TA = u.nA;
    const bool hasB = u.nB > 0;
    CP_EV(lane == 0, q, 200);                                                // unit received
    if (!mbar_wait(&bars->q_full, n_units & 1, bars, a.st, 41)) return;
    CP_EV(lane == 0, q, 201);                                                // Q ready
    if (!full_wait(item0)) return;
    CP_EV(lane == 0, q, 202);                                                // K0 ready
    tc_fence_after();
    issue_qk<kF16>(tS[0], qA, slot_addr(item0)); umma_commit(&bars->s_full[0]);
    if (hasB) { issue_qk<kF16>(tS[1], qB, slot_addr(item0)); umma_commit(&bars->s_full[1]); }
    umma_commit(&bars->kv_empty[item0 % kSlots]);
    if (T == 1) umma_commit(&bars->q_empty);               // a one-tile unit has no further QK^T
    for (int jt = 0; jt < T; ++jt) {
      const bool has_next = jt + 1 < T;
      const uint32_t iv = item0 + 2 * jt + 1, ik = item0 + 2 * (jt + 1);
      if (has_next && !full_wait(ik)) return;
      if (!full_wait(iv)) return;
      const uint32_t v_smem = slot_addr(iv), kn_smem = slot_addr(ik);
      if (jt < TA) {
        if (!mbar_wait(&bars->p_full[0], nA & 1, bars, a.st, 42)) return;
        CP_EV(lane == 0, q, 210);                                            // P_A ready
        ++nA;
        tc_fence_after();
        issue_pv<kF16>(tO[0], tS[0], v_smem, jt > 0);
        if (jt + 1 < TA) { issue_qk<kF16>(tS[0], qA, kn_smem); umma_commit(&bars->s_full[0]); }
        else umma_commit(&bars->o_done[0]);
      }
      if (hasB) {
        CP_EV(lane == 0, q, 211);                                            // group A issued
        if (!mbar_wait(&bars->p_full[1], nB & 1, bars, a.st, 43)) return;
        CP_EV(lane == 0, q, 212);                                            // P_B ready
        ++nB;
        tc_fence_after();
        issue_pv<kF16>(tO[1], tS[1], v_smem, jt > 0);
      }
      umma_commit(&bars->kv_empty[iv % kSlots]);             // every PV that reads this V tile has been issued
      if (has_next) {
        if (hasB) { issue_qk<kF16>(tS[1], qB, kn_smem); umma_commit(&bars->s_full[1]); }
        umma_commit(&bars->kv_empty[ik % kSlots]);
        if (jt + 1 == T - 1) umma_commit(&bars->q_empty);   // that was the unit's last QK^T: Q may be replaced
      } else if (hasB) {
        umma_commit(&bars->o_done[1]);
      }
      CP_EV(lane == 0, q, 213);                                              // tile step issued
    }
    item0 += 2 * T;
    ++n_units;
  }
}

// ---------------------------------------------------------------- kernel
template <bool kF16>
__global__ void __launch_bounds__(kThreads, 1)
attention_sm100_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKb,
                       const __grid_constant__ CUtensorMap tmVb, const __grid_constant__ CUtensorMap tmKt,
                       const __grid_constant__ CUtensorMap tmVt, const Args a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t smem_base = (raw + 1023u) & ~1023u;
  static_assert(sizeof(Bars) <= kBarBytes, "barrier block too small");
  Bars* bars = reinterpret_cast<Bars*>(smem_raw + (smem_base - raw) + kSmemBar);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    mbar_init(&bars->q_full, 1);
    mbar_init(&bars->q_empty, 1);
    for (int i = 0; i < kSlots; ++i) { mbar_init(&bars->kv_full[i], 1); mbar_init(&bars->kv_empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&bars->s_full[i], 1); mbar_init(&bars->p_full[i], 128); mbar_init(&bars->o_done[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&bars->sched_full[i], 1); mbar_init(&bars->sched_empty[i], 9); }
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 8 && lane == 0) {
    prefetch_tmap(&tmQ); prefetch_tmap(&tmKb); prefetch_tmap(&tmVb); prefetch_tmap(&tmKt); prefetch_tmap(&tmVt);
  }
  if (warp == 9) { tmem_alloc(&bars->tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  // Register re-partition.  The pool is what the CTA was launched with (384 threads x 168):
  // 256 x 216 + 128 x 64 = 63488 fits; asking for more than the pool would block forever.
  static_assert(kRegPoolNeeded <= kThreads * 168, "setmaxnreg budget exceeds the launch allocation");
  if (warp < 8) {
    reg_inc<216>();
    softmax_role<kF16>(a, bars, warp >> 2, warp & 3, lane);
  } else {
    reg_dec<64>();
    if (warp == 8) producer_role(a, bars, smem_base, &tmQ, &tmKb, &tmVb, &tmKt, &tmVt, lane);
    else if (warp == 9) mma_role<kF16>(a, bars, smem_base, lane);
  }
  if (bars->abort_flag) {
    // give copies and MMAs still in flight time to land before the CTA's resources go away
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 9) tmem_dealloc(bars->tmem_base, 512);
}

// ---------------------------------------------------------------- host side
// [B, H, n, 128] bf16 with element strides (sb, sh, st); box = 64 columns x `rows` tokens
bool make_map(CUtensorMap* map, const void* base, int B, int H, int n, const int64_t* s, int rows, bool f16) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[4] = {cuuint64_t(kD), cuuint64_t(n), cuuint64_t(H), cuuint64_t(B)};
  cuuint64_t strides[3] = {cuuint64_t(s[2]) * 2, cuuint64_t(s[1]) * 2, cuuint64_t(s[0]) * 2};
  cuuint32_t box[4] = {64, cuuint32_t(rows), 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool sm100_path_applies(const cp_params& p, const Dims& m) {
  return (p.dtype == CP_BF16 || p.dtype == CP_F16) && m.d == 128 && m.seg % kTile == 0 && (m.blk == 32 || m.blk == 64 || m.blk == 128) &&
         !(p.flags & CP_FLAG_FORCE_SIMT);
}

int launch_attention_sm100(const cp_params& p, const Dims& m, const void* Q, const void* K, const void* V,
                           const int32_t* idx, const int32_t* cnt, void* O, float* lse, DeviceStatus* st,
                           bool dense, cudaStream_t s) {
  CUtensorMap tmQ, tmKb, tmVb, tmKt, tmVt;
  const bool f16 = p.dtype == CP_F16;
  if (!make_map(&tmQ, Q, m.B, m.Hq, m.n, p.q_stride, kTile, f16) || !make_map(&tmKb, K, m.B, m.Hkv, m.n, p.k_stride, m.blk, f16) ||
      !make_map(&tmVb, V, m.B, m.Hkv, m.n, p.v_stride, m.blk, f16) || !make_map(&tmKt, K, m.B, m.Hkv, m.n, p.k_stride, kTile, f16) ||
      !make_map(&tmVt, V, m.B, m.Hkv, m.n, p.v_stride, kTile, f16))
    return CP_ERR_CUDA;
  Args a;
  a.idx = idx; a.cnt = cnt; a.O = static_cast<uint16_t*>(O); a.lse = lse; a.st = st;
  a.B = m.B; a.Hq = m.Hq; a.Hkv = m.Hkv; a.g = m.g; a.n = m.n; a.seg = m.seg; a.blk = m.blk; a.k = m.k;
  a.r = m.r; a.n1 = m.n1; a.n2 = m.n2;
  a.osb = p.o_stride[0]; a.osh = p.o_stride[1]; a.ost = p.o_stride[2];
  a.sm_scale = p.sm_scale; a.dense = dense ? 1 : 0;
  // a unit is two 128-row query tiles (one when a segment, or the sequence, has an odd tile count)
  const long long units = dense ? (long long)m.B * m.Hq * (((m.n + kTile - 1) / kTile + 1) / 2)
                                : (long long)m.B * m.Hq * m.n1 * ((m.seg / kTile + 1) / 2);
  if (units > 0x7fffffffLL) return CP_ERR_UNSUPPORTED;
  auto kern = f16 ? attention_sm100_kernel<true> : attention_sm100_kernel<false>;
  // setmaxnreg.inc blocks forever when the CTA's register pool (threads x registers the kernel was compiled
  // to) is smaller than what the roles ask for, and no bounded wait covers that: check the real allocation of
  // this build once per variant and refuse to launch instead.
  static int regs_ok[2] = {0, 0};   // 0 = not checked yet, 1 = fits, -1 = does not fit
  if (regs_ok[f16] == 0) {
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, kern) != cudaSuccess) return CP_ERR_CUDA;
    regs_ok[f16] = (fa.numRegs * kThreads >= kRegPoolNeeded) ? 1 : -1;
  }
  if (regs_ok[f16] < 0) return CP_ERR_UNSUPPORTED;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTotal) != cudaSuccess)
    return CP_ERR_CUDA;
  a.n_units = int(units);
  a.withhold_v = (p.flags & CP_FLAG_TEST_WITHHOLD_V) ? 1 : 0;
  // Moving every kEmulEvery-th pair of exponentials from the MUFU to the FMA pipes pays where units are long and the
  // kernel sits at the power cap (measured in 60-step loops: 1.6 % at 32 K/V tiles per unit) and costs where units are
  // short (3 % at 8 tiles per unit, the paper's operating point); a unit streams at most k*blk/128 tiles.
  a.emul = (dense || (long long)m.k * m.blk >= 12 * kTile) ? 1 : 0;
  a.o_vec32 = (reinterpret_cast<uintptr_t>(O) % 32 == 0 && p.o_stride[0] % 16 == 0 && p.o_stride[1] % 16 == 0 && p.o_stride[2] % 16 == 0) ? 1 : 0;
  a.work_counter = reinterpret_cast<unsigned int*>(reinterpret_cast<char*>(st) + 128);   // inside the status block
  if (cudaMemsetAsync(a.work_counter, 0, sizeof(unsigned int), s) != cudaSuccess) return CP_ERR_CUDA;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return CP_ERR_CUDA;
  // persistent CTAs, one per SM (the kernel takes all of an SM's tensor memory and shared memory)
  const unsigned grid = unsigned(units < sms ? units : sms);
  kern<<<grid, kThreads, kSmemTotal, s>>>(tmQ, tmKb, tmVb, tmKt, tmVt, a);
  return check_launch();
}

}  // namespace cp

// Upstream fusion: the projections of Eq. 1 (Q = W_Q X, K = W_K X, optionally V = W_V X) with rotary position embedding on Q and K, whose
// epilogue also produces the representatives of Algorithm 1, lines 3-8 (per-channel max / min of every query segment and
// key block), so that critiprefill_estimate can skip its own pass over Q and K.
//
// GEMM on the tcgen05 tensor cores: D[128 tokens x 128 channels] = X_tile[128 x d_model] * W_head[128 x d_model]^T per
// head; an output tile is 128 tokens of two adjacent heads of one kind (one head where a kind has an odd head count),
// so that both heads share the X operand of every MMA.  A work unit is (batch, head group, segment): its seg/128 token
// tiles run back to back on one CTA, so the segment's running max / min stay on chip.  Warps 0-3: epilogue (one thread
// per token row: tensor-memory load, rotation, rounding, stores; then one thread per channel for the column scans), warp 4:
// TMA producer (X and W tiles of 64 d_model columns, 128-byte swizzle), warp 5: MMA issuer; the accumulator stages in
// tensor memory let the epilogue of one tile run under the main loop of the next.  The value heads (Eq. 1, no rotation, no
// representatives) follow the query / key units as a pass of their own.  Every wait is bounded.
#include "sm100_ptx.cuh"

namespace cp {
namespace {

constexpr int kThreads = 192;
constexpr int kD = 128;                       // head_dim = channels per output tile
constexpr int kTileM = 128;                   // tokens per output tile
constexpr int kKB = 64;                       // d_model columns per pipeline stage (one 128-byte swizzled row)
constexpr int kOpBytes = 128 * kKB * 2;       // one operand tile of a stage: 128 rows x 64 columns, 16-bit
constexpr int kTStride = 132;                 // row stride (16-bit elements) of the transposition tile: conflict-free column reads
constexpr int kMaxRing = 5, kMaxAcc = 4;
// kNH = heads per output tile.  Two adjacent heads of one kind share the X operand of every MMA (M128 N256 K16): a stage
// then carries 16 KB of X for 32 KB of W instead of 16 + 16, which takes a quarter off the shared-memory and L2 traffic per
// FLOP; the ring has 4 stages of 48 KB instead of 5 of 32 KB and tensor memory holds 2 accumulator stages of 256 columns.
template <int kNH> struct Geo {
  static constexpr int kStageBytes = (1 + kNH) * kOpBytes;     // X tile + W tile(s)
  static constexpr int kRing = kNH == 2 ? 4 : 5;
  static constexpr int kAcc = 4 / kNH;                         // accumulator stages (512 columns in all)
  static constexpr int kSmemT = kRing * kStageBytes;
  static constexpr int kSmemBar = kSmemT + kTileM * kTStride * 2;
};

struct ProjBars {
  unsigned long long full[kMaxRing], empty[kMaxRing], acc_full[kMaxAcc], acc_empty[kMaxAcc];
  uint32_t tmem_base;
  volatile int abort_flag;
  float red[4];
};

struct ProjArgs {
  uint16_t *Q, *K, *V;                        // outputs, 16-bit elements (V nullable: no value projection)
  int64_t qsb, qsh, qst, ksb, ksh, kst, vsb, vsh, vst;   // element strides (batch, head, token)
  const float *cosT, *sinT;                   // [n, 64] fp32, nullable together: no rotation
  uint16_t *Qmax, *Qmin, *Kmax, *Kmin;        // summaries in the workspace
  float* kabs;
  DeviceStatus* st;
  int B, Hq, Hkv, Hv, n, seg, blk, n1, n2, d_model;   // Hv = Hkv when values are projected too, else 0
  long long n_units;
};

__device__ __forceinline__ float bf16_bits_to_f32(uint16_t v) { return __uint_as_float(uint32_t(v) << 16); }
template <bool kF16> __device__ __forceinline__ float elem_to_f32(uint16_t v) {
  if (kF16) return __half2float(*reinterpret_cast<const __half*>(&v));
  return bf16_bits_to_f32(v);
}

__device__ __forceinline__ void bar_sync_epilogue() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

template <bool kF16, int kNH>
__global__ void __launch_bounds__(kThreads, 1)
project_sm100_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmWq,
                     const __grid_constant__ CUtensorMap tmWk, const __grid_constant__ CUtensorMap tmWv, const ProjArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t smem_base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (smem_base - raw);
  constexpr int kStageBytes = Geo<kNH>::kStageBytes, kRing = Geo<kNH>::kRing, kAcc = Geo<kNH>::kAcc;
  uint16_t* tileT = reinterpret_cast<uint16_t*>(sm + Geo<kNH>::kSmemT);
  ProjBars* bars = reinterpret_cast<ProjBars*>(sm + Geo<kNH>::kSmemBar);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int i = 0; i < kRing; ++i) { mbar_init(&bars->full[i], 1); mbar_init(&bars->empty[i], 1); }
    for (int i = 0; i < kAcc; ++i) { mbar_init(&bars->acc_full[i], 1); mbar_init(&bars->acc_empty[i], 128); }
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 4 && lane == 0) { prefetch_tmap(&tmX); prefetch_tmap(&tmWq); prefetch_tmap(&tmWk); prefetch_tmap(&tmWv); }
  if (warp == 5) { tmem_alloc(&bars->tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = bars->tmem_base;

  const int Hqk = (a.Hq + a.Hkv) / kNH;    // head groups (kNH adjacent heads of one kind) in the order query, key, value
  const long long n_qk_units = (long long)a.B * Hqk * a.n1;
  const int tiles_per_seg = a.seg / kTileM;
  const int n_kb = a.d_model / kKB;
  // unit -> (segment j, batch b, head hh); heads of one segment are adjacent so that its X rows stay in L2.  The value
  // heads follow in a pass of their own after all query / key units: with all three weight matrices live at once
  // the weights and the X tiles in flight no longer fit the L2 share of a die and every head slows down
  auto decode = [&](long long u, int* b, int* hh, int* j) {
    const bool vpass = u >= n_qk_units;
    if (vpass) u -= n_qk_units;
    const int H = vpass ? a.Hv / kNH : Hqk;
    *hh = (int(u % H) + (vpass ? Hqk : 0)) * kNH; u /= H;      // first head of the group
    *b = int(u % a.B); u /= a.B;
    *j = int(u);
  };
  auto n_tiles_of = [&](int j) { return min(tiles_per_seg, (a.n - j * a.seg + kTileM - 1) / kTileM); };

  if (warp == 4) {
    // ---------------- TMA producer
    uint32_t it = 0;
    for (long long u = blockIdx.x; u < a.n_units; u += gridDim.x) {
      int b, hh, j;
      decode(u, &b, &hh, &j);
      const CUtensorMap* tw = hh < a.Hq ? &tmWq : (hh < a.Hq + a.Hkv ? &tmWk : &tmWv);
      const int wrow = (hh < a.Hq ? hh : (hh < a.Hq + a.Hkv ? hh - a.Hq : hh - a.Hq - a.Hkv)) * kD;
      const int nt = n_tiles_of(j);
      for (int t = 0; t < nt; ++t) {
        const int tok0 = j * a.seg + t * kTileM;
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const uint32_t s = it % kRing, use = it / kRing;
          if (use > 0 && !mbar_wait(&bars->empty[s], (use - 1) & 1, &bars->abort_flag, a.st, 70)) return;
          if (lane == 0) {
            const uint32_t dst = smem_base + s * kStageBytes;
            mbar_expect_tx(&bars->full[s], kStageBytes);
            tma_load_3d(dst, &tmX, &bars->full[s], kb * kKB, tok0, b);            // rows past n arrive as zeros
            tma_load_3d(dst + kOpBytes, tw, &bars->full[s], kb * kKB, wrow, 0);   // 128 * kNH weight rows
          }
          __syncwarp();
        }
      }
    }
  } else if (warp == 5) {
    // ---------------- MMA issuer
    uint32_t it = 0, tile_no = 0;
    const uint64_t base = desc_base(16);
    // M = 128, N = 128 * kNH (bits 17-22 hold N / 8)
    constexpr uint32_t kIdesc = (Idesc<kF16>::qk & ~(0x3fu << 17)) | ((uint32_t(kD * kNH) >> 3) << 17);
    for (long long u = blockIdx.x; u < a.n_units; u += gridDim.x) {
      int b, hh, j;
      decode(u, &b, &hh, &j);
      const int nt = n_tiles_of(j);
      for (int t = 0; t < nt; ++t, ++tile_no) {
        const uint32_t as = tile_no % kAcc;
        if (tile_no >= kAcc && !mbar_wait(&bars->acc_empty[as], ((tile_no / kAcc) - 1) & 1, &bars->abort_flag, a.st, 71)) return;
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const uint32_t s = it % kRing;
          if (!mbar_wait(&bars->full[s], (it / kRing) & 1, &bars->abort_flag, a.st, 72)) return;
          tc_fence_after();
          const uint32_t xa = smem_base + s * kStageBytes, wa = xa + kOpBytes;
#pragma unroll
          for (int kk = 0; kk < kKB / 16; ++kk)
            umma_ss(tm + as * kD * kNH, desc_at(base, xa + kk * 32), desc_at(base, wa + kk * 32), kIdesc, (kb > 0 || kk > 0) ? 1u : 0u);
          umma_commit(&bars->empty[s]);
        }
        umma_commit(&bars->acc_full[as]);
      }
    }
  } else {
    // ---------------- epilogue: thread = token row for the rotation and the stores, then thread = channel for the scans
    const int row = tid;                         // 0..127
    const uint32_t t_row = tm + (uint32_t(warp * 32) << 16);
    uint32_t tile_no = 0;
    for (long long u = blockIdx.x; u < a.n_units; u += gridDim.x) {
      int b, hh, j;
      decode(u, &b, &hh, &j);
      const bool is_q = hh < a.Hq, is_v = hh >= a.Hq + a.Hkv;
      const int h0 = is_q ? hh : (is_v ? hh - a.Hq - a.Hkv : hh - a.Hq);   // first head of the group within its kind
      const int nt = n_tiles_of(j);
      float seg_max[kNH], seg_min[kNH];                            // channel `tid` over the segment (query heads)
#pragma unroll
      for (int sub = 0; sub < kNH; ++sub) { seg_max[sub] = -CUDART_INF_F; seg_min[sub] = CUDART_INF_F; }
      for (int t = 0; t < nt; ++t, ++tile_no) {
        const uint32_t as = tile_no % kAcc;
        const int tok0 = j * a.seg + t * kTileM;
        const int tok = tok0 + row;
        if (!mbar_wait(&bars->acc_full[as], (tile_no / kAcc) & 1, &bars->abort_flag, a.st, 73)) return;
        tc_fence_after();
#pragma unroll
       for (int sub = 0; sub < kNH; ++sub) {                       // the heads of the group, 128 accumulator columns each
        const int h = h0 + sub;
        uint32_t acc[128];
        tmem_ld128(t_row + as * kD * kNH + sub * kD, acc);
        tmem_wait_ld();
        if (sub == kNH - 1) {
          tc_fence_before();
          mbar_arrive(&bars->acc_empty[as]);                       // the accumulator is in registers: its stage is free
        }
        float* x = reinterpret_cast<float*>(acc);
        if (a.cosT != nullptr && !is_v && tok < a.n) {
          // rotary embedding, rotate-half form: channel i pairs with channel i + 64
          const float4* c4 = reinterpret_cast<const float4*>(a.cosT + size_t(tok) * 64);
          const float4* s4 = reinterpret_cast<const float4*>(a.sinT + size_t(tok) * 64);
#pragma unroll
          for (int q = 0; q < 16; ++q) {
            const float4 c = __ldg(c4 + q), s = __ldg(s4 + q);
            const float cc[4] = {c.x, c.y, c.z, c.w}, ss[4] = {s.x, s.y, s.z, s.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int i = q * 4 + e;
              const float lo = x[i], hi = x[i + 64];
              x[i] = lo * cc[e] - hi * ss[e];
              x[i + 64] = hi * cc[e] + lo * ss[e];
            }
          }
        }
        uint32_t w[64];
#pragma unroll
        for (int i = 0; i < 64; ++i) w[i] = pack2<kF16>(x[2 * i], x[2 * i + 1]);
        if (tok < a.n) {
          uint16_t* orow = is_q ? a.Q + b * a.qsb + h * a.qsh + int64_t(tok) * a.qst
                         : (is_v ? a.V + b * a.vsb + h * a.vsh + int64_t(tok) * a.vst : a.K + b * a.ksb + h * a.ksh + int64_t(tok) * a.kst);
          uint4* dst = reinterpret_cast<uint4*>(orow);
#pragma unroll
          for (int i = 0; i < 16; ++i) dst[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
        }
        if (is_v) continue;                                        // values: Eq. 1 alone, Algorithm 1 takes nothing from them
        // the rounded row goes to shared memory; then every thread scans one channel over the tile's rows
        uint32_t* trow = reinterpret_cast<uint32_t*>(tileT + row * kTStride);
#pragma unroll
        for (int i = 0; i < 64; ++i) trow[i] = w[i];
        bar_sync_epilogue();
        const int rows_valid = min(kTileM, a.n - tok0);
        const int c = tid;
        if (is_q) {
          for (int r = 0; r < rows_valid; ++r) {
            const float v = elem_to_f32<kF16>(tileT[r * kTStride + c]);
            seg_max[sub] = fmaxf(seg_max[sub], v); seg_min[sub] = fminf(seg_min[sub], v);
          }
        } else {
          // key heads: one (max, min) per block of blk tokens, written straight away; kabs = largest magnitude of the block's summaries
          for (int g0 = 0; g0 < rows_valid; g0 += a.blk) {
            float mx = -CUDART_INF_F, mn = CUDART_INF_F;
            const int g1 = min(g0 + a.blk, rows_valid);
            for (int r = g0; r < g1; ++r) {
              const float v = elem_to_f32<kF16>(tileT[r * kTStride + c]);
              mx = fmaxf(mx, v); mn = fminf(mn, v);
            }
            const long long blkid = (long long)(b * a.Hkv + h) * a.n2 + (tok0 + g0) / a.blk;
            const uint16_t hmx = uint16_t(pack2<kF16>(mx, 0.f) & 0xffffu), hmn = uint16_t(pack2<kF16>(mn, 0.f) & 0xffffu);
            a.Kmax[blkid * kD + c] = hmx;
            a.Kmin[blkid * kD + c] = hmn;
            float am = fmaxf(fabsf(mx), fabsf(mn));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, o));
            if (lane == 0) bars->red[warp] = am;
            bar_sync_epilogue();
            if (tid == 0) a.kabs[blkid] = fmaxf(fmaxf(bars->red[0], bars->red[1]), fmaxf(bars->red[2], bars->red[3]));
            bar_sync_epilogue();
          }
        }
        bar_sync_epilogue();                                       // the tile may be overwritten by the next one
       }
      }
      if (is_q) {
#pragma unroll
        for (int sub = 0; sub < kNH; ++sub) {
          const long long unit = ((long long)b * a.Hq + h0 + sub) * a.n1 + j;
          a.Qmax[unit * kD + tid] = uint16_t(pack2<kF16>(seg_max[sub], 0.f) & 0xffffu);
          a.Qmin[unit * kD + tid] = uint16_t(pack2<kF16>(seg_min[sub], 0.f) & 0xffffu);
        }
      }
    }
  }
  if (bars->abort_flag) {
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) tmem_dealloc(bars->tmem_base, 512);
}

// rows x d_model 16-bit matrix, row-major; box = 64 columns x 128 rows; third dimension = batches of `rows` rows
bool make_map3(CUtensorMap* map, const void* base, int d_model, long long rows, long long batches, bool f16, int box_rows = 128) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[3] = {cuuint64_t(d_model), cuuint64_t(rows), cuuint64_t(batches)};
  cuuint64_t strides[2] = {cuuint64_t(d_model) * 2, cuuint64_t(rows) * cuuint64_t(d_model) * 2};
  cuuint32_t box[3] = {cuuint32_t(kKB), cuuint32_t(rows < box_rows ? rows : box_rows), 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides,
            box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

int launch_project(const cp_params& p, const Dims& m, const void* X, const void* Wq, const void* Wk, const void* Wv,
                   const float* cosT, const float* sinT, int d_model, void* Q, void* K, void* V, char* ws, cudaStream_t st) {
  const bool f16 = p.dtype == CP_F16;
  if (!((p.dtype == CP_BF16 || f16) && m.d == kD && m.seg % kTileM == 0 && (m.blk == 32 || m.blk == 64 || m.blk == 128) &&
        d_model % kKB == 0 && d_model >= kKB && m.n >= kTileM))
    return CP_ERR_UNSUPPORTED;
  const WsLayout w = ws_layout(m);
  ProjArgs a;
  a.Q = static_cast<uint16_t*>(Q); a.K = static_cast<uint16_t*>(K); a.V = static_cast<uint16_t*>(V);
  a.vsb = p.v_stride[0]; a.vsh = p.v_stride[1]; a.vst = p.v_stride[2];
  a.Hv = (Wv != nullptr) ? m.Hkv : 0;
  a.qsb = p.q_stride[0]; a.qsh = p.q_stride[1]; a.qst = p.q_stride[2];
  a.ksb = p.k_stride[0]; a.ksh = p.k_stride[1]; a.kst = p.k_stride[2];
  a.cosT = cosT; a.sinT = sinT;
  a.Qmax = reinterpret_cast<uint16_t*>(ws + w.qmax); a.Qmin = reinterpret_cast<uint16_t*>(ws + w.qmin);
  a.Kmax = reinterpret_cast<uint16_t*>(ws + w.kmax); a.Kmin = reinterpret_cast<uint16_t*>(ws + w.kmin);
  a.kabs = reinterpret_cast<float*>(ws + w.kabs);
  a.st = reinterpret_cast<DeviceStatus*>(ws);
  a.B = m.B; a.Hq = m.Hq; a.Hkv = m.Hkv; a.n = m.n; a.seg = m.seg; a.blk = m.blk; a.n1 = m.n1; a.n2 = m.n2; a.d_model = d_model;
  // two heads per output tile where every kind has an even head count (see Geo)
  const int nh = (m.Hq % 2 == 0 && m.Hkv % 2 == 0) ? 2 : 1;
  a.n_units = (long long)m.B * ((m.Hq + m.Hkv + a.Hv) / nh) * m.n1;
  CUtensorMap tmX, tmWq, tmWk, tmWv;
  if (!make_map3(&tmX, X, d_model, m.n, m.B, f16) || !make_map3(&tmWq, Wq, d_model, (long long)m.Hq * kD, 1, f16, 128 * nh) ||
      !make_map3(&tmWk, Wk, d_model, (long long)m.Hkv * kD, 1, f16, 128 * nh))
    return CP_ERR_CUDA;
  if (Wv == nullptr) tmWv = tmWk;
  else if (!make_map3(&tmWv, Wv, d_model, (long long)m.Hkv * kD, 1, f16, 128 * nh)) return CP_ERR_CUDA;
  auto kern = nh == 2 ? (f16 ? project_sm100_kernel<true, 2> : project_sm100_kernel<false, 2>)
                      : (f16 ? project_sm100_kernel<true, 1> : project_sm100_kernel<false, 1>);
  const int smem = (nh == 2 ? Geo<2>::kSmemBar : Geo<1>::kSmemBar) + int(sizeof(ProjBars)) + 1024;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return CP_ERR_CUDA;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return CP_ERR_CUDA;
  const unsigned grid = unsigned(a.n_units < sms ? a.n_units : sms);
  kern<<<grid, kThreads, smem, st>>>(tmX, tmWq, tmWk, tmWv, a);
  return check_launch();
}

}  // namespace cp

// Persistent warp-specialised GEMM for sm_100a:  C[M,N] = A[M,K] * Wt[N,K]^T  (+ fused epilogue).
//
// A (activations, fp16, row-major [M,K]) and Wt (weights, fp16, row-major [N,K]) are both K-major.
// Two CTAs on neighbouring SMs (a cluster of 2) share one 256x256 output tile: each CTA loads its own
// 128 rows of A and one half (128 rows) of the Wt tile per 64-wide K step (TMA, 128-byte swizzle,
// 6-stage ring of 32 KB), and one thread of the leader CTA issues tcgen05.mma.cta_group::2
// (256x256x16, kind::f16, fp32 accumulate).  Each CTA ends up with its 128 rows x 256 columns in one of
// two TMEM accumulators, so the epilogue of a tile overlaps the main loop of the next.  Compared with
// one CTA per 128x256 tile this halves the shared-memory and L2 traffic for the weight operand.
// No TMA multicast is used: both CTAs' loads report their bytes to the leader's barrier, and
// tcgen05.commit (multicast over the pair) releases stages and publishes accumulators in both CTAs.
// Warp roles (12 warps = 3 warpgroups): 0 = TMA producer, 1 = MMA issuer (leader CTA only) and TMEM owner,
// 2..3 = none (they fill the first warpgroup, so that registers can be re-balanced per warpgroup), 4..11 =
// epilogue: two warps per TMEM lane quarter, one for each half of the tile's columns.  In the steady state the
// epilogue is hidden under the next tile's main loop; it is exposed in a launch's last wave, which is the whole
// launch for a small batch, and there eight warps with their requests issued ahead (residual rows before the
// accumulator is complete, bias / gate / scale vectors one chunk ahead) finish it in half the time of four.
// Tiles are taken in a fixed order and every output element is accumulated over K in the same order whatever
// M is: a row's result does not depend on where it sits in the batch.
//
// Epilogues (the fused parts of the adaLN-Zero block):
//   kEpiBiasF16      out16 = acc + bias                                   (QKV projection)
//   kEpiBiasGeluF16  out16 = gelu_tanh(acc + bias)                        (MLP up-projection)
//   kEpiGateResidF32 out32 = resid + gate[request(row)] * (acc + bias)    (attention / MLP output)
//   kEpiBiasF32      out32 = acc + bias                                   (output projection of the final layer)
//   kEpiQkvF16       out16 = acc + bias, then per head of HD columns, for the Q and K thirds only:
//                    optional RMS-norm with a learned [HD] scale and optional 2-D rotary term
//                    (a head's columns sit in one thread, so both are thread-local)
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace dit {

enum GemmEpilogue : int { kEpiBiasF16 = 0, kEpiBiasGeluF16 = 1, kEpiGateResidF32 = 2, kEpiBiasF32 = 3, kEpiQkvF16 = 4 };

struct GemmParams {
  int M, N, K;
  int band;                 // > 0: row tiles (of 256 rows) per band of the tile order; < 0: column tiles per band
  const float* bias;        // [N]
  __half* out16;            // [M, N] with row stride ld16 elements (0 = N)
  const float* resid;       // [M, N]
  float* out32;             // [M, N]
  const float* gate;        // gate vector of request 0 for this block; request r at gate + r * gate_stride
  long long gate_stride;
  int ld16;
  int row0;                 // packed row index of row 0 of A / out (a launch may cover a slice of the batch's rows)
  int* status;              // device status word
  // kEpiQkvF16 only
  const float* q_norm;      // [HD] RMS-norm scale of the queries, NULL = no RMS-norm
  const float* k_norm;      // [HD] same for the keys
  const float* rope_theta;  // [(HD - HD/8) / 4] pair frequencies of one axis group, NULL = no rotary term
  int hidden;               // H: columns [0,H) are Q, [H,2H) K, [2H,3H) V
  float eps;
  // two-stream launches (DUAL) only: row-tile items, and the text stream's epilogue tensors
  const int* items;         // item i = row tile (low 24 bits) | stream << 24; a tile holding rows of both
                            // streams appears twice and each pass stores only its own stream's rows
  const int* num_items;
  const float* bias2;       // text stream's bias
  const float* q_norm2;
  const float* k_norm2;
  long long gate_kind_stride;   // text stream's gate vector = gate + gate_kind_stride
  // FP8 launches only: A and Wt hold e4m3 codes; out = acc * row_scale[m] * col_scale[n] + bias
  const float* row_scale;   // [M]
  const float* col_scale;   // [N]
  int operand_bf16;         // A and Wt hold bf16 instead of fp16 (same tensor maps: 16-bit elements)
  int* probe;               // measurement hook, NULL normally: [0] SM clock in MHz seen by a CTA of this launch
                            // (cycle counter against the global nanosecond timer over the CTA's life)
};

namespace gemm_cfg {
constexpr int BM = 128, BN = 256, BK = 64, STAGES = 6;     // BM: rows per CTA; the pair covers 2*BM x BN
constexpr int A_BYTES = BM * BK * 2;
constexpr int B_BYTES = (BN / 2) * BK * 2;                  // this CTA's half of the weight tile
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int EPI_WARPS = 8;                       // two per quarter of the accumulator's rows, each takes half of the columns
// Warpgroup 0 = {TMA warp, MMA warp, two warps without a role}, warpgroups 1 and 2 = epilogue.  Registers are
// re-balanced per warpgroup (setmaxnreg): each scheduler of the SM hosts one warp of each warpgroup, and ten warps
// at one common budget would leave the epilogue 168 registers, too few for its residual rows in flight.
constexpr int THREADS = 128 + 32 * EPI_WARPS;
constexpr int REGS_ISSUE = 56, REGS_EPILOGUE = 224;   // (56 + 2 * 224) * 32 <= 16384 per scheduler
// per epilogue warp: 16 rows x 32 fp32 columns with rows padded to 144 bytes (the fp32 epilogues pass their 32 rows
// through in two halves), or 32 rows x 32 16-bit columns with rows padded to 80 bytes
constexpr int EPI_STAGE_FLOATS = 640;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/ + EPI_WARPS * EPI_STAGE_FLOATS * 4;
}  // namespace gemm_cfg

__device__ __forceinline__ float gelu_tanh_f32(float z) {
  const float k0 = 0.7978845608028654f, k1 = 0.044715f;
  float y = k0 * (z + k1 * z * z * z);
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(y));
  return 0.5f * z * (1.0f + t);
}
// The same function on two values with packed fp32 arithmetic (the epilogue shares its scheduler with
// the MMA-issuing and the TMA-issuing warps: fewer instructions leave them more issue slots).
__device__ __forceinline__ float2 gelu_tanh_f32x2(float2 z) {
  const float k0 = 0.7978845608028654f, k1 = 0.044715f;
  const float2 inner = ffma2(fmul2(z, z), make_float2(k0 * k1, k0 * k1), make_float2(k0, k0));
  const float2 y = fmul2(inner, z);
  float2 t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t.x) : "f"(y.x));
  asm("tanh.approx.f32 %0, %1;" : "=f"(t.y) : "f"(y.y));
  const float2 hz = fmul2(z, make_float2(0.5f, 0.5f));
  return ffma2(hz, t, hz);
}

// Tile order.  band > 0: row tiles are grouped in bands of `band`; inside a band the row index runs fastest and
// every column tile is visited before the next band starts.  The tiles in flight then share one band of A (sized
// by the host to stay in L2) while the weight tiles stream past, each read from DRAM once per band.
// band < 0: the same with the roles swapped: column tiles in bands of -band whose weight tiles stay in L2 while
// the rows of A stream past, each read once per band.  The host picks whichever reads less from DRAM.
__device__ __forceinline__ void tile_coords(int t, int num_m, int num_n, int band, int& mb, int& nb) {
  if (band > 0) {
    const int per_band = band * num_n;
    const int b = t / per_band, r = t - b * per_band;
    const int rows = min(band, num_m - b * band);               // the last band may be shorter
    nb = r / rows;
    mb = b * band + (r - nb * rows);
  } else {
    const int cb = -band;
    const int per_band = cb * num_m;
    const int b = t / per_band, r = t - b * per_band;
    const int cols = min(cb, num_n - b * cb);
    mb = r / cols;
    nb = b * cb + (r - mb * cols);
  }
}

// DUAL: two-stream launch.  The weight operand comes from tmB for image-token rows and from tmB2 for
// text-token rows; the row tiles to visit are listed in p.items (built on the device from the batch's
// geometry), everything else is unchanged.
// FP8: both operands are e4m3 (1 byte per element, 128 elements per 128-byte swizzled row, K = 32
// per MMA); the row and column scales that map the codes back are applied in the epilogue.
// BF16: the 16-bit outputs are written as bf16 instead of fp16 (bf16-operand mode; the operands' format
// itself is a run-time field of the instruction descriptor, p.operand_bf16).
template <int EPI, int HD = 0, bool DUAL = false, bool FP8 = false, bool BF16 = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(gemm_cfg::THREADS, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmB2, const GemmParams p,
                    const __grid_constant__ SeqInfo seq, const __grid_constant__ RowGeom geo) {
  using namespace gemm_cfg;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* aligned = smem_raw + (base - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(aligned + STAGES * STAGE_BYTES);
  // bars: [0,S) full (used in the leader), [S,2S) empty, [2S,2S+2) tmem_full, [2S+2,2S+4) tmem_empty (leader)
  const uint32_t bar0 = base + STAGES * STAGE_BYTES;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + 2 + a); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* epi_stage = reinterpret_cast<float*>(aligned + STAGES * STAGE_BYTES + 256);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  long long probe_c0 = 0; uint64_t probe_t0 = 0;
  if (p.probe && threadIdx.x == 0) { probe_c0 = clock64(); probe_t0 = global_ns(); }
  const uint32_t rank = cluster_ctarank();                    // 0 = leader of the pair
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int num_m = DUAL ? *p.num_items : (p.M + 2 * BM - 1) / (2 * BM);   // row tiles (DUAL: row-tile items)
  const int num_n = (p.N + BN - 1) / BN;
  const int num_tiles = num_m * num_n;                        // 256 x 256 tiles
  // row tile and stream of item ib
  auto item_of = [&](int ib, int& mb, int& kind) {
    if (DUAL) { const int it = __ldg(p.items + ib); mb = it & 0xFFFFFF; kind = it >> 24; }
    else { mb = ib; kind = 0; }
  };
  constexpr int BKE = FP8 ? 2 * BK : BK;                      // elements of K per stage (128 bytes per row)
  const int num_k = (p.K + BKE - 1) / BKE;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 2 * EPI_WARPS); }
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0 && lane == 0) { prefetch_tmap(&tmA); prefetch_tmap(&tmB); if (DUAL) prefetch_tmap(&tmB2); }
  if (warp == 1) { tmem_alloc_pair(smem_u32(tmem_slot), 512); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                         // both CTAs' barriers exist before any remote arrive
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp < 4) {
    DIT_SETMAXNREG_DEC(REGS_ISSUE);
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      for (int t = pair; t < num_tiles; t += num_pairs) {
        int ib, mb, nb, kind;
        tile_coords(t, num_m, num_n, p.band, ib, nb);
        item_of(ib, mb, kind);
        const CUtensorMap* tb = (DUAL && kind) ? &tmB2 : &tmB;
        const int m0 = mb * (2 * BM) + rank * BM;             // this CTA's rows of A
        const int n0 = nb * BN + rank * (BN / 2);             // this CTA's half of the weight tile
        for (int kb = 0; kb < num_k; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) goto done;
          const uint32_t full_leader = map_to_cta(full_bar(stage), 0);
          if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), 2 * STAGE_BYTES);   // both CTAs' bytes
          const uint32_t sa = base + stage * STAGE_BYTES;
          tma_load_2d_pair(sa, &tmA, kb * BKE, m0, full_leader);
          tma_load_2d_pair(sa + A_BYTES, tb, kb * BKE, n0, full_leader);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = FP8 ? idesc_e4m3(2 * BM, BN) : idesc_f16(2 * BM, BN, false, p.operand_bf16 != 0);
      int stage = 0; uint32_t phase = 0; int it = 0;
      for (int t = pair; t < num_tiles; t += num_pairs, ++it) {
        const int acc = it & 1; const uint32_t acc_phase = (it >> 1) & 1u;
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) goto done;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; kb < num_k; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) goto done;
          tc_fence_after();
          const uint32_t sa = base + stage * STAGE_BYTES;
          const uint64_t adesc = smem_desc_sw128(sa, 16, 1024);
          const uint64_t bdesc = smem_desc_sw128(sa + A_BYTES, 16, 1024);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) { // 32 bytes further along K inside the swizzled row
            if (FP8) umma_f8_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0);
            else umma_f16_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0);
          }
          umma_commit_pair(empty_bar(stage), 3);   // frees the stage in both CTAs once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        umma_commit_pair(tfull_bar(acc), 3);       // accumulator complete in both CTAs
      }
    }
  }
  } else {
    DIT_SETMAXNREG_INC(REGS_EPILOGUE);
    // ------------------------------------------------------------------ epilogue (8 warps)
    // Two warps share each quarter of the accumulator's rows; the first takes the tile's columns 0..127, the
    // second 128..255.  When a launch is a single wave (small batches), or in every launch's last wave, the
    // epilogue is not hidden under a next main loop: twice the warps keep twice the memory requests in flight.
    const int quarter = warp & 3;              // TMEM lanes this warp may read: [32*quarter, +32)
    const int chalf = (warp - 4) >> 2;         // which half of the tile's columns
    constexpr int kChunks = BN / 32 / 2;       // 32-column chunks per warp
    int it = 0;
    const uint32_t tempty_leader0 = map_to_cta(tempty_bar(0), 0), tempty_leader1 = map_to_cta(tempty_bar(1), 0);
    for (int t = pair; t < num_tiles; t += num_pairs, ++it) {
      const int acc = it & 1; const uint32_t acc_phase = (it >> 1) & 1u;
      int ib, mb, nb, kind;
      tile_coords(t, num_m, num_n, p.band, ib, nb);
      item_of(ib, mb, kind);
      const int m0 = mb * (2 * BM) + rank * BM, n0 = nb * BN;
      const int row = m0 + quarter * 32 + lane;
      // gated-residual epilogue: request of this lane's row, and whether the warp's rows share it
      int my_req = -1;
      if ((EPI == kEpiGateResidF32 || DUAL) && row < p.M) my_req = find_request(seq, row + p.row0);
      // two-stream launch: this pass stores only the rows of its own stream
      int my_kind = -1;
      if (DUAL && row < p.M) my_kind = row_kind(seq, geo, my_req, row + p.row0);
      const bool row_ok = row < p.M && (!DUAL || my_kind == kind);
      const float sa = (FP8 && row < p.M) ? p.row_scale[row] : 1.0f;
      const float* bias = (DUAL && kind) ? p.bias2 : p.bias;
      const float* gate = p.gate + ((DUAL && kind) ? p.gate_kind_stride : 0);
      const int req0 = __shfl_sync(0xffffffffu, my_req, 0);
      const bool one_req = __all_sync(0xffffffffu, my_req == req0 || my_req < 0);
      // fp32 epilogues: this lane stores columns (lane % 8) * 4 .. + 3 of rows it * 4 + lane / 8, it < 8
      int row_req[8];
      float row_sa[8];                       // FP8: the row scales of the rows this lane stores
      unsigned store_rows = 0;
      if (EPI == kEpiGateResidF32 || EPI == kEpiBiasF32) {
#pragma unroll
        for (int i8 = 0; i8 < 8; ++i8) {
          const int rr = i8 * 4 + (lane >> 3);
          row_req[i8] = __shfl_sync(0xffffffffu, my_req, rr);
          if (FP8) row_sa[i8] = __shfl_sync(0xffffffffu, sa, rr);
          const int rk = DUAL ? __shfl_sync(0xffffffffu, my_kind, rr) : 0;
          if (m0 + quarter * 32 + rr < p.M && (!DUAL || rk == kind)) store_rows |= 1u << i8;
        }
      }
      // Residual rows of this tile do not depend on the accumulator: three of this warp's four 32-column
      // chunks are requested before waiting for the MMAs, the fourth when the first has been consumed
      // (four at once would not fit the register file beside the accumulator chunk).
      const int cg = (lane & 7) * 4;
      constexpr int kResDepth = 3;
      float4 xres[kResDepth][8];
      auto load_resid = [&](int c, float4 (&x)[8]) {
        const int col = n0 + c * 32 + cg;
        if (EPI == kEpiGateResidF32 && col < p.N) {
#pragma unroll
          for (int it = 0; it < 8; ++it) {
            const int grow = m0 + quarter * 32 + it * 4 + (lane >> 3);
            if (grow < p.M) x[it] = *reinterpret_cast<const float4*>(p.resid + static_cast<size_t>(grow) * p.N + col);
          }
        }
      };
#pragma unroll
      for (int d = 0; d < kResDepth; ++d) load_resid(chalf * kChunks + d, xres[d]);
      if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(acc), acc_phase, abort_flag))) goto done;
      tc_fence_after();
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * BN;
      if constexpr (EPI == kEpiQkvF16) {
        // patch row and column of this lane's token (text tokens and rows past M: (0, 0))
        int py = 0, px = 0;
        if (p.rope_theta && row_ok) {
          const int rq = find_request(seq, row + p.row0);
          const int local = row + p.row0 - seq.cu[rq];
          if (local < geo.img_cu[rq + 1] - geo.img_cu[rq]) { py = local / geo.gw[rq]; px = local - py * geo.gw[rq]; }
        }
#pragma unroll 1
        for (int hl = 0; hl < BN / HD / 2; ++hl) {
          const int hc = chalf * (BN / HD / 2) + hl;
          const int colh = n0 + hc * HD;       // first column of this head; heads never straddle Q | K | V
          if (colh >= p.N) break;              // warp-uniform
          float v[HD];
#pragma unroll
          for (int q = 0; q < HD / 32; ++q) {
            uint32_t r[32];
            __syncwarp();                      // tcgen05.ld is warp-collective: reconverge first
            tmem_ld32(t_row + hc * HD + q * 32, r);
            tmem_ld_wait();
            const float4* bias4 = reinterpret_cast<const float4*>(bias + colh + q * 32);   // colh is a multiple of HD
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              const float4 b4 = __ldg(bias4 + (i >> 2));
              float2 a0 = make_float2(__uint_as_float(r[i]), __uint_as_float(r[i + 1]));
              float2 a1 = make_float2(__uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
              if (FP8) {
                const float4 cs = __ldg(reinterpret_cast<const float4*>(p.col_scale + colh + q * 32 + i));
                a0 = fmul2(a0, make_float2(sa * cs.x, sa * cs.y));
                a1 = fmul2(a1, make_float2(sa * cs.z, sa * cs.w));
              }
              a0 = fadd2(a0, make_float2(b4.x, b4.y));
              a1 = fadd2(a1, make_float2(b4.z, b4.w));
              v[q * 32 + i] = a0.x; v[q * 32 + i + 1] = a0.y; v[q * 32 + i + 2] = a1.x; v[q * 32 + i + 3] = a1.y;
            }
          }
          if (row_ok) {
            const int part = colh / p.hidden;  // 0 = Q, 1 = K, 2 = V
            if (part < 2) {
              const float* g = (DUAL && kind) ? (part == 0 ? p.q_norm2 : p.k_norm2) : (part == 0 ? p.q_norm : p.k_norm);
              if (g) {
                float2 ss2 = make_float2(0.f, 0.f);
#pragma unroll
                for (int i = 0; i < HD; i += 2) { const float2 t = make_float2(v[i], v[i + 1]); ss2 = ffma2(t, t, ss2); }
                const float rstd = rsqrtf((ss2.x + ss2.y) * (1.0f / HD) + p.eps);
                const float2 rs = make_float2(rstd, rstd);
#pragma unroll
                for (int i = 0; i < HD; i += 4) {
                  const float4 g4 = __ldg(reinterpret_cast<const float4*>(g + i));
                  const float2 o0 = fmul2(make_float2(v[i], v[i + 1]), fmul2(rs, make_float2(g4.x, g4.y)));
                  const float2 o1 = fmul2(make_float2(v[i + 2], v[i + 3]), fmul2(rs, make_float2(g4.z, g4.w)));
                  v[i] = o0.x; v[i + 1] = o0.y; v[i + 2] = o1.x; v[i + 3] = o1.y;
                }
              }
              if (p.rope_theta && (py | px)) {
                constexpr int DT = HD / 8, NA = (HD - DT) / 2;   // unrotated channels, channels per axis group
#pragma unroll
                for (int i = 0; i < NA / 2; ++i) {
                  const float th = __ldg(p.rope_theta + i);
                  float sy, cy, sx, cx;
                  // hardware sine/cosine: angles stay below a few hundred radians (patch index times a
                  // frequency <= 1), where their absolute error (~1e-5) is far below the fp16 output step
                  __sincosf(static_cast<float>(py) * th, &sy, &cy);
                  __sincosf(static_cast<float>(px) * th, &sx, &cx);
                  const float a = v[DT + 2 * i], b = v[DT + 2 * i + 1];
                  v[DT + 2 * i] = a * cy - b * sy;
                  v[DT + 2 * i + 1] = a * sy + b * cy;
                  const float c2 = v[DT + NA + 2 * i], d2 = v[DT + NA + 2 * i + 1];
                  v[DT + NA + 2 * i] = c2 * cx - d2 * sx;
                  v[DT + NA + 2 * i + 1] = c2 * sx + d2 * cx;
                }
              }
            }
            uint4* dst = reinterpret_cast<uint4*>(p.out16 + static_cast<size_t>(row) * p.N + colh);
#pragma unroll
            for (int q = 0; q < HD / 8; ++q) {
              uint32_t w[4];
#pragma unroll
              for (int h = 0; h < 4; ++h) {
                w[h] = pack16x2<BF16>(v[8 * q + 2 * h], v[8 * q + 2 * h + 1]);
              }
              dst[q] = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      } else {
      // fp32 epilogues: the bias, gate and column-scale values of a chunk are requested one chunk ahead, so
      // that their latency passes under the previous chunk's work instead of in front of every chunk
      float4 nb4 = make_float4(0.f, 0.f, 0.f, 0.f), ng4 = nb4, ncs4 = make_float4(1.f, 1.f, 1.f, 1.f);
      auto load_vectors = [&](int c) {
        const int col = n0 + c * 32 + cg;
        if ((EPI == kEpiGateResidF32 || EPI == kEpiBiasF32) && c < BN / 32 && col < p.N) {
          nb4 = __ldg(reinterpret_cast<const float4*>(bias + col));
          if (FP8) ncs4 = __ldg(reinterpret_cast<const float4*>(p.col_scale + col));
          if (EPI == kEpiGateResidF32 && one_req && req0 >= 0) ng4 = __ldg(reinterpret_cast<const float4*>(gate + req0 * p.gate_stride + col));
        }
      };
      // 16-bit epilogues: the 32 bias values of the next chunk, the same way
      float4 nbias[8];
      auto load_bias16 = [&](int c) {
        const int col0 = n0 + c * 32;
        if ((EPI == kEpiBiasF16 || EPI == kEpiBiasGeluF16) && c < BN / 32 && col0 + 32 <= p.N) {
#pragma unroll
          for (int v = 0; v < 8; ++v) nbias[v] = __ldg(reinterpret_cast<const float4*>(bias + col0) + v);
        }
      };
      load_vectors(chalf * kChunks);
      load_bias16(chalf * kChunks);
#pragma unroll
      for (int cl = 0; cl < kChunks; ++cl) {
        const int c = chalf * kChunks + cl;
        uint32_t r[32];
        const float4 b = nb4, g_one = ng4, cs = ncs4;
        float4 bias_now[8];
        if (EPI == kEpiBiasF16 || EPI == kEpiBiasGeluF16) {
#pragma unroll
          for (int v = 0; v < 8; ++v) bias_now[v] = nbias[v];
        }
        if (cl + 1 < kChunks) { load_vectors(c + 1); load_bias16(c + 1); }
        __syncwarp();                          // tcgen05.ld is warp-collective: reconverge first
        tmem_ld32(t_row + c * 32, r);
        tmem_ld_wait();
        const int col0 = n0 + c * 32;
        if (col0 >= p.N) continue;             // warp-uniform
        if (EPI == kEpiGateResidF32 || EPI == kEpiBiasF32) {
          // Transpose through shared memory so that each global access covers whole 128-byte row
          // segments: lane -> (row it*4 + lane/8, columns (lane%8)*4 .. +3).
          // Rows are padded to 36 floats: 16-byte accesses of both phases are free of bank conflicts.
          float* st = epi_stage + (warp - 4) * EPI_STAGE_FLOATS;
          const int col = col0 + cg;                        // N is a multiple of 64: the whole chunk is inside
          float4 g = g_one;
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {                  // rows 0..15 of the warp's 32, then rows 16..31
            if ((lane >> 4) == hf) {
#pragma unroll
              for (int i = 0; i < 32; i += 4)
                *reinterpret_cast<uint4*>(st + (lane & 15) * 36 + i) = make_uint4(r[i], r[i + 1], r[i + 2], r[i + 3]);
            }
            __syncwarp();
#pragma unroll
            for (int it = hf * 4; it < hf * 4 + 4; ++it) {
              const int rr = it * 4 + (lane >> 3);
              const int grow = m0 + quarter * 32 + rr;
              if ((store_rows >> it) & 1u) {
                if (EPI == kEpiGateResidF32 && !one_req) g = __ldg(reinterpret_cast<const float4*>(gate + row_req[it] * p.gate_stride + col));
                const float4 a = *reinterpret_cast<const float4*>(st + (rr & 15) * 36 + cg);
                float2 s0, s1;
                if (FP8) {     // codes back to values: row scale of the activations, column scale of the weights
                  const float sr = row_sa[it];
                  s0 = ffma2(make_float2(a.x, a.y), make_float2(sr * cs.x, sr * cs.y), make_float2(b.x, b.y));
                  s1 = ffma2(make_float2(a.z, a.w), make_float2(sr * cs.z, sr * cs.w), make_float2(b.z, b.w));
                } else {
                  s0 = fadd2(make_float2(a.x, a.y), make_float2(b.x, b.y));
                  s1 = fadd2(make_float2(a.z, a.w), make_float2(b.z, b.w));
                }
                float4 o;
                if (EPI == kEpiGateResidF32) {
                  const float4 x = xres[cl % kResDepth][it];
                  const float2 o0 = ffma2(make_float2(g.x, g.y), s0, make_float2(x.x, x.y));
                  const float2 o1 = ffma2(make_float2(g.z, g.w), s1, make_float2(x.z, x.w));
                  o = make_float4(o0.x, o0.y, o1.x, o1.y);
                } else {
                  o = make_float4(s0.x, s0.y, s1.x, s1.y);
                }
                *reinterpret_cast<float4*>(p.out32 + static_cast<size_t>(grow) * p.N + col) = o;
              }
            }
            __syncwarp();                      // the staging buffer is reused by the next half and the next chunk
          }
          if (EPI == kEpiGateResidF32 && cl + kResDepth < kChunks) load_resid(c + kResDepth, xres[cl % kResDepth]);
        } else {
          const bool full = (col0 + 32 <= p.N);            // warp-uniform
          const int ld = p.ld16 ? p.ld16 : p.N;
          if (full) {
            // fp16 results go through shared memory so that a store instruction covers 64 contiguous
            // bytes of each of 8 rows (whole sectors) instead of 16 bytes of each of 32 rows
            uint8_t* stb = reinterpret_cast<uint8_t*>(epi_stage + (warp - 4) * EPI_STAGE_FLOATS);
            uint4* srow = reinterpret_cast<uint4*>(stb + lane * 80);
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              uint32_t w[4];
              const float4 b0 = bias_now[2 * v], b1 = bias_now[2 * v + 1];   // col0 is a multiple of 32
              const float2 bb[4] = {make_float2(b0.x, b0.y), make_float2(b0.z, b0.w), make_float2(b1.x, b1.y), make_float2(b1.z, b1.w)};
#pragma unroll
              for (int h = 0; h < 4; ++h) {
                const int i = 8 * v + 2 * h;
                float2 ab = make_float2(__uint_as_float(r[i]), __uint_as_float(r[i + 1]));
                if (FP8) { ab.x *= sa * __ldg(p.col_scale + col0 + i); ab.y *= sa * __ldg(p.col_scale + col0 + i + 1); }
                ab = fadd2(ab, bb[h]);
                if (EPI == kEpiBiasGeluF16) ab = gelu_tanh_f32x2(ab);
                w[h] = pack16x2<BF16>(ab.x, ab.y);
              }
              srow[v] = make_uint4(w[0], w[1], w[2], w[3]);
            }
            __syncwarp();
            const unsigned ok_rows = __ballot_sync(0xffffffffu, row_ok);
#pragma unroll
            for (int it = 0; it < 4; ++it) {
              const int rr = it * 8 + (lane >> 2), part = lane & 3;
              if ((ok_rows >> rr) & 1u) {
                const uint4 val = *reinterpret_cast<const uint4*>(stb + rr * 80 + part * 16);
                *reinterpret_cast<uint4*>(p.out16 + static_cast<size_t>(m0 + quarter * 32 + rr) * ld + col0 + part * 8) = val;
              }
            }
            __syncwarp();                      // staging buffer is reused by the next chunk
          } else if (row_ok) {
            __half* dst = p.out16 + static_cast<size_t>(row) * ld + col0;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              if (col0 + i < p.N) {
                float a = __uint_as_float(r[i]);
                if (FP8) a *= sa * p.col_scale[col0 + i];
                a += bias[col0 + i];
                if (EPI == kEpiBiasGeluF16) a = gelu_tanh_f32(a);
                reinterpret_cast<uint16_t*>(dst)[i] = pack16<BF16>(a);
              }
            }
          }
        }
      }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster_light(acc ? tempty_leader1 : tempty_leader0);   // 16 arrivals: 8 warps x 2 CTAs
    }
  }

done:
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();        // the peer may still signal this CTA's barriers or read its operands until here
  if (warp == 1) { tc_fence_after(); tmem_dealloc_pair(tmem_base, 512); }
  if (threadIdx.x == 0 && *abort_flag) atomicMax(p.status, kStatusGemmTimeout);
  if (p.probe && threadIdx.x == 0) {
    const long long dc = clock64() - probe_c0;
    const uint64_t dt = global_ns() - probe_t0;
    if (dt > 20000) p.probe[0] = static_cast<int>(dc * 1000 / static_cast<long long>(dt));   // CTAs that lived 20 us or more
  }
}

}  // namespace dit

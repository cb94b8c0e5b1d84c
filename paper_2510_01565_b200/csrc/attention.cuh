// Variable-length multi-head softmax attention for sm_100a, block-diagonal per request.
//
// One CTA owns (request, head, 256 query rows) as two 128-row tiles, each served by its own softmax
// warpgroup.  Tiles are cut relative to the request's first row, never relative to the packed
// offset, so a request sees the same tiling whether it runs alone or packed with others.  Q, K and
// V tiles are TMA boxes cut straight out of the packed [T, 3H] fp16 qkv buffer (columns head*d,
// H + head*d, 2H + head*d); V is consumed as an MN-major B operand, so no transpose is ever
// materialised.  Rows past the end of the batch are zero-filled by TMA, rows past the end of the
// request belong to the next request (finite values); both are masked out of the softmax before the
// row maximum is taken.
//
// Per KV tile j (128 keys) and query tile i (online softmax, fp32 statistics):
//   MMA warp      S_i = Q_i K_j^T              -> TMEM S (one buffer, used by the two tiles in turn)
//   softmax WG i  reads S into registers and hands the buffer back at once;
//                 m, alpha, P = exp2(c*(S-m))  -> fp16 P[i] in its own TMEM columns (tcgen05.st)
//   MMA warp      O_i += P_i V_j               -> TMEM O[i]            (TS tcgen05.mma, A = P in TMEM)
// Because P does not overwrite S, the scores of a tile's NEXT key block are computed while its
// softmax warpgroup is still busy with the current one: S uses run one and a half key blocks ahead
// of the P V products (order on the tensor pipe: P V of tile 0, scores of tile 1, P V of tile 1,
// scores of tile 0, ...), so a warpgroup finds its next scores waiting instead of standing idle for a
// P V + Q K^T round trip.  TMEM: S 128 columns, P[0], P[1] 64 each, O[0], O[1] 128 each = 512.
// O is rescaled in TMEM only when a row maximum has grown by more than 2^8 since the reference was
// set (rare after the first tiles); P is bounded by 2^8, and O and l share the reference, so the
// normalised result is the same.  Output = acc / l, written as fp16 [T, H]; a warp passes its 32 rows through
// the shared memory of the tile's (by then unused) Q so that its stores cover whole rows.
//
// Thread layout (384): warpgroup 0 = {warp 0: TMA producer, warp 1: score MMAs + TMEM owner, warp 2: P V MMAs},
// warpgroups 1 and 2 = softmax for query tile 0 and 1.  Registers are re-balanced with setmaxnreg.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace dit {

struct AttnParams {
  __half* out;        // [T, H] with row stride ld_out (elements)
  int ld_out;
  int H;
  int n_heads;
  float scale_log2;   // log2(e) / sqrt(d)
  int* status;
  int* probe;         // test hook, NULL normally: [0] SM clock in MHz seen by a CTA of this launch (cycle counter
                      // against the global nanosecond timer over the CTA's life), [1] its cycles per key block
};

template <int D>
struct AttnCfg {
  static constexpr int NP = D / 64;              // 64-column panels per head slice
  static constexpr int PANEL = 128 * 128;        // bytes of one [128 rows x 64 fp16] swizzled panel
  static constexpr int TILE_BYTES = NP * PANEL;  // one 128-row Q, K or V tile
  static constexpr int KV_STAGES = 2;
  static constexpr int OFF_Q = 0;                                    // two query tiles
  static constexpr int OFF_K = OFF_Q + 2 * TILE_BYTES;
  static constexpr int OFF_V = OFF_K + KV_STAGES * TILE_BYTES;
  static constexpr int OFF_BAR = OFF_V + KV_STAGES * TILE_BYTES;
  // Every CTA takes all 512 tensor-memory columns, so two CTAs on one SM would only queue in tcgen05.alloc:
  // the request is padded past half of the SM's shared memory so that exactly one CTA is resident (matters for
  // head_dim 64, whose tiles alone need under 100 KB).
  static constexpr int SMEM_USED = OFF_BAR + 256 + 1024;
  static constexpr int SMEM_BYTES = SMEM_USED > 116 * 1024 ? SMEM_USED : 116 * 1024;
  static constexpr int THREADS = 384;
  static constexpr int Q_ROWS = 256;             // query rows per CTA
};

__device__ __forceinline__ float exp2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// BF16: q, k, v, P and the output are bf16 instead of fp16 (bf16-operand mode).
template <int D, bool BF16 = false>
__global__ void __launch_bounds__(AttnCfg<D>::THREADS, 1)
attention_tcgen05_kernel(const __grid_constant__ CUtensorMap tmQKV, const AttnParams p,
                         const __grid_constant__ SeqInfo seq) {
  using C = AttnCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* aligned = smem_raw + (base - raw);
  const uint32_t bar0 = base + C::OFF_BAR;
  // barrier slots
  const uint32_t q_full = bar0;
  auto k_full = [&](int s) { return bar0 + 8u * (1 + s); };
  auto k_empty = [&](int s) { return bar0 + 8u * (3 + s); };
  auto v_full = [&](int s) { return bar0 + 8u * (5 + s); };
  auto v_empty = [&](int s) { return bar0 + 8u * (7 + s); };
  auto s_full = [&](int i) { return bar0 + 8u * (9 + i); };
  auto p_full = [&](int i) { return bar0 + 8u * (11 + i); };
  auto o_full = [&](int i) { return bar0 + 8u * (13 + i); };
  const uint32_t s_free = bar0 + 8u * 15;      // the warpgroup that was handed S has read it into registers
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aligned + C::OFF_BAR + 8 * 16);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  long long probe_c0 = 0; uint64_t probe_t0 = 0;
  if (p.probe && threadIdx.x == 0) { probe_c0 = clock64(); probe_t0 = global_ns(); }

  // ---- which (request, head, 256-row query block) this CTA owns: requests longest first, and within a
  // request head-major, so that the CTAs resident at one time share the K/V of a few heads (a long
  // request's K/V over all heads is larger than L2)
  int head = 0, qb = blockIdx.x;
  int row_begin = 0, len = 0;
  for (int i = 0; i < seq.n; ++i) {
    const int r = seq.order[i];
    const int l = seq.cu[r + 1] - seq.cu[r];
    const int nb = (l + C::Q_ROWS - 1) / C::Q_ROWS;
    if (qb < nb * p.n_heads) { row_begin = seq.cu[r]; len = l; head = qb / nb; qb -= head * nb; break; }
    qb -= nb * p.n_heads;
  }
  const int q_row0 = row_begin + qb * C::Q_ROWS;
  const int nkv = (len + 127) >> 7;
  const bool tile1_valid = qb * C::Q_ROWS + 128 < len;     // second query tile has at least one row
  const int xq = head * D, xk = p.H + head * D, xv = 2 * p.H + head * D;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    mbar_init(s_free, 4);                      // one arrival per warp of the warpgroup
    for (int s = 0; s < 2; ++s) {
      mbar_init(k_full(s), 1); mbar_init(k_empty(s), 1);
      mbar_init(v_full(s), 1); mbar_init(v_empty(s), 1);
      mbar_init(s_full(s), 1); mbar_init(p_full(s), 4); mbar_init(o_full(s), 1);
    }
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0 && lane == 0) prefetch_tmap(&tmQKV);
  if (warp == 1) { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // TMEM columns: S 0..127 (shared by the two query tiles in turn), P[0] 128..191, P[1] 192..255,
  // O[0] 256.., O[1] 384..
  const uint32_t tS = tmem_base, tP = tmem_base + 128, tO = tmem_base + 256;

  if (warp < 4) {
    DIT_SETMAXNREG_DEC(96);
    if (len == 0) goto done;   // grid padding (cannot happen with an exact grid)
    if (warp == 0 && lane == 0) {
      // ------------------------------------------------------------------ TMA producer
      mbar_arrive_expect_tx(q_full, 2 * C::TILE_BYTES);
      for (int i = 0; i < 2; ++i)
        for (int pn = 0; pn < C::NP; ++pn)
          tma_load_2d(base + C::OFF_Q + i * C::TILE_BYTES + pn * C::PANEL, &tmQKV, xq + pn * 64, q_row0 + i * 128, q_full);
      for (int j = 0; j < nkv; ++j) {
        const int s = j % C::KV_STAGES; const uint32_t ph = (j / C::KV_STAGES) & 1u;
        const int y = row_begin + j * 128;
        if (!mbar_wait(k_empty(s), ph ^ 1u, abort_flag)) goto done;
        mbar_arrive_expect_tx(k_full(s), C::TILE_BYTES);
        for (int pn = 0; pn < C::NP; ++pn)
          tma_load_2d(base + C::OFF_K + s * C::TILE_BYTES + pn * C::PANEL, &tmQKV, xk + pn * 64, y, k_full(s));
        if (!mbar_wait(v_empty(s), ph ^ 1u, abort_flag)) goto done;
        mbar_arrive_expect_tx(v_full(s), C::TILE_BYTES);
        for (int pn = 0; pn < C::NP; ++pn)
          tma_load_2d(base + C::OFF_V + s * C::TILE_BYTES + pn * C::PANEL, &tmQKV, xv + pn * 64, y, v_full(s));
      }
    } else if (warp == 1 && lane == 0) {
      // ------------------------------------------------------------------ MMA issuer 1: scores
      // Uses of the S buffer run in the order (j, i) = (0,0), (0,1), (1,0), ...; use u = j * ntile + i.
      // A use waits for its K tile (first query tile) and for the warpgroup of use u - 1 to have read
      // the buffer out; the K stage is released after the last query tile.  This thread and the P V
      // issuer wait independently, so neither hand-off keeps the other's MMAs off the tensor pipe.
      constexpr uint32_t idesc_s = idesc_f16(128, 128, false, BF16);
      const int ntile = tile1_valid ? 2 : 1;
      static_assert(C::KV_STAGES == 2, "descriptor selection below assumes two stages");
      const uint64_t qdesc0 = smem_desc_sw128(base + C::OFF_Q, 16, 1024);
      const uint64_t kdesc0 = smem_desc_sw128(base + C::OFF_K, 16, 1024);
      constexpr uint32_t kTileStep = C::TILE_BYTES >> 4;
      if (!mbar_wait(q_full, 0, abort_flag)) goto done;
      const int total = ntile * nkv;
      for (int u = 0, j = 0, i = 0; u < total; ++u) {
        const int s = j % C::KV_STAGES;
        if (i == 0 && !mbar_wait(k_full(s), (j / C::KV_STAGES) & 1u, abort_flag)) goto done;
        if (u > 0 && !mbar_wait(s_free, (u - 1) & 1u, abort_flag)) goto done;
        tc_fence_after();
        const uint64_t qd = qdesc0 + i * kTileStep, kd = kdesc0 + s * kTileStep;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = ((kk >> 2) * C::PANEL + (kk & 3) * 32) >> 4;
          umma_f16(tS, qd + off, kd + off, idesc_s, kk != 0);
        }
        if (i == ntile - 1) umma_commit(k_empty(s));
        umma_commit(s_full(i));
        if (++i == ntile) { i = 0; ++j; }
      }
    } else if (warp == 2 && lane == 0) {
      // ------------------------------------------------------------------ MMA issuer 2: P V
      constexpr uint32_t idesc_pv = idesc_f16(128, D, true, BF16);
      const int ntile = tile1_valid ? 2 : 1;
      // V: MN-major B.  16 keys = two 8-row groups (stride 1024 B); the next 64 head columns live
      // one panel further (leading byte offset).
      const uint64_t vdesc0 = smem_desc_sw128(base + C::OFF_V, C::PANEL, 1024);
      constexpr uint32_t kTileStep = C::TILE_BYTES >> 4;
      for (int j = 0; j < nkv; ++j) {
        const int s = j % C::KV_STAGES;
        if (!mbar_wait(v_full(s), (j / C::KV_STAGES) & 1u, abort_flag)) goto done;
        const uint64_t vd = vdesc0 + s * kTileStep;
        for (int i = 0; i < ntile; ++i) {
          if (!mbar_wait(p_full(i), j & 1u, abort_flag)) goto done;
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)         // 16 keys per MMA: 8 TMEM columns of packed fp16 P
            umma_f16_ts(tO + i * 128, tP + i * 64 + kk * 8, vd + kk * (2048 >> 4), idesc_pv, (j | kk) != 0);
          if (i == ntile - 1) umma_commit(v_empty(s));
          umma_commit(o_full(i));
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + accumulate (2 warpgroups)
    DIT_SETMAXNREG_INC(200);
    const int tile = (warp >> 2) - 1;                            // query tile of this warpgroup
    const int quarter = warp & 3;
    if (len == 0 || (tile == 1 && !tile1_valid)) goto done;
    const uint32_t lane_sel = static_cast<uint32_t>(quarter * 32) << 16;
    const uint32_t tSi = tS + lane_sel, tPi = tP + tile * 64 + lane_sel, tOi = tO + tile * 128 + lane_sel;
    const float c = p.scale_log2;
    const float2 c2 = make_float2(c, c);
    // Running reference maximum m_ref (scores are exponentiated relative to it) and row sum l.
    // O accumulates in TMEM; it is rescaled only when a row's maximum has grown by more than
    // kRescaleLog2 in the exponent, so P stays <= 2^kRescaleLog2 and the result is unchanged
    // (both O and l carry the same reference).
    constexpr float kRescaleLog2 = 8.0f;
    float m_ref = -INFINITY, l = 0.f;

    for (int j = 0; j < nkv; ++j) {
      const uint32_t ph = j & 1u;
      if (!__all_sync(0xffffffffu, mbar_wait(s_full(tile), ph, abort_flag))) goto done;
      tc_fence_after();
      const int valid = len - j * 128;                           // keys of this tile inside the request
      uint32_t sv[128];                                          // this row's 128 scores
      __syncwarp();
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) tmem_ld32p(tSi + ch * 32, sv + ch * 32);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(s_free);                        // the scores are in registers: S may be overwritten
      if (valid < 128) {
#pragma unroll
        for (int i = 0; i < 128; ++i)
          if (i >= valid) sv[i] = 0xff800000u;                   // -inf: drops out of max and sum
      }
      float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
      for (int i = 0; i < 128; i += 8) {
        mx0 = fmax3(mx0, __uint_as_float(sv[i]), __uint_as_float(sv[i + 1]));
        mx1 = fmax3(mx1, __uint_as_float(sv[i + 2]), __uint_as_float(sv[i + 3]));
        mx2 = fmax3(mx2, __uint_as_float(sv[i + 4]), __uint_as_float(sv[i + 5]));
        mx3 = fmax3(mx3, __uint_as_float(sv[i + 6]), __uint_as_float(sv[i + 7]));
      }
      const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
      if (j == 0) {
        m_ref = mx;
      } else {
        const bool grow = (mx - m_ref) * c > kRescaleLog2;
        if (__any_sync(0xffffffffu, grow)) {
          // rare: rescale this warp's rows of O (rows that did not grow are multiplied by 1); the
          // previous P V, which accumulates into O, must have finished
          if (!__all_sync(0xffffffffu, mbar_wait(o_full(tile), (j - 1) & 1u, abort_flag))) goto done;
          tc_fence_after();
          const float alpha = grow ? exp2_approx((m_ref - mx) * c) : 1.0f;
          if (grow) { m_ref = mx; l *= alpha; }
#pragma unroll 1
          for (int ch = 0; ch < D / 32; ++ch) {
            uint32_t r[32];
            __syncwarp();
            tmem_ld32(tOi + ch * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
            tmem_st32(tOi + ch * 32, r);
          }
          tmem_st_wait();
        }
      }
      const float neg_mc = -m_ref * c;
      const float2 nm2 = make_float2(neg_mc, neg_mc);
      // P = exp2(c*s - c*m_ref) as fp16, packed in place over the score registers (pair k lands in
      // word k, which has been consumed by then); row sum in fp32
      float2 rs0 = make_float2(0.f, 0.f), rs1 = make_float2(0.f, 0.f);
#pragma unroll
      for (int i = 0; i < 128; i += 2) {
        const float2 x = ffma2(make_float2(__uint_as_float(sv[i]), __uint_as_float(sv[i + 1])), c2, nm2);
        const float2 e = make_float2(exp2_approx(x.x), exp2_approx(x.y));
        if (i & 2) rs1 = fadd2(rs1, e); else rs0 = fadd2(rs0, e);
        sv[i >> 1] = pack16x2<BF16>(e.x, e.y);
      }
      // P[tile] is still being read by the previous key block's P V until that product has finished;
      // by now (a whole tile of exponentials later) it normally has
      if (j > 0) {
        if (!__all_sync(0xffffffffu, mbar_wait(o_full(tile), (j - 1) & 1u, abort_flag))) goto done;
        tc_fence_after();
      }
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) tmem_st16(tPi + ch * 16, *reinterpret_cast<const uint32_t(*)[16]>(sv + ch * 16));
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_full(tile));
      l += (rs0.x + rs0.y) + (rs1.x + rs1.y);
    }
    {
      // the last P V product has landed: normalise and write this row
      if (!__all_sync(0xffffffffu, mbar_wait(o_full(tile), (nkv - 1) & 1u, abort_flag))) goto done;
      tc_fence_after();
      // Far outside any sane range (|score * scale| beyond 2^24 or so, i.e. operands that were clamped
      // at the edge of the 16-bit format) the fused multiply-add of the exponent no longer cancels the
      // reference exactly and a row's probabilities can all underflow or overflow: such a row is written
      // as zeros, never as NaN or infinity
      const float inv = l > 0.f ? 1.0f / l : 0.f;
      // The rows go out through shared memory, so that a store instruction covers 256 contiguous bytes of
      // each of two rows instead of 16 bytes of each of 32 rows.  The staging area is this tile's Q (all
      // score products that read it finished before the last P V did); each warp stages its own 32 rows,
      // 16-byte units XOR-swizzled by the row so that both phases are free of bank conflicts.
      constexpr int ROW_BYTES = D * 2, UNITS = ROW_BYTES / 16;       // 256 bytes = 16 units for d = 128
      uint8_t* stage = smem_raw + (((smem_u32(smem_raw) + 1023u) & ~1023u) - smem_u32(smem_raw)) + C::OFF_Q + tile * C::TILE_BYTES + quarter * 32 * ROW_BYTES;
#pragma unroll 1
      for (int ch = 0; ch < D / 32; ++ch) {
        uint32_t r[32];
        __syncwarp();
        tmem_ld32(tOi + ch * 32, r);
        tmem_ld_wait();
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint32_t w[4];
#pragma unroll
          for (int h = 0; h < 4; ++h) {
            const int i = 8 * v + 2 * h;
            float o0 = __uint_as_float(r[i]) * inv, o1 = __uint_as_float(r[i + 1]) * inv;
            if (!(fabsf(o0) <= 3.0e38f)) o0 = 0.f;
            if (!(fabsf(o1) <= 3.0e38f)) o1 = 0.f;
            w[h] = pack16x2<BF16>(o0, o1);
          }
          const int unit = ch * 4 + v;
          *reinterpret_cast<uint4*>(stage + lane * ROW_BYTES + ((unit ^ (lane & (UNITS - 1))) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      __syncwarp();
      {
        constexpr int ROWS_PER_STORE = 32 / UNITS;                   // 2 rows per instruction for d = 128, 4 for d = 64
        const int unit = lane % UNITS, sub = lane / UNITS;
        const int row0_in_req = qb * C::Q_ROWS + tile * 128 + quarter * 32;
        __half* out0 = p.out + static_cast<size_t>(row_begin + row0_in_req) * p.ld_out + head * D;
#pragma unroll 4
        for (int it = 0; it < 32 / ROWS_PER_STORE; ++it) {
          const int rr = it * ROWS_PER_STORE + sub;
          if (row0_in_req + rr < len) {
            const uint4 val = *reinterpret_cast<const uint4*>(stage + rr * ROW_BYTES + ((unit ^ (rr & (UNITS - 1))) << 4));
            *(reinterpret_cast<uint4*>(out0 + static_cast<size_t>(rr) * p.ld_out) + unit) = val;
          }
        }
      }
    }
  }

done:
  tc_fence_before();
  __syncthreads();
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 512); }
  if (threadIdx.x == 0 && *abort_flag) atomicMax(p.status, kStatusAttnTimeout);
  if (p.probe && threadIdx.x == 0 && nkv >= 16) {      // long enough for the two timers to resolve the clock
    const long long dc = clock64() - probe_c0;
    const uint64_t dt = global_ns() - probe_t0;
    p.probe[0] = static_cast<int>(dc * 1000 / static_cast<long long>(dt ? dt : 1));
    p.probe[1] = static_cast<int>(dc / nkv);
  }
}

}  // namespace dit

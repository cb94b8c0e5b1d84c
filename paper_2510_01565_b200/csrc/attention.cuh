// Variable-length multi-head softmax attention for sm_100a, block-diagonal per request.
//
// One CTA owns (request, head, 128 query rows).  Tiles are cut relative to the request's first row,
// never relative to the packed offset, so a request sees the same tiling whether it runs alone or
// packed with others.  Q, K and V tiles are TMA boxes cut straight out of the packed [T, 3H] fp16
// qkv buffer (columns head*d, H + head*d, 2H + head*d); V is consumed as an MN-major B operand, so
// no transpose is ever materialised.  Rows past the end of the batch are zero-filled by TMA, rows
// past the end of the request belong to the next request (finite values); both are masked out of
// the softmax before the row maximum is taken.
//
// Pipeline per KV tile j (online softmax, fp32 statistics):
//   MMA warp     S_j = Q K_j^T            -> TMEM S[j&1]            (tcgen05.mma, fp32 accumulate)
//   softmax WG   m_j, alpha_j, P_j = exp2(c*(S_j - m_j)) -> fp16 P[j&1] in shared memory (swizzled)
//   MMA warp     O_j = P_j V_j            -> TMEM O[j&1]            (fresh, not accumulated)
//   softmax WG   acc = acc * alpha_j + O_j   (fp32 registers, one thread per query row)
// S_{j+1} is issued before P_j V_j, so the tensor core works on the next scores while the softmax
// warps exponentiate the current ones.  Output = acc / l, written as fp16 [T, H].
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace dit {

struct AttnParams {
  __half* out;        // [T, H]
  int H;
  int n_heads;
  float scale_log2;   // log2(e) / sqrt(d)
  int* status;
};

template <int D>
struct AttnCfg {
  static constexpr int NP = D / 64;              // 64-column panels per head slice
  static constexpr int PANEL = 128 * 128;        // bytes of one [128 rows x 64 fp16] swizzled panel
  static constexpr int Q_BYTES = NP * PANEL;
  static constexpr int KV_BYTES = NP * PANEL;
  static constexpr int P_BYTES = 2 * PANEL;      // 128 rows x 128 keys fp16
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = OFF_Q + Q_BYTES;
  static constexpr int OFF_V = OFF_K + 2 * KV_BYTES;
  static constexpr int OFF_P = OFF_V + 2 * KV_BYTES;
  static constexpr int OFF_BAR = OFF_P + 2 * P_BYTES;
  static constexpr int SMEM_BYTES = OFF_BAR + 256 + 1024;
  static constexpr int THREADS = 192;
};

__device__ __forceinline__ float exp2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int D>
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
  auto s_full = [&](int s) { return bar0 + 8u * (9 + s); };
  auto p_full = [&](int s) { return bar0 + 8u * (11 + s); };
  auto o_full = [&](int s) { return bar0 + 8u * (13 + s); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aligned + C::OFF_BAR + 8 * 15);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- which (request, head, query tile) this CTA owns
  const int head = blockIdx.x % p.n_heads;
  int qt = blockIdx.x / p.n_heads;
  int row_begin = 0, len = 0;
  for (int i = 0; i < seq.n; ++i) {
    const int r = seq.order[i];
    const int l = seq.cu[r + 1] - seq.cu[r];
    const int nt = (l + 127) >> 7;
    if (qt < nt) { row_begin = seq.cu[r]; len = l; break; }
    qt -= nt;
  }
  const int q_row0 = row_begin + qt * 128;
  const int nkv = (len + 127) >> 7;
  const int xq = head * D, xk = p.H + head * D, xv = 2 * p.H + head * D;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(k_full(s), 1); mbar_init(k_empty(s), 1);
      mbar_init(v_full(s), 1); mbar_init(v_empty(s), 1);
      mbar_init(s_full(s), 1); mbar_init(p_full(s), 128); mbar_init(o_full(s), 1);
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
  // TMEM columns: S[0] 0..127, S[1] 128..255, O[0] 256.., O[1] 384..
  const uint32_t tS = tmem_base, tO = tmem_base + 256;

  if (len == 0) goto done;   // grid padding (cannot happen with an exact grid)

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_arrive_expect_tx(q_full, C::Q_BYTES);
      for (int pn = 0; pn < C::NP; ++pn)
        tma_load_2d(base + C::OFF_Q + pn * C::PANEL, &tmQKV, xq + pn * 64, q_row0, q_full);
      for (int j = 0; j < nkv; ++j) {
        const int s = j & 1; const uint32_t ph = (j >> 1) & 1u;
        const int y = row_begin + j * 128;
        if (!mbar_wait(k_empty(s), ph ^ 1u, abort_flag)) goto done;
        mbar_arrive_expect_tx(k_full(s), C::KV_BYTES);
        for (int pn = 0; pn < C::NP; ++pn)
          tma_load_2d(base + C::OFF_K + s * C::KV_BYTES + pn * C::PANEL, &tmQKV, xk + pn * 64, y, k_full(s));
        if (!mbar_wait(v_empty(s), ph ^ 1u, abort_flag)) goto done;
        mbar_arrive_expect_tx(v_full(s), C::KV_BYTES);
        for (int pn = 0; pn < C::NP; ++pn)
          tma_load_2d(base + C::OFF_V + s * C::KV_BYTES + pn * C::PANEL, &tmQKV, xv + pn * 64, y, v_full(s));
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_f16(128, 128, false);
      constexpr uint32_t idesc_pv = idesc_f16(128, D, true);
      bool ok = true;
      auto issue_s = [&](int j) {
        const int s = j & 1;
        if (!mbar_wait(k_full(s), (j >> 1) & 1u, abort_flag)) { ok = false; return; }
        tc_fence_after();
        const uint32_t qa = base + C::OFF_Q, ka = base + C::OFF_K + s * C::KV_BYTES;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk >> 2) * C::PANEL + (kk & 3) * 32;
          umma_f16(tS + s * 128, smem_desc_sw128(qa + off, 16, 1024), smem_desc_sw128(ka + off, 16, 1024),
                   idesc_s, kk != 0);
        }
        umma_commit(k_empty(s));
        umma_commit(s_full(s));
      };
      if (!mbar_wait(q_full, 0, abort_flag)) goto done;
      issue_s(0);
      if (nkv > 1 && ok) issue_s(1);
      for (int j = 0; j < nkv && ok; ++j) {
        const int s = j & 1; const uint32_t ph = (j >> 1) & 1u;
        if (!mbar_wait(p_full(s), ph, abort_flag)) goto done;
        if (!mbar_wait(v_full(s), ph, abort_flag)) goto done;
        tc_fence_after();
        const uint32_t pa = base + C::OFF_P + s * C::P_BYTES, va = base + C::OFF_V + s * C::KV_BYTES;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {       // 16 keys per MMA
          const uint64_t adesc = smem_desc_sw128(pa + (kk >> 2) * C::PANEL + (kk & 3) * 32, 16, 1024);
          // V: MN-major B.  16 keys = two 8-row groups (stride 1024 B); the next 64 head columns
          // live one panel further (leading byte offset).
          const uint64_t bdesc = smem_desc_sw128(va + kk * 2048, C::PANEL, 1024);
          umma_f16(tO + s * 128, adesc, bdesc, idesc_pv, kk != 0);
        }
        umma_commit(v_empty(s));
        umma_commit(o_full(s));
        if (j + 2 < nkv) issue_s(j + 2);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + accumulate (4 warps)
    const int quarter = warp & 3;
    const int prow = quarter * 32 + lane;                        // query row inside the tile
    const uint32_t lane_sel = static_cast<uint32_t>(quarter * 32) << 16;
    const float c = p.scale_log2;
    float m = -INFINITY, l = 0.f, alpha_prev = 0.f;
    float acc[D];
#pragma unroll
    for (int i = 0; i < D; ++i) acc[i] = 0.f;

    for (int j = 0; j < nkv; ++j) {
      const int s = j & 1; const uint32_t ph = (j >> 1) & 1u;
      if (!__all_sync(0xffffffffu, mbar_wait(s_full(s), ph, abort_flag))) goto done;
      tc_fence_after();
      const int valid = len - j * 128;                           // keys of this tile inside the request
      // pass 1: row maximum
      float mx = m;
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t r[32];
        __syncwarp();
        tmem_ld32(tS + lane_sel + s * 128 + ch * 32, r);
        tmem_ld_wait();
        if (valid >= ch * 32 + 32) {
#pragma unroll
          for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(r[i]));
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (ch * 32 + i < valid) mx = fmaxf(mx, __uint_as_float(r[i]));
        }
      }
      const float alpha = exp2_approx((m - mx) * c);             // m = -inf on the first tile -> 0
      const float neg_mc = -mx * c;
      // pass 2: P = exp2(c*s - c*m), row sum, fp16 P into swizzled shared memory
      float rowsum = 0.f;
      const uint32_t p_row = base + C::OFF_P + s * C::P_BYTES + prow * 128;
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t r[32];
        __syncwarp();
        tmem_ld32(tS + lane_sel + s * 128 + ch * 32, r);
        tmem_ld_wait();
        uint32_t w[16];
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          float e0 = exp2_approx(fmaf(__uint_as_float(r[i]), c, neg_mc));
          float e1 = exp2_approx(fmaf(__uint_as_float(r[i + 1]), c, neg_mc));
          if (ch * 32 + i >= valid) e0 = 0.f;
          if (ch * 32 + i + 1 >= valid) e1 = 0.f;
          rowsum += e0 + e1;
          const __half2 hh = __floats2half2_rn(e0, e1);
          w[i >> 1] = *reinterpret_cast<const uint32_t*>(&hh);
        }
        const uint32_t panel = p_row + (ch >> 1) * C::PANEL;
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const uint32_t chunk = static_cast<uint32_t>(((ch & 1) * 4 + v) ^ (prow & 7));
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(panel + chunk * 16), "r"(w[4 * v]),
                       "r"(w[4 * v + 1]), "r"(w[4 * v + 2]), "r"(w[4 * v + 3]) : "memory");
        }
      }
      fence_proxy_async_smem();     // make this thread's P writes visible to the tensor core
      tc_fence_before();            // and order its TMEM reads of S before the next S MMA
      mbar_arrive(p_full(s));
      l = l * alpha + rowsum;
      // fold in the previous tile's P V product
      if (j > 0) {
        const int sp = (j - 1) & 1; const uint32_t php = ((j - 1) >> 1) & 1u;
        if (!__all_sync(0xffffffffu, mbar_wait(o_full(sp), php, abort_flag))) goto done;
        tc_fence_after();
#pragma unroll
        for (int ch = 0; ch < D / 32; ++ch) {
          uint32_t r[32];
          __syncwarp();
          tmem_ld32(tO + lane_sel + sp * 128 + ch * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) acc[ch * 32 + i] = fmaf(acc[ch * 32 + i], alpha_prev, __uint_as_float(r[i]));
        }
      }
      alpha_prev = alpha;
      m = mx;
    }
    {
      const int sp = (nkv - 1) & 1; const uint32_t php = ((nkv - 1) >> 1) & 1u;
      if (!__all_sync(0xffffffffu, mbar_wait(o_full(sp), php, abort_flag))) goto done;
      tc_fence_after();
      const float inv = 1.0f / l;
      const bool row_ok = qt * 128 + prow < len;
      __half* dst = p.out + static_cast<size_t>(q_row0 + prow) * p.H + head * D;
#pragma unroll
      for (int ch = 0; ch < D / 32; ++ch) {
        uint32_t r[32];
        __syncwarp();
        tmem_ld32(tO + lane_sel + sp * 128 + ch * 32, r);
        tmem_ld_wait();
        if (row_ok) {
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint32_t w[4];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
              const int i = 8 * v + 2 * h;
              const float a = fmaf(acc[ch * 32 + i], alpha_prev, __uint_as_float(r[i])) * inv;
              const float b = fmaf(acc[ch * 32 + i + 1], alpha_prev, __uint_as_float(r[i + 1])) * inv;
              const __half2 hh = __floats2half2_rn(a, b);
              w[h] = *reinterpret_cast<const uint32_t*>(&hh);
            }
            *(reinterpret_cast<uint4*>(dst + ch * 32) + v) = make_uint4(w[0], w[1], w[2], w[3]);
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
}

}  // namespace dit

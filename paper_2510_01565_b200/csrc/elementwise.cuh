// HBM-bound kernels of the step: adaLN modulation GEMV, LayerNorm + modulate, token gather,
// and the one-off weight re-layout done at load time.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace dit {

// ------------------------------------------------------------------------------------------------
// adaLN modulation for all blocks at once:
//   mod[r, b, j] = sum_c SiLU(cond[r, c]) * W_ada_b[c, j] + b_ada_b[j],   j in [0, 6H)
// Bound by reading W_ada once (C x 6H bf16 per block).  A CTA owns kModCols consecutive columns of one
// block: kModCols / 8 column groups (8 bf16 = 16 B per load) x 256 / (kModCols / 8) slices of the C range;
// slice partials are combined in shared memory in slice order, so the result does not depend on the
// number of requests.  The strip width is chosen per launch: the widest that still gives every SM about two
// CTAs (wide strips read 1-2 KB runs of a row instead of 256 B, which DRAM serves much better).
// The partials reuse the activation buffer, which keeps two CTAs resident per SM.
// Requests are processed in groups of kModReqGroup to bound registers.
// ------------------------------------------------------------------------------------------------
constexpr int kModReqGroup = 8;
constexpr int kModThreads = 256;
constexpr int kModColsMin = 128;   // narrowest strip of columns a CTA owns; wider strips (template argument) read longer
                                   // contiguous runs of each W_ada row and are used when there are CTAs to spare
constexpr int kModBatch = 12;

struct ModParams {
  const __nv_bfloat16* cond;     // [R, C]
  const __nv_bfloat16* w_ada0;   // block 0's W_ada [C, 6H]; block b at + b * w_block_stride (elements)
  const float* b_ada0;           // block 0's bias [6H] fp32; block b at + b * b_block_stride
  long long w_block_stride, b_block_stride;
  float* mod;                    // [R, NB, 6H]
  int R, C, N6, NB;
  // Used by the small linear layers around the block stack (NB = 1), NULL otherwise:
  const float* in32;             // fp32 input [R, C] instead of `cond` (kIn = 1, 2)
  const float* addend;           // [R, N6] added to the result
  __nv_bfloat16* out16;          // result written as bf16 [R, N6] instead of `mod`
};

// kIn selects the input of the layer: 0 = SiLU(bf16 cond) (the adaLN modulation), 1 = SiLU(fp32 in32),
// 2 = fp32 in32 as it is.
enum ModInput : int { kModInCondSilu = 0, kModInF32Silu = 1, kModInF32 = 2 };

template <int kIn, int kModCols = kModColsMin>
__global__ void __launch_bounds__(kModThreads) modulation_kernel(const ModParams p) {
  constexpr int kModSlices = kModThreads / (kModCols / 8);
  extern __shared__ float sm[];                       // silu(cond) [G][C]; afterwards reused for partials [16][G][128]
  const int cols_per_block = (p.N6 + kModCols - 1) / kModCols;
  const int blk = blockIdx.x / cols_per_block;
  const int col_base = (blockIdx.x % cols_per_block) * kModCols;
  const int cg = threadIdx.x % (kModCols / 8), slice = threadIdx.x / (kModCols / 8);
  const int col = col_base + cg * 8;
  const __nv_bfloat16* w = p.w_ada0 + blk * p.w_block_stride;
  const float* bias = p.b_ada0 + blk * p.b_block_stride;
  float* s_act = sm;
  float* s_part = sm;
  const int c_per = (p.C + kModSlices - 1) / kModSlices;
  const int c0 = slice * c_per, c1 = min(p.C, c0 + c_per);

  for (int r0 = 0; r0 < p.R; r0 += kModReqGroup) {
    const int g = min(kModReqGroup, p.R - r0);
    __syncthreads();
    for (int i = threadIdx.x; i < kModReqGroup * p.C; i += kModThreads) {
      const int rr = i / p.C, cc = i % p.C;
      float v = 0.f;
      if (rr < g) {
        const size_t at = static_cast<size_t>(r0 + rr) * p.C + cc;
        const float x = kIn == kModInCondSilu ? __bfloat162float(p.cond[at]) : p.in32[at];
        v = kIn == kModInF32 ? x : x / (1.0f + __expf(-x));
      }
      s_act[i] = v;
    }
    __syncthreads();
    float acc[kModReqGroup][8];
#pragma unroll
    for (int rr = 0; rr < kModReqGroup; ++rr)
#pragma unroll
      for (int k = 0; k < 8; ++k) acc[rr][k] = 0.f;
    if (col < p.N6) {
      // batches of kModBatch rows of W_ada: all loads of a batch are issued before any is used, so
      // each thread keeps kModBatch x 16 bytes in flight (the kernel is bound by reading W_ada)
      uint4 nxt[kModBatch];
      auto fetch = [&](int cb) {
#pragma unroll
        for (int j = 0; j < kModBatch; ++j)
          if (cb + j < c1) nxt[j] = __ldg(reinterpret_cast<const uint4*>(w + static_cast<size_t>(cb + j) * p.N6 + col));
      };
      fetch(c0);
      for (int cb = c0; cb < c1; cb += kModBatch) {
        uint4 raw[kModBatch];
#pragma unroll
        for (int j = 0; j < kModBatch; ++j) raw[j] = nxt[j];
        if (cb + kModBatch < c1) fetch(cb + kModBatch);          // next batch flies while this one is used
#pragma unroll
        for (int j = 0; j < kModBatch; ++j) {
          if (cb + j < c1) {
            const int c = cb + j;
            const uint32_t u[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
            float wf[8];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              wf[2 * k] = __uint_as_float(u[k] << 16);
              wf[2 * k + 1] = __uint_as_float(u[k] & 0xFFFF0000u);
            }
#pragma unroll
            for (int rr = 0; rr < kModReqGroup; ++rr) {
              const float a = s_act[rr * p.C + c];
#pragma unroll
              for (int k = 0; k < 8; ++k) acc[rr][k] = fmaf(a, wf[k], acc[rr][k]);
            }
          }
        }
      }
    }
    __syncthreads();                           // every thread is done with the activations: reuse the buffer
#pragma unroll
    for (int rr = 0; rr < kModReqGroup; ++rr)
#pragma unroll
      for (int k = 0; k < 8; ++k) s_part[(slice * kModReqGroup + rr) * kModCols + cg * 8 + k] = acc[rr][k];
    __syncthreads();
    for (int i = threadIdx.x; i < g * kModCols; i += kModThreads) {
      const int rr = i / kModCols, cc = i % kModCols;
      if (col_base + cc < p.N6) {
        float v = 0.f;
#pragma unroll
        for (int sl = 0; sl < kModSlices; ++sl) v += s_part[(sl * kModReqGroup + rr) * kModCols + cc];
        v += bias[col_base + cc];
        const size_t at = (static_cast<size_t>(r0 + rr) * p.NB + blk) * p.N6 + col_base + cc;
        if (kIn != kModInCondSilu && p.addend) v += p.addend[at];
        if (kIn != kModInCondSilu && p.out16) p.out16[at] = __float2bfloat16_rn(v);
        else p.mod[at] = v;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// The same modulation with W_ada streamed by TMA (for the adaLN modulation of a whole stack,
// kModInCondSilu only).  Per-thread loads keep about 48 KB in flight per SM; here a CTA owns a strip of
// 512 columns of one block; its four slices of the C range (two compute warps each) each have a
// two-stage ring of 15-row groups, 120 KB in flight per SM, refilled by a ninth warp that does nothing
// else (lane s serves slice s), so a compute warp only ever waits for data.  A group arrives as two
// boxes of 256 columns x 15 rows of a 3-D tensor map over every block's W_ada (measured: 10-row groups
// in three stages 0.38 ms, 6-row groups in five 0.40 ms, 15-row groups in two 0.36 ms; one 1 KB bulk
// copy per row 0.56 ms; the register-load kernel 0.48-0.51 ms).  The activations sit in shared memory
// request-minor ([c][8]) so that a row costs two 16-byte loads, and the products use packed fp32
// pairs.  Summation order: that of modulation_kernel<.., 512>.
// ------------------------------------------------------------------------------------------------
constexpr int kModTmaCols = 512, kModTmaSlices = 4, kModTmaStages = 2, kModTmaRows = 15;
constexpr int kModTmaComputeThreads = 256, kModTmaThreads = kModTmaComputeThreads + 32;
constexpr int kModTmaRingBytes = kModTmaSlices * kModTmaStages * kModTmaRows * kModTmaCols * 2;

__host__ __device__ inline size_t mod_tma_act_floats(int C, int G) {      // activations [C][G], later the slice partials
  const size_t a = static_cast<size_t>(G) * C, b = static_cast<size_t>(kModTmaSlices) * G * kModTmaCols;
  return ((a > b ? a : b) + 31) & ~static_cast<size_t>(31);      // the ring that follows must start on a 128-byte boundary
}

// G = requests handled per pass over W_ada (1, 2, 4 or 8; the host takes the smallest that covers the batch, so
// that a small batch does not pay the multiply-adds of eight).  Every request has its own accumulators, so
// its result does not depend on G or on the other requests.
template <int G>
__global__ void __launch_bounds__(kModTmaThreads, 1)
modulation_tma_kernel(const __grid_constant__ CUtensorMap tmW, const ModParams p, int* __restrict__ status) {
  static_assert(G == 1 || G == 2 || G == 4 || G == 8, "the activation layout packs G requests per row");
  extern __shared__ __align__(128) uint8_t mod_smem[];
  float* s_act = reinterpret_cast<float*>(mod_smem);               // [C][G]
  float* s_part = s_act;
  uint8_t* ring = mod_smem + mod_tma_act_floats(p.C, G) * sizeof(float);
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring + kModTmaRingBytes);      // full[slice][stage], then empty[slice][stage]
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * kModTmaSlices * kModTmaStages);
  const int cols_per_block = (p.N6 + kModTmaCols - 1) / kModTmaCols;
  const int blk = blockIdx.x / cols_per_block;
  const int col_base = (blockIdx.x % cols_per_block) * kModTmaCols;
  const int ncols = min(kModTmaCols, p.N6 - col_base);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool is_producer_warp = warp == kModTmaComputeThreads / 32;
  const int cg = threadIdx.x % (kModTmaCols / 8);
  const int slice = is_producer_warp ? lane : threadIdx.x / (kModTmaCols / 8);      // producer lane s serves slice s
  const bool col_ok = cg * 8 < ncols;
  const float* bias = p.b_ada0 + blk * p.b_block_stride;
  const int c_per = (p.C + kModTmaSlices - 1) / kModTmaSlices;
  const int c0 = min(p.C, slice * c_per), c1 = min(p.C, c0 + c_per);
  const int n_groups = (is_producer_warp && lane >= kModTmaSlices) ? 0 : (c1 - c0 + kModTmaRows - 1) / kModTmaRows;
  uint8_t* my_ring = ring + static_cast<size_t>(slice & (kModTmaSlices - 1)) * kModTmaStages * kModTmaRows * kModTmaCols * 2;
  auto full_bar = [&](int st) { return smem_u32(bars + (slice & (kModTmaSlices - 1)) * kModTmaStages + st); };
  auto empty_bar = [&](int st) { return smem_u32(bars + (kModTmaSlices + (slice & (kModTmaSlices - 1))) * kModTmaStages + st); };
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int i = 0; i < kModTmaSlices * kModTmaStages; ++i) {
      mbar_init(smem_u32(bars + i), 1);                                   // full: the producer's expect_tx arrival
      mbar_init(smem_u32(bars + kModTmaSlices * kModTmaStages + i), 2);    // empty: the slice's two warps
    }
    fence_mbar_init();
  }
  int used = 0;                                // stage uses so far (keeps the barrier phases across request groups)
  bool ok = true;
  for (int r0 = 0; r0 < p.R; r0 += G) {
    const int g = min(G, p.R - r0);
    __syncthreads();                           // barriers exist; previous group's partials have been read
    for (int i = threadIdx.x; i < G * p.C; i += kModTmaThreads) {
      const int cc = i / G, rr = i % G;
      float v = 0.f;
      if (rr < g) {
        const float x = __bfloat162float(p.cond[static_cast<size_t>(r0 + rr) * p.C + cc]);
        v = x / (1.0f + __expf(-x));
      }
      s_act[i] = v;
    }
    __syncthreads();
    if (is_producer_warp) {
      // ------------------------------------------------------------------ producer (lanes 0..3, one slice each)
      for (int k = 0; k < n_groups && ok; ++k) {
        const int u = used + k, st = u % kModTmaStages;
        if (k >= kModTmaStages && !mbar_wait(empty_bar(st), ((u / kModTmaStages) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        const int r_first = c0 + k * kModTmaRows, n = min(kModTmaRows, c1 - r_first);
        // two boxes of 256 columns x kModTmaRows rows (rows past C and columns past 6H arrive as zeros; rows that
        // belong to the next slice are simply not used)
        (void)n;
        const int halves = ncols > 256 ? 2 : 1;
        mbar_arrive_expect_tx(full_bar(st), static_cast<uint32_t>(halves) * kModTmaRows * 512u);
        for (int hf = 0; hf < halves; ++hf)
          tma_load_3d(smem_u32(my_ring + (static_cast<size_t>(st) * 2 + hf) * kModTmaRows * 512), &tmW, col_base + hf * 256, r_first, blk,
                      full_bar(st));
      }
      used += n_groups;
    } else {
      // ------------------------------------------------------------------ compute warps
      float2 acc[G][4];
#pragma unroll
      for (int rr = 0; rr < G; ++rr)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[rr][q] = make_float2(0.f, 0.f);
      for (int k = 0; k < n_groups; ++k, ++used) {
        const int st = used % kModTmaStages; const uint32_t ph = (used / kModTmaStages) & 1u;
        if (ok && !__all_sync(0xffffffffu, mbar_wait(full_bar(st), ph, abort_flag))) ok = false;
        if (ok && col_ok) {
          const int r_first = c0 + k * kModTmaRows, n = min(kModTmaRows, c1 - r_first);
          const uint8_t* rows = my_ring + (static_cast<size_t>(st) * 2 + (cg >> 5)) * kModTmaRows * 512 + (cg & 31) * 16;
#pragma unroll
          for (int j = 0; j < kModTmaRows; ++j) {
            if (j < n) {
              const uint4 raw = *reinterpret_cast<const uint4*>(rows + static_cast<size_t>(j) * 512);
              const uint32_t u4[4] = {raw.x, raw.y, raw.z, raw.w};
              float2 wf[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) wf[q] = make_float2(__uint_as_float(u4[q] << 16), __uint_as_float(u4[q] & 0xFFFF0000u));
              float a[G];
              const float* ap = s_act + static_cast<size_t>(r_first + j) * G;
              if constexpr (G == 8) {
                const float4 a_lo = *reinterpret_cast<const float4*>(ap), a_hi = *reinterpret_cast<const float4*>(ap + 4);
                a[0] = a_lo.x; a[1] = a_lo.y; a[2] = a_lo.z; a[3] = a_lo.w; a[4] = a_hi.x; a[5] = a_hi.y; a[6] = a_hi.z; a[7] = a_hi.w;
              } else if constexpr (G == 4) {
                const float4 a4 = *reinterpret_cast<const float4*>(ap);
                a[0] = a4.x; a[1] = a4.y; a[2] = a4.z; a[3] = a4.w;
              } else if constexpr (G == 2) {
                const float2 a2 = *reinterpret_cast<const float2*>(ap);
                a[0] = a2.x; a[1] = a2.y;
              } else {
                a[0] = *ap;
              }
#pragma unroll
              for (int rr = 0; rr < G; ++rr) {
                const float2 aa = make_float2(a[rr], a[rr]);
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[rr][q] = ffma2(aa, wf[q], acc[rr][q]);
              }
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar(st));         // this warp is done with the stage
      }
      __syncwarp();
      // the partials go into the activation buffer once every compute warp has finished with it (below)
      asm volatile("bar.sync 1, %0;" ::"n"(kModTmaComputeThreads));
#pragma unroll
      for (int rr = 0; rr < G; ++rr)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          s_part[(slice * G + rr) * kModTmaCols + cg * 8 + 2 * q] = acc[rr][q].x;
          s_part[(slice * G + rr) * kModTmaCols + cg * 8 + 2 * q + 1] = acc[rr][q].y;
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < g * kModTmaCols; i += kModTmaThreads) {
      const int rr = i / kModTmaCols, cc = i % kModTmaCols;
      if (col_base + cc < p.N6) {
        float v = 0.f;
#pragma unroll
        for (int sl = 0; sl < kModTmaSlices; ++sl) v += s_part[(sl * G + rr) * kModTmaCols + cc];
        p.mod[(static_cast<size_t>(r0 + rr) * p.NB + blk) * p.N6 + col_base + cc] = v + bias[col_base + cc];
      }
    }
  }
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicMax(status, kStatusModTimeout);
}

// ------------------------------------------------------------------------------------------------
// LayerNorm (over H, biased variance, eps inside the root, no affine) + adaLN modulate:
//   h[row, :] = (x - mean) * rstd * (1 + scale[req]) + shift[req]        -> fp16 (bf16 with out_bf16)
// One warp per row, the row held in registers (kVec float4 per lane: H <= 128 * kVec), two-pass
// statistics, fixed shuffle order.  Small CTAs (4 rows) and a register budget that lets several CTAs
// share an SM keep enough loads in flight to cover HBM latency.
// kFromBf16 = true reads the packed bf16 tokens (first block) and also writes the fp32 residual stream.
// kind_stride != 0: two-stream block, the modulation vectors are chosen per row by image/text.
// ------------------------------------------------------------------------------------------------
constexpr int kLnWarps = 4;

// One row by one warp.  `src` points at the row's input (fp32, or bf16 with kFromBf16), in global or
// shared memory.  kOutFp8: h is written as e4m3 codes (1 byte per element, `h` then points at bytes) with
// one scale per row, largest magnitude of the row -> 448; the scale goes to row_scale[row].
template <bool kFromBf16, int kLnMaxVec, bool kOutFp8>
__device__ __forceinline__ void ln_modulate_row(const void* src, int row, int lane, float* __restrict__ stream_out,
                                                __half* __restrict__ h, const float4* sh, const float4* sc, int H,
                                                float eps, float* __restrict__ row_scale, bool out_bf16) {
  const int nvec = H >> 2;
  float4 v[kLnMaxVec];
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < kLnMaxVec; ++i) {
    const int idx = i * 32 + lane;
    if (idx < nvec) {
      if (kFromBf16) {
        const uint2 raw = *(reinterpret_cast<const uint2*>(src) + idx);
        v[i] = make_float4(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xFFFF0000u),
                           __uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xFFFF0000u));
        reinterpret_cast<float4*>(stream_out + static_cast<size_t>(row) * H)[idx] = v[i];
      } else {
        v[i] = reinterpret_cast<const float4*>(src)[idx];
      }
      sum += (v[i].x + v[i].y) + (v[i].z + v[i].w);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const float mean = sum / static_cast<float>(H);
  float sq = 0.f;
#pragma unroll
  for (int i = 0; i < kLnMaxVec; ++i) {
    if (i * 32 + lane < nvec) {
      const float a = v[i].x - mean, b = v[i].y - mean, c = v[i].z - mean, d = v[i].w - mean;
      sq += (a * a + b * b) + (c * c + d * d);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  const float rstd = rsqrtf(sq / static_cast<float>(H) + eps);
  if (kOutFp8) {
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < kLnMaxVec; ++i) {
      const int idx = i * 32 + lane;
      if (idx < nvec) {
        const float4 s1 = sc[idx], s0 = sh[idx];
        v[i].x = (v[i].x - mean) * rstd * (1.f + s1.x) + s0.x;
        v[i].y = (v[i].y - mean) * rstd * (1.f + s1.y) + s0.y;
        v[i].z = (v[i].z - mean) * rstd * (1.f + s1.z) + s0.z;
        v[i].w = (v[i].w - mean) * rstd * (1.f + s1.w) + s0.w;
        amax = fmaxf(fmaxf(amax, fmaxf(fabsf(v[i].x), fabsf(v[i].y))), fmaxf(fabsf(v[i].z), fabsf(v[i].w)));
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const float inv = amax > 0.f ? 448.0f / amax : 1.0f;
    if (lane == 0) row_scale[row] = amax > 0.f ? amax / 448.0f : 1.0f;
    uint32_t* dst8 = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(h) + static_cast<size_t>(row) * H);
#pragma unroll
    for (int i = 0; i < kLnMaxVec; ++i) {
      const int idx = i * 32 + lane;
      if (idx < nvec) {
        const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(v[i].x * inv, v[i].y * inv), __NV_SATFINITE, __NV_E4M3);
        const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(v[i].z * inv, v[i].w * inv), __NV_SATFINITE, __NV_E4M3);
        dst8[idx] = lo | (hi << 16);
      }
    }
    return;
  }
  uint2* dst = reinterpret_cast<uint2*>(h + static_cast<size_t>(row) * H);
#pragma unroll
  for (int i = 0; i < kLnMaxVec; ++i) {
    const int idx = i * 32 + lane;
    if (idx < nvec) {
      const float4 s1 = sc[idx], s0 = sh[idx];
      const float a = (v[i].x - mean) * rstd * (1.f + s1.x) + s0.x;
      const float b = (v[i].y - mean) * rstd * (1.f + s1.y) + s0.y;
      const float c = (v[i].z - mean) * rstd * (1.f + s1.z) + s0.z;
      const float d = (v[i].w - mean) * rstd * (1.f + s1.w) + s0.w;
      // warp-uniform choice of the 16-bit format (the kernel is bound by HBM, not by issue slots)
      dst[idx] = out_bf16 ? make_uint2(pack16x2<true>(a, b), pack16x2<true>(c, d)) : make_uint2(pack16x2<false>(a, b), pack16x2<false>(c, d));
    }
  }
}

// Offset (floats) of the modulation vectors of `row`: its request's, and for two-stream blocks
// (kind_stride != 0) the text stream's set for text tokens, kind_stride floats further on.
__device__ __forceinline__ long long ln_vector_offset(const SeqInfo& seq, const RowGeom& geo, int row, long long req_stride,
                                                      long long kind_stride) {
  const int req = find_request(seq, row);
  return req * req_stride + (kind_stride ? row_kind(seq, geo, req, row) * kind_stride : 0);
}

template <bool kFromBf16, int kLnMaxVec, bool kOutFp8 = false>
__global__ void __launch_bounds__(kLnWarps * 32, (kLnMaxVec <= 8 ? 6 : (kLnMaxVec <= 24 ? 4 : 3)))
ln_modulate_kernel(const void* __restrict__ xin, float* __restrict__ stream_out, __half* __restrict__ h,
                   const float* __restrict__ shift0, const float* __restrict__ scale0, long long req_stride,
                   int T, int H, float eps, const __grid_constant__ SeqInfo seq,
                   long long kind_stride, const __grid_constant__ RowGeom geo, float* __restrict__ row_scale, int row0,
                   int out_bf16) {
  // rows are local to the launch (a launch may cover a slice of the batch starting at packed row row0:
  // the data pointers are already offset, only the request lookup needs the packed index)
  const int row = blockIdx.x * kLnWarps + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= T) return;
  const uint8_t* src = static_cast<const uint8_t*>(xin) + static_cast<size_t>(row) * H * (kFromBf16 ? 2 : 4);
  const long long voff = ln_vector_offset(seq, geo, row + row0, req_stride, kind_stride);
  ln_modulate_row<kFromBf16, kLnMaxVec, kOutFp8>(src, row, lane, stream_out, h, reinterpret_cast<const float4*>(shift0 + voff),
                                                 reinterpret_cast<const float4*>(scale0 + voff), H, eps, row_scale, out_bf16 != 0);
}

// The same rows fed by bulk copies.  Per-thread loads keep at most a few tens of KB in flight per SM
// (they go through the L1's request tracking), which holds the kernel above at about half of the
// HBM bandwidth; here every warp owns `slots` row buffers in shared memory that its lane 0 fills with
// cp.async.bulk (one copy per row), so an SM has 8 x slots rows in flight.  A warp waits for a row,
// processes it as above from shared memory and refills the buffer with its next row.
// Persistent grid: CTA c owns the contiguous rows [c * chunk, (c + 1) * chunk), its warps take them
// in turn.  Contiguous rows mostly share a request, so the CTA also keeps that request's shift and
// scale vectors in shared memory (`cache_vectors`; with only 8 warps per SM their global loads would
// otherwise sit on the critical path) and reloads them when its rows move on to the next request.
constexpr int kLnTmaWarps = 8;

template <bool kFromBf16, int kLnMaxVec, bool kOutFp8 = false>
__global__ void __launch_bounds__(kLnTmaWarps * 32, 1)
ln_modulate_tma_kernel(const void* __restrict__ xin, float* __restrict__ stream_out, __half* __restrict__ h,
                       const float* __restrict__ shift0, const float* __restrict__ scale0, long long req_stride,
                       int T, int H, float eps, const __grid_constant__ SeqInfo seq,
                       long long kind_stride, const __grid_constant__ RowGeom geo, float* __restrict__ row_scale,
                       int slots, int cache_vectors, int* __restrict__ status, int row0, int out_bf16) {
  extern __shared__ __align__(128) uint8_t ln_smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t row_bytes = static_cast<uint32_t>(H) * (kFromBf16 ? 2u : 4u);
  uint8_t* my_rows = ln_smem + static_cast<size_t>(warp) * slots * row_bytes;
  uint8_t* after_rows = ln_smem + static_cast<size_t>(kLnTmaWarps) * slots * row_bytes;
  float4* s_shift = reinterpret_cast<float4*>(after_rows);                     // [H] then scale [H] when cached
  float4* s_scale = s_shift + (H >> 2);
  uint8_t* after_vec = after_rows + (cache_vectors ? static_cast<size_t>(H) * 8 : 0);
  uint64_t* bars = reinterpret_cast<uint64_t*>(after_vec) + warp * slots;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(after_vec + kLnTmaWarps * slots * 8);
  if (threadIdx.x == 0) *abort_flag = 0;
  if (lane == 0) {
    for (int s = 0; s < slots; ++s) mbar_init(smem_u32(bars + s), 1);
    fence_mbar_init();
  }
  __syncthreads();
  const int chunk = (T + gridDim.x - 1) / gridDim.x;
  const int r0 = blockIdx.x * chunk, r1 = min(T, r0 + chunk);
  auto fetch = [&](int row, int slot) {       // lane 0 only
    mbar_arrive_expect_tx(smem_u32(bars + slot), row_bytes);
    bulk_load(smem_u32(my_rows + static_cast<size_t>(slot) * row_bytes),
              static_cast<const uint8_t*>(xin) + static_cast<size_t>(row) * row_bytes, row_bytes, smem_u32(bars + slot));
  };
  if (lane == 0)
    for (int s = 0; s < slots; ++s)
      if (r0 + warp + s * kLnTmaWarps < r1) fetch(r0 + warp + s * kLnTmaWarps, s);
  int slot = 0; uint32_t phase = 0;
  bool ok = true;
  int row = r0 + warp;
  // segments of the chunk that share one set of modulation vectors
  for (int seg0 = r0; seg0 < r1;) {
    int seg1 = r1;
    if (cache_vectors) {
      const int req = find_request(seq, seg0 + row0);
      seg1 = min(r1, seq.cu[req + 1] - row0);
      __syncthreads();                              // every warp is done with the previous vectors
      const float4* gsh = reinterpret_cast<const float4*>(shift0 + req * req_stride);
      const float4* gsc = reinterpret_cast<const float4*>(scale0 + req * req_stride);
      for (int i = threadIdx.x; i < (H >> 2); i += kLnTmaWarps * 32) { s_shift[i] = __ldg(gsh + i); s_scale[i] = __ldg(gsc + i); }
      __syncthreads();
    }
    for (; row < seg1; row += kLnTmaWarps) {
      if (ok && !__all_sync(0xffffffffu, mbar_wait(smem_u32(bars + slot), phase, abort_flag))) ok = false;
      if (ok) {
        const float4 *sh = s_shift, *sc = s_scale;
        if (!cache_vectors) {
          const long long voff = ln_vector_offset(seq, geo, row + row0, req_stride, kind_stride);
          sh = reinterpret_cast<const float4*>(shift0 + voff);
          sc = reinterpret_cast<const float4*>(scale0 + voff);
        }
        ln_modulate_row<kFromBf16, kLnMaxVec, kOutFp8>(my_rows + static_cast<size_t>(slot) * row_bytes, row, lane, stream_out, h,
                                                       sh, sc, H, eps, row_scale, out_bf16 != 0);
        __syncwarp();                               // every lane has read the buffer: refill it
        const int next = row + slots * kLnTmaWarps;
        if (lane == 0 && next < r1) fetch(next, slot);
        if (++slot == slots) { slot = 0; phase ^= 1u; }
      }
    }
    seg0 = seg1;
  }
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicMax(status, kStatusLnTimeout);
}

// ------------------------------------------------------------------------------------------------
// Row-tile items of a two-stream GEMM launch: for every tile of `tile_rows` packed rows, one item per
// stream (image = 0, text = 1) that has at least one row in the tile, in row order.  One small CTA;
// the compaction is serial (a batch has at most a few thousand row tiles).
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
build_row_items_kernel(const __grid_constant__ SeqInfo seq, const __grid_constant__ RowGeom geo, int tile_rows,
                       int* __restrict__ flags, int* __restrict__ items, int* __restrict__ num_items) {
  const int num_m = (seq.total + tile_rows - 1) / tile_rows;
  for (int mb = threadIdx.x; mb < num_m; mb += blockDim.x) {
    const int lo = mb * tile_rows, hi = min(seq.total, lo + tile_rows);
    int f = 0;
    for (int r = find_request(seq, lo); r < seq.n && seq.cu[r] < hi; ++r) {
      const int img_end = seq.cu[r] + (geo.img_cu[r + 1] - geo.img_cu[r]);
      if (max(lo, seq.cu[r]) < min(hi, img_end)) f |= 1;
      if (max(lo, img_end) < min(hi, seq.cu[r + 1])) f |= 2;
    }
    flags[mb] = f;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int n = 0;
    for (int mb = 0; mb < num_m; ++mb) {
      const int f = flags[mb];
      if (f & 1) items[n++] = mb;
      if (f & 2) items[n++] = mb | (1 << 24);
    }
    *num_items = n;
  }
}

// ------------------------------------------------------------------------------------------------
// Token gather: per-request [L_r, H] bf16 buffers -> one packed [T, H] bf16 buffer (16-byte copies).
// ------------------------------------------------------------------------------------------------
struct PtrList { const void* ptr[DIT_MAX_REQUESTS]; };

__global__ void __launch_bounds__(256)
pack_tokens_kernel(const __grid_constant__ PtrList src, const __grid_constant__ SeqInfo seq, void* __restrict__ dst, int row_vecs) {
  const long long total = static_cast<long long>(seq.total) * row_vecs;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < total; i += gridDim.x * 256ll) {
    const int row = static_cast<int>(i / row_vecs), vcol = static_cast<int>(i % row_vecs);
    const int r = find_request(seq, row);
    const uint4* s = static_cast<const uint4*>(src.ptr[r]) + static_cast<size_t>(row - seq.cu[r]) * row_vecs + vcol;
    static_cast<uint4*>(dst)[i] = __ldg(s);
  }
}

// ------------------------------------------------------------------------------------------------
// Weight load: bf16 [K, N] row-major -> fp16 [N, K] row-major (K-major B operand of the GEMMs).
// bf16 -> fp16 is exact for |w| >= 2^-17 (8 significant bits fit fp16's normal and subnormal range);
// larger magnitudes than fp16 holds clamp to its largest finite value.  kKeepBf16: the bf16 values are
// transposed as they are (bf16-operand mode).
// ------------------------------------------------------------------------------------------------
template <bool kKeepBf16 = false>
__global__ void __launch_bounds__(256)
transpose_bf16_to_f16_kernel(const __nv_bfloat16* __restrict__ in, __half* __restrict__ out, int K, int N) {
  __shared__ float tile[32][33];
  const int n0 = blockIdx.x * 32, k0 = blockIdx.y * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8
  for (int i = ty; i < 32; i += 8) {
    const int k = k0 + i, n = n0 + tx;
    tile[i][tx] = (k < K && n < N) ? __bfloat162float(in[static_cast<size_t>(k) * N + n]) : 0.f;
  }
  __syncthreads();
  for (int i = ty; i < 32; i += 8) {
    const int n = n0 + i, k = k0 + tx;
    if (n < N && k < K) reinterpret_cast<uint16_t*>(out)[static_cast<size_t>(n) * K + k] = pack16<kKeepBf16>(tile[tx][i]);
  }
}

// Widens a bf16 vector to fp32; a NULL input stands for a constant vector of `fill`.
// ------------------------------------------------------------------------------------------------
// FP8 weight load: per output channel n, scale[n] = max_k |W[k, n]| / 448, then
// bf16 [K, N] row-major -> e4m3 [N, K] row-major of W[k, n] / scale[n].
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
col_absmax_scale_kernel(const __nv_bfloat16* __restrict__ in, float* __restrict__ scale, int K, int N) {
  const int n = blockIdx.x * 256 + threadIdx.x;
  if (n >= N) return;
  float amax = 0.f;
  for (int k = 0; k < K; ++k) amax = fmaxf(amax, fabsf(__bfloat162float(in[static_cast<size_t>(k) * N + n])));
  scale[n] = amax > 0.f ? amax / 448.0f : 1.0f;
}

// ------------------------------------------------------------------------------------------------
// Row quantisation for the e4m3 mode: fp16 rows [T, K] (row stride ld elements) -> e4m3 codes [T, K]
// (dense) and one scale per row, largest magnitude of the row -> 448.  Used for the operands that are
// produced tile by tile (attention output, GELU output), where no kernel sees a whole row: one warp
// per row, two sweeps (the second one finds the row in L1/L2).  Bound by HBM: 3 bytes per element.
// ------------------------------------------------------------------------------------------------
constexpr int kQuantWarps = 8;

__global__ void __launch_bounds__(kQuantWarps * 32)
quantize_rows_e4m3_kernel(const __half* __restrict__ in, long long ld, uint8_t* __restrict__ out,
                          float* __restrict__ row_scale, int T, int K) {
  const int row = blockIdx.x * kQuantWarps + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= T) return;
  const uint4* src = reinterpret_cast<const uint4*>(in + static_cast<size_t>(row) * ld);   // 8 values per load
  const int nvec = K >> 3;
  __half2 m2 = __float2half2_rn(0.f);
  for (int i = lane; i < nvec; i += 32) {
    const uint4 v = src[i];
    const __half2* h2 = reinterpret_cast<const __half2*>(&v);
#pragma unroll
    for (int q = 0; q < 4; ++q) m2 = __hmax2(m2, __habs2(h2[q]));
  }
  float amax = fmaxf(__low2float(m2), __high2float(m2));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  const float inv = amax > 0.f ? 448.0f / amax : 1.0f;
  if (lane == 0) row_scale[row] = amax > 0.f ? amax / 448.0f : 1.0f;
  uint2* dst = reinterpret_cast<uint2*>(out + static_cast<size_t>(row) * K);
  for (int i = lane; i < nvec; i += 32) {
    const uint4 v = src[i];
    const __half2* h2 = reinterpret_cast<const __half2*>(&v);
    uint32_t c[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float2 f = __half22float2(h2[q]);
      c[q] = __nv_cvt_float2_to_fp8x2(make_float2(f.x * inv, f.y * inv), __NV_SATFINITE, __NV_E4M3);
    }
    dst[i] = make_uint2(c[0] | (c[1] << 16), c[2] | (c[3] << 16));
  }
}

__global__ void __launch_bounds__(256)
transpose_bf16_to_e4m3_kernel(const __nv_bfloat16* __restrict__ in, const float* __restrict__ scale,
                              uint8_t* __restrict__ out, int K, int N) {
  __shared__ float tile[32][33];
  const int n0 = blockIdx.x * 32, k0 = blockIdx.y * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8
  for (int i = ty; i < 32; i += 8) {
    const int k = k0 + i, n = n0 + tx;
    tile[i][tx] = (k < K && n < N) ? __bfloat162float(in[static_cast<size_t>(k) * N + n]) : 0.f;
  }
  __syncthreads();
  for (int i = ty; i < 32; i += 8) {
    const int n = n0 + i, k = k0 + tx;
    if (n < N && k < K)
      out[static_cast<size_t>(n) * K + k] = static_cast<uint8_t>(__nv_cvt_float_to_fp8(tile[tx][i] / scale[n], __NV_SATFINITE, __NV_E4M3));
  }
}

// Test hooks.  fill_u32_kernel writes a 32-bit pattern (guard areas of the workspace).
__global__ void fill_u32_kernel(uint32_t* __restrict__ dst, uint32_t value, int n) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) dst[i] = value;
}

// One warp waits with the library's bounded-wait routine on a barrier that nothing signals: a few
// parked attempts, then a 50 microsecond limit on the global timer.  The wait gives up, the kernel
// records it in the status word and returns; it holds no tensor memory and has no copy in flight.
__global__ void __launch_bounds__(32) expire_wait_kernel(int* __restrict__ status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    fence_mbar_init();
  }
  __syncwarp();
  const bool ok = mbar_wait_limited<2, 50000ull>(smem_u32(&bar), 0, &abort_flag);
  __syncwarp();
  if (threadIdx.x == 0 && (!ok || abort_flag)) atomicMax(status, kStatusTestTimeout);
}

__global__ void bf16_to_f32_kernel(const __nv_bfloat16* __restrict__ in, float* __restrict__ out, int n, float fill) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = in ? __bfloat162float(in[i]) : fill;
}

}  // namespace dit

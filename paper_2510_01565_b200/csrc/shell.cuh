// Kernels of the shell around the block stack: latent -> tokens, timestep embedding,
// token velocities -> latent update.  All are bound by memory traffic or plain ALU work and are a
// small share of a step; the contractions of the shell that are worth tensor cores (the output
// projection) run on the GEMM kernel.
#pragma once
#include "common.cuh"

namespace dit {

constexpr int kPatchDim = DIT_PATCH_DIM;       // 16 channels x 2 x 2
constexpr int kTEmbDim = DIT_T_EMB_DIM;

// Per-request geometry of a step, passed by value as a kernel parameter.
struct ShellInfo {
  int img_cu[DIT_MAX_REQUESTS + 1];   // prefix sums of image tokens over the requests of this launch
  long long lat_off[DIT_MAX_REQUESTS];// first float of request r's latent in the latent buffer (64 * its image-token prefix
                                      // in the caller's full request list, which may be longer than this launch's)
  int txt_row[DIT_MAX_REQUESTS];      // first row of request r's text tokens in the text buffer
  int gw[DIT_MAX_REQUESTS];           // patch columns (width / 16)
  float t[DIT_MAX_REQUESTS];          // diffusion time of this step
  float dsigma[DIT_MAX_REQUESTS];     // sigma_next - sigma_cur
};

// ------------------------------------------------------------------------------------------------
// Sinusoidal timestep embedding: e[r, :] = [cos(t_r f_k) | sin(t_r f_k)], f_k = 10000^(-k/128).
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kTEmbDim)
timestep_embed_kernel(const __grid_constant__ ShellInfo info, float* __restrict__ e) {
  const int r = blockIdx.x, j = threadIdx.x, half = kTEmbDim / 2;
  const int k = j < half ? j : j - half;
  // t reaches 1000, where an fp32 frequency would already cost 1e-3 rad: the R x 256 angles are taken in fp64
  const double f = exp2(-13.287712379549449 * static_cast<double>(k) / static_cast<double>(half));   // log2(10000)
  const double a = static_cast<double>(info.t[r]) * f;
  e[r * kTEmbDim + j] = static_cast<float>(j < half ? cos(a) : sin(a));
}

// ------------------------------------------------------------------------------------------------
// Patch embedding + 2-D sine/cosine position + text rows -> packed bf16 tokens.
//   image row (py, px) of request r:  tok = patch(py, px) W_in + b_in + pos(py, px)
//   text row i of request r:          tok = text[txt_row[r] + i]
// A CTA covers 64 packed rows x 128 channels: the 64 patches (fp32) and the 64 x 128 slice of W_in
// (bf16) sit in shared memory; a thread owns 4 rows x 8 channels.  The latent is read as float2
// (the two dx of a patch row), consecutive threads taking consecutive patches of a grid row.
// ------------------------------------------------------------------------------------------------
constexpr int kEmbRows = 64, kEmbCols = 128, kEmbThreads = 256;

__global__ void __launch_bounds__(kEmbThreads)
embed_latents_kernel(const float* __restrict__ latents, const __nv_bfloat16* __restrict__ text,
                     const __nv_bfloat16* __restrict__ w_in, const float* __restrict__ b_in,
                     __nv_bfloat16* __restrict__ tokens, int H, const __grid_constant__ SeqInfo seq,
                     const __grid_constant__ ShellInfo info) {
  __shared__ float s_patch[kEmbRows][kPatchDim + 1];
  __shared__ __align__(16) __nv_bfloat16 s_w[kPatchDim][kEmbCols];
  __shared__ int s_req[kEmbRows], s_py[kEmbRows], s_px[kEmbRows];      // s_py < 0: text row (s_px = row of the text buffer)
  const int row0 = blockIdx.x * kEmbRows, col0 = blockIdx.y * kEmbCols;
  const int tid = threadIdx.x;

  if (tid < kEmbRows) {
    const int row = row0 + tid;
    int req = -1, py = 0, px = 0;
    if (row < seq.total) {
      req = find_request(seq, row);
      const int local = row - seq.cu[req];
      const int n_img = info.img_cu[req + 1] - info.img_cu[req];
      if (local < n_img) { py = local / info.gw[req]; px = local - py * info.gw[req]; }
      else { py = -1; px = info.txt_row[req] + (local - n_img); }
    }
    s_req[tid] = req; s_py[tid] = py; s_px[tid] = px;
  }
  for (int i = tid; i < kPatchDim * kEmbCols / 8; i += kEmbThreads) {     // W_in slice, 16 bytes at a time
    const int k = i / (kEmbCols / 8), v = i % (kEmbCols / 8);
    uint4 val = make_uint4(0, 0, 0, 0);
    if (col0 + v * 8 < H) val = __ldg(reinterpret_cast<const uint4*>(w_in + static_cast<size_t>(k) * H + col0 + v * 8));
    *reinterpret_cast<uint4*>(&s_w[k][v * 8]) = val;
  }
  __syncthreads();
  for (int i = tid; i < kEmbRows * (kPatchDim / 2); i += kEmbThreads) {
    const int r = i % kEmbRows, pair = i / kEmbRows;                      // pair = (channel, dy)
    const int req = s_req[r], py = s_py[r];
    float2 v = make_float2(0.f, 0.f);
    if (req >= 0 && py >= 0) {
      const int gw = info.gw[req], w8 = 2 * gw;
      const long long plane = 4ll * (info.img_cu[req + 1] - info.img_cu[req]);
      const int c = pair >> 1, dy = pair & 1;
      const float* src = latents + info.lat_off[req] + c * plane + static_cast<long long>(2 * py + dy) * w8 + 2 * s_px[r];
      v = __ldg(reinterpret_cast<const float2*>(src));
    }
    s_patch[r][2 * pair] = v.x;
    s_patch[r][2 * pair + 1] = v.y;
  }
  __syncthreads();

  const int tc = tid & 15, tr = tid >> 4;          // 16 channel groups of 8, 16 row groups of 4
  const int col = col0 + tc * 8;
  if (col >= H) return;
  float acc[4][8];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
#pragma unroll 8
  for (int k = 0; k < kPatchDim; ++k) {
    const uint4 raw = *reinterpret_cast<const uint4*>(&s_w[k][tc * 8]);
    const uint32_t u[4] = {raw.x, raw.y, raw.z, raw.w};
    float wf[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) { wf[2 * j] = __uint_as_float(u[j] << 16); wf[2 * j + 1] = __uint_as_float(u[j] & 0xFFFF0000u); }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float a = s_patch[tr * 4 + i][k];
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a, wf[j], acc[i][j]);
    }
  }
  // position term: channels [0, H/2) encode the patch row, [H/2, H) the patch column; each half is
  // [sin | cos] over H/4 frequencies 10000^(-k / (H/4)).  The 8 channels of a thread share axis and function.
  const int quarter = H >> 2, halfH = H >> 1;
  const bool col_axis = col >= halfH;
  const int j0 = col_axis ? col - halfH : col;
  const bool use_cos = j0 >= quarter;
  float omega[8], bias[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int k = (use_cos ? j0 - quarter : j0) + j;
    omega[j] = exp2f(-13.287712379549449f * static_cast<float>(k) / static_cast<float>(quarter));
    bias[j] = b_in[col + j];
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = tr * 4 + i, row = row0 + r;
    if (row >= seq.total) continue;
    uint4 out;
    if (s_py[r] < 0) {
      out = __ldg(reinterpret_cast<const uint4*>(text + static_cast<size_t>(s_px[r]) * H + col));
    } else {
      const float p = static_cast<float>(col_axis ? s_px[r] : s_py[r]);
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float a0 = p * omega[2 * j], a1 = p * omega[2 * j + 1];
        const float v0 = acc[i][2 * j] + bias[2 * j] + (use_cos ? cosf(a0) : sinf(a0));
        const float v1 = acc[i][2 * j + 1] + bias[2 * j + 1] + (use_cos ? cosf(a1) : sinf(a1));
        const __nv_bfloat162 b2 = __floats2bfloat162_rn(v0, v1);
        w[j] = *reinterpret_cast<const uint32_t*>(&b2);
      }
      out = make_uint4(w[0], w[1], w[2], w[3]);
    }
    *reinterpret_cast<uint4*>(tokens + static_cast<size_t>(row) * H + col) = out;
  }
}

// ------------------------------------------------------------------------------------------------
// Token velocities [T, 64] (image rows only are used) -> velocity in latent layout and/or the
// Euler update of the latent:  z += dsigma_r * v.  One thread per (row, channel, dy): a float2 of the
// latent; consecutive threads take consecutive rows so that the latent accesses coalesce.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
unpatchify_update_kernel(const float* __restrict__ v_tok, float* __restrict__ velocity, float* __restrict__ latents,
                         const __grid_constant__ SeqInfo seq, const __grid_constant__ ShellInfo info) {
  const long long total = static_cast<long long>(seq.total) * (kPatchDim / 2);
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < total; i += gridDim.x * 256ll) {
    const int pair = static_cast<int>(i / seq.total), row = static_cast<int>(i % seq.total);
    const int req = find_request(seq, row);
    const int local = row - seq.cu[req];
    const int n_img = info.img_cu[req + 1] - info.img_cu[req];
    if (local >= n_img) continue;                                        // text rows produce no output
    const int gw = info.gw[req], w8 = 2 * gw;
    const int py = local / gw, px = local - py * gw;
    const int c = pair >> 1, dy = pair & 1;
    const long long off = info.lat_off[req] + c * (4ll * n_img) + static_cast<long long>(2 * py + dy) * w8 + 2 * px;
    const float2 v = *reinterpret_cast<const float2*>(v_tok + static_cast<size_t>(row) * kPatchDim + 2 * pair);
    if (velocity) *reinterpret_cast<float2*>(velocity + off) = v;
    if (latents) {
      float2 z = *reinterpret_cast<float2*>(latents + off);
      const float ds = info.dsigma[req];
      z.x = fmaf(ds, v.x, z.x);
      z.y = fmaf(ds, v.y, z.y);
      *reinterpret_cast<float2*>(latents + off) = z;
    }
  }
}

// z += dsigma_r * v over whole latents (both in latent layout); used by the stand-alone sampler call.
__global__ void __launch_bounds__(256)
euler_update_kernel(float* __restrict__ latents, const float* __restrict__ velocity, const __grid_constant__ ShellInfo info, int n) {
  const long long total = 64ll * info.img_cu[n];
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < total; i += gridDim.x * 256ll) {
    const int tokidx = static_cast<int>(i >> 6);
    int lo = 0, hi = n - 1;
    while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (info.img_cu[mid] <= tokidx) lo = mid; else hi = mid - 1; }
    latents[i] = fmaf(info.dsigma[lo], velocity[i], latents[i]);
  }
}

}  // namespace dit

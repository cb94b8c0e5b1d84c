// libdit: C ABI, context, host-side planning and kernel launches.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "attention.cuh"
#include "common.cuh"
#include "elementwise.cuh"
#include "gemm.cuh"
#include "shell.cuh"

using namespace dit;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr size_t kAlign = 1024;
constexpr int kMaxCondDim = 4096;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Offsets (bytes) inside one block's weight slot.
struct BlockLayout {
  size_t w_ada, b_ada, w_qkv, b_qkv, w_o, b_o, w_fc1, b_fc1, w_fc2, b_fc2, q_norm, k_norm;
  size_t s_qkv, s_fc1, s_o, s_fc2;   // per-output-channel scales of the e4m3 weights (DIT_FLAG_FP8_GEMM)
  size_t bytes;
};
// Offsets (bytes) inside the workspace.
struct Layout {
  BlockLayout blk;
  size_t weights, stream, h, qkv, a, u, mod, status, stage_tokens, stage_cond, stage_out;
  // tensors and intermediates of the shell around the block stack
  size_t sh_w_in, sh_b_in, sh_w_t1, sh_b_t1, sh_w_t2, sh_b_t2, sh_w_fa, sh_b_fa, sh_w_out, sh_b_out;
  size_t sh_temb, sh_pre1, sh_cond, sh_modfin, sh_vtok, sh_pooled;
  size_t rope_theta;   // pair frequencies of one rotary axis group, fp32
  size_t row_scale;    // per-row scales of the e4m3 activations (DIT_FLAG_FP8_GEMM)
  size_t q8, row_scale2;   // e4m3 codes [T, H + F] and row scales of the operands quantised by a pass of their own
                           // (attention output, GELU output, or both side by side); empty without DIT_FLAG_FP8_GEMM
  size_t items;        // two-stream launches: [0] item count, then per-tile flags, then the items
  // test hooks: 1 KiB guard areas after the activation regions, and the [begin, end) ranges that
  // dit_debug_poison fills
  static constexpr int kMaxGuards = 16;
  size_t guard[kMaxGuards];
  int n_guards;
  size_t poison_begin[kMaxGuards], poison_end[kMaxGuards];
  int n_poison;
  size_t bytes;
};
constexpr size_t kGuardBytes = 1024;
constexpr uint32_t kGuardPattern = 0xC3A55A3Cu;
constexpr int kWoutRows = 256;   // W_out^T is stored zero-padded to one full weight tile of the GEMM

bool config_ok(const dit_config* c) {
  if (!c) return false;
  if (c->hidden < 64 || c->hidden % 64 || c->hidden > 4096) return false;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->n_heads < 1 || static_cast<long long>(c->n_heads) * c->head_dim != c->hidden) return false;
  if (c->mlp_hidden < 64 || c->mlp_hidden % 64) return false;
  if (c->cond_dim < 1 || c->cond_dim > kMaxCondDim) return false;
  if (c->max_blocks < 1 || c->max_total_tokens < 1) return false;
  if (c->max_requests < 1 || c->max_requests > DIT_MAX_REQUESTS) return false;
  if (!(c->ln_eps >= 0.f) || (c->flags & ~static_cast<uint32_t>(DIT_FLAG_QK_RMSNORM | DIT_FLAG_ROPE_2D | DIT_FLAG_FP8_GEMM | DIT_FLAG_BF16_OPERANDS))) return false;
  // the bf16-operand mode is built for the plain sequential and parallel blocks only
  if ((c->flags & DIT_FLAG_BF16_OPERANDS) && (c->flags & (DIT_FLAG_QK_RMSNORM | DIT_FLAG_ROPE_2D | DIT_FLAG_FP8_GEMM))) return false;
  return true;
}

Layout make_layout(const dit_config& c) {
  const size_t H = c.hidden, F = c.mlp_hidden, C = c.cond_dim, T = c.max_total_tokens, R = c.max_requests;
  Layout L{};
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes); return at; };
  L.blk.w_ada = take(C * 6 * H * 2);
  L.blk.b_ada = take(6 * H * 4);
  L.blk.w_qkv = take(3 * H * H * 2);
  L.blk.b_qkv = take(3 * H * 4);
  L.blk.b_o = take(H * 4);
  L.blk.w_fc1 = take(F * H * 2);
  L.blk.b_fc1 = take(F * 4);
  // W_o and W_fc2 are neighbours with no gap (H * H * 2 is a multiple of the alignment): a parallel
  // block stores its single output projection [H, H + F] over both
  L.blk.w_o = take(H * H * 2);
  L.blk.w_fc2 = take(H * F * 2);
  L.blk.b_fc2 = take(H * 4);
  L.blk.q_norm = take(c.head_dim * 4);
  L.blk.k_norm = take(c.head_dim * 4);
  L.blk.s_qkv = take(3 * H * 4);
  L.blk.s_fc1 = take(F * 4);
  L.blk.s_o = take(H * 4);
  L.blk.s_fc2 = take(H * 4);
  L.blk.bytes = o;
  o = 0;
  // every activation region (or run of regions) is followed by a guard area and is listed as a poison range
  auto guard = [&](size_t begin) {
    L.poison_begin[L.n_poison] = begin; L.poison_end[L.n_poison++] = o;
    L.guard[L.n_guards++] = take(kGuardBytes);
  };
  L.weights = take(L.blk.bytes * c.max_blocks);
  L.stream = take(T * H * 4);
  guard(L.stream);
  L.h = take(T * H * 2);
  guard(L.h);
  L.qkv = take(T * 3 * H * 2);
  guard(L.qkv);
  L.a = take(T * H * 2);             // a and u stay neighbours: a parallel block uses them as one [T, H + F] buffer
  L.u = take(T * F * 2);
  guard(L.a);
  L.mod = take(R * c.max_blocks * 6 * H * 4);
  guard(L.mod);
  L.status = take(256);
  L.stage_tokens = take(T * H * 2);
  guard(L.stage_tokens);
  L.stage_cond = take(R * C * 2);
  guard(L.stage_cond);
  L.stage_out = take(T * H * 4);
  guard(L.stage_out);
  L.sh_w_in = take(DIT_PATCH_DIM * H * 2);
  L.sh_b_in = take(H * 4);
  L.sh_w_t1 = take(DIT_T_EMB_DIM * C * 2);
  L.sh_b_t1 = take(C * 4);
  L.sh_w_t2 = take(C * C * 2);
  L.sh_b_t2 = take(C * 4);
  L.sh_w_fa = take(C * 2 * H * 2);
  L.sh_b_fa = take(2 * H * 4);
  L.sh_w_out = take(kWoutRows * H * 2);
  L.sh_b_out = take(DIT_PATCH_DIM * 4);
  L.sh_temb = take(R * DIT_T_EMB_DIM * 4);
  L.sh_pre1 = take(R * C * 4);
  L.sh_cond = take(R * C * 2);
  L.sh_modfin = take(R * 2 * H * 4);
  L.sh_vtok = take(T * DIT_PATCH_DIM * 4);
  L.sh_pooled = take(R * C * 4);
  guard(L.sh_temb);
  L.rope_theta = take(64 * 4);
  L.row_scale = take(T * 4);
  const bool fp8_mode = (c.flags & DIT_FLAG_FP8_GEMM) != 0;
  L.row_scale2 = take(fp8_mode ? T * 4 : 0);
  L.q8 = take(fp8_mode ? T * (H + F) : 0);
  guard(L.row_scale);
  L.items = take((16 + 3 * (T / (2 * 128) + 2)) * 4);
  L.bytes = o;
  return L;
}

struct BlockState {
  bool loaded = false;
  bool parallel = false;                   // parallel form: tm_o is unused, tm_fc2 maps W_out^T [H, H + F]
  bool dual = false;                       // image stream of a two-stream block; the text stream is the next slot
  bool dual_second = false;                // text stream of a two-stream block (run together with the slot before)
  CUtensorMap tm_qkv, tm_o, tm_fc1, tm_fc2;
};

}  // namespace

constexpr int kHostOutSlices = 4;

// Tensor maps of the activation buffers for one batch length T (a8, u8, cat8: the e4m3 mode's quantised copies).
struct ActMaps { CUtensorMap h, a, u, qkv, cat, a8, u8, cat8; };

struct dit_ctx {
  dit_config cfg;
  Layout lay;
  uint8_t* ws;
  EncodeTiledFn encode;
  int num_sms;
  int gemm_pairs;                          // CTA pairs of the GEMM kernel that fit on the device at once
  BlockState* blocks;
  bool shell_loaded;
  CUtensorMap tm_wout;                     // W_out^T, fp16 [kWoutRows, H]
  CUtensorMap tm_wada;                     // every block's W_ada as one 3-D tensor [max_blocks, C, 6H] bf16, boxes of 10 x 256
  bool tm_wada_ok;
  bool attn_probe;                         // test hook: attention CTAs record the SM clock they ran at
  ActMaps maps;                            // valid for batch length maps_T (-1: none yet)
  int maps_T;
  int64_t last_launches;
  int last_T, last_R, last_nb;
  bool last_parallel;                      // the last block of the last step was a parallel block
  char err[256];
  // optional per-kernel timing (CUDA events recorded around every launch of a step)
  bool timing;
  // dit_step_forward_host: the output goes back to the host in row slices while the last GEMM still runs
  cudaStream_t copy_stream;                // device -> host copies of the output slices
  cudaStream_t h2d_stream;                 // host -> device copies of the token slices (the link is full duplex)
  cudaEvent_t slice_done[kHostOutSlices], tok_ready[kHostOutSlices];
  cudaEvent_t tok_consumed;                // block 0 of the last host-buffer step has read the staging tokens
  cudaEvent_t st_entry;                    // everything enqueued on the caller's stream before a host-buffer call
  bool last_step_from_host;                // the last step on this context was a host-buffer step
  cudaEvent_t d2h_done[2];                 // output of host-buffer call c has arrived: d2h_done[c & 1]
  uint64_t host_calls;                     // host-buffer calls so far
  bool host_copied;                        // the last step_impl call sent its output to the host itself
  std::vector<cudaEvent_t> ev_pool;        // pairs: [2i] start, [2i+1] stop
  std::vector<int> ev_kind;                // kind of pair i
  size_t ev_used;                          // pairs recorded since the last read

  template <class T> T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
  uint8_t* block_base(int b) const { return ws + lay.weights + lay.blk.bytes * static_cast<size_t>(b); }
};

namespace {

dit_status fail(dit_ctx* ctx, dit_status s, const char* fmt, const char* detail = "") {
  if (ctx) snprintf(ctx->err, sizeof(ctx->err), fmt, detail);
  return s;
}

// A failed CUDA call: the message holds the call's text (never used as a format string: it may contain
// a '%') and the runtime's error string.
dit_status fail_cuda(dit_ctx* ctx, const char* what, cudaError_t e) {
  if (ctx) snprintf(ctx->err, sizeof(ctx->err), "%.160s: %s", what, cudaGetErrorString(e));
  return DIT_ERR_CUDA;
}

#define DIT_CUDA_TRY(ctx, expr)                                                        \
  do {                                                                                 \
    cudaError_t e_ = (expr);                                                           \
    if (e_ != cudaSuccess) return fail_cuda(ctx, #expr, e_);                           \
  } while (0)

// 2-D fp16 tensor map: `inner` contiguous elements per row, `rows` rows, box 64 x box_rows, 128-byte swizzle,
// out-of-bounds elements read as zero.
bool make_map(const dit_ctx* ctx, CUtensorMap* m, const void* ptr, uint64_t inner, uint64_t rows, uint32_t box_rows) {
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {inner * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = ctx->encode(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// The same for e4m3 operands: 1 byte per element, box 128 bytes x box_rows.
bool make_map8(const dit_ctx* ctx, CUtensorMap* m, const void* ptr, uint64_t inner, uint64_t rows, uint32_t box_rows) {
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {inner};
  cuuint32_t box[2] = {128, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = ctx->encode(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool build_seq(const int32_t* lens, int n, SeqInfo* s) {
  s->n = n;
  s->cu[0] = 0;
  for (int r = 0; r < n; ++r) {
    if (lens[r] < 1) return false;
    s->cu[r + 1] = s->cu[r] + lens[r];
    s->order[r] = r;
  }
  s->total = s->cu[n];
  std::stable_sort(s->order, s->order + n, [&](int a, int b) { return lens[a] > lens[b]; });
  return true;
}

const RowGeom kNoGeom{};

template <int EPI, int HD = 0, bool DUAL = false, bool FP8 = false, bool BF16 = false>
cudaError_t launch_gemm(const dit_ctx* ctx, const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmParams& p,
                        const SeqInfo& seq, cudaStream_t st, const RowGeom& geo = kNoGeom, const CUtensorMap* tmB2 = nullptr) {
  // Band of the tile order: as many 256-row panels of one operand as fit in about 38 MB of L2 are held there
  // while the other operand streams past.  Holding A costs A + W * (row bands) bytes of DRAM reads, holding the
  // weights W + A * (column bands); the cheaper one is taken (long batches: the weights stay, the rows stream).
  GemmParams q = p;
  {
    const long long esz = FP8 ? 1 : 2;
    const long long panel = 2ll * gemm_cfg::BM * p.K * esz;                 // one 256-row panel of either operand
    const long long num_m = (p.M + 2 * gemm_cfg::BM - 1) / (2 * gemm_cfg::BM), num_n = (p.N + gemm_cfg::BN - 1) / gemm_cfg::BN;
    const long long fit = std::max(1ll, (38ll << 20) / panel);
    const long long rb = std::min(fit, num_m), cb = std::min(fit, num_n);
    const long long a_bytes = num_m * panel, w_bytes = num_n * panel;
    const long long cost_rows = a_bytes + w_bytes * ((num_m + rb - 1) / rb);
    const long long cost_cols = w_bytes + a_bytes * ((num_n + cb - 1) / cb);
    q.band = (!DUAL && cost_cols < cost_rows) ? -static_cast<int>(cb) : static_cast<int>(rb);
  }
  // 256 x 256 tiles, one per CTA pair; persistent grid of as many pairs as can be resident
  const int tiles = ((p.M + 2 * gemm_cfg::BM - 1) / (2 * gemm_cfg::BM)) * ((p.N + gemm_cfg::BN - 1) / gemm_cfg::BN);
  const int grid = 2 * std::min(tiles, ctx->gemm_pairs);   // a two-stream launch may have more items than row tiles: the loop covers them
  q.operand_bf16 = (ctx->cfg.flags & DIT_FLAG_BF16_OPERANDS) ? 1 : 0;
  q.probe = (ctx->attn_probe && p.status) ? p.status + 6 : nullptr;
  gemm_tcgen05_kernel<EPI, HD, DUAL, FP8, BF16><<<grid, gemm_cfg::THREADS, gemm_cfg::SMEM_BYTES, st>>>(tmA, tmB, tmB2 ? *tmB2 : tmB, q, seq, geo);
  return cudaGetLastError();
}

template <int D, bool BF16 = false>
cudaError_t launch_attention(const CUtensorMap& tmQKV, const AttnParams& p, const SeqInfo& seq, cudaStream_t st) {
  int qblocks = 0;
  for (int r = 0; r < seq.n; ++r) qblocks += (seq.cu[r + 1] - seq.cu[r] + AttnCfg<D>::Q_ROWS - 1) / AttnCfg<D>::Q_ROWS;
  attention_tcgen05_kernel<D, BF16><<<qblocks * p.n_heads, AttnCfg<D>::THREADS, AttnCfg<D>::SMEM_BYTES, st>>>(tmQKV, p, seq);
  return cudaGetLastError();
}

// LayerNorm + modulate launch: picks the register-resident row width (float4 per lane) for H.
// Shared memory of the bulk-copy LayerNorm: 8 warps x slots row buffers, the cached shift and scale
// vectors of one request (not for two-stream blocks), the barriers and the abort flag.
constexpr size_t kLnTmaBudget = 224 * 1024;
int ln_tma_slots(int H, bool from_bf16, bool cache_vectors) {
  const size_t row_bytes = static_cast<size_t>(H) * (from_bf16 ? 2 : 4);
  const size_t fixed = (cache_vectors ? static_cast<size_t>(H) * 8 : 0) + kLnTmaWarps * 4 * 8 + 16;
  return static_cast<int>(std::min<size_t>(4, (kLnTmaBudget - fixed) / (kLnTmaWarps * row_bytes)));
}
size_t ln_tma_smem(int H, bool from_bf16, bool cache_vectors, int slots) {
  const size_t row_bytes = static_cast<size_t>(H) * (from_bf16 ? 2 : 4);
  return kLnTmaWarps * slots * (row_bytes + 8) + (cache_vectors ? static_cast<size_t>(H) * 8 : 0) + 16;
}

// LayerNorm + modulate launch: picks the register-resident row width (float4 per lane) for H.  Batches
// of at least a few rows per SM take the bulk-copy kernel (one persistent CTA per SM), tiny ones the
// plain one.  `num_sms` = 0 forces the plain kernel.
template <bool kFromBf16, bool kOutFp8 = false>
cudaError_t launch_ln(const void* xin, float* stream_out, __half* h, const float* shift0, const float* scale0,
                      long long req_stride, int T, int H, float eps, const SeqInfo& seq, cudaStream_t st,
                      long long kind_stride = 0, const RowGeom& geo = kNoGeom, float* row_scale = nullptr,
                      int num_sms = 0, int* status = nullptr, int row0 = 0, bool out_bf16 = false) {
  const bool cache_vectors = kind_stride == 0;
  const int ob = out_bf16 ? 1 : 0;
  const int slots = ln_tma_slots(H, kFromBf16, cache_vectors);
  if (num_sms > 0 && status && slots >= 1 && T >= 4 * num_sms) {
    const int grid = std::min(num_sms, (T + kLnTmaWarps - 1) / kLnTmaWarps), block = kLnTmaWarps * 32;
    const size_t smem = ln_tma_smem(H, kFromBf16, cache_vectors, slots);
    const int cv = cache_vectors ? 1 : 0;
    if (H <= 1024) ln_modulate_tma_kernel<kFromBf16, 8, kOutFp8><<<grid, block, smem, st>>>(xin, stream_out, h, shift0, scale0, req_stride, T, H, eps, seq, kind_stride, geo, row_scale, slots, cv, status, row0, ob);
    else if (H <= 3072) ln_modulate_tma_kernel<kFromBf16, 24, kOutFp8><<<grid, block, smem, st>>>(xin, stream_out, h, shift0, scale0, req_stride, T, H, eps, seq, kind_stride, geo, row_scale, slots, cv, status, row0, ob);
    else ln_modulate_tma_kernel<kFromBf16, 32, kOutFp8><<<grid, block, smem, st>>>(xin, stream_out, h, shift0, scale0, req_stride, T, H, eps, seq, kind_stride, geo, row_scale, slots, cv, status, row0, ob);
    return cudaGetLastError();
  }
  const int grid = (T + kLnWarps - 1) / kLnWarps, block = kLnWarps * 32;
  if (H <= 1024) ln_modulate_kernel<kFromBf16, 8, kOutFp8><<<grid, block, 0, st>>>(xin, stream_out, h, shift0, scale0, req_stride, T, H, eps, seq, kind_stride, geo, row_scale, row0, ob);
  else if (H <= 3072) ln_modulate_kernel<kFromBf16, 24, kOutFp8><<<grid, block, 0, st>>>(xin, stream_out, h, shift0, scale0, req_stride, T, H, eps, seq, kind_stride, geo, row_scale, row0, ob);
  else ln_modulate_kernel<kFromBf16, 32, kOutFp8><<<grid, block, 0, st>>>(xin, stream_out, h, shift0, scale0, req_stride, T, H, eps, seq, kind_stride, geo, row_scale, row0, ob);
  return cudaGetLastError();
}

size_t mod_smem_bytes(int C) {   // activations [G][C], later reused for the slice partials [slices][G][cols] (slices * cols = 8 * threads)
  return std::max<size_t>(static_cast<size_t>(kModReqGroup) * C, static_cast<size_t>(8) * kModThreads * kModReqGroup) * sizeof(float);
}

size_t mod_tma_smem_bytes(int C, int G) {
  return mod_tma_act_floats(C, G) * sizeof(float) + kModTmaRingBytes + 2 * kModTmaSlices * kModTmaStages * 8 + 16;
}
constexpr size_t kModTmaSmemMax = 224 * 1024;

// adaLN modulation of all blocks.  With enough strips of 512 columns to give every SM about two CTAs, and
// a cond width whose activations leave room for the ring, W_ada is streamed by bulk copies; otherwise the
// register-load kernel runs with the widest column strip that still leaves about two CTAs per SM
// (measured on the 8-block mixed step: 0.72 / 0.57 / 0.48 ms for 128 / 256 / 512 columns).
cudaError_t launch_modulation(const ModParams& mp, int num_sms, size_t smem, cudaStream_t st, int* status, const CUtensorMap* tmW) {
  auto ctas = [&](int cols) { return mp.NB * ((mp.N6 + cols - 1) / cols); };
  const int enough = 3 * num_sms / 2;
  // the bulk-copy kernel keeps 120 KB in flight per CTA and holds an SM alone: about one CTA per SM is already enough
  if (status && tmW && ctas(kModTmaCols) >= num_sms * 9 / 10 && mod_tma_smem_bytes(mp.C, 8) <= kModTmaSmemMax) {
    // requests per pass over W_ada: the smallest group that covers the batch
    if (mp.R <= 1) modulation_tma_kernel<1><<<ctas(kModTmaCols), kModTmaThreads, mod_tma_smem_bytes(mp.C, 1), st>>>(*tmW, mp, status);
    else if (mp.R <= 2) modulation_tma_kernel<2><<<ctas(kModTmaCols), kModTmaThreads, mod_tma_smem_bytes(mp.C, 2), st>>>(*tmW, mp, status);
    else if (mp.R <= 4) modulation_tma_kernel<4><<<ctas(kModTmaCols), kModTmaThreads, mod_tma_smem_bytes(mp.C, 4), st>>>(*tmW, mp, status);
    else modulation_tma_kernel<8><<<ctas(kModTmaCols), kModTmaThreads, mod_tma_smem_bytes(mp.C, 8), st>>>(*tmW, mp, status);
    return cudaGetLastError();
  }
  if (ctas(1024) >= enough) modulation_kernel<kModInCondSilu, 1024><<<ctas(1024), kModThreads, smem, st>>>(mp);
  else if (ctas(512) >= enough) modulation_kernel<kModInCondSilu, 512><<<ctas(512), kModThreads, smem, st>>>(mp);
  else if (ctas(256) >= enough) modulation_kernel<kModInCondSilu, 256><<<ctas(256), kModThreads, smem, st>>>(mp);
  else modulation_kernel<kModInCondSilu, kModColsMin><<<ctas(kModColsMin), kModThreads, smem, st>>>(mp);
  return cudaGetLastError();
}

// `geo` (image geometry of the requests) is needed by the rotary term only; NULL otherwise.
// `host_out` (dit_step_forward_host): the last block's row-wise part (everything after attention; for the
// parallel form and the e4m3 mode only its last GEMM) runs in row slices and every finished slice of `out` is
// copied to the host on the context's copy stream while the next slice computes.  `tokens_in_slices`: the
// tokens are being copied in by the same slices (events tok_ready) and block 0 starts on each as it lands.
dit_status step_impl(dit_ctx* ctx, const void* tokens, const int32_t* lens, int n, const void* cond, int n_blocks,
                     float* out, cudaStream_t st, const RowGeom* geo = nullptr, float* host_out = nullptr,
                     bool tokens_in_slices = false) {
  const dit_config& c = ctx->cfg;
  SeqInfo seq{};
  if (!build_seq(lens, n, &seq)) return fail(ctx, DIT_ERR_INVALID_ARG, "every request needs at least one token");
  const bool qk_variant = (c.flags & (DIT_FLAG_QK_RMSNORM | DIT_FLAG_ROPE_2D)) != 0;
  const bool fp8 = (c.flags & DIT_FLAG_FP8_GEMM) != 0;     // QKV and up-projection read e4m3 h and weights
  const bool bf = (c.flags & DIT_FLAG_BF16_OPERANDS) != 0; // h, qkv, a, u and the weights are bf16 instead of fp16
  if ((c.flags & DIT_FLAG_ROPE_2D) && !geo)
    return fail(ctx, DIT_ERR_INVALID_ARG, "the rotary term needs the requests' geometry: use dit_step_forward_requests");
  const int T = seq.total, H = c.hidden, F = c.mlp_hidden;
  if (T > c.max_total_tokens) return fail(ctx, DIT_ERR_CAPACITY, "packed batch exceeds max_total_tokens");
  for (int b = 0; b < n_blocks; ++b)
    if (!ctx->blocks[b].loaded) return fail(ctx, DIT_ERR_NOT_LOADED, "a block in [0, n_blocks) has no weights");

  float* stream = ctx->at<float>(ctx->lay.stream);
  __half* h = ctx->at<__half>(ctx->lay.h);
  __half* qkv = ctx->at<__half>(ctx->lay.qkv);
  __half* a = ctx->at<__half>(ctx->lay.a);
  __half* u = ctx->at<__half>(ctx->lay.u);
  float* mod = ctx->at<float>(ctx->lay.mod);
  int* status = ctx->at<int>(ctx->lay.status);

  // a parallel block writes attention and MLP outputs side by side into one [T, H + F] buffer that
  // starts where `a` starts and runs on into `u` (the two regions are consecutive)
  __half* cat = a;
  // The activation tensor maps depend on the workspace (fixed) and on T only: they are encoded when T changes and
  // kept in the context (a serving loop repeats the same batch shape for every step of a round).
  float* row_scale = ctx->at<float>(ctx->lay.row_scale);
  // e4m3 mode: the operands that are produced tile by tile (attention output, GELU output, or the two side by
  // side in a parallel block) are quantised row by row into q8 by a pass of their own before the GEMM that reads them
  uint8_t* q8 = ctx->at<uint8_t>(ctx->lay.q8);
  float* row_scale2 = ctx->at<float>(ctx->lay.row_scale2);
  if (ctx->maps_T != T) {
    ActMaps& m = ctx->maps;
    ctx->maps_T = -1;
    if (!make_map(ctx, &m.h, h, H, T, gemm_cfg::BM) || !make_map(ctx, &m.a, a, H, T, gemm_cfg::BM) ||
        !make_map(ctx, &m.u, u, F, T, gemm_cfg::BM) || !make_map(ctx, &m.qkv, qkv, 3 * H, T, 128) ||
        !make_map(ctx, &m.cat, cat, H + F, T, gemm_cfg::BM))
      return fail(ctx, DIT_ERR_CUDA, "cuTensorMapEncodeTiled failed for an activation buffer");
    if (fp8 && (!make_map8(ctx, &m.h, h, H, T, gemm_cfg::BM) ||       // h holds e4m3 codes in this mode
                !make_map8(ctx, &m.a8, q8, H, T, gemm_cfg::BM) || !make_map8(ctx, &m.u8, q8, F, T, gemm_cfg::BM) ||
                !make_map8(ctx, &m.cat8, q8, H + F, T, gemm_cfg::BM)))
      return fail(ctx, DIT_ERR_CUDA, "cuTensorMapEncodeTiled failed for an activation buffer");
    ctx->maps_T = T;
  }
  const CUtensorMap &tm_h = ctx->maps.h, &tm_a = ctx->maps.a, &tm_u = ctx->maps.u, &tm_qkv = ctx->maps.qkv, &tm_cat = ctx->maps.cat;
  const CUtensorMap &tm_a8 = ctx->maps.a8, &tm_u8 = ctx->maps.u8, &tm_cat8 = ctx->maps.cat8;
  auto quantise_rows = [&](const __half* src, long long ld, int K) -> cudaError_t {
    quantize_rows_e4m3_kernel<<<(T + kQuantWarps - 1) / kQuantWarps, kQuantWarps * 32, 0, st>>>(src, ld, q8, row_scale2, T, K);
    return cudaGetLastError();
  };

  int64_t launches = 0;
  const long long req_stride = static_cast<long long>(n_blocks) * 6 * H;
  // Runs one launch; with timing enabled, brackets it with a pair of events on the stream.
  auto timed = [&](int kind, auto&& launch) -> cudaError_t {
    ++launches;
    if (!ctx->timing) return launch();
    if (ctx->ev_used * 2 + 2 > ctx->ev_pool.size()) {
      for (int i = 0; i < 2; ++i) {
        cudaEvent_t e;
        cudaError_t ce = cudaEventCreate(&e);
        if (ce != cudaSuccess) return ce;
        ctx->ev_pool.push_back(e);
      }
      ctx->ev_kind.push_back(kind);
    }
    const size_t i = ctx->ev_used++;
    ctx->ev_kind[i] = kind;
    cudaError_t ce = cudaEventRecord(ctx->ev_pool[2 * i], st);
    if (ce != cudaSuccess) return ce;
    ce = launch();
    if (ce != cudaSuccess) return ce;
    return cudaEventRecord(ctx->ev_pool[2 * i + 1], st);
  };

  // The gated-residual GEMM that writes `out`, sliced by rows when the result goes to the host.  A slice is a
  // whole number of 256-row tiles; every output element is computed exactly as in the unsliced launch.
  // In the e4m3 mode A is the quantised copy q8 (1 byte per element) and g carries the row and column scales.
  auto last_gemm = [&](const __half* a_ptr, int K, const CUtensorMap& tmA_full, const CUtensorMap& tmB, const GemmParams& g) -> dit_status {
    auto launch = [&](const CUtensorMap& tmA, const GemmParams& q) {
      return fp8 ? launch_gemm<kEpiGateResidF32, 0, false, true>(ctx, tmA, tmB, q, seq, st)
                 : launch_gemm<kEpiGateResidF32>(ctx, tmA, tmB, q, seq, st);
    };
    if (!host_out) {
      DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_GEMM_FC2, [&] { return launch(tmA_full, g); }));
      return DIT_OK;
    }
    const int tile_rows = 2 * gemm_cfg::BM;
    const int per = ((T + tile_rows - 1) / tile_rows + kHostOutSlices - 1) / kHostOutSlices * tile_rows;   // rows per slice
    // the previous host-buffer call may still be copying its output out of the same device buffer
    DIT_CUDA_TRY(ctx, cudaStreamWaitEvent(st, ctx->d2h_done[(ctx->host_calls & 1) ^ 1], 0));
    for (int sidx = 0, r0 = 0; r0 < T; ++sidx, r0 += per) {
      const int rows = std::min(per, T - r0);
      CUtensorMap tmA;
      if (!(fp8 ? make_map8(ctx, &tmA, q8 + static_cast<size_t>(r0) * K, K, rows, gemm_cfg::BM)
                : make_map(ctx, &tmA, a_ptr + static_cast<size_t>(r0) * K, K, rows, gemm_cfg::BM)))
        return fail(ctx, DIT_ERR_CUDA, "cuTensorMapEncodeTiled failed for an activation buffer");
      GemmParams q = g;
      q.M = rows; q.row0 = r0;
      q.resid = g.resid + static_cast<size_t>(r0) * g.N;
      q.out32 = g.out32 + static_cast<size_t>(r0) * g.N;
      if (fp8) q.row_scale = g.row_scale + r0;
      DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_GEMM_FC2, [&] { return launch(tmA, q); }));
      DIT_CUDA_TRY(ctx, cudaEventRecord(ctx->slice_done[sidx], st));
      DIT_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->slice_done[sidx], 0));
      DIT_CUDA_TRY(ctx, cudaMemcpyAsync(host_out + static_cast<size_t>(r0) * g.N, g.out32 + static_cast<size_t>(r0) * g.N,
                                        static_cast<size_t>(rows) * g.N * 4, cudaMemcpyDeviceToHost, ctx->copy_stream));
    }
    DIT_CUDA_TRY(ctx, cudaEventRecord(ctx->d2h_done[ctx->host_calls & 1], ctx->copy_stream));
    ctx->host_copied = true;
    return DIT_OK;
  };

  {  // adaLN modulation vectors of every block
    ModParams mp{};
    mp.cond = static_cast<const __nv_bfloat16*>(cond);
    mp.w_ada0 = reinterpret_cast<const __nv_bfloat16*>(ctx->block_base(0) + ctx->lay.blk.w_ada);
    mp.b_ada0 = reinterpret_cast<const float*>(ctx->block_base(0) + ctx->lay.blk.b_ada);
    mp.w_block_stride = static_cast<long long>(ctx->lay.blk.bytes / 2);
    mp.b_block_stride = static_cast<long long>(ctx->lay.blk.bytes / 4);
    mp.mod = mod; mp.R = n; mp.C = c.cond_dim; mp.N6 = 6 * H; mp.NB = n_blocks;
    DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_MODULATION, [&] { return launch_modulation(mp, ctx->num_sms, mod_smem_bytes(c.cond_dim), st, status, ctx->tm_wada_ok ? &ctx->tm_wada : nullptr); }));
  }

  // two-stream blocks: validate the pairing and list the row tiles of each stream once per step
  bool any_dual = false;
  for (int b = 0; b < n_blocks; ++b) {
    if (!ctx->blocks[b].dual) continue;
    any_dual = true;
    if (b + 1 >= n_blocks || !ctx->blocks[b + 1].dual_second)
      return fail(ctx, DIT_ERR_INVALID_ARG, "n_blocks ends between the two slots of a two-stream block");
  }
  if (ctx->blocks[0].dual_second) return fail(ctx, DIT_ERR_INVALID_ARG, "slot 0 holds the second half of a two-stream block");
  if (any_dual && !geo)
    return fail(ctx, DIT_ERR_INVALID_ARG, "two-stream blocks need the requests' geometry: use dit_step_forward_requests");
  const RowGeom& rg = geo ? *geo : kNoGeom;
  int* item_count = ctx->at<int>(ctx->lay.items);
  int* item_flags = item_count + 16;
  int* items = item_flags + (c.max_total_tokens / (2 * gemm_cfg::BM) + 2);
  if (any_dual) {
    build_row_items_kernel<<<1, 256, 0, st>>>(seq, rg, 2 * gemm_cfg::BM, item_flags, items, item_count);
    DIT_CUDA_TRY(ctx, cudaGetLastError());
    ++launches;
  }

  for (int b = 0; b < n_blocks; ++b) {
    const BlockState& bs = ctx->blocks[b];
    if (bs.dual_second) continue;                      // ran together with the slot before
    const bool dual = bs.dual;
    const BlockState& bt = ctx->blocks[dual ? b + 1 : b];     // text stream's slot of a two-stream block
    const uint8_t* wb = ctx->block_base(b);
    const uint8_t* wt = ctx->block_base(dual ? b + 1 : b);
    const long long ks = dual ? 6ll * H : 0;           // text stream's modulation vectors follow the image stream's
    const bool last = (dual ? b + 1 : b) == n_blocks - 1;
    const float* modb = mod + static_cast<size_t>(b) * 6 * H;   // request 0; request r at + r * req_stride
    auto two_stream = [&](GemmParams& gp, size_t bias_off) {
      if (!dual) return;
      gp.items = items; gp.num_items = item_count;
      gp.bias2 = reinterpret_cast<const float*>(wt + bias_off);
      gp.gate_kind_stride = ks;
    };
    // LN1 + modulate (block 0 also widens the bf16 tokens into the fp32 residual stream) and the QKV projection,
    // over packed rows [r0, r0 + rows): the whole batch, or one slice of it while the host's tokens still arrive
    GemmParams g{};
    g.status = status;
    g.M = T; g.N = 3 * H; g.K = H;
    g.bias = reinterpret_cast<const float*>(wb + ctx->lay.blk.b_qkv);
    g.out16 = qkv;
    two_stream(g, ctx->lay.blk.b_qkv);
    if (fp8) { g.row_scale = row_scale; g.col_scale = reinterpret_cast<const float*>(wb + ctx->lay.blk.s_qkv); }
    if (qk_variant) {
      g.hidden = H; g.eps = c.ln_eps;
      if (c.flags & DIT_FLAG_QK_RMSNORM) {
        g.q_norm = reinterpret_cast<const float*>(wb + ctx->lay.blk.q_norm);
        g.k_norm = reinterpret_cast<const float*>(wb + ctx->lay.blk.k_norm);
        g.q_norm2 = reinterpret_cast<const float*>(wt + ctx->lay.blk.q_norm);
        g.k_norm2 = reinterpret_cast<const float*>(wt + ctx->lay.blk.k_norm);
      }
      if (c.flags & DIT_FLAG_ROPE_2D) g.rope_theta = ctx->at<float>(ctx->lay.rope_theta);
    }
    auto ln1_qkv = [&](int r0, int rows, const CUtensorMap& tmA) -> dit_status {
      const size_t e0 = static_cast<size_t>(r0) * H;      // first element of the slice in a [T, H] buffer
      DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_LN_MODULATE, [&] {
        if (fp8)
          return b == 0 ? launch_ln<true, true>(tokens, stream, h, modb, modb + H, req_stride, T, H, c.ln_eps, seq, st, ks, rg, row_scale, ctx->num_sms, status)
                        : launch_ln<false, true>(stream, nullptr, h, modb, modb + H, req_stride, T, H, c.ln_eps, seq, st, ks, rg, row_scale, ctx->num_sms, status);
        return b == 0 ? launch_ln<true>(static_cast<const __nv_bfloat16*>(tokens) + e0, stream + e0, h + e0, modb, modb + H, req_stride, rows, H,
                                        c.ln_eps, seq, st, ks, rg, nullptr, ctx->num_sms, status, r0, bf)
                      : launch_ln<false>(stream, nullptr, h, modb, modb + H, req_stride, T, H, c.ln_eps, seq, st, ks, rg, nullptr, ctx->num_sms, status, 0, bf);
      }));
      GemmParams q = g;
      q.M = rows; q.row0 = r0; q.out16 = qkv + static_cast<size_t>(r0) * 3 * H;
      if (qk_variant) {
        DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_GEMM_QKV, [&] {
          if (fp8)
            return c.head_dim == 128 ? launch_gemm<kEpiQkvF16, 128, false, true>(ctx, tmA, bs.tm_qkv, q, seq, st, rg)
                                     : launch_gemm<kEpiQkvF16, 64, false, true>(ctx, tmA, bs.tm_qkv, q, seq, st, rg);
          if (dual)
            return c.head_dim == 128 ? launch_gemm<kEpiQkvF16, 128, true>(ctx, tmA, bs.tm_qkv, q, seq, st, rg, &bt.tm_qkv)
                                     : launch_gemm<kEpiQkvF16, 64, true>(ctx, tmA, bs.tm_qkv, q, seq, st, rg, &bt.tm_qkv);
          return c.head_dim == 128 ? launch_gemm<kEpiQkvF16, 128>(ctx, tmA, bs.tm_qkv, q, seq, st, rg)
                                   : launch_gemm<kEpiQkvF16, 64>(ctx, tmA, bs.tm_qkv, q, seq, st, rg);
        }));
      } else {
        DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_GEMM_QKV, [&] {
          if (fp8) return launch_gemm<kEpiBiasF16, 0, false, true>(ctx, tmA, bs.tm_qkv, q, seq, st);
          if (bf) return launch_gemm<kEpiBiasF16, 0, false, false, true>(ctx, tmA, bs.tm_qkv, q, seq, st);
          return dual ? launch_gemm<kEpiBiasF16, 0, true>(ctx, tmA, bs.tm_qkv, q, seq, st, rg, &bt.tm_qkv)
                      : launch_gemm<kEpiBiasF16>(ctx, tmA, bs.tm_qkv, q, seq, st);
        }));
      }
      return DIT_OK;
    };
    if (b == 0 && tokens_in_slices && !fp8 && !dual) {
      // dit_step_forward_host: the tokens are on their way in row slices on the copy stream; each slice is
      // normalised and projected as soon as it has landed
      const int tile_rows = 2 * gemm_cfg::BM;
      const int per = ((T + tile_rows - 1) / tile_rows + kHostOutSlices - 1) / kHostOutSlices * tile_rows;
      for (int sidx = 0, r0 = 0; r0 < T; ++sidx, r0 += per) {
        const int rows = std::min(per, T - r0);
        DIT_CUDA_TRY(ctx, cudaStreamWaitEvent(st, ctx->tok_ready[sidx], 0));
        CUtensorMap tmA;
        if (!make_map(ctx, &tmA, h + static_cast<size_t>(r0) * H, H, rows, gemm_cfg::BM))
          return fail(ctx, DIT_ERR_CUDA, "cuTensorMapEncodeTiled failed for an activation buffer");
        const dit_status ls = ln1_qkv(r0, rows, tmA);
        if (ls != DIT_OK) return ls;
      }
    } else {
      if (b == 0 && tokens_in_slices)
        for (int sidx = 0; sidx < kHostOutSlices; ++sidx) DIT_CUDA_TRY(ctx, cudaStreamWaitEvent(st, ctx->tok_ready[sidx], 0));
      const dit_status ls = ln1_qkv(0, T, tm_h);
      if (ls != DIT_OK) return ls;
    }
    // the packed tokens are read by block 0's LayerNorm only: from here on the staging buffer may be refilled for
    // the next host-buffer step (recorded for those steps only: they are never part of a stream capture, and an
    // event recorded inside a capture could not be waited for outside it)
    if (b == 0 && host_out) DIT_CUDA_TRY(ctx, cudaEventRecord(ctx->tok_consumed, st));
    // attention (one pass over all tokens of a request, whatever their stream)
    AttnParams ap{};
    ap.out = bs.parallel ? cat : a; ap.ld_out = bs.parallel ? H + F : H;
    ap.H = H; ap.n_heads = c.n_heads; ap.status = status;
    ap.probe = ctx->attn_probe ? status + 4 : nullptr;
    ap.scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(c.head_dim));
    DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_ATTENTION, [&] {
      if (bf) return c.head_dim == 128 ? launch_attention<128, true>(tm_qkv, ap, seq, st) : launch_attention<64, true>(tm_qkv, ap, seq, st);
      return c.head_dim == 128 ? launch_attention<128>(tm_qkv, ap, seq, st) : launch_attention<64>(tm_qkv, ap, seq, st);
    }));
    if (bs.parallel) {
      // MLP up-projection + GELU-tanh from the same h, written beside the attention output
      g = GemmParams{};
      g.status = status;
      g.M = T; g.N = F; g.K = H;
      g.bias = reinterpret_cast<const float*>(wb + ctx->lay.blk.b_fc1);
      g.out16 = cat + H; g.ld16 = H + F;
      if (fp8) { g.row_scale = row_scale; g.col_scale = reinterpret_cast<const float*>(wb + ctx->lay.blk.s_fc1); }
      DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_GEMM_FC1, [&] {
        if (bf) return launch_gemm<kEpiBiasGeluF16, 0, false, false, true>(ctx, tm_h, bs.tm_fc1, g, seq, st);
        return fp8 ? launch_gemm<kEpiBiasGeluF16, 0, false, true>(ctx, tm_h, bs.tm_fc1, g, seq, st)
                   : launch_gemm<kEpiBiasGeluF16>(ctx, tm_h, bs.tm_fc1, g, seq, st);
      }));
      // one output projection over [attention | MLP] + gate + residual
      g = GemmParams{};
      g.status = status;
      g.M = T; g.N = H; g.K = H + F;
      g.bias = reinterpret_cast<const float*>(wb + ctx->lay.blk.b_fc2);
      g.resid = stream; g.out32 = last ? out : stream;
      g.gate = modb + 2 * H; g.gate_stride = req_stride;
      if (fp8) {
        DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_QUANTIZE, [&] { return quantise_rows(cat, H + F, H + F); }));
        g.row_scale = row_scale2; g.col_scale = reinterpret_cast<const float*>(wb + ctx->lay.blk.s_fc2);
      }
      if (last) {
        const dit_status ls = last_gemm(cat, H + F, fp8 ? tm_cat8 : tm_cat, bs.tm_fc2, g);
        if (ls != DIT_OK) return ls;
      } else {
        DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_GEMM_FC2, [&] {
          return fp8 ? launch_gemm<kEpiGateResidF32, 0, false, true>(ctx, tm_cat8, bs.tm_fc2, g, seq, st)
                     : launch_gemm<kEpiGateResidF32>(ctx, tm_cat, bs.tm_fc2, g, seq, st);
        }));
      }
      continue;
    }
    if (last && host_out && !dual && !fp8) {
      // dit_step_forward_host, last block: after attention every row is independent, so projection, LayerNorm,
      // up- and down-projection run slice by slice and a finished slice of the output goes to the host while
      // the next one is computed.  A slice is a whole number of 256-row tiles: every element is computed
      // exactly as in the unsliced launches.
      const int tile_rows = 2 * gemm_cfg::BM;
      const int per = ((T + tile_rows - 1) / tile_rows + kHostOutSlices - 1) / kHostOutSlices * tile_rows;
      // the previous host-buffer call may still be copying its output out of the same device buffer
      DIT_CUDA_TRY(ctx, cudaStreamWaitEvent(st, ctx->d2h_done[(ctx->host_calls & 1) ^ 1], 0));
      for (int sidx = 0, r0 = 0; r0 < T; ++sidx, r0 += per) {
        const int rows = std::min(per, T - r0);
        const size_t eH = static_cast<size_t>(r0) * H, eF = static_cast<size_t>(r0) * F;
        CUtensorMap tm_as, tm_hs, tm_us;
        if (!make_map(ctx, &tm_as, a + eH, H, rows, gemm_cfg::BM) || !make_map(ctx, &tm_hs, h + eH, H, rows, gemm_cfg::BM) ||
            !make_map(ctx, &tm_us, u + eF, F, rows, gemm_cfg::BM))
          return fail(ctx, DIT_ERR_CUDA, "cuTensorMapEncodeTiled failed for an activation buffer");
        GemmParams q{};
        q.status = status;
        q.M = rows; q.row0 = r0; q.N = H; q.K = H;
        q.bias = reinterpret_cast<const float*>(wb + ctx->lay.blk.b_o);
        q.resid = stream + eH; q.out32 = stream + eH;
        q.gate = modb + 2 * H; q.gate_stride = req_stride;
        DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_GEMM_PROJ, [&] { return launch_gemm<kEpiGateResidF32>(ctx, tm_as, bs.tm_o, q, seq, st); }));
        DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_LN_MODULATE, [&] {
          return launch_ln<false>(stream + eH, nullptr, h + eH, modb + 3 * H, modb + 4 * H, req_stride, rows, H, c.ln_eps, seq, st, ks, rg,
                                  nullptr, ctx->num_sms, status, r0, bf);
        }));
        q = GemmParams{};
        q.status = status;
        q.M = rows; q.row0 = r0; q.N = F; q.K = H;
        q.bias = reinterpret_cast<const float*>(wb + ctx->lay.blk.b_fc1);
        q.out16 = u + eF;
        DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_GEMM_FC1, [&] {
          return bf ? launch_gemm<kEpiBiasGeluF16, 0, false, false, true>(ctx, tm_hs, bs.tm_fc1, q, seq, st)
                    : launch_gemm<kEpiBiasGeluF16>(ctx, tm_hs, bs.tm_fc1, q, seq, st);
        }));
        q = GemmParams{};
        q.status = status;
        q.M = rows; q.row0 = r0; q.N = H; q.K = F;
        q.bias = reinterpret_cast<const float*>(wb + ctx->lay.blk.b_fc2);
        q.resid = stream + eH; q.out32 = out + eH;
        q.gate = modb + 5 * H; q.gate_stride = req_stride;
        DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_GEMM_FC2, [&] { return launch_gemm<kEpiGateResidF32>(ctx, tm_us, bs.tm_fc2, q, seq, st); }));
        DIT_CUDA_TRY(ctx, cudaEventRecord(ctx->slice_done[sidx], st));
        DIT_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->slice_done[sidx], 0));
        DIT_CUDA_TRY(ctx, cudaMemcpyAsync(host_out + eH, out + eH, static_cast<size_t>(rows) * H * 4, cudaMemcpyDeviceToHost, ctx->copy_stream));
      }
      DIT_CUDA_TRY(ctx, cudaEventRecord(ctx->d2h_done[ctx->host_calls & 1], ctx->copy_stream));
      ctx->host_copied = true;
      continue;
    }
    // output projection + gate + residual
    g = GemmParams{};
    g.status = status;
    g.M = T; g.N = H; g.K = H;
    g.bias = reinterpret_cast<const float*>(wb + ctx->lay.blk.b_o);
    g.resid = stream; g.out32 = stream;
    g.gate = modb + 2 * H; g.gate_stride = req_stride;
    two_stream(g, ctx->lay.blk.b_o);
    if (fp8) {
      DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_QUANTIZE, [&] { return quantise_rows(a, H, H); }));
      g.row_scale = row_scale2; g.col_scale = reinterpret_cast<const float*>(wb + ctx->lay.blk.s_o);
    }
    DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_GEMM_PROJ, [&] {
      if (fp8) return launch_gemm<kEpiGateResidF32, 0, false, true>(ctx, tm_a8, bs.tm_o, g, seq, st);
      return dual ? launch_gemm<kEpiGateResidF32, 0, true>(ctx, tm_a, bs.tm_o, g, seq, st, rg, &bt.tm_o)
                  : launch_gemm<kEpiGateResidF32>(ctx, tm_a, bs.tm_o, g, seq, st);
    }));
    // LN2 + modulate
    DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_LN_MODULATE, [&] {
      return fp8 ? launch_ln<false, true>(stream, nullptr, h, modb + 3 * H, modb + 4 * H, req_stride, T, H, c.ln_eps, seq, st, ks, rg, row_scale, ctx->num_sms, status)
                 : launch_ln<false>(stream, nullptr, h, modb + 3 * H, modb + 4 * H, req_stride, T, H, c.ln_eps, seq, st, ks, rg, nullptr, ctx->num_sms, status, 0, bf);
    }));
    // MLP up-projection + GELU-tanh
    g = GemmParams{};
    g.status = status;
    g.M = T; g.N = F; g.K = H;
    g.bias = reinterpret_cast<const float*>(wb + ctx->lay.blk.b_fc1);
    g.out16 = u;
    two_stream(g, ctx->lay.blk.b_fc1);
    if (fp8) { g.row_scale = row_scale; g.col_scale = reinterpret_cast<const float*>(wb + ctx->lay.blk.s_fc1); }
    DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_GEMM_FC1, [&] {
      if (fp8) return launch_gemm<kEpiBiasGeluF16, 0, false, true>(ctx, tm_h, bs.tm_fc1, g, seq, st);
      if (bf) return launch_gemm<kEpiBiasGeluF16, 0, false, false, true>(ctx, tm_h, bs.tm_fc1, g, seq, st);
      return dual ? launch_gemm<kEpiBiasGeluF16, 0, true>(ctx, tm_h, bs.tm_fc1, g, seq, st, rg, &bt.tm_fc1)
                  : launch_gemm<kEpiBiasGeluF16>(ctx, tm_h, bs.tm_fc1, g, seq, st);
    }));
    // MLP down-projection + gate + residual (last block writes the caller's output)
    g = GemmParams{};
    g.status = status;
    g.M = T; g.N = H; g.K = F;
    g.bias = reinterpret_cast<const float*>(wb + ctx->lay.blk.b_fc2);
    g.resid = stream; g.out32 = last ? out : stream;
    g.gate = modb + 5 * H; g.gate_stride = req_stride;
    two_stream(g, ctx->lay.blk.b_fc2);
    if (fp8) {
      DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_QUANTIZE, [&] { return quantise_rows(u, F, F); }));
      g.row_scale = row_scale2; g.col_scale = reinterpret_cast<const float*>(wb + ctx->lay.blk.s_fc2);
    }
    if (last && !dual) {
      const dit_status ls = last_gemm(u, F, fp8 ? tm_u8 : tm_u, bs.tm_fc2, g);
      if (ls != DIT_OK) return ls;
    } else if (fp8) {
      DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_GEMM_FC2, [&] { return launch_gemm<kEpiGateResidF32, 0, false, true>(ctx, tm_u8, bs.tm_fc2, g, seq, st); }));
    } else {
      DIT_CUDA_TRY(ctx, timed(DIT_KERNEL_GEMM_FC2, [&] {
        return dual ? launch_gemm<kEpiGateResidF32, 0, true>(ctx, tm_u, bs.tm_fc2, g, seq, st, rg, &bt.tm_fc2)
                    : launch_gemm<kEpiGateResidF32>(ctx, tm_u, bs.tm_fc2, g, seq, st);
      }));
    }
  }
  ctx->last_launches = launches;
  ctx->last_T = T; ctx->last_R = n; ctx->last_nb = n_blocks;
  ctx->last_parallel = ctx->blocks[n_blocks - 1].parallel;
  ctx->last_step_from_host = host_out != nullptr;
  return DIT_OK;
}

// Loading one slot on its own dissolves a two-stream pair it was part of: the other half must be
// loaded again before it can run.
void unpair_slot(dit_ctx* ctx, int b) {
  BlockState& bs = ctx->blocks[b];
  if (bs.dual && b + 1 < ctx->cfg.max_blocks) { ctx->blocks[b + 1].dual_second = false; ctx->blocks[b + 1].loaded = false; }
  if (bs.dual_second && b > 0) { ctx->blocks[b - 1].dual = false; ctx->blocks[b - 1].loaded = false; }
  bs.dual = bs.dual_second = false;
}

dit_status check_step_args(dit_ctx* ctx, const void* tokens, const int32_t* lens, int n, const void* cond, int n_blocks,
                           const float* out) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  if (n < 0) return fail(ctx, DIT_ERR_INVALID_ARG, "n_requests is negative");
  if (n == 0) return DIT_OK;
  if (!tokens || !lens || !cond || !out) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL pointer argument");
  if (n > ctx->cfg.max_requests) return fail(ctx, DIT_ERR_CAPACITY, "n_requests exceeds max_requests");
  if (n_blocks < 1) return fail(ctx, DIT_ERR_INVALID_ARG, "n_blocks must be at least 1");
  if (n_blocks > ctx->cfg.max_blocks) return fail(ctx, DIT_ERR_CAPACITY, "n_blocks exceeds max_blocks");
  for (int b = 0; b < n_blocks; ++b)
    if (!ctx->blocks[b].loaded) return fail(ctx, DIT_ERR_NOT_LOADED, "a block in [0, n_blocks) has no weights");
  long long total = 0;
  for (int r = 0; r < n; ++r) {
    if (lens[r] < 1) return fail(ctx, DIT_ERR_INVALID_ARG, "every request needs at least one token");
    total += lens[r];
  }
  if (total > ctx->cfg.max_total_tokens) return fail(ctx, DIT_ERR_CAPACITY, "packed batch exceeds max_total_tokens");
  return DIT_OK;
}

}  // namespace

// =============================================================================================== C ABI
extern "C" {

size_t dit_workspace_bytes(const dit_config* cfg) {
  if (!config_ok(cfg)) return 0;
  return make_layout(*cfg).bytes;
}

dit_status dit_ctx_create(const dit_config* cfg, void* workspace, size_t workspace_bytes, dit_ctx** out) {
  if (!out) return DIT_ERR_INVALID_ARG;
  *out = nullptr;
  if (!cfg || !workspace) return DIT_ERR_INVALID_ARG;
  if (!config_ok(cfg)) return DIT_ERR_SHAPE;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return DIT_ERR_INVALID_ARG;
  const Layout lay = make_layout(*cfg);
  if (workspace_bytes < lay.bytes) return DIT_ERR_CAPACITY;

  int dev = 0, major = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return DIT_ERR_CUDA;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return DIT_ERR_CUDA;
  if (major != 10) return DIT_ERR_UNSUPPORTED_ARCH;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return DIT_ERR_CUDA;

  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess)
    return DIT_ERR_CUDA;

  dit_ctx* ctx = new (std::nothrow) dit_ctx();
  if (!ctx) return DIT_ERR_INTERNAL;
  ctx->cfg = *cfg;
  ctx->lay = lay;
  ctx->ws = static_cast<uint8_t*>(workspace);
  ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
  ctx->num_sms = sms;
  ctx->blocks = new (std::nothrow) BlockState[cfg->max_blocks];
  ctx->shell_loaded = false;
  ctx->last_launches = 0;
  ctx->maps_T = -1;
  ctx->attn_probe = false;
  ctx->last_T = ctx->last_R = ctx->last_nb = 0;
  ctx->last_parallel = false;
  ctx->timing = false;
  ctx->ev_used = 0;
  ctx->err[0] = 0;
  if (!ctx->blocks) { delete ctx; return DIT_ERR_INTERNAL; }

  cudaError_t e = cudaSuccess;
  auto opt_in = [&](const void* f, size_t bytes) {
    if (e == cudaSuccess) e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
  };
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiBiasF16>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiBiasGeluF16>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiGateResidF32>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiBiasF32>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiQkvF16, 64>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiQkvF16, 128>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiBiasF16, 0, true>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiBiasGeluF16, 0, true>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiGateResidF32, 0, true>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiQkvF16, 64, true>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiQkvF16, 128, true>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiGateResidF32, 0, false, true>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiBiasF16, 0, false, true>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiBiasGeluF16, 0, false, true>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiQkvF16, 64, false, true>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiQkvF16, 128, false, true>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiBiasF16, 0, false, false, true>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiBiasGeluF16, 0, false, false, true>), gemm_cfg::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&attention_tcgen05_kernel<128, true>), AttnCfg<128>::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&attention_tcgen05_kernel<64, true>), AttnCfg<64>::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&attention_tcgen05_kernel<128>), AttnCfg<128>::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&attention_tcgen05_kernel<64>), AttnCfg<64>::SMEM_BYTES);
  opt_in(reinterpret_cast<const void*>(&modulation_kernel<kModInCondSilu>), mod_smem_bytes(kMaxCondDim));  // same for every context
  opt_in(reinterpret_cast<const void*>(&modulation_kernel<kModInCondSilu, 256>), mod_smem_bytes(kMaxCondDim));
  opt_in(reinterpret_cast<const void*>(&modulation_kernel<kModInCondSilu, 512>), mod_smem_bytes(kMaxCondDim));
  opt_in(reinterpret_cast<const void*>(&modulation_kernel<kModInCondSilu, 1024>), mod_smem_bytes(kMaxCondDim));
  opt_in(reinterpret_cast<const void*>(&modulation_tma_kernel<1>), kModTmaSmemMax);
  opt_in(reinterpret_cast<const void*>(&modulation_tma_kernel<2>), kModTmaSmemMax);
  opt_in(reinterpret_cast<const void*>(&modulation_tma_kernel<4>), kModTmaSmemMax);
  opt_in(reinterpret_cast<const void*>(&modulation_tma_kernel<8>), kModTmaSmemMax);
  opt_in(reinterpret_cast<const void*>(&modulation_kernel<kModInF32Silu>), mod_smem_bytes(kMaxCondDim));
  opt_in(reinterpret_cast<const void*>(&modulation_kernel<kModInF32>), mod_smem_bytes(kMaxCondDim));
  {
    auto ln_opt = [&](auto kernel) { opt_in(reinterpret_cast<const void*>(kernel), kLnTmaBudget); };
    ln_opt(&ln_modulate_tma_kernel<false, 8, false>);  ln_opt(&ln_modulate_tma_kernel<false, 24, false>);  ln_opt(&ln_modulate_tma_kernel<false, 32, false>);
    ln_opt(&ln_modulate_tma_kernel<true, 8, false>);   ln_opt(&ln_modulate_tma_kernel<true, 24, false>);   ln_opt(&ln_modulate_tma_kernel<true, 32, false>);
    ln_opt(&ln_modulate_tma_kernel<false, 8, true>);   ln_opt(&ln_modulate_tma_kernel<false, 24, true>);   ln_opt(&ln_modulate_tma_kernel<false, 32, true>);
    ln_opt(&ln_modulate_tma_kernel<true, 8, true>);    ln_opt(&ln_modulate_tma_kernel<true, 24, true>);    ln_opt(&ln_modulate_tma_kernel<true, 32, true>);
  }
  if (e == cudaSuccess) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(sms & ~1); lc.blockDim = dim3(gemm_cfg::THREADS); lc.dynamicSmemBytes = gemm_cfg::SMEM_BYTES;
    cudaLaunchAttribute at;
    at.id = cudaLaunchAttributeClusterDimension;
    at.val.clusterDim.x = 2; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
    lc.attrs = &at; lc.numAttrs = 1;
    int clusters = 0;
    e = cudaOccupancyMaxActiveClusters(&clusters, reinterpret_cast<const void*>(&gemm_tcgen05_kernel<kEpiBiasF16>), &lc);
    ctx->gemm_pairs = std::max(1, std::min(clusters, sms / 2));
  }
  ctx->copy_stream = nullptr;
  ctx->h2d_stream = nullptr;
  ctx->host_copied = false;
  ctx->host_calls = 0;
  ctx->tok_consumed = nullptr;
  ctx->st_entry = nullptr;
  ctx->last_step_from_host = false;
  ctx->d2h_done[0] = ctx->d2h_done[1] = nullptr;
  for (int i = 0; i < kHostOutSlices; ++i) { ctx->slice_done[i] = nullptr; ctx->tok_ready[i] = nullptr; }
  {
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(6) * cfg->hidden, static_cast<cuuint64_t>(cfg->cond_dim), static_cast<cuuint64_t>(cfg->max_blocks)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(6) * cfg->hidden * 2, static_cast<cuuint64_t>(lay.blk.bytes)};
    const cuuint32_t box[3] = {256, kModTmaRows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    ctx->tm_wada_ok = ctx->encode(&ctx->tm_wada, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, ctx->ws + lay.weights + lay.blk.w_ada, dims, strides, box,
                                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  }
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->h2d_stream, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->tok_consumed, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->st_entry, cudaEventDisableTiming);
  for (int i = 0; i < 2 && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&ctx->d2h_done[i], cudaEventDisableTiming);
  for (int i = 0; i < kHostOutSlices && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&ctx->slice_done[i], cudaEventDisableTiming);
  for (int i = 0; i < kHostOutSlices && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&ctx->tok_ready[i], cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaMemset(ctx->ws + lay.status, 0, 256);
  for (int g = 0; g < lay.n_guards && e == cudaSuccess; ++g) {
    fill_u32_kernel<<<1, 256>>>(reinterpret_cast<uint32_t*>(ctx->ws + lay.guard[g]), kGuardPattern, static_cast<int>(kGuardBytes / 4));
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) {
    // rotary pair frequencies of one axis group of n = (d - d/8) / 2 channels: 10000^(-2i/n), i < n/2
    float theta[64] = {};
    const int n_axis = (cfg->head_dim - cfg->head_dim / 8) / 2;
    for (int i = 0; i < n_axis / 2; ++i) theta[i] = static_cast<float>(pow(10000.0, -2.0 * i / n_axis));
    e = cudaMemcpy(ctx->ws + lay.rope_theta, theta, sizeof(theta), cudaMemcpyHostToDevice);
  }
  if (e != cudaSuccess) { dit_ctx_destroy(ctx); return DIT_ERR_CUDA; }
  *out = ctx;
  return DIT_OK;
}

dit_status dit_ctx_destroy(dit_ctx* ctx) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  for (cudaEvent_t e : ctx->ev_pool) cudaEventDestroy(e);
  for (int i = 0; i < kHostOutSlices; ++i) if (ctx->slice_done[i]) cudaEventDestroy(ctx->slice_done[i]);
  for (int i = 0; i < kHostOutSlices; ++i) if (ctx->tok_ready[i]) cudaEventDestroy(ctx->tok_ready[i]);
  if (ctx->tok_consumed) cudaEventDestroy(ctx->tok_consumed);
  if (ctx->st_entry) cudaEventDestroy(ctx->st_entry);
  for (int i = 0; i < 2; ++i) if (ctx->d2h_done[i]) cudaEventDestroy(ctx->d2h_done[i]);
  if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  if (ctx->h2d_stream) cudaStreamDestroy(ctx->h2d_stream);
  delete[] ctx->blocks;
  delete ctx;
  return DIT_OK;
}

dit_status dit_load_block_weights(dit_ctx* ctx, int32_t b, const dit_block_weights* w, void* stream) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  if (!w) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL weights");
  if (b < 0 || b >= ctx->cfg.max_blocks) return fail(ctx, DIT_ERR_CAPACITY, "block index outside [0, max_blocks)");
  if (!w->w_ada || !w->w_qkv || !w->w_o || !w->w_fc1 || !w->w_fc2) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL weight matrix");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int H = ctx->cfg.hidden, F = ctx->cfg.mlp_hidden, C = ctx->cfg.cond_dim;
  uint8_t* base = ctx->block_base(b);
  const BlockLayout& L = ctx->lay.blk;
  BlockState& bs = ctx->blocks[b];
  unpair_slot(ctx, b);
  bs.loaded = false;
  bs.parallel = false;

  DIT_CUDA_TRY(ctx, cudaMemcpyAsync(base + L.w_ada, w->w_ada, static_cast<size_t>(C) * 6 * H * 2, cudaMemcpyDeviceToDevice, st));
  auto bias = [&](const void* src, size_t off, int n, float fill = 0.f) {
    bf16_to_f32_kernel<<<(n + 255) / 256, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(src), reinterpret_cast<float*>(base + off), n, fill);
    return cudaGetLastError();
  };
  auto weight = [&](const void* src, size_t off, int K, int N) {   // [K, N] bf16 -> [N, K] fp16
    dim3 grid((N + 31) / 32, (K + 31) / 32);
    if (ctx->cfg.flags & DIT_FLAG_BF16_OPERANDS)
      transpose_bf16_to_f16_kernel<true><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(src), reinterpret_cast<__half*>(base + off), K, N);
    else
      transpose_bf16_to_f16_kernel<false><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(src), reinterpret_cast<__half*>(base + off), K, N);
    return cudaGetLastError();
  };
  const bool fp8 = (ctx->cfg.flags & DIT_FLAG_FP8_GEMM) != 0;
  auto weight8 = [&](const void* src, size_t off, size_t scale_off, int K, int N) {   // [K, N] bf16 -> e4m3 [N, K] + scales [N]
    col_absmax_scale_kernel<<<(N + 255) / 256, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(src), reinterpret_cast<float*>(base + scale_off), K, N);
    dim3 grid((N + 31) / 32, (K + 31) / 32);
    transpose_bf16_to_e4m3_kernel<<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(src), reinterpret_cast<const float*>(base + scale_off), base + off, K, N);
    return cudaGetLastError();
  };
  DIT_CUDA_TRY(ctx, bias(w->b_ada, L.b_ada, 6 * H));
  DIT_CUDA_TRY(ctx, fp8 ? weight8(w->w_qkv, L.w_qkv, L.s_qkv, H, 3 * H) : weight(w->w_qkv, L.w_qkv, H, 3 * H));
  DIT_CUDA_TRY(ctx, bias(w->b_qkv, L.b_qkv, 3 * H));
  DIT_CUDA_TRY(ctx, fp8 ? weight8(w->w_o, L.w_o, L.s_o, H, H) : weight(w->w_o, L.w_o, H, H));
  DIT_CUDA_TRY(ctx, bias(w->b_o, L.b_o, H));
  DIT_CUDA_TRY(ctx, fp8 ? weight8(w->w_fc1, L.w_fc1, L.s_fc1, H, F) : weight(w->w_fc1, L.w_fc1, H, F));
  DIT_CUDA_TRY(ctx, bias(w->b_fc1, L.b_fc1, F));
  DIT_CUDA_TRY(ctx, fp8 ? weight8(w->w_fc2, L.w_fc2, L.s_fc2, F, H) : weight(w->w_fc2, L.w_fc2, F, H));
  DIT_CUDA_TRY(ctx, bias(w->b_fc2, L.b_fc2, H));
  DIT_CUDA_TRY(ctx, bias(w->q_norm, L.q_norm, ctx->cfg.head_dim, 1.f));   // NULL scale = ones
  DIT_CUDA_TRY(ctx, bias(w->k_norm, L.k_norm, ctx->cfg.head_dim, 1.f));

  if (!(fp8 ? make_map8(ctx, &bs.tm_qkv, base + L.w_qkv, H, 3 * H, gemm_cfg::BN / 2) : make_map(ctx, &bs.tm_qkv, base + L.w_qkv, H, 3 * H, gemm_cfg::BN / 2)) ||
      !(fp8 ? make_map8(ctx, &bs.tm_o, base + L.w_o, H, H, gemm_cfg::BN / 2) : make_map(ctx, &bs.tm_o, base + L.w_o, H, H, gemm_cfg::BN / 2)) ||
      !(fp8 ? make_map8(ctx, &bs.tm_fc1, base + L.w_fc1, H, F, gemm_cfg::BN / 2) : make_map(ctx, &bs.tm_fc1, base + L.w_fc1, H, F, gemm_cfg::BN / 2)) ||
      !(fp8 ? make_map8(ctx, &bs.tm_fc2, base + L.w_fc2, F, H, gemm_cfg::BN / 2) : make_map(ctx, &bs.tm_fc2, base + L.w_fc2, F, H, gemm_cfg::BN / 2)))
    return fail(ctx, DIT_ERR_CUDA, "cuTensorMapEncodeTiled failed for a weight matrix");
  bs.loaded = true;
  return DIT_OK;
}

dit_status dit_load_dual_block_weights(dit_ctx* ctx, int32_t b, const dit_block_weights* image_stream,
                                       const dit_block_weights* text_stream, void* stream) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  if (b < 0 || b + 1 >= ctx->cfg.max_blocks) return fail(ctx, DIT_ERR_CAPACITY, "a two-stream block needs slots b and b + 1 inside [0, max_blocks)");
  if (ctx->cfg.flags & DIT_FLAG_FP8_GEMM) return fail(ctx, DIT_ERR_SHAPE, "two-stream blocks are not available with DIT_FLAG_FP8_GEMM");
  if (ctx->cfg.flags & DIT_FLAG_BF16_OPERANDS) return fail(ctx, DIT_ERR_SHAPE, "two-stream blocks are not available with DIT_FLAG_BF16_OPERANDS");
  dit_status s = dit_load_block_weights(ctx, b, image_stream, stream);
  if (s != DIT_OK) return s;
  s = dit_load_block_weights(ctx, b + 1, text_stream, stream);
  if (s != DIT_OK) return s;
  ctx->blocks[b].dual = true;
  ctx->blocks[b + 1].dual_second = true;
  return DIT_OK;
}

dit_status dit_load_parallel_block_weights(dit_ctx* ctx, int32_t b, const dit_parallel_block_weights* w, void* stream) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  if (!w) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL weights");
  if (b < 0 || b >= ctx->cfg.max_blocks) return fail(ctx, DIT_ERR_CAPACITY, "block index outside [0, max_blocks)");
  if (!w->w_ada || !w->w_qkv || !w->w_fc1 || !w->w_out) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL weight matrix");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int H = ctx->cfg.hidden, F = ctx->cfg.mlp_hidden, C = ctx->cfg.cond_dim;
  uint8_t* base = ctx->block_base(b);
  const BlockLayout& L = ctx->lay.blk;
  BlockState& bs = ctx->blocks[b];
  unpair_slot(ctx, b);
  bs.loaded = false;
  bs.parallel = true;

  // The modulation kernel produces six H-wide vectors per block for the whole stack in one launch; a
  // parallel block has three (shift, scale, gate): its W_ada / b_ada fill the first three, the rest is zero.
  DIT_CUDA_TRY(ctx, cudaMemsetAsync(base + L.w_ada, 0, static_cast<size_t>(C) * 6 * H * 2, st));
  DIT_CUDA_TRY(ctx, cudaMemcpy2DAsync(base + L.w_ada, static_cast<size_t>(6) * H * 2, w->w_ada, static_cast<size_t>(3) * H * 2,
                                      static_cast<size_t>(3) * H * 2, C, cudaMemcpyDeviceToDevice, st));
  auto bias = [&](const void* src, size_t off, int n, float fill = 0.f) {
    bf16_to_f32_kernel<<<(n + 255) / 256, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(src), reinterpret_cast<float*>(base + off), n, fill);
    return cudaGetLastError();
  };
  auto weight = [&](const void* src, size_t off, int K, int N) {   // [K, N] bf16 -> [N, K] fp16
    dim3 grid((N + 31) / 32, (K + 31) / 32);
    if (ctx->cfg.flags & DIT_FLAG_BF16_OPERANDS)
      transpose_bf16_to_f16_kernel<true><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(src), reinterpret_cast<__half*>(base + off), K, N);
    else
      transpose_bf16_to_f16_kernel<false><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(src), reinterpret_cast<__half*>(base + off), K, N);
    return cudaGetLastError();
  };
  DIT_CUDA_TRY(ctx, cudaMemsetAsync(base + L.b_ada, 0, static_cast<size_t>(6) * H * 4, st));
  const bool fp8 = (ctx->cfg.flags & DIT_FLAG_FP8_GEMM) != 0;
  auto weight8 = [&](const void* src, size_t off, size_t scale_off, int K, int N) {   // [K, N] bf16 -> e4m3 [N, K] + scales [N]
    col_absmax_scale_kernel<<<(N + 255) / 256, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(src), reinterpret_cast<float*>(base + scale_off), K, N);
    dim3 grid((N + 31) / 32, (K + 31) / 32);
    transpose_bf16_to_e4m3_kernel<<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(src), reinterpret_cast<const float*>(base + scale_off), base + off, K, N);
    return cudaGetLastError();
  };
  DIT_CUDA_TRY(ctx, bias(w->b_ada, L.b_ada, 3 * H));
  DIT_CUDA_TRY(ctx, fp8 ? weight8(w->w_qkv, L.w_qkv, L.s_qkv, H, 3 * H) : weight(w->w_qkv, L.w_qkv, H, 3 * H));
  DIT_CUDA_TRY(ctx, bias(w->b_qkv, L.b_qkv, 3 * H));
  DIT_CUDA_TRY(ctx, fp8 ? weight8(w->w_fc1, L.w_fc1, L.s_fc1, H, F) : weight(w->w_fc1, L.w_fc1, H, F));
  DIT_CUDA_TRY(ctx, bias(w->b_fc1, L.b_fc1, F));
  DIT_CUDA_TRY(ctx, fp8 ? weight8(w->w_out, L.w_o, L.s_fc2, H + F, H) : weight(w->w_out, L.w_o, H + F, H));   // runs on over the W_fc2 region
  DIT_CUDA_TRY(ctx, bias(w->b_out, L.b_fc2, H));
  DIT_CUDA_TRY(ctx, bias(w->q_norm, L.q_norm, ctx->cfg.head_dim, 1.f));
  DIT_CUDA_TRY(ctx, bias(w->k_norm, L.k_norm, ctx->cfg.head_dim, 1.f));
  if (!(fp8 ? make_map8(ctx, &bs.tm_qkv, base + L.w_qkv, H, 3 * H, gemm_cfg::BN / 2) : make_map(ctx, &bs.tm_qkv, base + L.w_qkv, H, 3 * H, gemm_cfg::BN / 2)) ||
      !(fp8 ? make_map8(ctx, &bs.tm_fc1, base + L.w_fc1, H, F, gemm_cfg::BN / 2) : make_map(ctx, &bs.tm_fc1, base + L.w_fc1, H, F, gemm_cfg::BN / 2)) ||
      !(fp8 ? make_map8(ctx, &bs.tm_fc2, base + L.w_o, H + F, H, gemm_cfg::BN / 2) : make_map(ctx, &bs.tm_fc2, base + L.w_o, H + F, H, gemm_cfg::BN / 2)))
    return fail(ctx, DIT_ERR_CUDA, "cuTensorMapEncodeTiled failed for a weight matrix");
  bs.loaded = true;
  return DIT_OK;
}

dit_status dit_pack_requests(const dit_request* reqs, int32_t n, int32_t* token_lens, int32_t* cu_seqlens,
                             int32_t* row_req, int32_t* row_local, int32_t* total_tokens) {
  if (n < 0 || (n > 0 && !reqs) || !token_lens || !cu_seqlens || !total_tokens) return DIT_ERR_INVALID_ARG;
  long long cu = 0;
  for (int r = 0; r < n; ++r) {
    const dit_request& q = reqs[r];
    if (q.height <= 0 || q.width <= 0 || q.height % 16 || q.width % 16 || q.n_text_tokens < 0) return DIT_ERR_SHAPE;
    const long long l = static_cast<long long>(q.height / 16) * (q.width / 16) + q.n_text_tokens;
    if (cu + l > INT32_MAX) return DIT_ERR_CAPACITY;
    cu += l;
  }
  cu = 0;
  cu_seqlens[0] = 0;
  for (int r = 0; r < n; ++r) {
    const int32_t l = (reqs[r].height / 16) * (reqs[r].width / 16) + reqs[r].n_text_tokens;
    token_lens[r] = l;
    for (int32_t i = 0; i < l; ++i) {
      if (row_req) row_req[cu + i] = r;
      if (row_local) row_local[cu + i] = i;
    }
    cu += l;
    cu_seqlens[r + 1] = static_cast<int32_t>(cu);
  }
  *total_tokens = static_cast<int32_t>(cu);
  return DIT_OK;
}

dit_status dit_pack_tokens(dit_ctx* ctx, const void* const* per_request_tokens, const int32_t* token_lens, int32_t n,
                           void* packed_tokens, void* stream) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  if (n < 0) return fail(ctx, DIT_ERR_INVALID_ARG, "n is negative");
  if (n == 0) return DIT_OK;
  if (!per_request_tokens || !token_lens || !packed_tokens) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL pointer argument");
  if (n > ctx->cfg.max_requests) return fail(ctx, DIT_ERR_CAPACITY, "n exceeds max_requests");
  SeqInfo seq{};
  if (!build_seq(token_lens, n, &seq)) return fail(ctx, DIT_ERR_INVALID_ARG, "every request needs at least one token");
  PtrList pl{};
  for (int r = 0; r < n; ++r) {
    if (!per_request_tokens[r]) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL request buffer");
    pl.ptr[r] = per_request_tokens[r];
  }
  const int row_vecs = ctx->cfg.hidden * 2 / 16;
  const long long total = static_cast<long long>(seq.total) * row_vecs;
  const int grid = static_cast<int>(std::min<long long>((total + 255) / 256, static_cast<long long>(ctx->num_sms) * 16));
  pack_tokens_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(pl, seq, packed_tokens, row_vecs);
  DIT_CUDA_TRY(ctx, cudaGetLastError());
  return DIT_OK;
}

dit_status dit_step_forward(dit_ctx* ctx, const void* packed_tokens, const int32_t* lens, int32_t n, const void* cond,
                            int32_t n_blocks, float* out, void* stream) {
  dit_status s = check_step_args(ctx, packed_tokens, lens, n, cond, n_blocks, out);
  if (s != DIT_OK || n == 0) return s;
  if (reinterpret_cast<uintptr_t>(packed_tokens) % 16 || reinterpret_cast<uintptr_t>(out) % 16)
    return fail(ctx, DIT_ERR_INVALID_ARG, "packed_tokens and out must be 16-byte aligned");
  return step_impl(ctx, packed_tokens, lens, n, cond, n_blocks, out, static_cast<cudaStream_t>(stream));
}

dit_status dit_step_forward_host_async(dit_ctx* ctx, const void* host_tokens, const int32_t* lens, int32_t n,
                                       const void* host_cond, int32_t n_blocks, float* host_out, void* stream) {
  dit_status s = check_step_args(ctx, host_tokens, lens, n, host_cond, n_blocks, host_out);
  if (s != DIT_OK || n == 0) return s;            // an empty batch is a no-op and does not count as a call
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  size_t T = 0;
  for (int r = 0; r < n; ++r) T += lens[r];
  const size_t H = ctx->cfg.hidden, C = ctx->cfg.cond_dim;
  void* d_tok = ctx->ws + ctx->lay.stage_tokens;
  void* d_cond = ctx->ws + ctx->lay.stage_cond;
  float* d_out = ctx->at<float>(ctx->lay.stage_out);
  // cond first (the modulation kernel needs nothing else; it follows the previous step on `st`), then the
  // tokens in row slices on the host-to-device stream: they may go in as soon as block 0 of the PREVIOUS step
  // has read the staging buffer, i.e. under that step's remaining blocks; block 0 of this step starts on a
  // slice as soon as it has landed
  DIT_CUDA_TRY(ctx, cudaMemcpyAsync(d_cond, host_cond, n * C * 2, cudaMemcpyHostToDevice, st));
  {
    if (ctx->last_step_from_host) {
      DIT_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->h2d_stream, ctx->tok_consumed, 0));
    } else {
      // some other step (or a replayed graph of one) may still be reading the staging buffer: wait for all of it
      DIT_CUDA_TRY(ctx, cudaEventRecord(ctx->st_entry, st));
      DIT_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->h2d_stream, ctx->st_entry, 0));
    }
    const size_t tile_rows = 2 * gemm_cfg::BM;
    const size_t per = ((T + tile_rows - 1) / tile_rows + kHostOutSlices - 1) / kHostOutSlices * tile_rows;
    for (size_t sidx = 0, r0 = 0; sidx < static_cast<size_t>(kHostOutSlices); ++sidx, r0 += per) {
      if (r0 < T) {
        const size_t rows = std::min(per, T - r0);
        DIT_CUDA_TRY(ctx, cudaMemcpyAsync(static_cast<uint8_t*>(d_tok) + r0 * H * 2, static_cast<const uint8_t*>(host_tokens) + r0 * H * 2,
                                          rows * H * 2, cudaMemcpyHostToDevice, ctx->h2d_stream));
      }
      DIT_CUDA_TRY(ctx, cudaEventRecord(ctx->tok_ready[sidx], ctx->h2d_stream));
    }
  }
  ctx->host_copied = false;
  const uint64_t call = ctx->host_calls;           // step_impl records this call's arrival event d2h_done[call & 1]
  s = step_impl(ctx, d_tok, lens, n, d_cond, n_blocks, d_out, st, nullptr, host_out, true);
  if (s != DIT_OK) return s;
  // the output normally goes back slice by slice on the copy stream (see step_impl); otherwise in one piece here
  if (!ctx->host_copied) {
    DIT_CUDA_TRY(ctx, cudaStreamWaitEvent(st, ctx->d2h_done[(call & 1) ^ 1], 0));
    DIT_CUDA_TRY(ctx, cudaMemcpyAsync(host_out, d_out, T * H * 4, cudaMemcpyDeviceToHost, st));
    DIT_CUDA_TRY(ctx, cudaEventRecord(ctx->d2h_done[call & 1], st));
  }
  ctx->host_calls = call + 1;
  return DIT_OK;
}

dit_status dit_host_wait(dit_ctx* ctx, int32_t calls_back) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  if (calls_back < 0 || calls_back > 1) return fail(ctx, DIT_ERR_INVALID_ARG, "calls_back must be 0 (the latest call) or 1 (the one before)");
  if (ctx->host_calls <= static_cast<uint64_t>(calls_back)) return DIT_OK;        // no such call yet
  DIT_CUDA_TRY(ctx, cudaEventSynchronize(ctx->d2h_done[(ctx->host_calls - 1 - calls_back) & 1]));
  return DIT_OK;
}

dit_status dit_step_forward_host(dit_ctx* ctx, const void* host_tokens, const int32_t* lens, int32_t n,
                                 const void* host_cond, int32_t n_blocks, float* host_out, void* stream) {
  const dit_status s = dit_step_forward_host_async(ctx, host_tokens, lens, n, host_cond, n_blocks, host_out, stream);
  if (s != DIT_OK || n == 0) return s;
  return dit_host_wait(ctx, 0);
}

dit_status dit_ctx_poll_status(dit_ctx* ctx) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  int word[4] = {0, 0, 0, 0};
  DIT_CUDA_TRY(ctx, cudaDeviceSynchronize());
  DIT_CUDA_TRY(ctx, cudaMemcpy(word, ctx->ws + ctx->lay.status, sizeof(word), cudaMemcpyDeviceToHost));
  if (word[0] == kStatusOk) return DIT_OK;
  DIT_CUDA_TRY(ctx, cudaMemset(ctx->ws + ctx->lay.status, 0, sizeof(word)));
  return fail(ctx, DIT_ERR_TIMEOUT, "a bounded wait ran out in the %s kernel",
              word[0] == kStatusGemmTimeout ? "GEMM" : (word[0] == kStatusAttnTimeout ? "attention" : (word[0] == kStatusLnTimeout ? "LayerNorm" :
              (word[0] == kStatusTestTimeout ? "wait-expiry test" : "modulation"))));
}

dit_status dit_debug_tap(dit_ctx* ctx, dit_tap which, const void** ptr, int64_t* rows, int64_t* cols, int32_t* elem_bytes) {
  if (!ctx || !ptr || !rows || !cols || !elem_bytes) return DIT_ERR_INVALID_ARG;
  const int64_t H = ctx->cfg.hidden, F = ctx->cfg.mlp_hidden, T = ctx->last_T;
  if (ctx->last_parallel && (which == DIT_TAP_ATTN || which == DIT_TAP_U))
    return fail(ctx, DIT_ERR_INVALID_ARG, "a parallel block keeps attention and MLP outputs interleaved: no dense tap");
  switch (which) {
    case DIT_TAP_H: *ptr = ctx->ws + ctx->lay.h; *rows = T; *cols = H; *elem_bytes = 2; break;
    case DIT_TAP_QKV: *ptr = ctx->ws + ctx->lay.qkv; *rows = T; *cols = 3 * H; *elem_bytes = 2; break;
    case DIT_TAP_ATTN: *ptr = ctx->ws + ctx->lay.a; *rows = T; *cols = H; *elem_bytes = 2; break;
    case DIT_TAP_U: *ptr = ctx->ws + ctx->lay.u; *rows = T; *cols = F; *elem_bytes = 2; break;
    case DIT_TAP_MOD: *ptr = ctx->ws + ctx->lay.mod; *rows = static_cast<int64_t>(ctx->last_R) * ctx->last_nb; *cols = 6 * H; *elem_bytes = 4; break;
    case DIT_TAP_STREAM: *ptr = ctx->ws + ctx->lay.stream; *rows = T; *cols = H; *elem_bytes = 4; break;
    default: return DIT_ERR_INVALID_ARG;
  }
  return DIT_OK;
}

dit_status dit_debug_poison(dit_ctx* ctx, void* stream) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Layout& L = ctx->lay;
  for (int i = 0; i < L.n_poison; ++i)
    DIT_CUDA_TRY(ctx, cudaMemsetAsync(ctx->ws + L.poison_begin[i], 0xFF, L.poison_end[i] - L.poison_begin[i], st));
  for (int g = 0; g < L.n_guards; ++g) {
    fill_u32_kernel<<<1, 256, 0, st>>>(reinterpret_cast<uint32_t*>(ctx->ws + L.guard[g]), kGuardPattern, static_cast<int>(kGuardBytes / 4));
    DIT_CUDA_TRY(ctx, cudaGetLastError());
  }
  return DIT_OK;
}

dit_status dit_debug_check_guards(dit_ctx* ctx, int32_t* n_damaged) {
  if (!ctx || !n_damaged) return DIT_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  *n_damaged = 0;
  DIT_CUDA_TRY(ctx, cudaDeviceSynchronize());
  uint32_t host[kGuardBytes / 4];
  for (int g = 0; g < ctx->lay.n_guards; ++g) {
    DIT_CUDA_TRY(ctx, cudaMemcpy(host, ctx->ws + ctx->lay.guard[g], kGuardBytes, cudaMemcpyDeviceToHost));
    for (size_t i = 0; i < kGuardBytes / 4; ++i)
      if (host[i] != kGuardPattern) { ++*n_damaged; break; }
  }
  return DIT_OK;
}

dit_status dit_debug_clock_probe(dit_ctx* ctx, int32_t enabled, int32_t* attention_mhz, int32_t* cycles_per_key_block,
                                 int32_t* gemm_mhz) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  DIT_CUDA_TRY(ctx, cudaDeviceSynchronize());
  int word[3] = {0, 0, 0};
  DIT_CUDA_TRY(ctx, cudaMemcpy(word, ctx->at<int>(ctx->lay.status) + 4, sizeof(word), cudaMemcpyDeviceToHost));
  DIT_CUDA_TRY(ctx, cudaMemset(ctx->at<int>(ctx->lay.status) + 4, 0, sizeof(word)));
  if (attention_mhz) *attention_mhz = word[0];
  if (cycles_per_key_block) *cycles_per_key_block = word[1];
  if (gemm_mhz) *gemm_mhz = word[2];
  ctx->attn_probe = enabled != 0;
  return DIT_OK;
}

dit_status dit_debug_expire_wait(dit_ctx* ctx, void* stream) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  expire_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ctx->at<int>(ctx->lay.status));
  DIT_CUDA_TRY(ctx, cudaGetLastError());
  return DIT_OK;
}

dit_status dit_ctx_set_timing(dit_ctx* ctx, int32_t enabled) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  ctx->timing = enabled != 0;
  ctx->ev_used = 0;
  return DIT_OK;
}

dit_status dit_ctx_read_timing(dit_ctx* ctx, double* ms_by_kernel, int64_t* launches_by_kernel) {
  if (!ctx || !ms_by_kernel || !launches_by_kernel) return DIT_ERR_INVALID_ARG;
  for (int k = 0; k < DIT_KERNEL_KINDS; ++k) { ms_by_kernel[k] = 0.0; launches_by_kernel[k] = 0; }
  DIT_CUDA_TRY(ctx, cudaDeviceSynchronize());
  for (size_t i = 0; i < ctx->ev_used; ++i) {
    float ms = 0.f;
    DIT_CUDA_TRY(ctx, cudaEventElapsedTime(&ms, ctx->ev_pool[2 * i], ctx->ev_pool[2 * i + 1]));
    ms_by_kernel[ctx->ev_kind[i]] += ms;
    launches_by_kernel[ctx->ev_kind[i]] += 1;
  }
  ctx->ev_used = 0;
  return DIT_OK;
}

int64_t dit_last_launch_count(const dit_ctx* ctx) { return ctx ? ctx->last_launches : 0; }

const char* dit_status_string(dit_status s) {
  switch (s) {
    case DIT_OK: return "ok";
    case DIT_ERR_INVALID_ARG: return "invalid argument";
    case DIT_ERR_SHAPE: return "unsupported shape";
    case DIT_ERR_CAPACITY: return "capacity exceeded";
    case DIT_ERR_NOT_LOADED: return "block weights not loaded";
    case DIT_ERR_UNSUPPORTED_ARCH: return "device is not sm_100";
    case DIT_ERR_CUDA: return "CUDA error";
    case DIT_ERR_TIMEOUT: return "device wait timed out";
    case DIT_ERR_INTERNAL: return "internal error";
  }
  return "unknown status";
}

const char* dit_last_error(const dit_ctx* ctx) { return ctx ? ctx->err : ""; }

}  // extern "C"

// =============================================================================================== shell around the block stack
namespace {

// Packed-batch and per-request geometry from a HOST request array (same rules as dit_pack_requests).
dit_status build_shell(dit_ctx* ctx, const dit_request* reqs, int n, const float* dsigma, SeqInfo* seq, ShellInfo* info,
                       int* total_text = nullptr) {
  if (n > ctx->cfg.max_requests) return fail(ctx, DIT_ERR_CAPACITY, "n exceeds max_requests");
  int32_t lens[DIT_MAX_REQUESTS];
  long long total = 0;
  info->img_cu[0] = 0;
  int txt_rows = 0;
  for (int r = 0; r < n; ++r) {
    const dit_request& q = reqs[r];
    if (q.height <= 0 || q.width <= 0 || q.height % 16 || q.width % 16 || q.n_text_tokens < 0)
      return fail(ctx, DIT_ERR_SHAPE, "resolution must be a positive multiple of 16 and the text length non-negative");
    const long long n_img = static_cast<long long>(q.height / 16) * (q.width / 16);
    total += n_img + q.n_text_tokens;
    if (total > ctx->cfg.max_total_tokens) return fail(ctx, DIT_ERR_CAPACITY, "packed batch exceeds max_total_tokens");
    lens[r] = static_cast<int32_t>(n_img + q.n_text_tokens);
    info->lat_off[r] = 64ll * info->img_cu[r];
    info->txt_row[r] = txt_rows;
    info->img_cu[r + 1] = info->img_cu[r] + static_cast<int>(n_img);
    txt_rows += q.n_text_tokens;
    info->gw[r] = q.width / 16;
    info->t[r] = q.timestep;
    info->dsigma[r] = dsigma ? dsigma[r] : 0.f;
  }
  if (!build_seq(lens, n, seq)) return fail(ctx, DIT_ERR_INTERNAL, "empty request");
  if (total_text) *total_text = txt_rows;
  return DIT_OK;
}

RowGeom geom_of(const ShellInfo& info) {
  RowGeom g{};
  memcpy(g.img_cu, info.img_cu, sizeof(g.img_cu));
  memcpy(g.gw, info.gw, sizeof(g.gw));
  return g;
}

// out[r, :] = act(in[r, :]) W + b (+ addend[r, :]): the modulation kernel with one "block".
template <int kIn>
cudaError_t launch_small_linear(const void* in, const void* w, const float* b, const float* addend, float* out32,
                                __nv_bfloat16* out16, int R, int K, int N, cudaStream_t st) {
  ModParams mp{};
  if (kIn == kModInCondSilu) mp.cond = static_cast<const __nv_bfloat16*>(in); else mp.in32 = static_cast<const float*>(in);
  mp.w_ada0 = static_cast<const __nv_bfloat16*>(w);
  mp.b_ada0 = b;
  mp.mod = out32; mp.out16 = out16; mp.addend = addend;
  mp.R = R; mp.C = K; mp.N6 = N; mp.NB = 1;
  modulation_kernel<kIn><<<(N + kModColsMin - 1) / kModColsMin, kModThreads, mod_smem_bytes(K), st>>>(mp);
  return cudaGetLastError();
}

dit_status cond_impl(dit_ctx* ctx, const ShellInfo& info, int n, const float* pooled, void* cond_out, cudaStream_t st) {
  const int Cd = ctx->cfg.cond_dim;
  float* temb = ctx->at<float>(ctx->lay.sh_temb);
  float* pre1 = ctx->at<float>(ctx->lay.sh_pre1);
  timestep_embed_kernel<<<n, kTEmbDim, 0, st>>>(info, temb);
  DIT_CUDA_TRY(ctx, cudaGetLastError());
  DIT_CUDA_TRY(ctx, launch_small_linear<kModInF32>(temb, ctx->ws + ctx->lay.sh_w_t1, ctx->at<float>(ctx->lay.sh_b_t1), nullptr,
                                                   pre1, nullptr, n, kTEmbDim, Cd, st));
  DIT_CUDA_TRY(ctx, launch_small_linear<kModInF32Silu>(pre1, ctx->ws + ctx->lay.sh_w_t2, ctx->at<float>(ctx->lay.sh_b_t2), pooled,
                                                       nullptr, static_cast<__nv_bfloat16*>(cond_out), n, Cd, Cd, st));
  return DIT_OK;
}

dit_status embed_impl(dit_ctx* ctx, const float* latents, const void* text, const SeqInfo& seq, const ShellInfo& info,
                      void* tokens, cudaStream_t st) {
  const int H = ctx->cfg.hidden;
  dim3 grid((seq.total + kEmbRows - 1) / kEmbRows, (H + kEmbCols - 1) / kEmbCols);
  embed_latents_kernel<<<grid, kEmbThreads, 0, st>>>(latents, static_cast<const __nv_bfloat16*>(text),
                                                     ctx->at<__nv_bfloat16>(ctx->lay.sh_w_in), ctx->at<float>(ctx->lay.sh_b_in),
                                                     static_cast<__nv_bfloat16*>(tokens), H, seq, info);
  DIT_CUDA_TRY(ctx, cudaGetLastError());
  return DIT_OK;
}

// Final adaLN + output projection, then un-patchify into `velocity` and/or the Euler update of `latents`.
dit_status final_impl(dit_ctx* ctx, const float* x, const SeqInfo& seq, const ShellInfo& info, int n, const void* cond,
                      float* velocity, float* latents, cudaStream_t st) {
  const dit_config& c = ctx->cfg;
  const int T = seq.total, H = c.hidden;
  float* modfin = ctx->at<float>(ctx->lay.sh_modfin);
  __half* h = ctx->at<__half>(ctx->lay.h);
  float* vtok = ctx->at<float>(ctx->lay.sh_vtok);
  CUtensorMap tm_h;
  if (!make_map(ctx, &tm_h, h, H, T, gemm_cfg::BM)) return fail(ctx, DIT_ERR_CUDA, "cuTensorMapEncodeTiled failed for an activation buffer");
  DIT_CUDA_TRY(ctx, launch_small_linear<kModInCondSilu>(cond, ctx->ws + ctx->lay.sh_w_fa, ctx->at<float>(ctx->lay.sh_b_fa), nullptr,
                                                        modfin, nullptr, n, c.cond_dim, 2 * H, st));
  DIT_CUDA_TRY(ctx, launch_ln<false>(x, nullptr, h, modfin, modfin + H, 2ll * H, T, H, c.ln_eps, seq, st, 0, kNoGeom, nullptr, ctx->num_sms, ctx->at<int>(ctx->lay.status),
                                     0, (c.flags & DIT_FLAG_BF16_OPERANDS) != 0));
  GemmParams g{};
  g.status = ctx->at<int>(ctx->lay.status);
  g.M = T; g.N = DIT_PATCH_DIM; g.K = H;
  g.bias = ctx->at<float>(ctx->lay.sh_b_out);
  g.out32 = vtok;
  DIT_CUDA_TRY(ctx, launch_gemm<kEpiBiasF32>(ctx, tm_h, ctx->tm_wout, g, seq, st));
  const long long work = static_cast<long long>(T) * (DIT_PATCH_DIM / 2);
  const int grid = static_cast<int>(std::min<long long>((work + 255) / 256, static_cast<long long>(ctx->num_sms) * 16));
  unpatchify_update_kernel<<<grid, 256, 0, st>>>(vtok, velocity, latents, seq, info);
  DIT_CUDA_TRY(ctx, cudaGetLastError());
  return DIT_OK;
}

dit_status check_shell_args(dit_ctx* ctx, const dit_request* reqs, int n) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  if (n < 0) return fail(ctx, DIT_ERR_INVALID_ARG, "n is negative");
  if (n > 0 && !reqs) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL requests");
  if (n > 0 && !ctx->shell_loaded) return fail(ctx, DIT_ERR_NOT_LOADED, "dit_load_shell_weights has not been called");
  return DIT_OK;
}

}  // namespace

extern "C" {

dit_status dit_load_shell_weights(dit_ctx* ctx, const dit_shell_weights* w, void* stream) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  if (!w) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL weights");
  if (!w->w_in || !w->w_t1 || !w->w_t2 || !w->w_fa || !w->w_out) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL weight matrix");
  const size_t H = ctx->cfg.hidden, Cd = ctx->cfg.cond_dim;
  if (Cd % 8) return fail(ctx, DIT_ERR_SHAPE, "the shell needs cond_dim to be a multiple of 8");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Layout& L = ctx->lay;
  ctx->shell_loaded = false;
  auto copy = [&](size_t off, const void* src, size_t bytes) {
    return cudaMemcpyAsync(ctx->ws + off, src, bytes, cudaMemcpyDeviceToDevice, st);
  };
  auto bias = [&](const void* src, size_t off, int n) {
    bf16_to_f32_kernel<<<(n + 255) / 256, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(src), ctx->at<float>(off), n, 0.f);
    return cudaGetLastError();
  };
  DIT_CUDA_TRY(ctx, copy(L.sh_w_in, w->w_in, DIT_PATCH_DIM * H * 2));
  DIT_CUDA_TRY(ctx, copy(L.sh_w_t1, w->w_t1, DIT_T_EMB_DIM * Cd * 2));
  DIT_CUDA_TRY(ctx, copy(L.sh_w_t2, w->w_t2, Cd * Cd * 2));
  DIT_CUDA_TRY(ctx, copy(L.sh_w_fa, w->w_fa, Cd * 2 * H * 2));
  DIT_CUDA_TRY(ctx, bias(w->b_in, L.sh_b_in, static_cast<int>(H)));
  DIT_CUDA_TRY(ctx, bias(w->b_t1, L.sh_b_t1, static_cast<int>(Cd)));
  DIT_CUDA_TRY(ctx, bias(w->b_t2, L.sh_b_t2, static_cast<int>(Cd)));
  DIT_CUDA_TRY(ctx, bias(w->b_fa, L.sh_b_fa, static_cast<int>(2 * H)));
  DIT_CUDA_TRY(ctx, bias(w->b_out, L.sh_b_out, DIT_PATCH_DIM));
  // W_out [H, 64] bf16 -> fp16 [64, H], padded with zero rows up to one weight tile
  DIT_CUDA_TRY(ctx, cudaMemsetAsync(ctx->ws + L.sh_w_out, 0, kWoutRows * H * 2, st));
  {
    dim3 grid((DIT_PATCH_DIM + 31) / 32, static_cast<unsigned>((H + 31) / 32));
    if (ctx->cfg.flags & DIT_FLAG_BF16_OPERANDS)
      transpose_bf16_to_f16_kernel<true><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(w->w_out), ctx->at<__half>(L.sh_w_out),
                                                               static_cast<int>(H), DIT_PATCH_DIM);
    else
      transpose_bf16_to_f16_kernel<false><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(w->w_out), ctx->at<__half>(L.sh_w_out),
                                                                static_cast<int>(H), DIT_PATCH_DIM);
    DIT_CUDA_TRY(ctx, cudaGetLastError());
  }
  if (!make_map(ctx, &ctx->tm_wout, ctx->ws + L.sh_w_out, H, kWoutRows, gemm_cfg::BN / 2))
    return fail(ctx, DIT_ERR_CUDA, "cuTensorMapEncodeTiled failed for a weight matrix");
  ctx->shell_loaded = true;
  return DIT_OK;
}

dit_status dit_timestep_cond(dit_ctx* ctx, const dit_request* reqs, int32_t n, const float* pooled, void* cond_out, void* stream) {
  dit_status s = check_shell_args(ctx, reqs, n);
  if (s != DIT_OK || n == 0) return s;
  if (!cond_out) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL pointer argument");
  SeqInfo seq{}; ShellInfo info{};
  s = build_shell(ctx, reqs, n, nullptr, &seq, &info);
  if (s != DIT_OK) return s;
  return cond_impl(ctx, info, n, pooled, cond_out, static_cast<cudaStream_t>(stream));
}

dit_status dit_embed_latents(dit_ctx* ctx, const float* latents, const void* text_tokens, const dit_request* reqs, int32_t n,
                             void* packed_tokens, void* stream) {
  dit_status s = check_shell_args(ctx, reqs, n);
  if (s != DIT_OK || n == 0) return s;
  if (!latents || !packed_tokens) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL pointer argument");
  SeqInfo seq{}; ShellInfo info{};
  int total_text = 0;
  s = build_shell(ctx, reqs, n, nullptr, &seq, &info, &total_text);
  if (s != DIT_OK) return s;
  if (total_text > 0 && !text_tokens) return fail(ctx, DIT_ERR_INVALID_ARG, "text_tokens is NULL but a request has text tokens");
  return embed_impl(ctx, latents, text_tokens, seq, info, packed_tokens, static_cast<cudaStream_t>(stream));
}

dit_status dit_final_layer(dit_ctx* ctx, const float* x, const dit_request* reqs, int32_t n, const void* cond, float* velocity,
                           void* stream) {
  dit_status s = check_shell_args(ctx, reqs, n);
  if (s != DIT_OK || n == 0) return s;
  if (!x || !cond || !velocity) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL pointer argument");
  if (reinterpret_cast<uintptr_t>(x) % 16) return fail(ctx, DIT_ERR_INVALID_ARG, "x must be 16-byte aligned");
  SeqInfo seq{}; ShellInfo info{};
  s = build_shell(ctx, reqs, n, nullptr, &seq, &info);
  if (s != DIT_OK) return s;
  return final_impl(ctx, x, seq, info, n, cond, velocity, nullptr, static_cast<cudaStream_t>(stream));
}

dit_status dit_sampler_update(dit_ctx* ctx, float* latents, const float* velocity, const dit_request* reqs, int32_t n,
                              const float* dsigma, void* stream) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  if (n < 0) return fail(ctx, DIT_ERR_INVALID_ARG, "n is negative");
  if (n == 0) return DIT_OK;
  if (!latents || !velocity || !reqs || !dsigma) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL pointer argument");
  SeqInfo seq{}; ShellInfo info{};
  dit_status s = build_shell(ctx, reqs, n, dsigma, &seq, &info);
  if (s != DIT_OK) return s;
  const long long total = 64ll * info.img_cu[n];
  const int grid = static_cast<int>(std::min<long long>((total + 255) / 256, static_cast<long long>(ctx->num_sms) * 16));
  euler_update_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(latents, velocity, info, n);
  DIT_CUDA_TRY(ctx, cudaGetLastError());
  return DIT_OK;
}

dit_status dit_step_forward_requests(dit_ctx* ctx, const void* packed_tokens, const dit_request* reqs, int32_t n,
                                     const void* cond, int32_t n_blocks, float* out, void* stream) {
  if (!ctx) return DIT_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  if (n < 0) return fail(ctx, DIT_ERR_INVALID_ARG, "n_requests is negative");
  if (n == 0) return DIT_OK;
  if (!reqs) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL pointer argument");
  SeqInfo seq{}; ShellInfo info{};
  dit_status s = build_shell(ctx, reqs, n, nullptr, &seq, &info);
  if (s != DIT_OK) return s;
  int32_t lens[DIT_MAX_REQUESTS];
  for (int r = 0; r < n; ++r) lens[r] = seq.cu[r + 1] - seq.cu[r];
  s = check_step_args(ctx, packed_tokens, lens, n, cond, n_blocks, out);
  if (s != DIT_OK) return s;
  if (reinterpret_cast<uintptr_t>(packed_tokens) % 16 || reinterpret_cast<uintptr_t>(out) % 16)
    return fail(ctx, DIT_ERR_INVALID_ARG, "packed_tokens and out must be 16-byte aligned");
  const RowGeom geo = geom_of(info);
  return step_impl(ctx, packed_tokens, lens, n, cond, n_blocks, out, static_cast<cudaStream_t>(stream), &geo);
}

dit_status dit_denoise_step(dit_ctx* ctx, float* latents, const void* text_tokens, const dit_request* reqs, int32_t n,
                            const float* dsigma, const float* pooled, int32_t n_blocks, float* velocity, void* stream) {
  dit_status s = check_shell_args(ctx, reqs, n);
  if (s != DIT_OK || n == 0) return s;
  if (!latents || !dsigma) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL pointer argument");
  if (n_blocks < 1) return fail(ctx, DIT_ERR_INVALID_ARG, "n_blocks must be at least 1");
  if (n_blocks > ctx->cfg.max_blocks) return fail(ctx, DIT_ERR_CAPACITY, "n_blocks exceeds max_blocks");
  for (int b = 0; b < n_blocks; ++b)
    if (!ctx->blocks[b].loaded) return fail(ctx, DIT_ERR_NOT_LOADED, "a block in [0, n_blocks) has no weights");
  SeqInfo seq{}; ShellInfo info{};
  int total_text = 0;
  s = build_shell(ctx, reqs, n, dsigma, &seq, &info, &total_text);
  if (s != DIT_OK) return s;
  if (total_text > 0 && !text_tokens) return fail(ctx, DIT_ERR_INVALID_ARG, "text_tokens is NULL but a request has text tokens");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  void* cond = ctx->ws + ctx->lay.sh_cond;
  void* tokens = ctx->ws + ctx->lay.stage_tokens;
  float* x = ctx->at<float>(ctx->lay.stream);
  int32_t lens[DIT_MAX_REQUESTS];
  for (int r = 0; r < n; ++r) lens[r] = seq.cu[r + 1] - seq.cu[r];
  s = cond_impl(ctx, info, n, pooled, cond, st);
  if (s != DIT_OK) return s;
  s = embed_impl(ctx, latents, text_tokens, seq, info, tokens, st);
  if (s != DIT_OK) return s;
  const RowGeom geo = geom_of(info);
  s = step_impl(ctx, tokens, lens, n, cond, n_blocks, x, st, &geo);   // the last block writes the residual stream in place
  if (s != DIT_OK) return s;
  s = final_impl(ctx, x, seq, info, n, cond, velocity, latents, st);
  if (s != DIT_OK) return s;
  ctx->last_launches += 3 + 1 + 4;
  return DIT_OK;
}

dit_status dit_denoise_round(dit_ctx* ctx, float* latents, const void* text_tokens, const dit_request* reqs, int32_t n,
                             const int32_t* steps_in_round, const float* sigmas, int32_t sigma_stride, const float* pooled,
                             int32_t n_blocks, void* stream) {
  dit_status s = check_shell_args(ctx, reqs, n);
  if (s != DIT_OK || n == 0) return s;
  if (!latents || !steps_in_round || !sigmas) return fail(ctx, DIT_ERR_INVALID_ARG, "NULL pointer argument");
  if (n_blocks < 1) return fail(ctx, DIT_ERR_INVALID_ARG, "n_blocks must be at least 1");
  if (n_blocks > ctx->cfg.max_blocks) return fail(ctx, DIT_ERR_CAPACITY, "n_blocks exceeds max_blocks");
  for (int b = 0; b < n_blocks; ++b)
    if (!ctx->blocks[b].loaded) return fail(ctx, DIT_ERR_NOT_LOADED, "a block in [0, n_blocks) has no weights");
  int max_steps = 0;
  for (int r = 0; r < n; ++r) {
    if (steps_in_round[r] < 0) return fail(ctx, DIT_ERR_INVALID_ARG, "negative step count");
    max_steps = std::max(max_steps, steps_in_round[r]);
  }
  if (sigma_stride < max_steps + 1) return fail(ctx, DIT_ERR_INVALID_ARG, "sigma_stride must be at least the largest step count + 1");
  SeqInfo full_seq{}; ShellInfo full{};
  int total_text = 0;
  s = build_shell(ctx, reqs, n, nullptr, &full_seq, &full, &total_text);     // also checks shapes and capacity
  if (s != DIT_OK) return s;
  if (total_text > 0 && !text_tokens) return fail(ctx, DIT_ERR_INVALID_ARG, "text_tokens is NULL but a request has text tokens");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t Cd = ctx->cfg.cond_dim;
  void* cond = ctx->ws + ctx->lay.sh_cond;
  void* tokens = ctx->ws + ctx->lay.stage_tokens;
  float* x = ctx->at<float>(ctx->lay.stream);
  float* pooled_stage = ctx->at<float>(ctx->lay.sh_pooled);
  int64_t launches = 0;
  for (int k = 0; k < max_steps; ++k) {
    // the requests that still have a step to run in this round, in their original order
    SeqInfo seq{}; ShellInfo info{};
    int32_t lens[DIT_MAX_REQUESTS];
    int active[DIT_MAX_REQUESTS];
    int na = 0;
    info.img_cu[0] = 0;
    for (int r = 0; r < n; ++r) {
      if (steps_in_round[r] <= k) continue;
      const int n_img = full.img_cu[r + 1] - full.img_cu[r];
      lens[na] = full_seq.cu[r + 1] - full_seq.cu[r];
      info.img_cu[na + 1] = info.img_cu[na] + n_img;
      info.lat_off[na] = full.lat_off[r];
      info.txt_row[na] = full.txt_row[r];
      info.gw[na] = full.gw[r];
      const float s0 = sigmas[static_cast<size_t>(r) * sigma_stride + k], s1 = sigmas[static_cast<size_t>(r) * sigma_stride + k + 1];
      info.t[na] = 1000.0f * s0;
      info.dsigma[na] = s1 - s0;
      active[na] = r;
      ++na;
    }
    if (!build_seq(lens, na, &seq)) return fail(ctx, DIT_ERR_INTERNAL, "empty request");
    const float* pooled_k = pooled;
    if (pooled && na != n) {   // the batch has shrunk: line the active requests' pooled rows up
      for (int i = 0; i < na; ++i)
        DIT_CUDA_TRY(ctx, cudaMemcpyAsync(pooled_stage + i * Cd, pooled + active[i] * Cd, Cd * 4, cudaMemcpyDeviceToDevice, st));
      pooled_k = pooled_stage;
    }
    s = cond_impl(ctx, info, na, pooled_k, cond, st);
    if (s != DIT_OK) return s;
    s = embed_impl(ctx, latents, text_tokens, seq, info, tokens, st);
    if (s != DIT_OK) return s;
    const RowGeom geo = geom_of(info);
    s = step_impl(ctx, tokens, lens, na, cond, n_blocks, x, st, &geo);
    if (s != DIT_OK) return s;
    s = final_impl(ctx, x, seq, info, na, cond, nullptr, latents, st);
    if (s != DIT_OK) return s;
    launches += ctx->last_launches + 3 + 1 + 4;
  }
  ctx->last_launches = launches;
  return DIT_OK;
}

}  // extern "C"

// =============================================================================================== no-allocation entry point
// adaLN modulation vectors without a context, a workspace or any allocation.  The context path keeps
// the fp32 copy of the modulation bias in the caller's workspace; here that scratch is a fixed
// array inside the library image, so the call works for hosts that must not allocate device
// memory.  See include/dit.h for the contract.
namespace {

constexpr int kNoAllocMaxHidden = 4096;                       // same bound as dit_config.hidden
constexpr int kNoAllocMaxCond = kMaxCondDim;
constexpr int kNoAllocScratchFloats = 6 * kNoAllocMaxHidden;  // 96 KiB per GPU that loads the library
constexpr int kNoAllocMaxDevices = 64;

static __device__ __align__(256) float g_noalloc_bias_scratch[kNoAllocScratchFloats];

// In host code the array's name is only a handle for the runtime; the device address is looked up
// once per device (with that device current) and cached.
std::mutex g_noalloc_mutex;
float* g_noalloc_scratch_ptr[kNoAllocMaxDevices] = {};

cudaError_t noalloc_scratch_for_current_device(float** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kNoAllocMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (!g_noalloc_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_bias_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    e = cudaFuncSetAttribute(reinterpret_cast<const void*>(&modulation_kernel<kModInCondSilu>),
                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(mod_smem_bytes(kNoAllocMaxCond)));
    if (e != cudaSuccess) return e;
    g_noalloc_scratch_ptr[dev] = static_cast<float*>(p);
  }
  *out = g_noalloc_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" dit_status dit_modulation_noalloc(const void* cond, const void* w_ada, const void* b_ada,
                                             int32_t n_requests, int32_t cond_dim, int32_t hidden, float* mod_out,
                                             void* stream) {
  if (n_requests < 0) return DIT_ERR_INVALID_ARG;
  if (n_requests == 0) return DIT_OK;
  if (!cond || !w_ada || !mod_out) return DIT_ERR_INVALID_ARG;
  // W_ada is read with 16-byte loads (rows are 6H bf16 = a multiple of 16 bytes, so the base decides)
  if (reinterpret_cast<uintptr_t>(w_ada) % 16 || reinterpret_cast<uintptr_t>(mod_out) % 4 ||
      reinterpret_cast<uintptr_t>(cond) % 2 || reinterpret_cast<uintptr_t>(b_ada) % 2)
    return DIT_ERR_INVALID_ARG;
  if (hidden < 64 || hidden % 64 || cond_dim < 1) return DIT_ERR_SHAPE;
  if (hidden > kNoAllocMaxHidden || cond_dim > kNoAllocMaxCond || n_requests > DIT_MAX_REQUESTS) return DIT_ERR_CAPACITY;
  float* scratch = nullptr;
  if (noalloc_scratch_for_current_device(&scratch) != cudaSuccess) return DIT_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int n6 = 6 * hidden;
  // The scratch still holds the previous call's bias: rewrite all of [0, 6H) (zeros for a NULL bias).
  bf16_to_f32_kernel<<<(n6 + 255) / 256, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(b_ada), scratch, n6, 0.f);
  if (cudaGetLastError() != cudaSuccess) return DIT_ERR_CUDA;
  ModParams mp{};
  mp.cond = static_cast<const __nv_bfloat16*>(cond);
  mp.w_ada0 = static_cast<const __nv_bfloat16*>(w_ada);
  mp.b_ada0 = scratch;
  mp.w_block_stride = 0; mp.b_block_stride = 0;
  mp.mod = mod_out; mp.R = n_requests; mp.C = cond_dim; mp.N6 = n6; mp.NB = 1;
  modulation_kernel<kModInCondSilu><<<(n6 + kModColsMin - 1) / kModColsMin, kModThreads, mod_smem_bytes(cond_dim), st>>>(mp);
  if (cudaGetLastError() != cudaSuccess) return DIT_ERR_CUDA;
  return DIT_OK;
}

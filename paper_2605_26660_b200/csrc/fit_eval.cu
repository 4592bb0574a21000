// windq_fit_eval: every group of a weight matrix fitted under all six bit-widths.
//
// Bound by the FP32 pipes, not by HBM: about 28*K + 40 binary32 operations per 2-byte weight
// (K clip ratios x 4 uniform bit-widths x 7 operations, plus the ternary / binary fits).  The
// design therefore spends nothing on data movement tricks -- each lane reads its 64 bytes of a
// row once with 128-bit loads, straight into registers -- and everything on keeping the inner
// loop at its minimum instruction count (see fit_device.cuh).
//
// Work is split into items = (unit, block of GPW consecutive rows), one warp per item, no
// block-level synchronisation.  The grid is persistent (one block of 16 warps per SM) and the warps
// claim items from a counter in scratch, in order.
// Per item the warp writes seven partial sums (six errors and the energy, added over its rows in
// double) to scratch; a second small kernel adds them per unit in a fixed order, so unit totals
// are reproducible from run to run.
#include <string.h>

#include "fit_device.cuh"

namespace windq {

constexpr int kFitWarpsPerBlock = 16;  // one block of 16 warps per SM: measured 5 % faster than four blocks of 4
constexpr int kFitPartials = 8;  // 6 errors + energy + pad

__host__ __device__ inline int fit_cand_chunk(int G) {
  // candidates per shared-memory chunk: GPW * stride * 16 bytes <= ~5.4 KB per warp
  const int gpw = 32 / (G / 32);
  int c = 336 / gpw;  // 8 rows -> 42, 16 -> 21, 32 -> 10, 4 -> 84, 2 -> 168
  return c > 64 ? 64 : c;
}
__host__ __device__ inline int fit_cand_stride(int chunk) { return chunk | 1; }  // odd: conflict-free rows

// Several matrices in one launch (windq_fit_eval_batch): what differs from matrix to matrix, by value in
// the kernel's parameters.  Items are numbered through all jobs; job j owns [first_item[j], first_item[j+1]).
constexpr int kFitMaxJobs = 16;
struct FitJobs {
  const __half* W[kFitMaxJobs];
  const float* s[kFitMaxJobs];
  uint8_t* clip_idx[kFitMaxJobs];
  float* group_err[kFitMaxJobs];
  float* err[kFitMaxJobs];
  float* energy[kFitMaxJobs];
  __half* lowbit[kFitMaxJobs];  // [3][U][R]: 1.58-bit scale, 1-bit scale, 1.58-bit threshold (rounded towards zero), or NULL
  long long ldw[kFitMaxJobs];
  int R[kFitMaxJobs];
  int U[kFitMaxJobs];
  unsigned int first_item[kFitMaxJobs + 1];
  unsigned int first_unit[kFitMaxJobs + 1];
  int n;
  unsigned int* hist;  // FEAT: one 32768-bin histogram of |w| bit patterns per unit of all jobs, in scratch
};

// PROTECT: salient weights (key |w| * scale_j >= thresh[u], scale_j = sqrt(s_j)) are taken out of
// the fits: in the lane's registers such a weight becomes a zero weight with zero activation weight,
// after which the fit is the ordinary one.  `never` is a NaN (see the masking step).
// PARTS: every item is handed out in five parts (one per uniform bit-width, one for the two low-bit fits and
// the energy), each of which reloads the group.  Used for matrices with fewer than a few items per warp, where
// whole items leave most warps idle at the end (or from the start); the code of the other instantiation is
// untouched by it.
// BATCH: the matrix of an item is looked up in `jobs` (the scalar matrix parameters are then unused).
// FEAT (with BATCH): the pass also gathers what the state features of Table 1 need from the weights -- every weight
// is counted in its unit's histogram of |w| bit patterns (integer atomics in global memory: exact and independent
// of the order) and the item's signed sum goes to the spare eighth partial -- so that the features cost no second
// read of the matrix and no pass of their own.
template <int G, bool PROTECT, bool PARTS, bool BATCH, bool FEAT = false>
__global__ void __launch_bounds__(kFitWarpsPerBlock * 32, 1)
fit_eval_kernel(const __half* __restrict__ W_one, int R_one, int U_one, int64_t ldw_one, const float* __restrict__ s_one,
                const float* __restrict__ clip, int K, double* __restrict__ partial, uint8_t* __restrict__ clip_idx_one,
                float* __restrict__ group_err_one, int rows_blocks_one, int chunk, int stride,
                const float* __restrict__ scale, const float* __restrict__ thresh, float never,
                unsigned int* __restrict__ next_item, unsigned long long* __restrict__ work, const FitJobs jobs) {
  constexpr int LG = Map<G>::LG, GPW = Map<G>::GPW;
  extern __shared__ float4 smem_f4[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  Cand* cand = reinterpret_cast<Cand*>(smem_f4) + (size_t)warp * GPW * stride;
  __shared__ float4 ext_all[kFitWarpsPerBlock][32];  // every lane's least and greatest weight, for those bounds
  float4* ext = ext_all[warp];
  const int g = lane / LG, q = lane % LG;

  const unsigned int n_items = (BATCH ? jobs.first_item[jobs.n] : (unsigned int)(U_one * rows_blocks_one)) * (PARTS ? 5u : 1u);

  unsigned int searches = 0, skipped = 0;  // clip searches of this warp (K candidates each), and candidates left out
  Lane32 sv;
  for (;;) {
    // items are claimed from a counter, in order: with equal static shares the warps of an SM do not
    // finish together (the schedulers are not fair), and the SM ends the kernel on a few warps that
    // cannot fill its issue slots; an item is about 100,000 cycles of work against one atomic
    unsigned int item = 0;
    if (lane == 0) item = atomicAdd(next_item, 1u);
    item = __shfl_sync(0xffffffffu, item, 0);
    if (item >= n_items) break;
    unsigned int parts = 0x1fu;
    if (PARTS) {
      parts = 1u << (item % 5u);
      item /= 5u;
    }
    const __half* W = W_one;
    const float* s = s_one;
    uint8_t* clip_idx_out = clip_idx_one;
    float* group_err_out = group_err_one;
    int R = R_one, U = U_one, rows_blocks = rows_blocks_one;
    int64_t ldw = ldw_one;
    unsigned int local = item;
    int jfeat = 0;
    if (BATCH) {
      int j = 0;
      while (j + 1 < jobs.n && item >= jobs.first_item[j + 1]) ++j;
      jfeat = j;
      W = jobs.W[j];
      s = jobs.s[j];
      clip_idx_out = jobs.clip_idx[j];
      group_err_out = jobs.group_err[j];
      R = jobs.R[j];
      U = jobs.U[j];
      ldw = jobs.ldw[j];
      rows_blocks = (R + GPW - 1) / GPW;
      local = item - jobs.first_item[j];
    }
    const int u = (int)(local / rows_blocks), rb = (int)(local % rows_blocks);
    load_stats(s + (int64_t)u * G + 32 * q, sv);
    const int row = rb * GPW + g;
    const bool live = row < R;
    const int row_ld = live ? row : R - 1;  // rows past the end repeat the last row and are not written
    Lane32 wv;
    if (FEAT) {
      const uint4* p4 = reinterpret_cast<const uint4*>(W + (int64_t)row_ld * ldw + (int64_t)u * G + 32 * q);
      uint4 raw[4];
#pragma unroll
      for (int l = 0; l < 4; ++l) raw[l] = __ldg(p4 + l);
      unpack_weights(raw, wv);
      if (!PARTS || (parts & 0x10u)) {
        // histogram and signed sum of the item's live rows (once per item: with PARTS, in the part of the low-bit fits)
        unsigned int* h = jobs.hist + (size_t)(jobs.first_unit[jfeat] + u) * 32768u;
        float part = 0.0f;
        if (live) {
          const unsigned int* r = reinterpret_cast<const unsigned int*>(raw);
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            atomicAdd(h + (r[i] & 0x7fffu), 1u);
            atomicAdd(h + ((r[i] >> 16) & 0x7fffu), 1u);
          }
#pragma unroll
          for (int hh = 0; hh < 2; ++hh)
#pragma unroll
            for (int i = 0; i < 8; ++i) part += wv.v[hh][i].x + wv.v[hh][i].y;
        }
        double ds = (double)part;
#pragma unroll
        for (int m = 16; m > 0; m >>= 1) ds += __shfl_xor_sync(0xffffffffu, ds, m);
        if (lane == 0) partial[(int64_t)item * kFitPartials + 7] = ds;
      }
    } else {
      load_weights(W + (int64_t)row_ld * ldw + (int64_t)u * G + 32 * q, wv);
    }
    {
      // Masking step.  PROTECT: a weight whose key |w| * scale_j reaches the unit's threshold becomes a
      // zero weight with zero activation weight.  Otherwise the same step runs against `never`, a NaN
      // that the host passes in, so no comparison is ever true and no value changes -- but with every
      // w and s going through a select here, ptxas schedules the candidate loop with far fewer
      // dependency stalls (measured: 7 % less time, same instruction count, same results bit for bit).
      Lane32 av;
      if (PROTECT) load_stats(scale + (int64_t)u * G + 32 * q, av);
      else av = sv;
      const float tau = PROTECT ? __ldg(thresh + u) : never;
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (__fmul_rn(fabsf(wv.v[h][i].x), av.v[h][i].x) >= tau) { wv.v[h][i].x = 0.0f; sv.v[h][i].x = 0.0f; }
          if (__fmul_rn(fabsf(wv.v[h][i].y), av.v[h][i].y) >= tau) { wv.v[h][i].y = 0.0f; sv.v[h][i].y = 0.0f; }
        }
    }

    float mn, mx;
    group_range<G>(wv, mn, mx);
    const float rng = __fsub_rn(mx, mn);
    __syncwarp();                       // the previous item's search has read its entries
    ext[lane] = lane_extremes(wv, sv);  // read by the eight-bit search, after its __syncwarp()

    float e[3] = {0.0f, 0.0f, 0.0f};
#pragma unroll 1
    for (int bi = 0; bi < 4; ++bi) {
      if (PARTS && !((parts >> bi) & 1u)) continue;
      float be;
      int bk;
      ++searches;
      if (bi == 0) {
        search_uniform_pruned<G>(wv, sv, ext, mn, rng, bi, clip, K, cand, chunk, stride, lane, be, bk, skipped);
      } else {
        search_uniform<G>(wv, sv, mn, rng, bi, clip, K, cand, chunk, stride, lane, be, bk);
      }
      {
        double d = live ? (double)be : 0.0;
#pragma unroll
        for (int m = LG; m < 32; m <<= 1) d += __shfl_xor_sync(0xffffffffu, d, m);
        if (lane == 0) partial[(int64_t)item * kFitPartials + bi] = d;
      }
      if (live && q == 0) {
        const int64_t o = ((int64_t)bi * U + u) * R + row;
        if (clip_idx_out) clip_idx_out[o] = (uint8_t)bk;
        if (group_err_out) group_err_out[o] = be;
      }
    }
    if (!PARTS || (parts & 0x10u)) {
      // group errors wanted: the term-by-term sums (bit-defined); unit sums only: from the sums of the fit
      const LowBitFit low = fit_low_bits<G>(wv, sv, group_err_out != nullptr);
      e[0] = low.err_t;
      e[1] = low.err_b;
      e[2] = low.energy;
      if (live && q == 0 && group_err_out) {
        group_err_out[((int64_t)4 * U + u) * R + row] = low.err_t;
        group_err_out[((int64_t)5 * U + u) * R + row] = low.err_b;
      }
      if (BATCH) {
        // the parameters of the two low-bit fits, for a plan application that wants to skip their sums
        __half* lb = jobs.lowbit[jfeat];
        if (lb && live && q == 0) {
          const int64_t o = (int64_t)u * R + row, plane = (int64_t)U * R;
          lb[o] = __float2half_rn(low.alpha_t);               // exact: the value of an fp16 number
          lb[plane + o] = __float2half_rn(low.alpha_b);
          lb[2 * plane + o] = __float2half_rz(low.delta);      // |w| > delta for an fp16 |w| is |w| > this
        }
      }
    }

    // add over the rows of this item in double; lanes of a group hold equal values
#pragma unroll
    for (int c = 0; c < 3; ++c) {
      double d = live ? (double)e[c] : 0.0;
#pragma unroll
      for (int m = LG; m < 32; m <<= 1) d += __shfl_xor_sync(0xffffffffu, d, m);
      if (lane == 0 && (!PARTS || (parts & 0x10u))) partial[(int64_t)item * kFitPartials + 4 + c] = d;
    }
  }
  if (lane == 0 && searches) {
    atomicAdd(work, (unsigned long long)searches * (unsigned long long)K - (unsigned long long)skipped);
    atomicAdd(work + 1, (unsigned long long)searches * (unsigned long long)K);
  }
}

// err_out[u][0..5], energy_out[u] = sum over the unit's row blocks, fixed order.
__global__ void __launch_bounds__(256)
fit_finalize_kernel(const double* __restrict__ partial, int rows_blocks, float* __restrict__ err_out,
                    float* __restrict__ energy_out) {
  __shared__ double red[256];
  const int u = blockIdx.x, t = threadIdx.x;
  const double* p = partial + (int64_t)u * rows_blocks * kFitPartials;
  for (int c = 0; c < 7; ++c) {
    double acc = 0.0;
    for (int rb = t; rb < rows_blocks; rb += 256) acc += p[(int64_t)rb * kFitPartials + c];
    red[t] = acc;
    __syncthreads();
    for (int n = 128; n > 0; n >>= 1) {
      if (t < n) red[t] += red[t + n];
      __syncthreads();
    }
    if (t == 0) {
      if (c < 6) err_out[(int64_t)u * 6 + c] = (float)red[0];
      else if (energy_out) energy_out[u] = (float)red[0];
    }
    __syncthreads();
  }
}

// The same for a batch: block b is unit b - first_unit[j] of job j.
__global__ void __launch_bounds__(256)
fit_finalize_batch_kernel(const double* __restrict__ partial, int gpw, const FitJobs jobs, double* __restrict__ unit_wsum) {
  __shared__ double red[256];
  const int b = blockIdx.x, t = threadIdx.x;
  int j = 0;
  while (j + 1 < jobs.n && (unsigned int)b >= jobs.first_unit[j + 1]) ++j;
  const int u = b - (int)jobs.first_unit[j];
  const int rows_blocks = (jobs.R[j] + gpw - 1) / gpw;
  const double* p = partial + ((int64_t)jobs.first_item[j] + (int64_t)u * rows_blocks) * kFitPartials;
  for (int c = 0; c < (unit_wsum ? 8 : 7); ++c) {
    double acc = 0.0;
    for (int rb = t; rb < rows_blocks; rb += 256) acc += p[(int64_t)rb * kFitPartials + c];
    red[t] = acc;
    __syncthreads();
    for (int n = 128; n > 0; n >>= 1) {
      if (t < n) red[t] += red[t + n];
      __syncthreads();
    }
    if (t == 0) {
      if (c < 6) jobs.err[j][(int64_t)u * 6 + c] = (float)red[0];
      else if (c == 6) { if (jobs.energy[j]) jobs.energy[j][u] = (float)red[0]; }
      else unit_wsum[b] = red[0];  // sum of the unit's weights, for the features
    }
    __syncthreads();
  }
}

// sqrt(s_j): the activation scale that the saliency key uses.
__global__ void fit_scale_kernel(const float* __restrict__ s, int C, float* __restrict__ scale) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < C) scale[j] = __fsqrt_rn(s[j]);
}

template <int G, bool PROTECT>
windq_status launch_fit(windq_ctx* ctx, const __half* W, int R, int U, int64_t ldw, const float* s,
                        const float* clip, int K, double* partial, float* err_out, float* energy_out,
                        uint8_t* clip_idx_out, float* group_err_out, float* scale, const float* thresh,
                        unsigned int* next_item, cudaStream_t st) {
  constexpr int GPW = Map<G>::GPW;
  const int rows_blocks = (R + GPW - 1) / GPW;
  const int chunk = fit_cand_chunk(G), stride = fit_cand_stride(chunk);
  const size_t smem = (size_t)kFitWarpsPerBlock * GPW * stride * sizeof(Cand);
  const int id = (PROTECT ? kFitProtectG32 : kFitG32) + g_index(G);
  if (windq_status rc = prepare_kernel(ctx, id, fit_eval_kernel<G, PROTECT, false, false>, kFitWarpsPerBlock * 32, smem, true)) return rc;
  const int blocks_per_sm = ctx->occupancy[id];
  const int64_t n_items = (int64_t)U * rows_blocks;
  WINDQ_REQUIRE(ctx, n_items < (1ll << 28), WINDQ_ERR_SHAPE, "windq_fit_eval: R * C is too large for one call");
  const int64_t full_grid = (int64_t)ctx->sm_count * blocks_per_sm;
  // fewer than one and a half items per warp of a full grid: hand the items out in parts.  (With more, whole
  // items are as fast: an SM whose warps run out one by one gives their issue slots to the rest, measured on
  // 2048 x 2048.  A 512 x 2048 matrix, whose 1024 items would fill less than half the warps, gains 1.5x.)
  const bool in_parts = 2 * n_items < 3 * full_grid * kFitWarpsPerBlock;
  if (in_parts)
    if (windq_status rc = prepare_kernel(ctx, id + kFitPartsOffset, fit_eval_kernel<G, PROTECT, true, false>, kFitWarpsPerBlock * 32, smem, false))
      return rc;
  int64_t grid = full_grid;
  const int64_t need = ((in_parts ? 5 : 1) * n_items + kFitWarpsPerBlock - 1) / kFitWarpsPerBlock;
  if (grid > need) grid = need;
  WINDQ_CUDA(ctx, cudaMemsetAsync(next_item, 0, sizeof(unsigned int), st));
  if (PROTECT) fit_scale_kernel<<<(unsigned)((U * G + 255) / 256), 256, 0, st>>>(s, U * G, scale);
  if (in_parts)
    fit_eval_kernel<G, PROTECT, true, false><<<(unsigned)grid, kFitWarpsPerBlock * 32, smem, st>>>(
        W, R, U, ldw, s, clip, K, partial, clip_idx_out, group_err_out, rows_blocks, chunk, stride, scale, thresh,
        __builtin_nanf(""), next_item, fit_work_counters(ctx), FitJobs());
  else
    fit_eval_kernel<G, PROTECT, false, false><<<(unsigned)grid, kFitWarpsPerBlock * 32, smem, st>>>(
        W, R, U, ldw, s, clip, K, partial, clip_idx_out, group_err_out, rows_blocks, chunk, stride, scale, thresh,
        __builtin_nanf(""), next_item, fit_work_counters(ctx), FitJobs());
  WINDQ_CUDA(ctx, cudaGetLastError());
  fit_finalize_kernel<<<(unsigned)U, 256, 0, st>>>(partial, rows_blocks, err_out, energy_out);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

// FEAT: jobs.hist (zeroed here) and unit_wsum receive what the features need (see the kernel).
template <int G, bool FEAT>
windq_status launch_fit_batch(windq_ctx* ctx, const FitJobs& jobs, const float* clip, int K, double* unit_wsum, cudaStream_t st) {
  constexpr int GPW = Map<G>::GPW;
  const int chunk = fit_cand_chunk(G), stride = fit_cand_stride(chunk);
  const size_t smem = (size_t)kFitWarpsPerBlock * GPW * stride * sizeof(Cand);
  const int id = (FEAT ? kFitFeatG32 : kFitBatchG32) + g_index(G);
  if (windq_status rc = prepare_kernel(ctx, id, fit_eval_kernel<G, false, false, true, FEAT>, kFitWarpsPerBlock * 32, smem, true)) return rc;
  const int64_t full_grid = (int64_t)ctx->sm_count * ctx->occupancy[id];
  const int64_t n_items = jobs.first_item[jobs.n];
  const bool in_parts = 2 * n_items < 3 * full_grid * kFitWarpsPerBlock;
  if (in_parts)
    if (windq_status rc = prepare_kernel(ctx, id + 5, fit_eval_kernel<G, false, true, true, FEAT>, kFitWarpsPerBlock * 32, smem, false))
      return rc;
  int64_t grid = full_grid;
  const int64_t need = ((in_parts ? 5 : 1) * n_items + kFitWarpsPerBlock - 1) / kFitWarpsPerBlock;
  if (grid > need) grid = need;
  unsigned int* next_item = (unsigned int*)ctx->scratch;
  double* partial = (double*)((char*)ctx->scratch + 16);
  WINDQ_CUDA(ctx, cudaMemsetAsync(next_item, 0, sizeof(unsigned int), st));
  if (FEAT) WINDQ_CUDA(ctx, cudaMemsetAsync(jobs.hist, 0, (size_t)jobs.first_unit[jobs.n] * 32768u * sizeof(unsigned int), st));
  if (in_parts)
    fit_eval_kernel<G, false, true, true, FEAT><<<(unsigned)grid, kFitWarpsPerBlock * 32, smem, st>>>(
        nullptr, 0, 0, 0, nullptr, clip, K, partial, nullptr, nullptr, 0, chunk, stride, nullptr, nullptr, __builtin_nanf(""),
        next_item, fit_work_counters(ctx), jobs);
  else
    fit_eval_kernel<G, false, false, true, FEAT><<<(unsigned)grid, kFitWarpsPerBlock * 32, smem, st>>>(
        nullptr, 0, 0, 0, nullptr, clip, K, partial, nullptr, nullptr, 0, chunk, stride, nullptr, nullptr, __builtin_nanf(""),
        next_item, fit_work_counters(ctx), jobs);
  WINDQ_CUDA(ctx, cudaGetLastError());
  fit_finalize_batch_kernel<<<jobs.first_unit[jobs.n], 256, 0, st>>>(partial, GPW, jobs, FEAT ? unit_wsum : nullptr);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

}  // namespace windq

extern "C" {

int64_t windq_scratch_bytes_fit_eval(int64_t R, int64_t C, int G) {
  if (!windq::valid_G(G) || R <= 0 || C <= 0) return 0;
  const int gpw = 32 / (G / 32);
  // the item counter (16 bytes, so that the doubles stay aligned), then eight doubles per item
  return 16 + (C / G) * ((R + gpw - 1) / gpw) * windq::kFitPartials * (int64_t)sizeof(double);
}

static windq_status fit_eval_any(windq_ctx* ctx, const char* who, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                 const float* s, const float* clip_grid, int K, const float* thresh, float* err_out,
                                 float* energy_out, uint8_t* clip_idx_out, float* group_err_out, void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "%s: ctx is NULL", who);
  if (windq_status st = check_matrix(ctx, who, W, R, C, ldw, G)) return st;
  if (windq_status st = check_K(ctx, who, K)) return st;
  WINDQ_REQUIRE(ctx, s && clip_grid && err_out, WINDQ_ERR_NULL, "%s: s, clip_grid or err_out is NULL", who);
  WINDQ_REQUIRE(ctx, aligned16(s), WINDQ_ERR_ALIGN, "%s: s is not 16-byte aligned", who);
  DeviceGuard guard(ctx->device);
  const int64_t part_bytes = windq_scratch_bytes_fit_eval(R, C, G);
  if (windq_status st = ensure_scratch(ctx, thresh ? windq_scratch_bytes_fit_eval_protected(R, C, G) : part_bytes)) return st;
  const int U = (int)(C / G);
  cudaStream_t st = (cudaStream_t)stream;
  const __half* Wh = (const __half*)W;
  unsigned int* next_item = (unsigned int*)ctx->scratch;
  double* partial = (double*)((char*)ctx->scratch + 16);
  float* scale = (float*)((char*)ctx->scratch + round_up(part_bytes, 16));
#define WINDQ_FIT_CASE(GG)                                                                                              \
  case GG:                                                                                                              \
    return thresh ? launch_fit<GG, true>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, partial, err_out, energy_out,         \
                                         clip_idx_out, group_err_out, scale, thresh, next_item, st)                                \
                  : launch_fit<GG, false>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, partial, err_out, energy_out,        \
                                          clip_idx_out, group_err_out, nullptr, nullptr, next_item, st);
  switch (G) {
    WINDQ_FIT_CASE(32)
    WINDQ_FIT_CASE(64)
    WINDQ_FIT_CASE(128)
    WINDQ_FIT_CASE(256)
    default:
      WINDQ_FIT_CASE(512)
  }
#undef WINDQ_FIT_CASE
}

int64_t windq_scratch_bytes_fit_eval_protected(int64_t R, int64_t C, int G) {
  const int64_t base = windq_scratch_bytes_fit_eval(R, C, G);
  return base ? windq::round_up(base, 16) + C * (int64_t)sizeof(float) : 0;
}

windq_status windq_fit_eval(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                            const float* clip_grid, int K, float* err_out, float* energy_out, uint8_t* clip_idx_out,
                            float* group_err_out, void* stream) {
  return fit_eval_any(ctx, "windq_fit_eval", W, R, C, ldw, G, s, clip_grid, K, nullptr, err_out, energy_out, clip_idx_out,
                      group_err_out, stream);
}

windq_status windq_fit_eval_protected(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                      const float* s, const float* clip_grid, int K, const float* thresh, float* err_out,
                                      float* energy_out, uint8_t* clip_idx_out, float* group_err_out, void* stream) {
  if (ctx && !thresh) return windq::fail(ctx, WINDQ_ERR_NULL, "windq_fit_eval_protected: thresh is NULL");
  return fit_eval_any(ctx, "windq_fit_eval_protected", W, R, C, ldw, G, s, clip_grid, K, thresh, err_out, energy_out,
                      clip_idx_out, group_err_out, stream);
}

int64_t windq_scratch_bytes_fit_eval_batch(const windq_fit_job* jobs, int n_jobs, int G) {
  if (!jobs || n_jobs <= 0 || !windq::valid_G(G)) return 0;
  const int gpw = 32 / (G / 32);
  int64_t items = 0;
  for (int j = 0; j < n_jobs; ++j) {
    if (jobs[j].R <= 0 || jobs[j].C <= 0) return 0;
    items += (jobs[j].C / G) * ((jobs[j].R + gpw - 1) / gpw);
  }
  return 16 + items * windq::kFitPartials * (int64_t)sizeof(double);
}

static windq_status fit_batch_any(windq_ctx* ctx, const char* who, const windq_fit_job* jobs, float* const* feat_out, int n_jobs,
                                  int G, const float* clip_grid, int K, void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "%s: ctx is NULL", who);
  WINDQ_REQUIRE(ctx, jobs && clip_grid, WINDQ_ERR_NULL, "%s: jobs or clip_grid is NULL", who);
  WINDQ_REQUIRE(ctx, n_jobs >= 1 && n_jobs <= kFitMaxJobs, WINDQ_ERR_SHAPE, "%s: n_jobs = %d is outside [1, %d]", who, n_jobs,
                kFitMaxJobs);
  if (windq_status st = check_K(ctx, who, K)) return st;
  FitJobs fj;
  memset(&fj, 0, sizeof(fj));
  fj.n = n_jobs;
  int64_t items = 0, units = 0;
  for (int j = 0; j < n_jobs; ++j) {
    const windq_fit_job& b = jobs[j];
    if (windq_status st = check_matrix(ctx, who, b.W, b.R, b.C, b.ldw, G)) return st;
    WINDQ_REQUIRE(ctx, b.s && b.err_out, WINDQ_ERR_NULL, "%s: job %d: s or err_out is NULL", who, j);
    WINDQ_REQUIRE(ctx, aligned16(b.s), WINDQ_ERR_ALIGN, "%s: job %d: s is not 16-byte aligned", who, j);
    const int gpw = 32 / (G / 32);
    fj.W[j] = (const __half*)b.W;
    fj.s[j] = b.s;
    fj.clip_idx[j] = b.clip_idx_out;
    fj.group_err[j] = b.group_err_out;
    fj.err[j] = b.err_out;
    fj.energy[j] = b.energy_out;
    fj.lowbit[j] = (__half*)b.lowbit_out;
    WINDQ_REQUIRE(ctx, ((uintptr_t)b.lowbit_out & 1) == 0, WINDQ_ERR_ALIGN, "%s: job %d: lowbit_out is misaligned", who, j);
    fj.ldw[j] = b.ldw;
    fj.R[j] = (int)b.R;
    fj.U[j] = (int)(b.C / G);
    fj.first_item[j] = (unsigned int)items;
    fj.first_unit[j] = (unsigned int)units;
    items += (b.C / G) * ((b.R + gpw - 1) / gpw);
    units += b.C / G;
    WINDQ_REQUIRE(ctx, items < (1ll << 28), WINDQ_ERR_SHAPE, "%s: the batch is too large for one call", who);
  }
  fj.first_item[n_jobs] = (unsigned int)items;
  fj.first_unit[n_jobs] = (unsigned int)units;
  DeviceGuard guard(ctx->device);
  const int64_t part_bytes = round_up(16 + items * kFitPartials * (int64_t)sizeof(double), 16);
  cudaStream_t st = (cudaStream_t)stream;
  if (!feat_out) {
    if (windq_status rc = ensure_scratch(ctx, part_bytes)) return rc;
    switch (G) {
      case 32: return launch_fit_batch<32, false>(ctx, fj, clip_grid, K, nullptr, st);
      case 64: return launch_fit_batch<64, false>(ctx, fj, clip_grid, K, nullptr, st);
      case 128: return launch_fit_batch<128, false>(ctx, fj, clip_grid, K, nullptr, st);
      case 256: return launch_fit_batch<256, false>(ctx, fj, clip_grid, K, nullptr, st);
      default: return launch_fit_batch<512, false>(ctx, fj, clip_grid, K, nullptr, st);
    }
  }
  // features too: scratch = counter and partials | one histogram per unit | one sum per unit
  for (int j = 0; j < n_jobs; ++j) {
    WINDQ_REQUIRE(ctx, feat_out[j], WINDQ_ERR_NULL, "%s: job %d: feat_out is NULL", who, j);
    WINDQ_REQUIRE(ctx, jobs[j].R * (int64_t)G < (1ll << 32), WINDQ_ERR_SHAPE, "%s: job %d: R * G must be below 2^32", who, j);
  }
  const int64_t hist_bytes = units * 32768 * (int64_t)sizeof(unsigned int);
  if (windq_status rc = ensure_scratch(ctx, part_bytes + hist_bytes + units * (int64_t)sizeof(double))) return rc;
  fj.hist = (unsigned int*)((char*)ctx->scratch + part_bytes);
  double* unit_wsum = (double*)((char*)ctx->scratch + part_bytes + hist_bytes);
  windq_status rc;
  switch (G) {
    case 32: rc = launch_fit_batch<32, true>(ctx, fj, clip_grid, K, unit_wsum, st); break;
    case 64: rc = launch_fit_batch<64, true>(ctx, fj, clip_grid, K, unit_wsum, st); break;
    case 128: rc = launch_fit_batch<128, true>(ctx, fj, clip_grid, K, unit_wsum, st); break;
    case 256: rc = launch_fit_batch<256, true>(ctx, fj, clip_grid, K, unit_wsum, st); break;
    default: rc = launch_fit_batch<512, true>(ctx, fj, clip_grid, K, unit_wsum, st); break;
  }
  if (rc != WINDQ_OK) return rc;
  int Rs[kFitMaxJobs], first_unit[kFitMaxJobs + 1];
  const float* ss[kFitMaxJobs];
  for (int j = 0; j < n_jobs; ++j) {
    Rs[j] = fj.R[j];
    first_unit[j] = (int)fj.first_unit[j];
    ss[j] = fj.s[j];
  }
  first_unit[n_jobs] = (int)fj.first_unit[n_jobs];
  return features_from_histograms(ctx, fj.hist, unit_wsum, n_jobs, Rs, first_unit, ss, feat_out, G, st);
}

windq_status windq_fit_eval_batch(windq_ctx* ctx, const windq_fit_job* jobs, int n_jobs, int G, const float* clip_grid, int K,
                                  void* stream) {
  return fit_batch_any(ctx, "windq_fit_eval_batch", jobs, nullptr, n_jobs, G, clip_grid, K, stream);
}

int64_t windq_scratch_bytes_features_fit_batch(const windq_featfit_job* jobs, int n_jobs, int G) {
  if (!jobs || n_jobs <= 0 || n_jobs > windq::kFitMaxJobs || !windq::valid_G(G)) return 0;
  const int gpw = 32 / (G / 32);
  int64_t items = 0, units = 0;
  for (int j = 0; j < n_jobs; ++j) {
    if (jobs[j].R <= 0 || jobs[j].C <= 0) return 0;
    items += (jobs[j].C / G) * ((jobs[j].R + gpw - 1) / gpw);
    units += jobs[j].C / G;
  }
  return windq::round_up(16 + items * windq::kFitPartials * (int64_t)sizeof(double), 16) + units * 32768 * (int64_t)sizeof(unsigned int) +
         units * (int64_t)sizeof(double);
}

windq_status windq_features_fit_batch(windq_ctx* ctx, const windq_featfit_job* jobs, int n_jobs, int G, const float* clip_grid,
                                      int K, void* stream) {
  const char* who = "windq_features_fit_batch";
  if (!ctx) return windq::fail(nullptr, WINDQ_ERR_NULL, "%s: ctx is NULL", who);
  if (!jobs) return windq::fail(ctx, WINDQ_ERR_NULL, "%s: jobs is NULL", who);
  if (n_jobs < 1 || n_jobs > windq::kFitMaxJobs)
    return windq::fail(ctx, WINDQ_ERR_SHAPE, "%s: n_jobs = %d is outside [1, %d]", who, n_jobs, windq::kFitMaxJobs);
  windq_fit_job fit[windq::kFitMaxJobs];
  float* feat[windq::kFitMaxJobs];
  for (int j = 0; j < n_jobs; ++j) {
    fit[j].W = jobs[j].W;
    fit[j].R = jobs[j].R;
    fit[j].C = jobs[j].C;
    fit[j].ldw = jobs[j].ldw;
    fit[j].s = jobs[j].s;
    fit[j].err_out = jobs[j].err_out;
    fit[j].energy_out = jobs[j].energy_out;
    fit[j].clip_idx_out = jobs[j].clip_idx_out;
    fit[j].group_err_out = jobs[j].group_err_out;
    fit[j].lowbit_out = jobs[j].lowbit_out;
    feat[j] = jobs[j].feat_out;
    if (!feat[j]) return windq::fail(ctx, WINDQ_ERR_NULL, "%s: job %d: feat_out is NULL", who, j);
  }
  return fit_batch_any(ctx, who, fit, feat, n_jobs, G, clip_grid, K, stream);
}

}  // extern "C"

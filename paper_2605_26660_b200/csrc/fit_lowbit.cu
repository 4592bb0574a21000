// windq_fit_ternary_search: the 1.58-bit fit with its assignment searched (App. "Per-unit Scale Optimization"
// and Sec. 3.5 name fitted low-bit operators without formulas).  For a fixed scale the best ternary code of a
// weight is its sign above half the scale and 0 below, so the best support is a threshold set; the call tries the
// caller's threshold ratios one after the other, each fitted and scored exactly like the single threshold of
// windq_fit_eval, and keeps the first of the least error.
//
// Bound by the FP32 pipes like the other fits: per threshold ratio six packed binary32 operations and four
// comparisons per pair of weights (the support sums, then the error with the scale those sums give).  Same layout: LG = G / 32 lanes per group hold 32
// magnitudes and 32 statistics in registers, one warp per item of GPW rows of a unit, persistent grid, items
// claimed from a counter; sums in PSUM8 order, so thresholds, scales and group errors are reproducible bit for bit.
#include "fit_device.cuh"

namespace windq {

constexpr int kTernaryWarpsPerBlock = 16;

__global__ void ternary_scale_kernel(const float* __restrict__ s, int C, float* __restrict__ scale) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < C) scale[j] = __fsqrt_rn(s[j]);
}

// PROTECT: a weight whose key |w| * act_scale_j reaches thresh[u] is taken out of its group (zero weight, zero
// activation weight), as in the protected fit.
template <int G, bool PROTECT>
__global__ void __launch_bounds__(kTernaryWarpsPerBlock * 32, 1)
fit_ternary_search_kernel(const __half* __restrict__ W, int R, int U, int64_t ldw, const float* __restrict__ s,
                          const float* __restrict__ thr_grid, int Kt, double* __restrict__ partial,
                          uint8_t* __restrict__ thr_idx_out, __half* __restrict__ alpha_out, float* __restrict__ group_err_out,
                          int rows_blocks, unsigned int* __restrict__ next_item, const float* __restrict__ act_scale,
                          const float* __restrict__ thresh, float never) {
  constexpr int LG = Map<G>::LG, GPW = Map<G>::GPW;
  __shared__ float thr_s[64];
  if (threadIdx.x < 64) thr_s[threadIdx.x] = threadIdx.x < Kt ? __ldg(thr_grid + threadIdx.x) : 0.0f;
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const int g = lane / LG, q = lane % LG;
  const unsigned int n_items = (unsigned int)(U * rows_blocks);

  for (;;) {
    unsigned int item = 0;
    if (lane == 0) item = atomicAdd(next_item, 1u);
    item = __shfl_sync(0xffffffffu, item, 0);
    if (item >= n_items) break;
    const int u = (int)(item / rows_blocks), rb = (int)(item % rows_blocks);
    Lane32 sv, av;  // statistics and magnitudes |w|
    load_stats(s + (int64_t)u * G + 32 * q, sv);
    const int row = rb * GPW + g;
    const bool live = row < R;
    const int row_ld = live ? row : R - 1;  // rows past the end repeat the last row and are not written
    load_weights(W + (int64_t)row_ld * ldw + (int64_t)u * G + 32 * q, av);
    {
      // magnitudes, and the masking step of the protected fit (against a NaN when nothing is protected, so that
      // no comparison is true)
      Lane32 ks;
      if (PROTECT) load_stats(act_scale + (int64_t)u * G + 32 * q, ks);
      else ks = sv;
      const float tau = PROTECT ? __ldg(thresh + u) : never;
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          av.v[h][i].x = fabsf(av.v[h][i].x);
          av.v[h][i].y = fabsf(av.v[h][i].y);
          if (__fmul_rn(av.v[h][i].x, ks.v[h][i].x) >= tau) { av.v[h][i].x = 0.0f; sv.v[h][i].x = 0.0f; }
          if (__fmul_rn(av.v[h][i].y, ks.v[h][i].y) >= tau) { av.v[h][i].y = 0.0f; sv.v[h][i].y = 0.0f; }
        }
    }
    const float sumA = group_abs_sum<G>(av);
    const float meanA = __fmul_rn(sumA, 1.0f / (float)G);
    const bool some = sumA > 0.0f;

    float best_e = __int_as_float(0x7f800000), best_alpha = 0.0f;
    int best_k = 0;
#pragma unroll 1
    for (int k = 0; k < Kt; ++k) {
      const float delta = __fmul_rn(thr_s[k], meanA);
      // support sums, weighted by s.  The support enters as a factor m = 1 or 0 per weight: s (|w| m) and s m are
      // exact products of the terms the definition adds, so the sums round as they do there; leaves 2 h and
      // 2 h + 1 run side by side in the two halves of the packed operations.
      const float2 zero2 = make_float2(0.0f, 0.0f);
      float2 bt[2] = {zero2, zero2}, ct[2] = {zero2, zero2};
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float2 aw = av.v[h][i], sj = sv.v[h][i];
          const float2 m = make_float2(aw.x > delta ? 1.0f : 0.0f, aw.y > delta ? 1.0f : 0.0f);
          bt[h] = fma2(sj, mul2(aw, m), bt[h]);
          ct[h] = fma2(sj, m, ct[h]);
        }
      float sumBt = group_tree<G>(bt[0], bt[1]);
      float sumCt = group_tree<G>(ct[0], ct[1]);
      // a weighted sum of zero: no activation weight on the support, or no support at all; the unweighted sums
      // decide which, and give the scale in the first case
      bool nonempty = some;
      if (__any_sync(0xffffffffu, some && sumCt == 0.0f)) {
        float Bu[4], Cu[4];
#pragma unroll
        for (int l = 0; l < 4; ++l) {
          float bu = 0.0f, cu = 0.0f;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float aw = av.get(l, i);
            const bool in = aw > delta;
            bu = __fadd_rn(bu, in ? aw : 0.0f);
            cu = __fadd_rn(cu, in ? 1.0f : 0.0f);
          }
          Bu[l] = bu; Cu[l] = cu;
        }
        const float sumBu = group_tree<G>(Bu[0], Bu[1], Bu[2], Bu[3]);
        const float sumCu = group_tree<G>(Cu[0], Cu[1], Cu[2], Cu[3]);
        if (sumCt == 0.0f) {
          sumBt = sumBu;
          sumCt = sumCu;
          nonempty = some && sumCu > 0.0f;
        }
      }
      const float alpha = nonempty ? __half2float(__float2half_rn(__fdiv_rn(sumBt, sumCt))) : 0.0f;
      // error: the difference between the reconstruction and the weight has the magnitude |alpha - |w|| on the
      // support and |w| off it; its sign does not matter to (s d) d, and rounding is symmetric in sign
      // (m alpha is alpha or 0 exactly, so |w| - m alpha rounds once, like the difference itself)
      const float2 nalpha2 = make_float2(-alpha, -alpha);
      float2 et[2] = {zero2, zero2};
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float2 aw = av.v[h][i];
          const float2 m = make_float2(aw.x > delta ? 1.0f : 0.0f, aw.y > delta ? 1.0f : 0.0f);
          const float2 d = fma2(m, nalpha2, aw);
          et[h] = fma2(mul2(sv.v[h][i], d), d, et[h]);
        }
      const float e = group_tree<G>(et[0], et[1]);
      if (e < best_e) {
        best_e = e;
        best_k = k;
        best_alpha = alpha;
      }
    }
    if (live && q == 0) {
      const int64_t o = (int64_t)u * R + row;
      thr_idx_out[o] = (uint8_t)best_k;
      alpha_out[o] = __float2half_rn(best_alpha);
      if (group_err_out) group_err_out[o] = best_e;
    }
    // add over the rows of this item in double; lanes of a group hold equal values
    double d = live ? (double)best_e : 0.0;
#pragma unroll
    for (int m = LG; m < 32; m <<= 1) d += __shfl_xor_sync(0xffffffffu, d, m);
    if (lane == 0) partial[item] = d;
  }
}

// err_out[u] = sum over the unit's row blocks, fixed order.
__global__ void __launch_bounds__(256)
ternary_finalize_kernel(const double* __restrict__ partial, int rows_blocks, float* __restrict__ err_out) {
  __shared__ double red[256];
  const int u = blockIdx.x, t = threadIdx.x;
  const double* p = partial + (int64_t)u * rows_blocks;
  double acc = 0.0;
  for (int rb = t; rb < rows_blocks; rb += 256) acc += p[rb];
  red[t] = acc;
  __syncthreads();
  for (int n = 128; n > 0; n >>= 1) {
    if (t < n) red[t] += red[t + n];
    __syncthreads();
  }
  if (t == 0) err_out[u] = (float)red[0];
}

template <int G>
windq_status launch_ternary_search(windq_ctx* ctx, const __half* W, int R, int U, int64_t ldw, const float* s,
                                   const float* thr_grid, int Kt, const float* thresh, float* err_out, uint8_t* thr_idx_out,
                                   __half* alpha_out, float* group_err_out, cudaStream_t st) {
  constexpr int GPW = Map<G>::GPW;
  const int rows_blocks = (R + GPW - 1) / GPW;
  const int64_t n_items = (int64_t)U * rows_blocks;
  WINDQ_REQUIRE(ctx, n_items < (1ll << 31), WINDQ_ERR_SHAPE, "windq_fit_ternary_search: R * C is too large for one call");
  unsigned int* next_item = (unsigned int*)ctx->scratch;
  double* partial = (double*)((char*)ctx->scratch + 16);
  int64_t grid = ctx->sm_count;
  const int64_t need = (n_items + kTernaryWarpsPerBlock - 1) / kTernaryWarpsPerBlock;
  if (grid > need) grid = need;
  WINDQ_CUDA(ctx, cudaMemsetAsync(next_item, 0, sizeof(unsigned int), st));
  if (thresh) {
    float* act_scale = (float*)((char*)ctx->scratch + round_up(16 + n_items * (int64_t)sizeof(double), 16));
    ternary_scale_kernel<<<(unsigned)((U * G + 255) / 256), 256, 0, st>>>(s, U * G, act_scale);
    fit_ternary_search_kernel<G, true><<<(unsigned)grid, kTernaryWarpsPerBlock * 32, 0, st>>>(
        W, R, U, ldw, s, thr_grid, Kt, partial, thr_idx_out, alpha_out, group_err_out, rows_blocks, next_item, act_scale, thresh,
        __builtin_nanf(""));
  } else {
    fit_ternary_search_kernel<G, false><<<(unsigned)grid, kTernaryWarpsPerBlock * 32, 0, st>>>(
        W, R, U, ldw, s, thr_grid, Kt, partial, thr_idx_out, alpha_out, group_err_out, rows_blocks, next_item, nullptr, nullptr,
        __builtin_nanf(""));
  }
  WINDQ_CUDA(ctx, cudaGetLastError());
  ternary_finalize_kernel<<<(unsigned)U, 256, 0, st>>>(partial, rows_blocks, err_out);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

}  // namespace windq

extern "C" {

int64_t windq_scratch_bytes_fit_ternary_search(int64_t R, int64_t C, int G) {
  if (!windq::valid_G(G) || R <= 0 || C <= 0) return 0;
  const int gpw = 32 / (G / 32);
  // the item counter, one double per item, and (with protection) C activation scales
  return windq::round_up(16 + (C / G) * ((R + gpw - 1) / gpw) * (int64_t)sizeof(double), 16) + C * (int64_t)sizeof(float);
}

windq_status windq_fit_ternary_search(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                                      const float* thr_grid, int thr_K, const float* thresh, float* err_out,
                                      uint8_t* thr_idx_out, void* alpha_out, float* group_err_out, void* stream) {
  using namespace windq;
  const char* who = "windq_fit_ternary_search";
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "%s: ctx is NULL", who);
  if (windq_status st = check_matrix(ctx, who, W, R, C, ldw, G)) return st;
  WINDQ_REQUIRE(ctx, s && thr_grid && err_out && thr_idx_out && alpha_out, WINDQ_ERR_NULL,
                "%s: s, thr_grid, err_out, thr_idx_out or alpha_out is NULL", who);
  WINDQ_REQUIRE(ctx, thr_K >= 1 && thr_K <= 64, WINDQ_ERR_ARG, "%s: thr_K = %d is outside [1, 64]", who, thr_K);
  WINDQ_REQUIRE(ctx, aligned16(s), WINDQ_ERR_ALIGN, "%s: s is not 16-byte aligned", who);
  WINDQ_REQUIRE(ctx, ((uintptr_t)alpha_out & 1) == 0, WINDQ_ERR_ALIGN, "%s: alpha_out is misaligned", who);
  DeviceGuard guard(ctx->device);
  if (windq_status st = ensure_scratch(ctx, windq_scratch_bytes_fit_ternary_search(R, C, G))) return st;
  const int U = (int)(C / G);
  cudaStream_t st = (cudaStream_t)stream;
  const __half* Wh = (const __half*)W;
  __half* ao = (__half*)alpha_out;
  switch (G) {
    case 32: return launch_ternary_search<32>(ctx, Wh, (int)R, U, ldw, s, thr_grid, thr_K, thresh, err_out, thr_idx_out, ao, group_err_out, st);
    case 64: return launch_ternary_search<64>(ctx, Wh, (int)R, U, ldw, s, thr_grid, thr_K, thresh, err_out, thr_idx_out, ao, group_err_out, st);
    case 128: return launch_ternary_search<128>(ctx, Wh, (int)R, U, ldw, s, thr_grid, thr_K, thresh, err_out, thr_idx_out, ao, group_err_out, st);
    case 256: return launch_ternary_search<256>(ctx, Wh, (int)R, U, ldw, s, thr_grid, thr_K, thresh, err_out, thr_idx_out, ao, group_err_out, st);
    default: return launch_ternary_search<512>(ctx, Wh, (int)R, U, ldw, s, thr_grid, thr_K, thresh, err_out, thr_idx_out, ao, group_err_out, st);
  }
}

}  // extern "C"

// windq_fit_refine: iterative refinement of every group's step size for the four uniform bit-widths
// (App. "Per-unit Scale Optimization": a few Adam steps on the reconstruction loss of the chunk, the
// step size learned with straight-through estimation of the rounding), warm-started from the clip-grid
// fit of windq_fit_eval.
//
// Bound by the FP32 pipes like windq_fit_eval: (T + 1) evaluations x 4 bit-widths x about 11 binary32
// operations per weight (loss and gradient share the code, the difference and s * d).  Same layout:
// LG = G / 32 lanes per group hold 32 weights and 32 statistics each in registers, one warp per item of
// GPW rows of a unit, persistent grid, items claimed from a counter.  Every lane of a group carries the
// group's Adam state; the arithmetic is a fixed sequence of binary32 operations, so scales and group
// errors are reproducible bit for bit.
#include "fit_device.cuh"

namespace windq {

constexpr int kRefineWarpsPerBlock = 16;
constexpr int kRefineMaxSteps = 32;

struct AdamTable {
  float c1[kRefineMaxSteps];  // 1 / (1 - 0.9^t),   t = 1..T
  float c2[kRefineMaxSteps];  // 1 / (1 - 0.999^t)
};

// Loss and (negated) gradient leaf sums of one step size over this lane's 32 elements.  The difference
// is taken as d' = w - c * scale = -d, so that the loss uses the operations of the clip search and the
// gradient sums come out exactly negated (rounding is symmetric in sign).
__device__ __forceinline__ void refine_leaf_sums(const Lane32& w, const Lane32& s, float scale, float inv, float lo,
                                                 float hi, float2& e01, float2& e23, float2& g01, float2& g23) {
  const float2 inv2 = make_float2(inv, inv);
  const float2 ns2 = make_float2(-scale, -scale);
  const float2 magic2 = make_float2(kMagic, kMagic);
  const float2 nmagic2 = make_float2(-kMagic, -kMagic);
  float2 acc[2] = {make_float2(0.0f, 0.0f), make_float2(0.0f, 0.0f)};
  float2 gacc[2] = {make_float2(0.0f, 0.0f), make_float2(0.0f, 0.0f)};
#pragma unroll
  for (int h = 0; h < 2; ++h) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float2 wv = w.v[h][i];
      const float2 r = add2(fma2(wv, inv2, magic2), nmagic2);
      float2 c;
      c.x = fminf(fmaxf(r.x, lo), hi);
      c.y = fminf(fmaxf(r.y, lo), hi);
      const float2 x = mul2(wv, inv2);
      float2 psi;
      psi.x = (c.x == r.x) ? __fsub_rn(r.x, x.x) : c.x;
      psi.y = (c.y == r.y) ? __fsub_rn(r.y, x.y) : c.y;
      const float2 d = fma2(c, ns2, wv);
      const float2 t = mul2(s.v[h][i], d);
      acc[h] = fma2(t, d, acc[h]);
      gacc[h] = fma2(t, psi, gacc[h]);
    }
  }
  e01 = acc[0];
  e23 = acc[1];
  g01 = gacc[0];
  g23 = gacc[1];
}

// sqrt(s_j): the activation scale that the saliency key uses.
__global__ void refine_scale_kernel(const float* __restrict__ s, int C, float* __restrict__ scale) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < C) scale[j] = __fsqrt_rn(s[j]);
}

// PROTECT: a weight whose key |w| * act_scale_j reaches thresh[u] is taken out of its group (zero weight,
// zero activation weight), exactly as in the protected fit whose clip indices this kernel starts from.
template <int G, bool PROTECT>
__global__ void __launch_bounds__(kRefineWarpsPerBlock * 32, 1)
fit_refine_kernel(const __half* __restrict__ W, int R, int U, int64_t ldw, const float* __restrict__ s,
                  const float* __restrict__ clip, int K, const uint8_t* __restrict__ clip_idx, int T, float lr,
                  AdamTable adam, double* __restrict__ partial, __half* __restrict__ scale_out,
                  float* __restrict__ group_err_out, int rows_blocks, unsigned int* __restrict__ next_item,
                  const float* __restrict__ act_scale, const float* __restrict__ thresh, float never) {
  constexpr int LG = Map<G>::LG, GPW = Map<G>::GPW;
  const int lane = threadIdx.x & 31;
  const int g = lane / LG, q = lane % LG;
  const unsigned int n_items = (unsigned int)(U * rows_blocks);

  for (;;) {
    unsigned int item = 0;
    if (lane == 0) item = atomicAdd(next_item, 1u);
    item = __shfl_sync(0xffffffffu, item, 0);
    if (item >= n_items) break;
    const int u = (int)(item / rows_blocks), rb = (int)(item % rows_blocks);
    Lane32 sv, wv;
    load_stats(s + (int64_t)u * G + 32 * q, sv);
    const int row = rb * GPW + g;
    const bool live = row < R;
    const int row_ld = live ? row : R - 1;  // rows past the end repeat the last row and are not written
    load_weights(W + (int64_t)row_ld * ldw + (int64_t)u * G + 32 * q, wv);
    {
      // Masking step.  Without PROTECT it runs against `never`, a NaN from the host, so that no comparison is
      // true and nothing changes; as in fit_eval_kernel, ptxas schedules the loops below better with every w
      // and s having gone through a select (measured: 5 % less time, same results bit for bit).
      Lane32 av;
      if (PROTECT) load_stats(act_scale + (int64_t)u * G + 32 * q, av);
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

    float best[4];
#pragma unroll 1
    for (int bi = 0; bi < 4; ++bi) {
      const int64_t o = ((int64_t)bi * U + u) * R + row_ld;
      int k = __ldg(clip_idx + o);
      k = k < K ? k : K - 1;
      const UniformSpec us = uniform_spec(bi);
      float scale0, zf;
      uniform_scale_zero(mn, rng, __ldg(clip + k), us, scale0, zf);
      const float lo = __fsub_rn(0.0f, zf), hi = __fsub_rn(us.qmax, zf);
      const float step = __fmul_rn(lr, scale0);
      float delta = scale0, m = 0.0f, v = 0.0f;
      float best_e = __int_as_float(0x7f800000), best_scale = scale0;
      bool active = true;
#pragma unroll 1
      for (int t = 0; t <= T; ++t) {
        float sh = __half2float(__float2half_rn(delta));
        active = active && sh > 0.0f && sh < __int_as_float(0x7f800000);
        if (!active) sh = 1.0f;  // a finished group idles on a harmless value
        float2 e01, e23, g01, g23;
        refine_leaf_sums(wv, sv, sh, __frcp_rn(sh), lo, hi, e01, e23, g01, g23);
        const float loss = group_tree<G>(e01, e23);
        const float grad = -group_tree<G>(g01, g23);
        if (active && loss < best_e) {
          best_e = loss;
          best_scale = sh;
        }
        if (t < T && active) {
          m = __fmaf_rn(0.9f, m, __fmul_rn(0.1f, grad));
          v = __fmaf_rn(0.999f, v, __fmul_rn(0.001f, __fmul_rn(grad, grad)));
          const float mhat = __fmul_rn(m, adam.c1[t]), vhat = __fmul_rn(v, adam.c2[t]);
          const float upd = __fdiv_rn(mhat, __fadd_rn(__fsqrt_rn(vhat), 1e-8f));
          delta = __fmaf_rn(-step, upd, delta);
        }
      }
      best[bi] = best_e;
      if (live && q == 0) {
        const int64_t oo = ((int64_t)bi * U + u) * R + row;
        scale_out[oo] = __float2half_rn(best_scale);
        if (group_err_out) group_err_out[oo] = best_e;
      }
    }

    // add over the rows of this item in double; lanes of a group hold equal values
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      double d = live ? (double)best[c] : 0.0;
#pragma unroll
      for (int mm = LG; mm < 32; mm <<= 1) d += __shfl_xor_sync(0xffffffffu, d, mm);
      if (lane == 0) partial[(int64_t)item * 4 + c] = d;
    }
  }
}

// err_out[u][0..3] = sum over the unit's row blocks, fixed order.
__global__ void __launch_bounds__(256)
refine_finalize_kernel(const double* __restrict__ partial, int rows_blocks, float* __restrict__ err_out) {
  __shared__ double red[256];
  const int u = blockIdx.x, t = threadIdx.x;
  const double* p = partial + (int64_t)u * rows_blocks * 4;
  for (int c = 0; c < 4; ++c) {
    double acc = 0.0;
    for (int rb = t; rb < rows_blocks; rb += 256) acc += p[(int64_t)rb * 4 + c];
    red[t] = acc;
    __syncthreads();
    for (int n = 128; n > 0; n >>= 1) {
      if (t < n) red[t] += red[t + n];
      __syncthreads();
    }
    if (t == 0) err_out[(int64_t)u * 4 + c] = (float)red[0];
    __syncthreads();
  }
}

template <int G>
windq_status launch_refine(windq_ctx* ctx, const __half* W, int R, int U, int64_t ldw, const float* s, const float* clip,
                           int K, const uint8_t* clip_idx, int T, float lr, const AdamTable& adam, float* err_out,
                           __half* scale_out, float* group_err_out, const float* thresh, cudaStream_t st) {
  constexpr int GPW = Map<G>::GPW;
  const int rows_blocks = (R + GPW - 1) / GPW;
  const int64_t n_items = (int64_t)U * rows_blocks;
  WINDQ_REQUIRE(ctx, n_items < (1ll << 31), WINDQ_ERR_SHAPE, "windq_fit_refine: R * C is too large for one call");
  unsigned int* next_item = (unsigned int*)ctx->scratch;
  double* partial = (double*)((char*)ctx->scratch + 16);
  int64_t grid = ctx->sm_count;
  const int64_t need = (n_items + kRefineWarpsPerBlock - 1) / kRefineWarpsPerBlock;
  if (grid > need) grid = need;
  WINDQ_CUDA(ctx, cudaMemsetAsync(next_item, 0, sizeof(unsigned int), st));
  if (thresh) {
    float* act_scale = (float*)((char*)ctx->scratch + round_up(16 + n_items * 4 * (int64_t)sizeof(double), 16));
    refine_scale_kernel<<<(unsigned)((U * G + 255) / 256), 256, 0, st>>>(s, U * G, act_scale);
    fit_refine_kernel<G, true><<<(unsigned)grid, kRefineWarpsPerBlock * 32, 0, st>>>(
        W, R, U, ldw, s, clip, K, clip_idx, T, lr, adam, partial, scale_out, group_err_out, rows_blocks, next_item, act_scale,
        thresh, __builtin_nanf(""));
  } else {
    fit_refine_kernel<G, false><<<(unsigned)grid, kRefineWarpsPerBlock * 32, 0, st>>>(
        W, R, U, ldw, s, clip, K, clip_idx, T, lr, adam, partial, scale_out, group_err_out, rows_blocks, next_item, nullptr,
        nullptr, __builtin_nanf(""));
  }
  WINDQ_CUDA(ctx, cudaGetLastError());
  refine_finalize_kernel<<<(unsigned)U, 256, 0, st>>>(partial, rows_blocks, err_out);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

}  // namespace windq

extern "C" {

int64_t windq_scratch_bytes_fit_refine(int64_t R, int64_t C, int G) {
  if (!windq::valid_G(G) || R <= 0 || C <= 0) return 0;
  const int gpw = 32 / (G / 32);
  // the item counter, four doubles per item, and (protected variant) C activation scales
  return windq::round_up(16 + (C / G) * ((R + gpw - 1) / gpw) * 4 * (int64_t)sizeof(double), 16) + C * (int64_t)sizeof(float);
}

static windq_status fit_refine_any(windq_ctx* ctx, const char* who, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                   const float* s, const float* clip_grid, int K, const uint8_t* clip_idx,
                                   const float* thresh, int n_steps, float lr, float* err_out, void* scale_out,
                                   float* group_err_out, void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "%s: ctx is NULL", who);
  if (windq_status st = check_matrix(ctx, who, W, R, C, ldw, G)) return st;
  if (windq_status st = check_K(ctx, who, K)) return st;
  WINDQ_REQUIRE(ctx, s && clip_grid && clip_idx && err_out && scale_out, WINDQ_ERR_NULL,
                "%s: s, clip_grid, clip_idx, err_out or scale_out is NULL", who);
  WINDQ_REQUIRE(ctx, aligned16(s), WINDQ_ERR_ALIGN, "%s: s is not 16-byte aligned", who);
  WINDQ_REQUIRE(ctx, n_steps >= 0 && n_steps <= kRefineMaxSteps, WINDQ_ERR_SHAPE, "%s: n_steps = %d is outside [0, %d]", who,
                n_steps, kRefineMaxSteps);
  WINDQ_REQUIRE(ctx, lr >= 0.0f && lr <= 1.0f, WINDQ_ERR_SHAPE, "%s: lr = %g is outside [0, 1]", who, (double)lr);
  DeviceGuard guard(ctx->device);
  if (windq_status st = ensure_scratch(ctx, windq_scratch_bytes_fit_refine(R, C, G))) return st;
  AdamTable adam;
  double p1 = 1.0, p2 = 1.0;
  for (int t = 0; t < kRefineMaxSteps; ++t) {
    p1 *= 0.9;
    p2 *= 0.999;
    adam.c1[t] = (float)(1.0 / (1.0 - p1));
    adam.c2[t] = (float)(1.0 / (1.0 - p2));
  }
  const int U = (int)(C / G);
  cudaStream_t st = (cudaStream_t)stream;
  const __half* Wh = (const __half*)W;
  __half* so = (__half*)scale_out;
  switch (G) {
    case 32: return launch_refine<32>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, clip_idx, n_steps, lr, adam, err_out, so, group_err_out, thresh, st);
    case 64: return launch_refine<64>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, clip_idx, n_steps, lr, adam, err_out, so, group_err_out, thresh, st);
    case 128: return launch_refine<128>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, clip_idx, n_steps, lr, adam, err_out, so, group_err_out, thresh, st);
    case 256: return launch_refine<256>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, clip_idx, n_steps, lr, adam, err_out, so, group_err_out, thresh, st);
    default: return launch_refine<512>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, clip_idx, n_steps, lr, adam, err_out, so, group_err_out, thresh, st);
  }
}

windq_status windq_fit_refine(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                              const float* clip_grid, int K, const uint8_t* clip_idx, int n_steps, float lr,
                              float* err_out, void* scale_out, float* group_err_out, void* stream) {
  return fit_refine_any(ctx, "windq_fit_refine", W, R, C, ldw, G, s, clip_grid, K, clip_idx, nullptr, n_steps, lr, err_out,
                        scale_out, group_err_out, stream);
}

windq_status windq_fit_refine_protected(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                        const float* s, const float* clip_grid, int K, const uint8_t* clip_idx,
                                        const float* thresh, int n_steps, float lr, float* err_out, void* scale_out,
                                        float* group_err_out, void* stream) {
  if (ctx && !thresh) return windq::fail(ctx, WINDQ_ERR_NULL, "windq_fit_refine_protected: thresh is NULL");
  return fit_refine_any(ctx, "windq_fit_refine_protected", W, R, C, ldw, G, s, clip_grid, K, clip_idx, thresh, n_steps, lr,
                        err_out, scale_out, group_err_out, stream);
}

}  // extern "C"

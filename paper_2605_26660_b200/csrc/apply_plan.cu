// windq_apply_plan: codes, packed bytes, fp16 scale / zero point and fake-quantised weights of a
// chosen plan.
//
// With clip indices supplied this is a streaming kernel bound by HBM: 2 bytes read per weight,
// 2 bytes written for the fake-quantised copy and bits/8 for the codes.  Thread mapping as in
// the fit (LG lanes per group, 32 values per lane in registers).  A block handles one tile =
// (unit, 64 or 128 consecutive rows); the action is uniform over the tile, so there is no
// divergence.  Each lane packs its own 32 codes into whole 32-bit words in registers (1, 2, 3, 4
// and 8 bit all give whole bytes per lane); the words are staged in shared memory so that the
// tile's packed bytes, which are contiguous in the output, leave with 128-bit stores.  Only the
// base-3 ternary packing crosses lanes (5 trits per byte): its trits are staged as bytes and the
// output bytes are assembled from shared memory.
#include "fit_device.cuh"

namespace windq {

constexpr int kApplyWarps = 4;

template <int G>
struct ApplyTile {
  static constexpr int GPW = Map<G>::GPW;
  static constexpr int ROWS = (kApplyWarps * GPW >= 64) ? kApplyWarps * GPW : 64;  // multiple of 16
  static constexpr int PASSES = ROWS / (kApplyWarps * GPW);
  static constexpr int STAGE_BYTES = ROWS * G;
};

// 32 small codes -> packed little-endian words; returns the number of words.
template <int BITS>
__device__ __forceinline__ void pack_words(const unsigned (&q)[32], unsigned (&out)[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) out[i] = 0u;
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const int pos = BITS * j, wd = pos >> 5, sh = pos & 31;
    out[wd] |= q[j] << sh;
    if (sh + BITS > 32) out[wd + 1] |= q[j] >> (32 - sh);
  }
}

__device__ __forceinline__ unsigned short half_bits(float x) { return __half_as_ushort(__float2half_rn(x)); }

template <int G>
__global__ void __launch_bounds__(kApplyWarps * 32)
apply_plan_kernel(const __half* __restrict__ W, int R, int U, int64_t ldw, const float* __restrict__ s,
                  const float* __restrict__ clip, int K, const uint8_t* __restrict__ actions,
                  const uint8_t* __restrict__ clip_idx, const long long* __restrict__ code_offsets,
                  uint8_t* __restrict__ codes_out, __half* __restrict__ scales_out, __half* __restrict__ zeros_out,
                  __half* __restrict__ Wq_out, int row_tiles, int chunk, int stride) {
  using T = ApplyTile<G>;
  constexpr int LG = Map<G>::LG, GPW = Map<G>::GPW;
  extern __shared__ uint4 smem_u4[];
  uint8_t* stage = reinterpret_cast<uint8_t*>(smem_u4);
  Cand* cand_all = reinterpret_cast<Cand*>(stage + T::STAGE_BYTES);

  const int u = blockIdx.x / row_tiles, rt = blockIdx.x % row_tiles;
  const int a = actions[u];
  if (a > 6) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane / LG, q = lane % LG;
  Cand* cand = cand_all + (size_t)warp * GPW * stride;
  const int r0 = rt * T::ROWS;
  const int rows_here = min(T::ROWS, R - r0);
  const int bpg = group_code_bytes(a, G);
  uint8_t* out_base = codes_out + code_offsets[u] + (long long)r0 * bpg;

  Lane32 sv;
  load_stats(s + (int64_t)u * G + 32 * q, sv);

#pragma unroll 1
  for (int pass = 0; pass < T::PASSES; ++pass) {
    const int rl = (pass * kApplyWarps + warp) * GPW + g;  // row inside the tile
    const int row = r0 + rl;
    const bool live = row < R;
    const int row_ld = live ? row : R - 1;
    const __half* wp = W + (int64_t)row_ld * ldw + (int64_t)u * G + 32 * q;
    if (a == 0) {  // skip: the raw fp16 values are the codes and the reconstruction
      if (live) {
        const uint4* src = reinterpret_cast<const uint4*>(wp);
        uint4* dst = reinterpret_cast<uint4*>(out_base + (long long)rl * bpg + 64 * q);
        uint4* wq = Wq_out ? reinterpret_cast<uint4*>(Wq_out + (int64_t)row * ldw + (int64_t)u * G + 32 * q) : nullptr;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint4 v = __ldg(src + i);
          dst[i] = v;
          if (wq) wq[i] = v;
        }
        if (q == 0) {
          scales_out[(int64_t)u * R + row] = __ushort_as_half(0);
          zeros_out[(int64_t)u * R + row] = __ushort_as_half(0);
        }
      }
      continue;
    }
    Lane32 wv;
    load_weights(wp, wv);
    unsigned code[32];
    unsigned short wq16[32];
    float scale_store, zero_store = 0.0f;
    if (a <= 4) {
      const int bi = a - 1;
      float mn, mx;
      group_range<G>(wv, mn, mx);
      const float rng = __fsub_rn(mx, mn);
      int k;
      if (clip_idx) {
        k = min((int)clip_idx[((int64_t)bi * U + u) * R + row_ld], K - 1);
      } else {
        float be;
        search_uniform<G>(wv, sv, mn, rng, bi, clip, K, cand, chunk, stride, lane, be, k);
      }
      const UniformSpec us = uniform_spec(bi);
      const float p = __ldg(clip + k);
      float scale, zf;
      uniform_scale_zero(mn, rng, p, us, scale, zf);
      const Cand c = make_cand(mn, rng, p, us);
#pragma unroll
      for (int l = 0; l < 4; ++l)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float cc = centred_code(wv.get(l, i), c);
          code[8 * l + i] = (unsigned)(int)__fadd_rn(cc, zf);
          wq16[8 * l + i] = half_bits(__fmul_rn(cc, scale));
        }
      scale_store = scale;
      zero_store = zf;
    } else {
      const LowBitFit f = fit_low_bits<G>(wv, sv);
      const float alpha = (a == 5) ? f.alpha_t : f.alpha_b;
      const unsigned short pos = half_bits(alpha), neg = half_bits(-alpha);
#pragma unroll
      for (int l = 0; l < 4; ++l)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float w = wv.get(l, i);
          const bool is_neg = w < 0.0f;
          if (a == 5) {
            const bool in = fabsf(w) > f.delta;
            code[8 * l + i] = in ? (is_neg ? 0u : 2u) : 1u;
            wq16[8 * l + i] = in ? (is_neg ? neg : pos) : (unsigned short)0;
          } else {
            code[8 * l + i] = is_neg ? 0u : 1u;
            wq16[8 * l + i] = is_neg ? neg : pos;
          }
        }
      scale_store = alpha;
    }
    if (live) {
      if (Wq_out) {
        uint4* wq = reinterpret_cast<uint4*>(Wq_out + (int64_t)row * ldw + (int64_t)u * G + 32 * q);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint4 v;
          v.x = wq16[8 * i + 0] | ((unsigned)wq16[8 * i + 1] << 16);
          v.y = wq16[8 * i + 2] | ((unsigned)wq16[8 * i + 3] << 16);
          v.z = wq16[8 * i + 4] | ((unsigned)wq16[8 * i + 5] << 16);
          v.w = wq16[8 * i + 6] | ((unsigned)wq16[8 * i + 7] << 16);
          wq[i] = v;
        }
      }
      if (q == 0) {
        scales_out[(int64_t)u * R + row] = __float2half_rn(scale_store);
        zeros_out[(int64_t)u * R + row] = __float2half_rn(zero_store);
      }
      unsigned words[8];
      int n_words;
      unsigned* dst;
      switch (a) {
        case 1: pack_words<8>(code, words); n_words = 8; break;
        case 2: pack_words<4>(code, words); n_words = 4; break;
        case 3: pack_words<3>(code, words); n_words = 3; break;
        case 4: pack_words<2>(code, words); n_words = 2; break;
        case 5: pack_words<8>(code, words); n_words = 8; break;  // trits as bytes
        default: pack_words<1>(code, words); n_words = 1; break;
      }
      if (a == 5) dst = reinterpret_cast<unsigned*>(stage + (size_t)rl * G + 32 * q);
      else dst = reinterpret_cast<unsigned*>(stage + (size_t)rl * bpg + 4 * n_words * q);
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (i < n_words) dst[i] = words[i];
    }
  }
  if (a == 0) return;
  __syncthreads();

  // the tile's packed bytes are contiguous in the output; the unit's last tile also writes the
  // zero padding up to the next 16-byte boundary
  const int total = rows_here * bpg;
  const int out_len = (total + 15) & ~15;
  for (int i = threadIdx.x * 16; i < out_len; i += kApplyWarps * 32 * 16) {
    uint4 v;
    if (a != 5) {
      v = *reinterpret_cast<const uint4*>(stage + i);
    } else {
      unsigned w4[4] = {0u, 0u, 0u, 0u};
#pragma unroll
      for (int b = 0; b < 16; ++b) {
        const int B = i + b;
        if (B < total) {
          const int rl = B / bpg, bi = B - rl * bpg;
          const uint8_t* t = stage + (size_t)rl * G + 5 * bi;
          unsigned val = 0u, p3 = 1u;
#pragma unroll
          for (int m = 0; m < 5; ++m) {
            if (5 * bi + m < G) val += t[m] * p3;
            p3 *= 3u;
          }
          w4[b >> 2] |= val << (8 * (b & 3));
        }
      }
      v = make_uint4(w4[0], w4[1], w4[2], w4[3]);
    }
    if (i + 16 > total) {  // mask the padding bytes of the last chunk
      unsigned* pv = reinterpret_cast<unsigned*>(&v);
#pragma unroll
      for (int b = 0; b < 16; ++b)
        if (i + b >= total) pv[b >> 2] &= ~(0xffu << (8 * (b & 3)));
    }
    *reinterpret_cast<uint4*>(out_base + i) = v;
  }
}

template <int G>
windq_status launch_apply(windq_ctx* ctx, const __half* W, int R, int U, int64_t ldw, const float* s, const float* clip,
                          int K, const uint8_t* actions, const uint8_t* clip_idx, const long long* code_offsets,
                          uint8_t* codes_out, __half* scales_out, __half* zeros_out, __half* Wq_out, cudaStream_t st) {
  using T = ApplyTile<G>;
  const int chunk = 336 / T::GPW > 64 ? 64 : 336 / T::GPW, stride = chunk | 1;
  const size_t smem = (size_t)T::STAGE_BYTES + (size_t)kApplyWarps * T::GPW * stride * sizeof(Cand);
  static bool configured = false;
  if (!configured) {
    WINDQ_CUDA(ctx, cudaFuncSetAttribute(apply_plan_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    configured = true;
  }
  const int row_tiles = (R + T::ROWS - 1) / T::ROWS;
  const int64_t blocks = (int64_t)U * row_tiles;
  WINDQ_REQUIRE(ctx, blocks < (1ll << 31), WINDQ_ERR_SHAPE, "windq_apply_plan: too many tiles");
  apply_plan_kernel<G><<<(unsigned)blocks, kApplyWarps * 32, smem, st>>>(W, R, U, ldw, s, clip, K, actions, clip_idx,
                                                                          code_offsets, codes_out, scales_out, zeros_out,
                                                                          Wq_out, row_tiles, chunk, stride);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

}  // namespace windq

extern "C" windq_status windq_apply_plan(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                         const float* s, const float* clip_grid, int K, const uint8_t* actions,
                                         const uint8_t* clip_idx, const int64_t* code_offsets, uint8_t* codes_out,
                                         void* scales_out, void* zeros_out, void* Wq_out, void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "windq_apply_plan: ctx is NULL");
  if (windq_status st = check_matrix(ctx, "windq_apply_plan", W, R, C, ldw, G)) return st;
  if (windq_status st = check_K(ctx, "windq_apply_plan", K)) return st;
  WINDQ_REQUIRE(ctx, s && clip_grid && actions && code_offsets && codes_out && scales_out && zeros_out, WINDQ_ERR_NULL,
                "windq_apply_plan: a required pointer is NULL");
  WINDQ_REQUIRE(ctx, aligned16(s) && aligned16(codes_out), WINDQ_ERR_ALIGN,
                "windq_apply_plan: s or codes_out is not 16-byte aligned");
  WINDQ_REQUIRE(ctx, ((uintptr_t)code_offsets & 7) == 0 && ((uintptr_t)scales_out & 1) == 0 && ((uintptr_t)zeros_out & 1) == 0,
                WINDQ_ERR_ALIGN, "windq_apply_plan: code_offsets, scales_out or zeros_out is misaligned");
  WINDQ_REQUIRE(ctx, Wq_out == nullptr || aligned16(Wq_out), WINDQ_ERR_ALIGN, "windq_apply_plan: Wq_out is not 16-byte aligned");
  WINDQ_REQUIRE(ctx, Wq_out != W, WINDQ_ERR_ARG, "windq_apply_plan: Wq_out must not alias W");
  DeviceGuard guard(ctx->device);
  const int U = (int)(C / G);
  cudaStream_t st = (cudaStream_t)stream;
  const __half* Wh = (const __half*)W;
  const long long* offs = (const long long*)code_offsets;
  __half *sc = (__half*)scales_out, *zp = (__half*)zeros_out, *wq = (__half*)Wq_out;
  switch (G) {
    case 32: return launch_apply<32>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, actions, clip_idx, offs, codes_out, sc, zp, wq, st);
    case 64: return launch_apply<64>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, actions, clip_idx, offs, codes_out, sc, zp, wq, st);
    case 128: return launch_apply<128>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, actions, clip_idx, offs, codes_out, sc, zp, wq, st);
    case 256: return launch_apply<256>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, actions, clip_idx, offs, codes_out, sc, zp, wq, st);
    default: return launch_apply<512>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, actions, clip_idx, offs, codes_out, sc, zp, wq, st);
  }
}

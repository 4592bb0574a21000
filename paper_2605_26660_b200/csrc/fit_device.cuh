// Device-side group fitting shared by windq_fit_eval and windq_apply_plan.
//
// Thread mapping.  A group (one row of one unit, G fp16 values) is owned by LG = G/32 adjacent
// lanes; each lane keeps its 32 consecutive values (four leaves of 8) and the matching 32
// activation statistics in registers as fp32 for the whole fit, so a weight is read from memory
// once and every clip candidate of every bit-width is evaluated from registers.  A warp therefore
// works on GPW = 32/LG consecutive rows of the same unit.
//
// Arithmetic.  Everything that decides a clip index, a code or a stored fp16 value is an explicit
// IEEE binary32 operation (round to nearest even, no flush to zero, no contraction beyond the
// fma's written here).  A sum over a group is taken as: each leaf of 8 consecutive elements
// accumulated left to right from +0, then a balanced tree that adds adjacent leaves first.  In
// this mapping the first two tree levels are inside a lane and the rest are xor-shuffles over
// 1, 2, ... LG/2, which perform exactly those additions.
//
// The inner loop uses the sm_100 packed binary32 instructions (fma/add/mul .f32x2): two leaves of
// a lane advance together, one instruction per pair, each half rounded exactly like the scalar
// instruction.  The clamp has no packed form and stays scalar (see Cand).
#pragma once

#include "windq_internal.cuh"

namespace windq {

constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23: adding it rounds to the nearest-even integer

template <int G>
struct Map {
  static constexpr int LG = G / 32;    // lanes per group
  static constexpr int GPW = 32 / LG;  // groups (rows) per warp
};

// ---- packed binary32 pairs --------------------------------------------------------------------
__device__ __forceinline__ unsigned long long as_u64(float2 v) {
  unsigned long long u;
  asm("mov.b64 %0, {%1, %2};" : "=l"(u) : "f"(v.x), "f"(v.y));
  return u;
}
__device__ __forceinline__ float2 as_f2(unsigned long long u) {
  float2 v;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(v.x), "=f"(v.y) : "l"(u));
  return v;
}
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(as_u64(a)), "l"(as_u64(b)), "l"(as_u64(c)));
  return as_f2(d);
}
__device__ __forceinline__ float2 add2(float2 a, float2 b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(as_u64(a)), "l"(as_u64(b)));
  return as_f2(d);
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b) {
  unsigned long long d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(as_u64(a)), "l"(as_u64(b)));
  return as_f2(d);
}

// ---- what a lane owns -------------------------------------------------------------------------
// Element e (0..31) of the lane = leaf l = e / 8, position i = e % 8, stored in
// v[l >> 1][i].x (even leaf) or .y (odd leaf): the two halves of a pair belong to different
// leaves, so their accumulations are independent.
struct Lane32 {
  float2 v[2][8];
  __device__ __forceinline__ float get(int l, int i) const { return (l & 1) ? v[l >> 1][i].y : v[l >> 1][i].x; }
  __device__ __forceinline__ void set(int l, int i, float x) {
    if (l & 1) v[l >> 1][i].y = x; else v[l >> 1][i].x = x;
  }
};

// 32 fp16 values, as four 128-bit words -> Lane32.
__device__ __forceinline__ void unpack_weights(const uint4 (&raw)[4], Lane32& w) {
#pragma unroll
  for (int l = 0; l < 4; ++l) {
    const __half2* h = reinterpret_cast<const __half2*>(&raw[l]);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __half22float2(h[i]);
      w.set(l, 2 * i, f.x);
      w.set(l, 2 * i + 1, f.y);
    }
  }
}

// 32 fp16 values (64 bytes, 16-byte aligned) -> Lane32.
__device__ __forceinline__ void load_weights(const __half* p, Lane32& w) {
  const uint4* p4 = reinterpret_cast<const uint4*>(p);
  uint4 raw[4];
#pragma unroll
  for (int l = 0; l < 4; ++l) raw[l] = __ldg(p4 + l);
  unpack_weights(raw, w);
}

// 32 fp32 statistics (128 bytes, 16-byte aligned) -> Lane32.
__device__ __forceinline__ void load_stats(const float* p, Lane32& s) {
  const float4* p4 = reinterpret_cast<const float4*>(p);
#pragma unroll
  for (int l = 0; l < 4; ++l) {
    const float4 a = __ldg(p4 + 2 * l), b = __ldg(p4 + 2 * l + 1);
    s.set(l, 0, a.x); s.set(l, 1, a.y); s.set(l, 2, a.z); s.set(l, 3, a.w);
    s.set(l, 4, b.x); s.set(l, 5, b.y); s.set(l, 6, b.z); s.set(l, 7, b.w);
  }
}

// Tree over the group: four leaf sums of this lane, then the lanes of the group.
template <int G>
__device__ __forceinline__ float group_tree(float l0, float l1, float l2, float l3) {
  float t = __fadd_rn(__fadd_rn(l0, l1), __fadd_rn(l2, l3));
#pragma unroll
  for (int m = 1; m < Map<G>::LG; m <<= 1) t = __fadd_rn(t, __shfl_xor_sync(0xffffffffu, t, m));
  return t;
}
template <int G>
__device__ __forceinline__ float group_tree(float2 a01, float2 a23) {
  return group_tree<G>(a01.x, a01.y, a23.x, a23.y);
}

// min(0, min w) and max(0, max w) over the group.
template <int G>
__device__ __forceinline__ void group_range(const Lane32& w, float& mn, float& mx) {
  float lo = 0.0f, hi = 0.0f;
#pragma unroll
  for (int h = 0; h < 2; ++h)
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      lo = fminf(lo, fminf(w.v[h][i].x, w.v[h][i].y));
      hi = fmaxf(hi, fmaxf(w.v[h][i].x, w.v[h][i].y));
    }
#pragma unroll
  for (int m = 1; m < Map<G>::LG; m <<= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, m));
    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, m));
  }
  mn = __fadd_rn(lo, 0.0f);  // -0 -> +0
  mx = hi;
}

// ---- uniform candidates -----------------------------------------------------------------------
// Parameters of one (bit-width, clip ratio) candidate of one group, as the inner loop wants them.
//
// Per element the loop computes, with the group's scale (an fp16 value), inv = 1 / scale and zero point z:
//   r    = fma(w, inv, M)            M = 1.5 * 2^23: r = M + rne(w * inv), one rounding of the exact product
//   x    = r + (z - M)               = rne(w * inv) + z, the code before clamping (exact: small integers)
//   code = clamp(x, 0, qmax)         ONE integer instruction on the bit patterns (min.s32.relu): a negative float
//                                    is a negative integer and is floored to 0 = +0.0f, non-negative floats
//                                    order like their bit patterns
//   e    = fma(code, -scale, z * scale)   = -(code - z) * scale exactly: an integer of at most 8 bits times an
//                                    11-bit significand, and z * scale is exact for the same reason
//   d    = e + w                     = w - c * scale with c = code - z, rounded once: the negative of the
//                                    difference fma(c, scale, -w) of the definition; (s d) d is the same either way
//   t = s * d;  acc = fma(t, d, acc)
// i.e. six FP32-pipe operations and one integer min per element.  The textbook form -- subtract M, max, min,
// fma(c, -scale, w) -- has five and two; on B200 a float min / max costs about two issue cycles of the pipe the
// FP32 operations need (measured: the loop ran at 9 cycles per element and candidate, 5 + 2 * 2), so trading one of
// them for an addition and folding the other into the relu form is 8 % faster, with the same bits.
struct Cand {
  float inv;     // 1 / scale
  float nscale;  // -scale
  float bias;    // z - M
  float kz;      // z * scale
};

struct UniformSpec {
  float qmax;
  float rq;  // fp32 nearest to 1 / qmax
};
__device__ __forceinline__ UniformSpec uniform_spec(int bi) {  // bi: 0..3 = 8, 4, 3, 2 bit
  switch (bi) {
    case 0: return {255.0f, (float)(1.0 / 255.0)};
    case 1: return {15.0f, (float)(1.0 / 15.0)};
    case 2: return {7.0f, (float)(1.0 / 7.0)};
    default: return {3.0f, (float)(1.0 / 3.0)};
  }
}

// 1 / x, correctly rounded, for x the value of a positive finite fp16 number (a stored scale, or the 1 that
// stands in for a scale of zero): the hardware approximation followed by one Newton step in fused arithmetic.
// For these 31,743 inputs the result equals IEEE division bit for bit (windq_selfcheck tests every one of them
// on the device); the general-purpose correctly rounded reciprocal costs about three times the instructions,
// and a fit forms one per candidate.
__device__ __forceinline__ float reciprocal_of_half_value(float x) {
  float r0;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r0) : "f"(x));
  return __fmaf_rn(r0, __fmaf_rn(-x, r0, 1.0f), r0);
}

// scale (value of the stored fp16 scale, 1 if that is zero), its reciprocal, and the zero point (float integer).
__device__ __forceinline__ void uniform_scale_zero(float mn, float rng, float p, UniformSpec us, float& scale, float& inv,
                                                   float& zf) {
  const float scale32 = __fmul_rn(__fmul_rn(p, rng), us.rq);
  scale = __half2float(__float2half_rn(scale32));
  if (scale == 0.0f) scale = 1.0f;
  inv = reciprocal_of_half_value(scale);
  // nearest-even integer of |p mn| / scale, which is at most about 1.5 qmax: adding and subtracting 1.5 * 2^23
  // rounds exactly like rint
  const float z = __fadd_rn(__fadd_rn(__fmul_rn(fabsf(__fmul_rn(p, mn)), inv), kMagic), -kMagic);
  zf = fminf(fmaxf(z, 0.0f), us.qmax);
}
__device__ __forceinline__ void uniform_scale_zero(float mn, float rng, float p, UniformSpec us, float& scale, float& zf) {
  float inv;
  uniform_scale_zero(mn, rng, p, us, scale, inv, zf);
}

__device__ __forceinline__ Cand make_cand(float mn, float rng, float p, UniformSpec us) {
  float scale, zf;
  Cand c;
  uniform_scale_zero(mn, rng, p, us, scale, c.inv, zf);
  c.nscale = -scale;
  c.bias = __fsub_rn(zf, kMagic);
  c.kz = __fmul_rn(zf, scale);
  return c;
}

// clamp(x, 0, qmax) of an integer-valued float, on the bit patterns (qmax_bits = the bit pattern of qmax).
__device__ __forceinline__ float clamp_code(float x, int qmax_bits) {
  int r;
  asm("min.s32.relu %0, %1, %2;" : "=r"(r) : "r"(__float_as_int(x)), "r"(qmax_bits));
  return __int_as_float(r);
}

// s-weighted squared error of one candidate over this lane's 32 elements: the four leaf sums,
// as two pairs.
__device__ __forceinline__ void cand_leaf_errors(const Lane32& w, const Lane32& s, const Cand& c, int qmax_bits, float2& e01,
                                                 float2& e23) {
  const float2 inv2 = make_float2(c.inv, c.inv);
  const float2 ns2 = make_float2(c.nscale, c.nscale);
  const float2 magic2 = make_float2(kMagic, kMagic);
  const float2 bias2 = make_float2(c.bias, c.bias);
  const float2 kz2 = make_float2(c.kz, c.kz);
  float2 acc[2] = {make_float2(0.0f, 0.0f), make_float2(0.0f, 0.0f)};
  // leaf pair by leaf pair (measured: this order schedules 2 % better than alternating the pairs)
#pragma unroll
  for (int h = 0; h < 2; ++h) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float2 wv = w.v[h][i];
      float2 q = add2(fma2(wv, inv2, magic2), bias2);  // rne(w * inv) + z
      q.x = clamp_code(q.x, qmax_bits);
      q.y = clamp_code(q.y, qmax_bits);
      const float2 d = add2(fma2(q, ns2, kz2), wv);     // w - (code - z) * scale
      const float2 t = mul2(s.v[h][i], d);
      acc[h] = fma2(t, d, acc[h]);
    }
  }
  e01 = acc[0];
  e23 = acc[1];
}

// Clip search for one bit-width.  `cand` is this warp's shared-memory parameter table with room
// for GPW rows of `stride` entries; candidates are processed in chunks of at most `chunk`.
// On return best_e / best_k hold the least error and the smallest index that reaches it; all
// lanes of a group hold the same values.  Must be called by all 32 lanes.
template <int G>
__device__ __forceinline__ void search_uniform(const Lane32& w, const Lane32& s, float mn, float rng, int bi,
                                               const float* __restrict__ clip, int K, Cand* cand, int chunk,
                                               int stride, int lane, float& best_e, int& best_k) {
  constexpr int LG = Map<G>::LG;
  const int g = lane / LG, q = lane % LG;
  const UniformSpec us = uniform_spec(bi);
  Cand* mine = cand + g * stride;
  best_e = __int_as_float(0x7f800000);  // +inf: the first candidate replaces it (or none does, if no error is finite)
  best_k = 0;
  for (int k0 = 0; k0 < K; k0 += chunk) {
    const int kc = min(chunk, K - k0);
    __syncwarp();
    for (int k = q; k < kc; k += LG) mine[k] = make_cand(mn, rng, __ldg(clip + k0 + k), us);
    __syncwarp();
    for (int k = 0; k < kc; ++k) {
      const Cand c = mine[k];
      float2 e01, e23;
      cand_leaf_errors(w, s, c, __float_as_int(us.qmax), e01, e23);
      const float e = group_tree<G>(e01, e23);
      if (e < best_e) {
        best_e = e;
        best_k = k0 + k;
      }
    }
  }
}

// This lane's least and greatest weight and their activation weights, as (least, greatest, s of least, s of
// greatest): the elements a narrower clip range cuts deepest, for the bound of search_uniform_pruned.
__device__ __forceinline__ float4 lane_extremes(const Lane32& w, const Lane32& s) {
  float lo = w.v[0][0].x, hi = lo, slo = s.v[0][0].x, shi = slo;
#pragma unroll
  for (int h = 0; h < 2; ++h)
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float2 wv = w.v[h][i], sv = s.v[h][i];
      if (wv.x < lo) { lo = wv.x; slo = sv.x; }
      if (wv.x > hi) { hi = wv.x; shi = sv.x; }
      if (wv.y < lo) { lo = wv.y; slo = sv.y; }
      if (wv.y > hi) { hi = wv.y; shi = sv.y; }
    }
  return make_float4(lo, hi, slo, shi);
}

// search_uniform with candidates left out that cannot win -- same best_e and best_k, bit for bit.
//
// Every term (s d) d of a candidate's error is >= 0 when s >= 0, and rounding to nearest is monotone, so the
// error of a group -- a tree of additions of such terms, each addition rounded -- is at least the rounded term
// fl(fl(s_j d_j) d_j) of any one element j.  A candidate whose term for some element already exceeds the least
// error found so far therefore cannot replace it, and if that holds in every group of the warp the warp skips the
// candidate.  The elements tried are every lane's least and greatest weight (`ext`, one entry per lane of the
// warp, in shared memory: the ones a narrower clip range cuts deepest).  Where a group has four lanes or more, the
// lane that forms a candidate's parameters also forms its bound -- the largest of those terms over the group's
// lanes -- and leaves it in the table entry in place of z * scale, which the scan forms again for the candidates
// it evaluates.  Where a group has one or two lanes, a lane would have to form ten bounds and more on its own, and
// every lane tries its own two elements inside the scan instead (a group is out if any of its lanes says so);
// measured, each form is the faster one on its side (chunk width 64: 0.72 against 0.80 ms on 11008 x 4096; 128:
// 0.71 against 0.74).  The scan runs from the last candidate to the first and replaces on <=, which ends on the
// same candidate as the forward scan with < (the first of the least error): clip grids usually end on the widest
// range and the wide ranges win at eight bits -- there four candidates in five are skipped on weight-like data.
// With activation weights below zero the premise fails; such input is outside the domain (s is a mean of squares).
// `skipped` is advanced by the number of candidates left out.
template <int G>
__device__ __forceinline__ void search_uniform_pruned(const Lane32& w, const Lane32& s, const float4* ext, float mn,
                                                      float rng, int bi, const float* __restrict__ clip, int K, Cand* cand,
                                                      int chunk, int stride, int lane, float& best_e, int& best_k,
                                                      unsigned int& skipped) {
  constexpr int LG = Map<G>::LG;
  const int g = lane / LG, q = lane % LG;
  const UniformSpec us = uniform_spec(bi);
  const int qmax_bits = __float_as_int(us.qmax);
  Cand* mine = cand + g * stride;
  best_e = __int_as_float(0x7f800000);
  best_k = 0;
  const float2 magic2 = make_float2(kMagic, kMagic);
  constexpr bool kInLoop = LG <= 2;  // bounds formed inside the scan, from the lane's own elements
  const float4 own = ext[lane];
  const float2 own_w = make_float2(own.x, own.y), own_s = make_float2(own.z, own.w);
  const int n_chunks = (K + chunk - 1) / chunk;
  for (int ci = n_chunks - 1; ci >= 0; --ci) {
    const int k0 = ci * chunk;
    const int kc = min(chunk, K - k0);
    __syncwarp();
    if (kInLoop) {
      for (int k = q; k < kc; k += LG) mine[k] = make_cand(mn, rng, __ldg(clip + k0 + k), us);
    } else
    for (int k = q; k < kc; k += LG) {
      Cand c = make_cand(mn, rng, __ldg(clip + k0 + k), us);
      float b = 0.0f;
#pragma unroll
      for (int j = 0; j < LG; ++j) {
        const float4 e = ext[g * LG + j];
        const float2 ew = make_float2(e.x, e.y);
        float2 x = add2(fma2(ew, make_float2(c.inv, c.inv), magic2), make_float2(c.bias, c.bias));
        x.x = clamp_code(x.x, qmax_bits);
        x.y = clamp_code(x.y, qmax_bits);
        const float2 d = add2(fma2(x, make_float2(c.nscale, c.nscale), make_float2(c.kz, c.kz)), ew);
        const float2 term = mul2(mul2(make_float2(e.z, e.w), d), d);
        b = fmaxf(b, fmaxf(term.x, term.y));
      }
      c.kz = b;  // the table entry carries the bound in place of z * scale, which the scan forms again
      mine[k] = c;
    }
    __syncwarp();
    for (int k = kc - 1; k >= 0; --k) {
      Cand c = mine[k];
      if (kInLoop) {
        // this lane's own two elements; a group is out if any of its lanes says so
        float2 x = add2(fma2(own_w, make_float2(c.inv, c.inv), magic2), make_float2(c.bias, c.bias));
        x.x = clamp_code(x.x, qmax_bits);
        x.y = clamp_code(x.y, qmax_bits);
        const float2 d = add2(fma2(x, make_float2(c.nscale, c.nscale), make_float2(c.kz, c.kz)), own_w);
        const float2 term = mul2(mul2(own_s, d), d);
        unsigned int out = __ballot_sync(0xffffffffu, fmaxf(term.x, term.y) > best_e);
#pragma unroll
        for (int m = 1; m < LG; m <<= 1) out |= out >> m;
        constexpr unsigned int kFirstLanes = LG == 1 ? 0xffffffffu : LG == 2 ? 0x55555555u : LG == 4 ? 0x11111111u
                                             : LG == 8 ? 0x01010101u : 0x00010001u;
        if ((out & kFirstLanes) == kFirstLanes) { ++skipped; continue; }
      } else {
        if (__all_sync(0xffffffffu, c.kz > best_e)) { ++skipped; continue; }  // ruled out in every group of the warp
        c.kz = __fmul_rn(__fadd_rn(c.bias, kMagic), -c.nscale);  // z * scale, as make_cand forms it
      }
      float2 e01, e23;
      cand_leaf_errors(w, s, c, qmax_bits, e01, e23);
      const float e = group_tree<G>(e01, e23);
      if (e <= best_e) {
        best_e = e;
        best_k = k0 + k;
      }
    }
  }
}

// ---- ternary and binary -----------------------------------------------------------------------
struct LowBitFit {
  float delta;    // ternary threshold 0.7 * mean |w|
  float alpha_t;  // ternary scale (value of the fp16 number), 0 if the support is empty
  float alpha_b;  // binary scale
  float err_t, err_b;
  float energy;   // sum_j s_j w_j^2 of the group (any order; tolerance output)
};

// Must be called by all 32 lanes.  exact_errors = false: err_t and err_b are wanted only for the unit sums (which
// are tolerance outputs); they are then taken from the sums already formed instead of a pass of their own.
template <int G>
__device__ __forceinline__ LowBitFit fit_low_bits(const Lane32& w, const Lane32& s, bool exact_errors) {
  LowBitFit f;
  const float2 zero2 = make_float2(0.0f, 0.0f);
  // leaves 2 h and 2 h + 1 side by side in the two halves of the packed operations
  float2 a2[2] = {zero2, zero2}, sb2[2] = {zero2, zero2}, bb2[2] = {zero2, zero2}, en2[2] = {zero2, zero2};
#pragma unroll
  for (int h = 0; h < 2; ++h)
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float2 wv = w.v[h][i], sv = s.v[h][i];
      const float2 aw = make_float2(fabsf(wv.x), fabsf(wv.y));
      a2[h] = add2(a2[h], aw);
      sb2[h] = add2(sb2[h], sv);
      bb2[h] = fma2(sv, aw, bb2[h]);
      en2[h] = fma2(mul2(sv, wv), wv, en2[h]);
    }
  const float sumA = group_tree<G>(a2[0], a2[1]);
  const float sumS = group_tree<G>(sb2[0], sb2[1]);
  const float sumB = group_tree<G>(bb2[0], bb2[1]);
  f.energy = group_tree<G>(en2[0], en2[1]);
  const float meanA = __fmul_rn(sumA, 1.0f / (float)G);
  f.delta = __fmul_rn(0.7f, meanA);
  f.alpha_b = __half2float(__float2half_rn(sumS == 0.0f ? meanA : __fdiv_rn(sumB, sumS)));

  // ternary sums over the support, weighted by s; the unweighted ones only if some group of the
  // warp has no activation weight on its support.  The support enters as a factor 1 or 0 per weight: s (|w| m)
  // and s m are exact products of the terms the definition adds, so the sums round as they do there.
  float2 bt2[2] = {zero2, zero2}, ct2[2] = {zero2, zero2};
#pragma unroll
  for (int h = 0; h < 2; ++h)
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float2 wv = w.v[h][i], sv = s.v[h][i];
      const float2 aw = make_float2(fabsf(wv.x), fabsf(wv.y));
      const float2 m = make_float2(aw.x > f.delta ? 1.0f : 0.0f, aw.y > f.delta ? 1.0f : 0.0f);
      bt2[h] = fma2(sv, mul2(aw, m), bt2[h]);
      ct2[h] = fma2(sv, m, ct2[h]);
    }
  float sumBt = group_tree<G>(bt2[0], bt2[1]);
  float sumCt = group_tree<G>(ct2[0], ct2[1]);
  const float wBt = sumBt, wCt = sumCt;  // the weighted sums, whatever the scale is taken from
  // delta < max |w| whenever some w is not zero (0.7 * mean <= 0.7 * max, roundings included), so
  // the support is empty exactly when every |w| is zero, i.e. when their sum is
  const bool nonempty = sumA > 0.0f;
  if (__any_sync(0xffffffffu, nonempty && sumCt == 0.0f)) {
    float Bu[4], Cu[4];
#pragma unroll
    for (int l = 0; l < 4; ++l) {
      float bu = 0.0f, cu = 0.0f;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float aw = fabsf(w.get(l, i));
        const bool in = aw > f.delta;
        bu = __fadd_rn(bu, in ? aw : 0.0f);
        cu = __fadd_rn(cu, in ? 1.0f : 0.0f);
      }
      Bu[l] = bu; Cu[l] = cu;
    }
    const float sumBu = group_tree<G>(Bu[0], Bu[1], Bu[2], Bu[3]);
    const float sumCu = group_tree<G>(Cu[0], Cu[1], Cu[2], Cu[3]);
    if (sumCt == 0.0f) { sumBt = sumBu; sumCt = sumCu; }
  }
  f.alpha_t = nonempty ? __half2float(__float2half_rn(__fdiv_rn(sumBt, sumCt))) : 0.0f;

  if (!exact_errors) {
    // sum_j s_j (alpha q_j - w_j)^2 = sum s w^2 - 2 alpha sum_I s |w| + alpha^2 sum_I s  over the support I (every
    // j for the binary fit), in double from the group sums (the weighted support sums, also when the scale came
    // from the unweighted ones).  The three sums carry binary32 rounding of about 1e-6 of the energy at worst, so
    // the difference is good to 2e-5 relative as long as the error is at least a sixteenth of the energy -- on
    // weight-like data it is a fifth or more.  Where a group of the warp falls below that (weights of nearly
    // equal magnitude, which a one-scale fit reproduces almost exactly), the warp takes the term-by-term pass.
    const double at = (double)f.alpha_t, ab = (double)f.alpha_b, en = (double)f.energy;
    const double et = en - 2.0 * at * (double)wBt + at * at * (double)wCt;
    const double eb = en - 2.0 * ab * (double)sumB + ab * ab * (double)sumS;
    const bool thin = et < 0.0625 * en || eb < 0.0625 * en;
    if (!__any_sync(0xffffffffu, thin)) {
      f.err_t = (float)et;
      f.err_b = (float)eb;
      return f;
    }
  }
  float Et[4], Eb[4];
#pragma unroll
  for (int l = 0; l < 4; ++l) {
    float et = 0.0f, eb = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float wv = w.get(l, i), sv = s.get(l, i);
      const bool neg = wv < 0.0f;
      const float rt = (fabsf(wv) > f.delta) ? (neg ? -f.alpha_t : f.alpha_t) : 0.0f;
      const float dt = __fsub_rn(rt, wv);
      et = __fmaf_rn(__fmul_rn(sv, dt), dt, et);
      const float db = __fsub_rn(neg ? -f.alpha_b : f.alpha_b, wv);
      eb = __fmaf_rn(__fmul_rn(sv, db), db, eb);
    }
    Et[l] = et; Eb[l] = eb;
  }
  f.err_t = group_tree<G>(Et[0], Et[1], Et[2], Et[3]);
  f.err_b = group_tree<G>(Eb[0], Eb[1], Eb[2], Eb[3]);
  return f;
}

// ---- scales only (plan application) ------------------------------------------------------------
// The binary and ternary scales as fit_low_bits computes them -- the same operations in the same
// order -- without the error sums, and without the sums that only a rare fallback needs unless
// some group of the warp takes that fallback.  Must be called by all 32 lanes.

// PSUM8 of |w| over the group.
template <int G>
__device__ __forceinline__ float group_abs_sum(const Lane32& w) {
  float A[4];
#pragma unroll
  for (int l = 0; l < 4; ++l) {
    float a = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) a = __fadd_rn(a, fabsf(w.get(l, i)));
    A[l] = a;
  }
  return group_tree<G>(A[0], A[1], A[2], A[3]);
}

template <int G>
__device__ __forceinline__ float binary_scale(const Lane32& w, const Lane32& s) {
  float Sb[4], Bb[4];
#pragma unroll
  for (int l = 0; l < 4; ++l) {
    float sb = 0.0f, bb = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float sv = s.get(l, i);
      sb = __fadd_rn(sb, sv);
      bb = __fmaf_rn(sv, fabsf(w.get(l, i)), bb);
    }
    Sb[l] = sb; Bb[l] = bb;
  }
  const float sumS = group_tree<G>(Sb[0], Sb[1], Sb[2], Sb[3]);
  const float sumB = group_tree<G>(Bb[0], Bb[1], Bb[2], Bb[3]);
  float meanA = 0.0f;
  if (__any_sync(0xffffffffu, sumS == 0.0f)) meanA = __fmul_rn(group_abs_sum<G>(w), 1.0f / (float)G);
  return __half2float(__float2half_rn(sumS == 0.0f ? meanA : __fdiv_rn(sumB, sumS)));
}

// delta = 0.7 * mean |w|; returns the scale (0 when the support is empty).
template <int G>
__device__ __forceinline__ float ternary_scale(const Lane32& w, const Lane32& s, float& delta) {
  const float sumA = group_abs_sum<G>(w);
  delta = __fmul_rn(0.7f, __fmul_rn(sumA, 1.0f / (float)G));
  float Bt[4], Ct[4];
#pragma unroll
  for (int l = 0; l < 4; ++l) {
    float bt = 0.0f, ct = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float aw = fabsf(w.get(l, i)), sv = s.get(l, i);
      const bool in = aw > delta;
      bt = __fmaf_rn(sv, in ? aw : 0.0f, bt);
      ct = __fadd_rn(ct, in ? sv : 0.0f);
    }
    Bt[l] = bt; Ct[l] = ct;
  }
  float sumBt = group_tree<G>(Bt[0], Bt[1], Bt[2], Bt[3]);
  float sumCt = group_tree<G>(Ct[0], Ct[1], Ct[2], Ct[3]);
  // delta < max |w| whenever some w is not zero (0.7 * mean <= 0.7 * max, roundings included), so
  // the support is empty exactly when every |w| is zero, i.e. when their sum is
  const bool nonempty = sumA > 0.0f;
  if (__any_sync(0xffffffffu, nonempty && sumCt == 0.0f)) {  // no activation weight on the support: unweighted mean
    float Bu[4], Cu[4];
#pragma unroll
    for (int l = 0; l < 4; ++l) {
      float bu = 0.0f, cu = 0.0f;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float aw = fabsf(w.get(l, i));
        const bool in = aw > delta;
        bu = __fadd_rn(bu, in ? aw : 0.0f);
        cu = __fadd_rn(cu, in ? 1.0f : 0.0f);
      }
      Bu[l] = bu; Cu[l] = cu;
    }
    const float sumBu = group_tree<G>(Bu[0], Bu[1], Bu[2], Bu[3]);
    const float sumCu = group_tree<G>(Cu[0], Cu[1], Cu[2], Cu[3]);
    if (sumCt == 0.0f) { sumBt = sumBu; sumCt = sumCu; }
  }
  return nonempty ? __half2float(__float2half_rn(__fdiv_rn(sumBt, sumCt))) : 0.0f;
}

}  // namespace windq

// windq_apply_plan: codes, packed bytes, fp16 scale / zero point and fake-quantised weights of a
// chosen plan.
//
// With clip indices supplied this is a streaming kernel bound by HBM: 2 bytes read per weight,
// 2 bytes written for the fake-quantised copy and bits/8 for the codes.  Thread mapping as in
// the fit (LG lanes per group, 32 values per lane in registers).  Work is split into items =
// (unit, GPW consecutive rows), one warp per item; the warps of a persistent grid walk the items
// with a stride of the number of warps, so that neighbouring warps read and write neighbouring
// rows.  What keeps HBM busy is that the weights of a warp's NEXT item are already on their way
// (cp.async into a 2 KB shared-memory buffer per warp, two buffers) while it fits, quantises
// and stores the current one.
//
// Packing.  Each lane packs its own 32 codes into whole 32-bit words in registers (1, 2, 3, 4
// and 8 bit all give whole words per lane) and the rows of an item are adjacent in the output, so
// the words of a warp form one contiguous run and go out with plain vector stores, no staging.
// Only the base-3 ternary packing crosses lanes (5 trits per byte): its trits are staged as 2-bit
// fields in shared memory and each output byte is looked up from the 10-bit window that holds its
// five trits.
#include <string.h>

#include "fit_device.cuh"

namespace windq {

constexpr int kApplyWarps = 4;

// 16 registers that each hold two small codes -- one in the low bits of each 16-bit half, anything
// above the low BITS bits ignored -- -> packed little-endian words.
template <int BITS>
__device__ __forceinline__ void pack_pairs(const unsigned (&p)[16], unsigned (&out)[8]) {
  constexpr unsigned mask = (1u << BITS) - 1u;
#pragma unroll
  for (int i = 0; i < 8; ++i) out[i] = 0u;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const unsigned f = (p[j] & mask) | (((p[j] >> 16) & mask) << BITS);  // codes 2j, 2j+1
    const int pos = 2 * BITS * j, wd = pos >> 5, sh = pos & 31;
    out[wd] |= f << sh;
    if (sh + 2 * BITS > 32) out[wd + 1] |= f >> (32 - sh);
  }
}

__device__ __forceinline__ unsigned h2_bits(__half2 h) { return *reinterpret_cast<unsigned*>(&h); }
__device__ __forceinline__ __half2 bits_h2(unsigned u) { return *reinterpret_cast<__half2*>(&u); }

// min(0, min w) and max(0, max w) over the group, from the lane's 32 halves: the comparisons are
// made on the fp16 values themselves (exact, two per instruction).
template <int G>
__device__ __forceinline__ void group_range_h(const uint4 (&raw)[4], float& mn, float& mx) {
  const unsigned* r = reinterpret_cast<const unsigned*>(raw);
  __half2 lo2 = bits_h2(r[0]), hi2 = lo2;
#pragma unroll
  for (int i = 1; i < 16; ++i) {
    lo2 = __hmin2(lo2, bits_h2(r[i]));
    hi2 = __hmax2(hi2, bits_h2(r[i]));
  }
  const float2 l = __half22float2(lo2), h = __half22float2(hi2);
  float lo = fminf(0.0f, fminf(l.x, l.y)), hi = fmaxf(0.0f, fmaxf(h.x, h.y));
#pragma unroll
  for (int m = 1; m < Map<G>::LG; m <<= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, m));
    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, m));
  }
  mn = __fadd_rn(lo, 0.0f);  // -0 -> +0
  mx = hi;
}

// Uniform grid with known parameters: codes and fake-quantised weights of the lane's 32 values.
// The centred code c = clamp(rne(w / scale), lo, hi) is formed in fp32 exactly as in the fit; being
// an integer of at most 8 bits it is exact in fp16, so the stored weight fp16(c * scale) is one
// half-precision product (scale is an fp16 value: the product is rounded once either way), and
// the code c + z comes out of a half-precision add of z + 1024, whose low bits are the integer.
__device__ __forceinline__ void quantise_uniform(const uint4 (&raw)[4], float scale, float zf, float qmax,
                                                 unsigned (&wq)[16], unsigned (&code)[16]) {
  const float inv = __frcp_rn(scale);
  const float lo = __fsub_rn(0.0f, zf), hi = __fsub_rn(qmax, zf);
  const __half2 scale2 = __float2half2_rn(scale);              // exact
  const __half2 zbias2 = __float2half2_rn(__fadd_rn(zf, 1024.0f));  // exact: an integer below 2048
  const unsigned* r = reinterpret_cast<const unsigned*>(raw);
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const float2 w = __half22float2(bits_h2(r[i]));
    const float cx = fminf(fmaxf(__fadd_rn(__fmaf_rn(w.x, inv, kMagic), -kMagic), lo), hi);
    const float cy = fminf(fmaxf(__fadd_rn(__fmaf_rn(w.y, inv, kMagic), -kMagic), lo), hi);
    const __half2 c2 = __floats2half2_rn(cx, cy);  // exact
    wq[i] = h2_bits(__hmul2(c2, scale2));
    code[i] = h2_bits(__hadd2(c2, zbias2));        // 0x6400 + code in each half
  }
}


__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

// Shared memory of a block: per warp two weight buffers (GPW rows x G halves = 2 KB each) and a
// staging area for the ternary packing (1 KB; 256 bytes of 2-bit fields are used); then, only when the clip search has to be repeated, the
// candidate tables of the warps.
constexpr int kApplyWarpBytes = 2 * 2048 + 1024;

template <int G>
__host__ __device__ inline int apply_cand_chunk() {
  return (336 / Map<G>::GPW > 64) ? 64 : 336 / Map<G>::GPW;
}

// n_words packed words of a lane -> dst (4-byte aligned; 8- or 16-byte aligned for 2, 4, 8 words).
__device__ __forceinline__ void store_words(uint8_t* dst, const unsigned (&w)[8], int n_words) {
  switch (n_words) {
    case 8:
      reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
      reinterpret_cast<uint4*>(dst)[1] = make_uint4(w[4], w[5], w[6], w[7]);
      break;
    case 4: reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]); break;
    case 3: {
      unsigned* d = reinterpret_cast<unsigned*>(dst);
      d[0] = w[0]; d[1] = w[1]; d[2] = w[2];
      break;
    }
    case 2: reinterpret_cast<uint2*>(dst)[0] = make_uint2(w[0], w[1]); break;
    default: reinterpret_cast<unsigned*>(dst)[0] = w[0]; break;
  }
}

// SEARCH = false: clip indices are supplied.  SEARCH = true: the clip search is repeated for the
// unit's bit-width (the candidate table follows the warp buffers in shared memory).
// Zero activation weight for the protected values of a lane (bit e of pm = value e = leaf e / 8, position e % 8).
__device__ __forceinline__ void mask_stats(Lane32& sv, unsigned int pm) {
#pragma unroll
  for (int e = 0; e < 32; ++e)
    if ((pm >> e) & 1u) sv.set(e >> 3, e & 7, 0.0f);
}

// What the protected variant needs beside the arguments of the plain one.
struct ProtectArgs {
  const float* scale;              // sqrt(s_j), [C]
  const float* thresh;             // saliency threshold per unit, [U]
  const unsigned int* row_off;     // [U][R] number of protected weights of the unit in the rows before this one
  const long long* prot_offsets;   // [U + 1] start of every unit's INT8 codes
  const __half* prot_scale;        // [U] INT8 scale of the unit's protected weights
  int8_t* prot_q;                  // INT8 codes
  long long capacity;              // entries of prot_q; nothing is written at or beyond it
  const __half* scale_in;          // [4][U][R] refined scales of the uniform groups, or NULL (any variant)
};

// Saliency mask of a lane's 32 values: bit e is set when |w_e| * scale_e >= tau.
__device__ __forceinline__ unsigned int protect_mask(const uint4 (&raw)[4], const float* __restrict__ scale, float tau) {
  const unsigned int* r = reinterpret_cast<const unsigned int*>(raw);
  const float4* a4 = reinterpret_cast<const float4*>(scale);
  unsigned int pm = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float4 a = __ldg(a4 + i);
    const float2 w0 = __half22float2(bits_h2(r[2 * i])), w1 = __half22float2(bits_h2(r[2 * i + 1]));
    pm |= (__fmul_rn(fabsf(w0.x), a.x) >= tau ? 1u : 0u) << (4 * i);
    pm |= (__fmul_rn(fabsf(w0.y), a.y) >= tau ? 1u : 0u) << (4 * i + 1);
    pm |= (__fmul_rn(fabsf(w1.x), a.z) >= tau ? 1u : 0u) << (4 * i + 2);
    pm |= (__fmul_rn(fabsf(w1.y), a.w) >= tau ? 1u : 0u) << (4 * i + 3);
  }
  return pm;
}

// Several plans in one launch (windq_apply_plan_batch): what differs from job to job, by value in the kernel's
// parameters.  Items are numbered through all jobs; job j owns [first_item[j], first_item[j + 1]).
constexpr int kApplyMaxJobs = 24;
struct ApplyJobs {
  const __half* W[kApplyMaxJobs];
  const float* s[kApplyMaxJobs];
  const uint8_t* actions[kApplyMaxJobs];
  const uint8_t* clip_idx[kApplyMaxJobs];
  const long long* code_offsets[kApplyMaxJobs];
  uint8_t* codes[kApplyMaxJobs];
  __half* scales[kApplyMaxJobs];
  __half* zeros[kApplyMaxJobs];
  __half* Wq[kApplyMaxJobs];
  long long ldw[kApplyMaxJobs];
  int R[kApplyMaxJobs];
  int U[kApplyMaxJobs];
  int first_item[kApplyMaxJobs + 1];
  int n;
};

constexpr int kApplyMinBlocks = 4;  // resident blocks per SM the register budget is held to
// PROTECT = true: salient weights (see ProtectArgs) are taken out of the group fits -- zero weight,
// zero activation weight, as in the protected fit -- and kept on one symmetric INT8 grid per unit.
// BATCH: the matrix and the plan of an item are looked up in `jobs` (the scalar parameters that describe one
// matrix are then unused).
template <int G, bool SEARCH, bool PROTECT, bool BATCH>
__global__ void __launch_bounds__(kApplyWarps * 32, kApplyMinBlocks)
apply_plan_kernel(const __half* __restrict__ W_one, int R_one, int U_one, int64_t ldw_one, const float* __restrict__ s_one,
                  const float* __restrict__ clip, int K, const uint8_t* __restrict__ actions_one,
                  const uint8_t* __restrict__ clip_idx_one, const long long* __restrict__ code_offsets_one,
                  uint8_t* __restrict__ codes_one, __half* __restrict__ scales_one, __half* __restrict__ zeros_one,
                  __half* __restrict__ Wq_one, int rows_blocks_one, ProtectArgs pa, const ApplyJobs jobs) {
  constexpr int LG = Map<G>::LG, GPW = Map<G>::GPW;
  extern __shared__ uint4 smem_u4[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane / LG, q = lane % LG;
  uint8_t* mine = reinterpret_cast<uint8_t*>(smem_u4) + (size_t)warp * kApplyWarpBytes;
  uint8_t* trits = mine + 4096;
  // base3[x] = sum over m < 5 of ((x >> 2m) & 3) * 3^m: five 2-bit trits -> one packed byte
  __shared__ uint8_t base3[1024];
  for (int x = threadIdx.x; x < 1024; x += kApplyWarps * 32)
    base3[x] = (uint8_t)((x & 3) + 3 * ((x >> 2) & 3) + 9 * ((x >> 4) & 3) + 27 * ((x >> 6) & 3) + 81 * ((x >> 8) & 3));
  __syncthreads();
  const int chunk = apply_cand_chunk<G>(), stride = chunk | 1;
  Cand* cand = reinterpret_cast<Cand*>(reinterpret_cast<uint8_t*>(smem_u4) + (size_t)kApplyWarps * kApplyWarpBytes) +
               (size_t)warp * GPW * stride;

  const int n_items = BATCH ? jobs.first_item[jobs.n] : U_one * rows_blocks_one;
  const int n_warps = gridDim.x * kApplyWarps;
  int item = blockIdx.x * kApplyWarps + warp;

  // asks for the lane's 64 bytes of `it` into buffer `buf` (rows past the end repeat the last row)
  auto prefetch = [&](int it, int buf) {
    if (it < n_items) {
      const __half* W = W_one;
      int R = R_one, rows_blocks = rows_blocks_one;
      int64_t ldw = ldw_one;
      if (BATCH) {
        int j = 0;
        while (j + 1 < jobs.n && it >= jobs.first_item[j + 1]) ++j;
        W = jobs.W[j];
        R = jobs.R[j];
        ldw = jobs.ldw[j];
        rows_blocks = (R + GPW - 1) / GPW;
        it -= jobs.first_item[j];
      }
      const int u = it / rows_blocks, rb = it - u * rows_blocks;
      const int row = min(rb * GPW + g, R - 1);
      const __half* src = W + (int64_t)row * ldw + (int64_t)u * G + 32 * q;
      uint8_t* dst = mine + buf * 2048 + lane * 64;
#pragma unroll
      for (int i = 0; i < 4; ++i) cp_async16(dst + 16 * i, src + 8 * i);
    }
    cp_async_commit();  // one group per call, possibly empty, so that the wait below counts right
  };

  prefetch(item, 0);
  for (int n = 0; item < n_items; item += n_warps, ++n) {
    prefetch(item + n_warps, (n + 1) & 1);
    cp_async_wait_all_but_one();  // this lane's 64 bytes of the current item have arrived
    const float* s = s_one;
    const uint8_t* actions = actions_one;
    const uint8_t* clip_idx = clip_idx_one;
    const long long* code_offsets = code_offsets_one;
    uint8_t* codes_out = codes_one;
    __half *scales_out = scales_one, *zeros_out = zeros_one, *Wq_out = Wq_one;
    int R = R_one, U = U_one, rows_blocks = rows_blocks_one, local = item;
    int64_t ldw = ldw_one;
    if (BATCH) {
      int j = 0;
      while (j + 1 < jobs.n && item >= jobs.first_item[j + 1]) ++j;
      s = jobs.s[j];
      actions = jobs.actions[j];
      clip_idx = jobs.clip_idx[j];
      code_offsets = jobs.code_offsets[j];
      codes_out = jobs.codes[j];
      scales_out = jobs.scales[j];
      zeros_out = jobs.zeros[j];
      Wq_out = jobs.Wq[j];
      R = jobs.R[j];
      U = jobs.U[j];
      ldw = jobs.ldw[j];
      rows_blocks = (R + GPW - 1) / GPW;
      local = item - jobs.first_item[j];
    }
    const int u = local / rows_blocks, rb = local - u * rows_blocks;
    const int a = actions[u];
    if (a > 6) continue;
    const int row = rb * GPW + g;
    const bool live = row < R;
    const int bpg = group_code_bytes(a, G);
    uint8_t* unit_codes = codes_out + code_offsets[u];
    uint8_t* row_codes = unit_codes + (long long)row * bpg;
    __half* wq_dst = Wq_out ? Wq_out + (int64_t)row * ldw + (int64_t)u * G + 32 * q : nullptr;

    uint4 raw[4];
    {
      const uint4* src = reinterpret_cast<const uint4*>(mine + (n & 1) * 2048 + lane * 64);
#pragma unroll
      for (int i = 0; i < 4; ++i) raw[i] = src[i];
    }
    // the unit's last rows also write the zero padding up to the next 16-byte boundary
    if (rb == rows_blocks - 1) {
      const long long total = (long long)R * bpg;
      const int pad = (int)(((total + 15) & ~15ll) - total);
      if (lane < pad) unit_codes[total + lane] = 0;
    }

    if (a == 0) {  // skip: the raw fp16 values are the codes and the reconstruction
      if (live) {
        uint4* dst = reinterpret_cast<uint4*>(row_codes + 64 * q);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          dst[i] = raw[i];
          if (wq_dst) reinterpret_cast<uint4*>(wq_dst)[i] = raw[i];
        }
        if (q == 0) {
          scales_out[(int64_t)u * R + row] = __ushort_as_half(0);
          zeros_out[(int64_t)u * R + row] = __ushort_as_half(0);
        }
      }
      continue;
    }

    unsigned int pm = 0;  // protected values of this lane
    uint4 raw_all[4];     // the lane's values before masking (PROTECT only)
    if (PROTECT) {
#pragma unroll
      for (int i = 0; i < 4; ++i) raw_all[i] = raw[i];
      pm = protect_mask(raw, pa.scale + (int64_t)u * G + 32 * q, __ldg(pa.thresh + u));
      unsigned int* r = reinterpret_cast<unsigned int*>(raw);
#pragma unroll
      for (int i = 0; i < 16; ++i)
        r[i] &= ~(((pm >> (2 * i)) & 1u ? 0x0000ffffu : 0u) | ((pm >> (2 * i + 1)) & 1u ? 0xffff0000u : 0u));
    }
    unsigned wq[16], code[16];  // two fp16 weights / two codes per register
    float scale_store, zero_store = 0.0f;
    if (a <= 4) {
      const int bi = a - 1;
      const UniformSpec us = uniform_spec(bi);
      float mn, mx;
      int k;
      if (!SEARCH) {
        group_range_h<G>(raw, mn, mx);
        k = min((int)clip_idx[((int64_t)bi * U + u) * R + min(row, R - 1)], K - 1);
      } else {
        Lane32 wv, sv;
        unpack_weights(raw, wv);
        load_stats(s + (int64_t)u * G + 32 * q, sv);
        if (PROTECT) mask_stats(sv, pm);
        group_range<G>(wv, mn, mx);
        float be;
        search_uniform<G>(wv, sv, mn, __fsub_rn(mx, mn), bi, clip, K, cand, chunk, stride, lane, be, k);
      }
      float scale, zf;
      uniform_scale_zero(mn, __fsub_rn(mx, mn), __ldg(clip + k), us, scale, zf);
      if (pa.scale_in) scale = __half2float(pa.scale_in[((int64_t)bi * U + u) * R + min(row, R - 1)]);
      quantise_uniform(raw, scale, zf, us.qmax, wq, code);
      scale_store = scale;
      zero_store = zf;
    } else {
      Lane32 wv, sv;
      unpack_weights(raw, wv);
      load_stats(s + (int64_t)u * G + 32 * q, sv);
      if (PROTECT) mask_stats(sv, pm);
      float delta = 0.0f;
      const float alpha = (a == 5) ? ternary_scale<G>(wv, sv, delta) : binary_scale<G>(wv, sv);
      const unsigned alpha2 = h2_bits(__float2half2_rn(alpha));
      const unsigned* r = reinterpret_cast<const unsigned*>(raw);
      if (a == 5) {
        // |w| > delta, with |w| an fp16 value, is |w| > (delta rounded towards zero to fp16)
        const __half2 delta2 = __half2half2(__float2half_rz(delta));
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const unsigned in = __hgt2_mask(__habs2(bits_h2(r[i])), delta2);  // 0xffff per value on the support
          wq[i] = ((r[i] & 0x80008000u) | alpha2) & in;                      // +-alpha on the support, +0 elsewhere
          const unsigned neg = (r[i] >> 14) & 0x00020002u;
          code[i] = (in & 0x00020002u & ~neg) | (~in & 0x00010001u);         // trit 2, 0 (negative) or 1 (off the support)
        }
      } else {
        const __half2 zero2 = __float2half2_rn(0.0f);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const unsigned neg = __hlt2_mask(bits_h2(r[i]), zero2);  // w < 0 (false for -0)
          wq[i] = (neg & 0x80008000u) | alpha2;
          code[i] = ~neg & 0x00010001u;
        }
      }
      scale_store = alpha;
    }

    if (PROTECT) {
      // place of this lane's INT8 codes: the unit's list, then the rows before, then the lanes before
      const int cnt = __popc(pm);
      int before = cnt;
#pragma unroll
      for (int m = 1; m < LG; m <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, before, m);
        if (q >= m) before += o;
      }
      before -= cnt;
      if (live && pm) {
        const float sigma = __half2float(pa.prot_scale[u]);
        const float inv8 = __frcp_rn(sigma);
        const long long base = pa.prot_offsets[u] + pa.row_off[(int64_t)u * R + row] + before;
        const unsigned int* ro = reinterpret_cast<const unsigned int*>(raw_all);
        int rank = 0;
#pragma unroll
        for (int e = 0; e < 32; ++e)
          if ((pm >> e) & 1u) {
            const float2 w2 = __half22float2(bits_h2(ro[e >> 1]));
            const float w = (e & 1) ? w2.y : w2.x;
            const float c = fminf(fmaxf(__fadd_rn(__fmaf_rn(w, inv8, kMagic), -kMagic), -127.0f), 127.0f);
            const unsigned int h = __half_as_ushort(__float2half_rn(__fmul_rn(c, sigma)));
            wq[e >> 1] = (e & 1) ? ((wq[e >> 1] & 0x0000ffffu) | (h << 16)) : ((wq[e >> 1] & 0xffff0000u) | h);
            if (base + rank < pa.capacity) pa.prot_q[base + rank] = (int8_t)(int)c;
            ++rank;
          }
      }
    }
    if (live) {
      if (wq_dst) {
        uint4* dst = reinterpret_cast<uint4*>(wq_dst);
#pragma unroll
        for (int i = 0; i < 4; ++i) dst[i] = make_uint4(wq[4 * i], wq[4 * i + 1], wq[4 * i + 2], wq[4 * i + 3]);
      }
      if (q == 0) {
        scales_out[(int64_t)u * R + row] = __float2half_rn(scale_store);
        zeros_out[(int64_t)u * R + row] = __float2half_rn(zero_store);
      }
    }
    unsigned words[8];
    if (a != 5) {
      int n_words;
      switch (a) {
        case 1: pack_pairs<8>(code, words); n_words = 8; break;
        case 2: pack_pairs<4>(code, words); n_words = 4; break;
        case 3: pack_pairs<3>(code, words); n_words = 3; break;
        case 4: pack_pairs<2>(code, words); n_words = 2; break;
        default: pack_pairs<1>(code, words); n_words = 1; break;
      }
      if (live) store_words(row_codes + 4 * n_words * q, words, n_words);
    } else {
      // codes as 2-bit fields into the warp's buffer; an output byte is the base-3 value of five
      // consecutive fields, i.e. of a 10-bit window, looked up in the block's table
      pack_pairs<2>(code, words);
      __syncwarp();  // the previous item's fields have been read
      *reinterpret_cast<uint2*>(trits + g * (G / 4) + 8 * q) = make_uint2(words[0], words[1]);
      __syncwarp();
      const int rows_here = min(GPW, R - rb * GPW);
      uint8_t* dst = unit_codes + (long long)rb * GPW * bpg;
      for (int B = lane; B < rows_here * bpg; B += 32) {
        const int rl = B / bpg, bj = B - rl * bpg;
        const uint8_t* t = trits + rl * (G / 4) + ((10 * bj) >> 3);
        unsigned x = ((unsigned)t[0] | ((unsigned)t[1] << 8)) >> ((10 * bj) & 7);
        const int valid = min(5, G - 5 * bj);  // the row's last byte holds fewer than five trits
        x &= (1u << (2 * valid)) - 1u;
        dst[B] = base3[x];
      }
    }
  }
}

template <int G, bool SEARCH, bool PROTECT>
windq_status launch_apply(windq_ctx* ctx, const __half* W, int R, int U, int64_t ldw, const float* s, const float* clip,
                          int K, const uint8_t* actions, const uint8_t* clip_idx, const long long* code_offsets,
                          uint8_t* codes_out, __half* scales_out, __half* zeros_out, __half* Wq_out, const ProtectArgs& pa,
                          cudaStream_t st) {
  constexpr int GPW = Map<G>::GPW;
  const int stride = apply_cand_chunk<G>() | 1;
  const size_t smem = (size_t)kApplyWarps * kApplyWarpBytes + (SEARCH ? (size_t)kApplyWarps * GPW * stride * sizeof(Cand) : 0);
  const int id = (PROTECT ? (SEARCH ? kApplyProtectSearchG32 : kApplyProtectG32) : (SEARCH ? kApplySearchG32 : kApplyG32)) +
                 g_index(G);
  if (windq_status rc = prepare_kernel(ctx, id, apply_plan_kernel<G, SEARCH, PROTECT, false>, kApplyWarps * 32, smem, true)) return rc;
  const int blocks_per_sm = ctx->occupancy[id];
  const int rows_blocks = (R + GPW - 1) / GPW;
  const int64_t n_items = (int64_t)U * rows_blocks;
  WINDQ_REQUIRE(ctx, n_items < (1ll << 30), WINDQ_ERR_SHAPE, "windq_apply_plan: R * C is too large for one call");
  int64_t grid = (int64_t)ctx->sm_count * blocks_per_sm;
  const int64_t need = (n_items + kApplyWarps - 1) / kApplyWarps;
  if (grid > need) grid = need;
  apply_plan_kernel<G, SEARCH, PROTECT, false><<<(unsigned)grid, kApplyWarps * 32, smem, st>>>(
      W, R, U, ldw, s, clip, K, actions, clip_idx, code_offsets, codes_out, scales_out, zeros_out, Wq_out, rows_blocks, pa,
      ApplyJobs());
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

// ---- protected variant: what has to be known before the plan can be applied -----------------------
__global__ void apply_scale_kernel(const float* __restrict__ s, int C, float* __restrict__ scale) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < C) scale[j] = __fsqrt_rn(s[j]);
}

// Per (unit, row): the number of protected weights; per unit: the largest protected magnitude.
// One warp per item (unit, GPW rows), as in the plan kernel.
template <int G>
__global__ void __launch_bounds__(kApplyWarps * 32)
protect_count_kernel(const __half* __restrict__ W, int R, int U, int64_t ldw, const uint8_t* __restrict__ actions,
                     const float* __restrict__ scale, const float* __restrict__ thresh, int rows_blocks,
                     unsigned int* __restrict__ row_cnt, unsigned int* __restrict__ unit_max_bits) {
  constexpr int LG = Map<G>::LG, GPW = Map<G>::GPW;
  const int lane = threadIdx.x & 31;
  const int g = lane / LG, q = lane % LG;
  const int n_items = U * rows_blocks;
  const int n_warps = gridDim.x * kApplyWarps;
  for (int item = blockIdx.x * kApplyWarps + (threadIdx.x >> 5); item < n_items; item += n_warps) {
    const int u = item / rows_blocks, rb = item - u * rows_blocks;
    const int row = rb * GPW + g;
    unsigned int cnt = 0, mx = 0;
    if (actions[u] != 0 && actions[u] <= 6 && row < R) {
      uint4 raw[4];
      const uint4* src = reinterpret_cast<const uint4*>(W + (int64_t)row * ldw + (int64_t)u * G + 32 * q);
#pragma unroll
      for (int i = 0; i < 4; ++i) raw[i] = __ldg(src + i);
      const unsigned int pm = protect_mask(raw, scale + (int64_t)u * G + 32 * q, __ldg(thresh + u));
      cnt = __popc(pm);
      const unsigned int* r = reinterpret_cast<const unsigned int*>(raw);
#pragma unroll
      for (int e = 0; e < 32; ++e)
        if ((pm >> e) & 1u) mx = max(mx, ((e & 1) ? (r[e >> 1] >> 16) : r[e >> 1]) & 0x7fffu);  // |fp16| bits order like values
    }
#pragma unroll
    for (int m = 1; m < LG; m <<= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, m);
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, m));
    if (q == 0 && row < R) row_cnt[(int64_t)u * R + row] = cnt;
    if (lane == 0 && mx) atomicMax(&unit_max_bits[u], mx);
  }
}

// One block per unit: row counts -> exclusive offsets inside the unit (in place), unit total.
__global__ void __launch_bounds__(1024)
protect_row_scan_kernel(unsigned int* __restrict__ row_cnt, int R, unsigned int* __restrict__ unit_total) {
  __shared__ unsigned int warp_sum[32];
  __shared__ unsigned int carry_s;
  const int u = blockIdx.x, t = threadIdx.x, lane = t & 31, wp = t >> 5;
  unsigned int* c = row_cnt + (int64_t)u * R;
  if (t == 0) carry_s = 0;
  __syncthreads();
  for (int base = 0; base < R; base += 1024) {
    const int r = base + t;
    const unsigned int v = r < R ? c[r] : 0u;
    unsigned int incl = v;
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) {
      const unsigned int o = __shfl_up_sync(0xffffffffu, incl, m);
      if (lane >= m) incl += o;
    }
    if (lane == 31) warp_sum[wp] = incl;
    __syncthreads();
    unsigned int before = carry_s;
    for (int i = 0; i < wp; ++i) before += warp_sum[i];
    if (r < R) c[r] = before + incl - v;
    __syncthreads();
    if (t == 1023) carry_s = before + incl;
    __syncthreads();
  }
  if (t == 0) unit_total[u] = carry_s;
}

// Unit totals -> start of every unit's list; largest protected magnitude -> the unit's INT8 scale.
__global__ void protect_unit_scan_kernel(const unsigned int* __restrict__ unit_total, const unsigned int* __restrict__ unit_max_bits,
                                         const uint8_t* __restrict__ actions, int U, long long* __restrict__ prot_offsets,
                                         __half* __restrict__ prot_scale) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    long long run = 0;
    for (int u = 0; u < U; ++u) {
      prot_offsets[u] = run;
      run += unit_total[u];
    }
    prot_offsets[U] = run;
  }
  for (int u = blockIdx.x * blockDim.x + threadIdx.x; u < U; u += gridDim.x * blockDim.x) {
    float sigma = 0.0f;
    if (actions[u] != 0 && actions[u] <= 6) {
      const float m = __half2float(__ushort_as_half((unsigned short)unit_max_bits[u]));
      sigma = __half2float(__float2half_rn(__fdiv_rn(m, 127.0f)));
      if (sigma == 0.0f) sigma = 1.0f;
    }
    prot_scale[u] = __float2half_rn(sigma);
  }
}

template <int G>
windq_status launch_apply_any(windq_ctx* ctx, const __half* W, int R, int U, int64_t ldw, const float* s,
                              const float* clip, int K, const uint8_t* actions, const uint8_t* clip_idx,
                              const long long* code_offsets, uint8_t* codes_out, __half* scales_out, __half* zeros_out,
                              __half* Wq_out, const __half* scale_in, cudaStream_t st) {
  ProtectArgs none = {};
  none.scale_in = scale_in;
  if (clip_idx)
    return launch_apply<G, false, false>(ctx, W, R, U, ldw, s, clip, K, actions, clip_idx, code_offsets, codes_out,
                                         scales_out, zeros_out, Wq_out, none, st);
  return launch_apply<G, true, false>(ctx, W, R, U, ldw, s, clip, K, actions, clip_idx, code_offsets, codes_out, scales_out,
                                      zeros_out, Wq_out, none, st);
}

template <int G>
windq_status launch_apply_protected(windq_ctx* ctx, const __half* W, int R, int U, int64_t ldw, const float* s,
                                    const float* clip, int K, const uint8_t* actions, const uint8_t* clip_idx,
                                    const long long* code_offsets, const float* thresh, uint8_t* codes_out,
                                    __half* scales_out, __half* zeros_out, __half* Wq_out, __half* prot_scale_out,
                                    long long* prot_offsets_out, int8_t* prot_q_out, long long capacity,
                                    const __half* scale_in, cudaStream_t st) {
  constexpr int GPW = Map<G>::GPW;
  const int C = U * G;
  // scratch: sqrt(s) [C] | row counts / offsets [U][R] | unit totals [U] | unit maxima [U]
  float* scale = (float*)ctx->scratch;
  unsigned int* row_cnt = (unsigned int*)((char*)ctx->scratch + round_up((int64_t)C * 4, 16));
  unsigned int* unit_total = row_cnt + (int64_t)U * R;
  unsigned int* unit_max = unit_total + U;
  const int rows_blocks = (R + GPW - 1) / GPW;
  const int64_t n_items = (int64_t)U * rows_blocks;
  WINDQ_REQUIRE(ctx, n_items < (1ll << 30), WINDQ_ERR_SHAPE, "windq_apply_plan_protected: R * C is too large for one call");
  int64_t grid = (int64_t)ctx->sm_count * 8;
  const int64_t need = (n_items + kApplyWarps - 1) / kApplyWarps;
  if (grid > need) grid = need;
  WINDQ_CUDA(ctx, cudaMemsetAsync(unit_max, 0, (size_t)U * sizeof(unsigned int), st));
  apply_scale_kernel<<<(unsigned)((C + 255) / 256), 256, 0, st>>>(s, C, scale);
  protect_count_kernel<G><<<(unsigned)grid, kApplyWarps * 32, 0, st>>>(W, R, U, ldw, actions, scale, thresh, rows_blocks, row_cnt,
                                                                      unit_max);
  protect_row_scan_kernel<<<(unsigned)U, 1024, 0, st>>>(row_cnt, R, unit_total);
  protect_unit_scan_kernel<<<(unsigned)((U + 255) / 256), 256, 0, st>>>(unit_total, unit_max, actions, U, prot_offsets_out,
                                                                       prot_scale_out);
  WINDQ_CUDA(ctx, cudaGetLastError());
  const ProtectArgs pa = {scale, thresh, row_cnt, prot_offsets_out, prot_scale_out, prot_q_out, capacity, scale_in};
  if (clip_idx)
    return launch_apply<G, false, true>(ctx, W, R, U, ldw, s, clip, K, actions, clip_idx, code_offsets, codes_out, scales_out,
                                        zeros_out, Wq_out, pa, st);
  return launch_apply<G, true, true>(ctx, W, R, U, ldw, s, clip, K, actions, clip_idx, code_offsets, codes_out, scales_out,
                                     zeros_out, Wq_out, pa, st);
}

}  // namespace windq

static windq_status apply_plan_plain(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                                     const float* clip_grid, int K, const uint8_t* actions, const uint8_t* clip_idx,
                                     const void* scale_in, const int64_t* code_offsets, uint8_t* codes_out,
                                     void* scales_out, void* zeros_out, void* Wq_out, void* stream) {
  using namespace windq;
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
  if (clip_idx) {  // clip indices supplied: the streaming kernel
    const windq_plan_out pl = {actions, code_offsets, codes_out, scales_out, zeros_out, Wq_out};
    return launch_apply_stream(ctx, G, W, R, C, ldw, s, clip_grid, K, clip_idx, scale_in, nullptr, 0, nullptr, nullptr, &pl, 1, st);
  }
  const __half* Wh = (const __half*)W;
  const long long* offs = (const long long*)code_offsets;
  __half *sc = (__half*)scales_out, *zp = (__half*)zeros_out, *wq = (__half*)Wq_out;
  const __half* si = (const __half*)scale_in;
  switch (G) {
    case 32: return launch_apply_any<32>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, actions, clip_idx, offs, codes_out, sc, zp, wq, si, st);
    case 64: return launch_apply_any<64>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, actions, clip_idx, offs, codes_out, sc, zp, wq, si, st);
    case 128: return launch_apply_any<128>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, actions, clip_idx, offs, codes_out, sc, zp, wq, si, st);
    case 256: return launch_apply_any<256>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, actions, clip_idx, offs, codes_out, sc, zp, wq, si, st);
    default: return launch_apply_any<512>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, actions, clip_idx, offs, codes_out, sc, zp, wq, si, st);
  }
}

extern "C" windq_status windq_apply_plan(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                         const float* s, const float* clip_grid, int K, const uint8_t* actions,
                                         const uint8_t* clip_idx, const int64_t* code_offsets, uint8_t* codes_out,
                                         void* scales_out, void* zeros_out, void* Wq_out, void* stream) {
  if (!ctx) return windq::fail(nullptr, WINDQ_ERR_NULL, "windq_apply_plan: ctx is NULL");
  return apply_plan_plain(ctx, W, R, C, ldw, G, s, clip_grid, K, actions, clip_idx, nullptr, code_offsets, codes_out,
                          scales_out, zeros_out, Wq_out, stream);
}

extern "C" windq_status windq_apply_plan_refined(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                                 const float* s, const float* clip_grid, int K, const uint8_t* actions,
                                                 const uint8_t* clip_idx, const void* scale_in, const int64_t* code_offsets,
                                                 uint8_t* codes_out, void* scales_out, void* zeros_out, void* Wq_out,
                                                 void* stream) {
  if (!ctx) return windq::fail(nullptr, WINDQ_ERR_NULL, "windq_apply_plan_refined: ctx is NULL");
  if (!clip_idx || !scale_in)
    return windq::fail(ctx, WINDQ_ERR_NULL, "windq_apply_plan_refined: clip_idx or scale_in is NULL");
  if ((uintptr_t)scale_in & 1) return windq::fail(ctx, WINDQ_ERR_ALIGN, "windq_apply_plan_refined: scale_in is misaligned");
  return apply_plan_plain(ctx, W, R, C, ldw, G, s, clip_grid, K, actions, clip_idx, scale_in, code_offsets, codes_out,
                          scales_out, zeros_out, Wq_out, stream);
}

extern "C" int64_t windq_scratch_bytes_apply_plan_protected(int64_t R, int64_t C, int G) {
  if (!windq::valid_G(G) || R <= 0 || C <= 0) return 0;
  const int64_t U = C / G;
  return windq::round_up(C * 4, 16) + (U * R + 2 * U) * (int64_t)sizeof(unsigned int);
}

static windq_status apply_plan_protected_any(windq_ctx* ctx, const char* who, const void* W, int64_t R, int64_t C, int64_t ldw,
                                             int G, const float* s, const float* clip_grid, int K, const uint8_t* actions,
                                             const uint8_t* clip_idx, const void* scale_in, const int64_t* code_offsets,
                                             const float* thresh, uint8_t* codes_out, void* scales_out, void* zeros_out,
                                             void* Wq_out, void* prot_scale_out, int64_t* prot_offsets_out,
                                             int8_t* prot_q_out, int64_t prot_q_capacity, void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "%s: ctx is NULL", who);
  if (windq_status st = check_matrix(ctx, who, W, R, C, ldw, G)) return st;
  if (windq_status st = check_K(ctx, who, K)) return st;
  WINDQ_REQUIRE(ctx, s && clip_grid && actions && code_offsets && codes_out && scales_out && zeros_out && thresh &&
                         prot_scale_out && prot_offsets_out && (prot_q_out || prot_q_capacity == 0),
                WINDQ_ERR_NULL, "%s: a required pointer is NULL", who);
  WINDQ_REQUIRE(ctx, prot_q_capacity >= 0, WINDQ_ERR_ARG, "%s: prot_q_capacity = %lld", who, (long long)prot_q_capacity);
  WINDQ_REQUIRE(ctx, aligned16(s) && aligned16(codes_out), WINDQ_ERR_ALIGN, "%s: s or codes_out is not 16-byte aligned", who);
  WINDQ_REQUIRE(ctx, ((uintptr_t)code_offsets & 7) == 0 && ((uintptr_t)prot_offsets_out & 7) == 0 && ((uintptr_t)scales_out & 1) == 0 &&
                         ((uintptr_t)zeros_out & 1) == 0 && ((uintptr_t)prot_scale_out & 1) == 0,
                WINDQ_ERR_ALIGN, "%s: an output array is misaligned", who);
  WINDQ_REQUIRE(ctx, Wq_out == nullptr || aligned16(Wq_out), WINDQ_ERR_ALIGN, "%s: Wq_out is not 16-byte aligned", who);
  WINDQ_REQUIRE(ctx, Wq_out != W, WINDQ_ERR_ARG, "%s: Wq_out must not alias W", who);
  WINDQ_REQUIRE(ctx, R * (int64_t)G < (1ll << 32), WINDQ_ERR_SHAPE, "%s: R * G must be below 2^32", who);
  DeviceGuard guard(ctx->device);
  if (windq_status rc = ensure_scratch(ctx, windq_scratch_bytes_apply_plan_protected(R, C, G))) return rc;
  const int U = (int)(C / G);
  cudaStream_t st = (cudaStream_t)stream;
  const __half* Wh = (const __half*)W;
  const long long* offs = (const long long*)code_offsets;
  __half *sc = (__half*)scales_out, *zp = (__half*)zeros_out, *wq = (__half*)Wq_out, *ps = (__half*)prot_scale_out;
  long long* po = (long long*)prot_offsets_out;
#define WINDQ_APPLY_CASE(GG)                                                                                             \
  case GG:                                                                                                               \
    return launch_apply_protected<GG>(ctx, Wh, (int)R, U, ldw, s, clip_grid, K, actions, clip_idx, offs, thresh, codes_out, \
                                      sc, zp, wq, ps, po, prot_q_out, (long long)prot_q_capacity, (const __half*)scale_in, st);
  switch (G) {
    WINDQ_APPLY_CASE(32)
    WINDQ_APPLY_CASE(64)
    WINDQ_APPLY_CASE(128)
    WINDQ_APPLY_CASE(256)
    default:
      WINDQ_APPLY_CASE(512)
  }
#undef WINDQ_APPLY_CASE
}

extern "C" windq_status windq_apply_plan_protected(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                                   const float* s, const float* clip_grid, int K, const uint8_t* actions,
                                                   const uint8_t* clip_idx, const int64_t* code_offsets, const float* thresh,
                                                   uint8_t* codes_out, void* scales_out, void* zeros_out, void* Wq_out,
                                                   void* prot_scale_out, int64_t* prot_offsets_out, int8_t* prot_q_out,
                                                   int64_t prot_q_capacity, void* stream) {
  return apply_plan_protected_any(ctx, "windq_apply_plan_protected", W, R, C, ldw, G, s, clip_grid, K, actions, clip_idx,
                                  nullptr, code_offsets, thresh, codes_out, scales_out, zeros_out, Wq_out, prot_scale_out,
                                  prot_offsets_out, prot_q_out, prot_q_capacity, stream);
}

extern "C" windq_status windq_apply_plan_protected_refined(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                                                           int G, const float* s, const float* clip_grid, int K,
                                                           const uint8_t* actions, const uint8_t* clip_idx,
                                                           const void* scale_in, const int64_t* code_offsets,
                                                           const float* thresh, uint8_t* codes_out, void* scales_out,
                                                           void* zeros_out, void* Wq_out, void* prot_scale_out,
                                                           int64_t* prot_offsets_out, int8_t* prot_q_out,
                                                           int64_t prot_q_capacity, void* stream) {
  const char* who = "windq_apply_plan_protected_refined";
  if (!ctx) return windq::fail(nullptr, WINDQ_ERR_NULL, "%s: ctx is NULL", who);
  if (!clip_idx || !scale_in) return windq::fail(ctx, WINDQ_ERR_NULL, "%s: clip_idx or scale_in is NULL", who);
  if ((uintptr_t)scale_in & 1) return windq::fail(ctx, WINDQ_ERR_ALIGN, "%s: scale_in is misaligned", who);
  return apply_plan_protected_any(ctx, who, W, R, C, ldw, G, s, clip_grid, K, actions, clip_idx, scale_in, code_offsets, thresh,
                                  codes_out, scales_out, zeros_out, Wq_out, prot_scale_out, prot_offsets_out, prot_q_out,
                                  prot_q_capacity, stream);
}

namespace windq {

template <int G>
windq_status launch_apply_batch(windq_ctx* ctx, const ApplyJobs& jobs, const float* clip, int K, cudaStream_t st) {
  const size_t smem = (size_t)kApplyWarps * kApplyWarpBytes;
  const int id = kApplyBatchG32 + g_index(G);
  if (windq_status rc = prepare_kernel(ctx, id, apply_plan_kernel<G, false, false, true>, kApplyWarps * 32, smem, true)) return rc;
  int64_t grid = (int64_t)ctx->sm_count * ctx->occupancy[id];
  const int64_t need = ((int64_t)jobs.first_item[jobs.n] + kApplyWarps - 1) / kApplyWarps;
  if (grid > need) grid = need;
  apply_plan_kernel<G, false, false, true><<<(unsigned)grid, kApplyWarps * 32, smem, st>>>(
      nullptr, 0, 0, 0, nullptr, clip, K, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, ProtectArgs(), jobs);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

}  // namespace windq

extern "C" windq_status windq_apply_plan_batch(windq_ctx* ctx, const windq_apply_job* jobs, int n_jobs, int G,
                                               const float* clip_grid, int K, void* stream) {
  using namespace windq;
  const char* who = "windq_apply_plan_batch";
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "%s: ctx is NULL", who);
  WINDQ_REQUIRE(ctx, jobs && clip_grid, WINDQ_ERR_NULL, "%s: jobs or clip_grid is NULL", who);
  WINDQ_REQUIRE(ctx, n_jobs >= 1 && n_jobs <= kApplyMaxJobs, WINDQ_ERR_SHAPE, "%s: n_jobs = %d is outside [1, %d]", who, n_jobs,
                kApplyMaxJobs);
  if (windq_status st = check_K(ctx, who, K)) return st;
  ApplyJobs aj;
  memset(&aj, 0, sizeof(aj));
  aj.n = n_jobs;
  int64_t items = 0;
  const int gpw = 32 / (G > 0 ? (G / 32 > 0 ? G / 32 : 1) : 1);
  for (int j = 0; j < n_jobs; ++j) {
    const windq_apply_job& b = jobs[j];
    if (windq_status st = check_matrix(ctx, who, b.W, b.R, b.C, b.ldw, G)) return st;
    WINDQ_REQUIRE(ctx, b.s && b.actions && b.clip_idx && b.code_offsets && b.codes_out && b.scales_out && b.zeros_out,
                  WINDQ_ERR_NULL, "%s: job %d: a required pointer is NULL (clip_idx is required in a batch)", who, j);
    WINDQ_REQUIRE(ctx, aligned16(b.s) && aligned16(b.codes_out), WINDQ_ERR_ALIGN, "%s: job %d: s or codes_out is not 16-byte aligned",
                  who, j);
    WINDQ_REQUIRE(ctx, ((uintptr_t)b.code_offsets & 7) == 0 && ((uintptr_t)b.scales_out & 1) == 0 && ((uintptr_t)b.zeros_out & 1) == 0,
                  WINDQ_ERR_ALIGN, "%s: job %d: code_offsets, scales_out or zeros_out is misaligned", who, j);
    WINDQ_REQUIRE(ctx, b.Wq_out == nullptr || aligned16(b.Wq_out), WINDQ_ERR_ALIGN, "%s: job %d: Wq_out is not 16-byte aligned", who, j);
    WINDQ_REQUIRE(ctx, b.Wq_out != b.W, WINDQ_ERR_ARG, "%s: job %d: Wq_out must not alias W", who, j);
    aj.W[j] = (const __half*)b.W;
    aj.s[j] = b.s;
    aj.actions[j] = b.actions;
    aj.clip_idx[j] = b.clip_idx;
    aj.code_offsets[j] = (const long long*)b.code_offsets;
    aj.codes[j] = b.codes_out;
    aj.scales[j] = (__half*)b.scales_out;
    aj.zeros[j] = (__half*)b.zeros_out;
    aj.Wq[j] = (__half*)b.Wq_out;
    aj.ldw[j] = b.ldw;
    aj.R[j] = (int)b.R;
    aj.U[j] = (int)(b.C / G);
    aj.first_item[j] = (int)items;
    items += (b.C / G) * ((b.R + gpw - 1) / gpw);
    WINDQ_REQUIRE(ctx, items < (1ll << 30), WINDQ_ERR_SHAPE, "%s: the batch is too large for one call", who);
  }
  aj.first_item[n_jobs] = (int)items;
  DeviceGuard guard(ctx->device);
  cudaStream_t st = (cudaStream_t)stream;
  switch (G) {
    case 32: return launch_apply_batch<32>(ctx, aj, clip_grid, K, st);
    case 64: return launch_apply_batch<64>(ctx, aj, clip_grid, K, st);
    case 128: return launch_apply_batch<128>(ctx, aj, clip_grid, K, st);
    case 256: return launch_apply_batch<256>(ctx, aj, clip_grid, K, st);
    default: return launch_apply_batch<512>(ctx, aj, clip_grid, K, st);
  }
}

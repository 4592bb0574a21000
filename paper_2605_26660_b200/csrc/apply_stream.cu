// Plan application with supplied clip indices, as a streaming kernel: windq_apply_plan (clip indices given),
// windq_apply_plan_refined, windq_apply_plan_searched and windq_apply_plan_multi (up to four plans of one
// matrix in one pass over its weights).
//
// Bound by HBM: per weight 2 bytes read once, and per plan 2 bytes of fake-quantised output, bits / 8 bytes of
// codes and 5 bytes per group (clip index in, scale and zero point out).  What decides the speed of such a kernel
// is the shape of its memory instructions and how much traffic each SM keeps in flight:
//   * lanes of a group are interleaved by 16-byte chunks: lane q of the LG = G / 32 lanes that own a row takes the
//     chunks q, q + LG, q + 2 LG, q + 3 LG of the row's G / 8 chunks (8 values each), so that every load and
//     store instruction of the warp covers whole 32-byte sectors (measured on B200: a lane that owns 64
//     contiguous bytes touches half a sector per instruction and the same copy runs at 0.7 of the speed);
//   * packed codes are collected per item in a shared-memory staging area and leave with contiguous 16-byte
//     stores (the rows of an item are adjacent in the output);
//   * a lane holds no more than 16 of its 32 values in registers at a time (the item's weights stay in the
//     warp's shared-memory buffer and each half is quantised, stored and packed before the next is read), which
//     keeps the kernel at 64 registers: 32 warps per SM;
//   * the weights of the warp's next item are already on their way (cp.async, two 2 KB buffers per warp), and
//     with them everything else the next item will need from global memory -- the plans' action codes and block
//     offsets (one lane per plan) and the clip indices of the item's rows for all four bit-widths (one byte per
//     lane) -- so that no load of the current item depends on another load of the current item;
//   * the clip ratios, the threshold ratios and the base-3 table sit in shared memory.
// Arithmetic is that of the fit (fit_device.cuh): a chunk is one leaf of the PSUM8 order, leaf sums are added
// adjacent leaves first (across the lanes of a group inside every chunk slot, then over the four slots of a
// lane), and every value that is stored is a fixed sequence of binary32 / binary16 operations.
#include <string.h>

#include "fit_device.cuh"

namespace windq {

constexpr int kStreamWarps = 4;
constexpr int kStreamMaxPlans = 4;
constexpr int kStreamStage = 1024 + 32;                       // packed codes of one item (at most 1 KB) + slack for the ternary window read
constexpr int kStreamWarpBytes = 2 * 2048 + kStreamStage;     // two weight buffers, then the staging area

struct StreamPlan {
  const uint8_t* actions;        // [U]
  const long long* code_offsets;  // [U + 1]
  uint8_t* codes;
  __half* scales;  // [U][R]
  __half* zeros;   // [U][R]
  __half* Wq;      // [R][ldw] or NULL
};

struct StreamArgs {
  const __half* W;
  const float* s;
  const float* clip;         // [K]
  const uint8_t* clip_idx;   // [4][U][R]
  const __half* scale_in;    // [4][U][R] or NULL: refined scales of the uniform groups
  const float* thr_grid;     // [thr_K] or NULL: threshold ratios of the ternary search
  const uint8_t* thr_idx;    // [U][R] or NULL
  const __half* lowbit;      // [3][U][R] or NULL: 1.58-bit scale, 1-bit scale, 1.58-bit threshold, as the fit left them
  long long ldw;
  int R, U, K, thr_K, rows_blocks, n_plans;
  StreamPlan plan[kStreamMaxPlans];
};

__device__ __forceinline__ unsigned sh2_bits(__half2 h) { return *reinterpret_cast<unsigned*>(&h); }
__device__ __forceinline__ __half2 sbits_h2(unsigned u) { return *reinterpret_cast<__half2*>(&u); }

__device__ __forceinline__ void stream_cp16(void* smem_dst, const void* gmem_src) {
  const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void stream_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void stream_wait_all_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

// What a lane fetched ahead for an item, beside the weights.
struct ItemMeta {
  unsigned act;    // lane p < n_plans: action code of the item's unit under plan p
  long long off;   // lane p < n_plans: byte offset of the unit's block under plan p
  unsigned clip;   // byte b (b = q, q + LG, ... < 4): clip index of this lane's row for bit-width column b
  unsigned thr;    // lanes with q == 0: threshold index of this lane's row (ternary search), else unused
};

// Chunk slot i (0..3) of lane q is chunk q + LG * i of the row: values 8 * (q + LG * i) .. + 7.
template <int G>
__device__ __forceinline__ int chunk_of(int q, int i) { return q + Map<G>::LG * i; }

// Leaf sums t[i] of the lane's four chunk slots -> PSUM8 total of the group: adjacent leaves first, which is
// the lanes of the group inside every slot (xor 1, 2, ...), then the slots (0 + 1) + (2 + 3).
template <int G>
__device__ __forceinline__ float slots_tree(float t0, float t1, float t2, float t3) {
#pragma unroll
  for (int m = 1; m < Map<G>::LG; m <<= 1) {
    t0 = __fadd_rn(t0, __shfl_xor_sync(0xffffffffu, t0, m));
    t1 = __fadd_rn(t1, __shfl_xor_sync(0xffffffffu, t1, m));
    t2 = __fadd_rn(t2, __shfl_xor_sync(0xffffffffu, t2, m));
    t3 = __fadd_rn(t3, __shfl_xor_sync(0xffffffffu, t3, m));
  }
  return __fadd_rn(__fadd_rn(t0, t1), __fadd_rn(t2, t3));
}

// Layout of a warp's 2 KB weight buffer: chunk slot i of lane l at byte (32 i + l) * 16, so that the 32 lanes of a
// cp.async or of a 128-bit shared load touch 512 contiguous bytes (no bank conflicts; with 64 contiguous bytes per
// lane every such access is a four-way conflict).  `lane_buf` points at the lane's slot 0; slot i is 512 i further.
__device__ __forceinline__ uint4 load_slot(const uint8_t* lane_buf, int i) {
  return *reinterpret_cast<const uint4*>(lane_buf + 512 * i);
}

// The eight registers of half H (chunk slots 2H and 2H + 1) of the lane's values.
__device__ __forceinline__ void load_half(const uint8_t* lane_buf, int H, unsigned (&r)[8]) {
  const uint4 a = load_slot(lane_buf, 2 * H), b = load_slot(lane_buf, 2 * H + 1);
  r[0] = a.x; r[1] = a.y; r[2] = a.z; r[3] = a.w;
  r[4] = b.x; r[5] = b.y; r[6] = b.z; r[7] = b.w;
}

__device__ __forceinline__ void load_stats8(const float* __restrict__ s_unit, int c, float (&sv)[8]) {
  const float4* s4 = reinterpret_cast<const float4*>(s_unit + 8 * c);
  const float4 a = __ldg(s4), b = __ldg(s4 + 1);
  sv[0] = a.x; sv[1] = a.y; sv[2] = a.z; sv[3] = a.w;
  sv[4] = b.x; sv[5] = b.y; sv[6] = b.z; sv[7] = b.w;
}

// Eight codes (two per register, one in the low bits of each 16-bit half, anything above the low BITS bits
// ignored) -> the chunk's 8 * BITS packed bits, little-endian.
template <int BITS>
__device__ __forceinline__ unsigned long long pack_chunk(const unsigned* p) {
  constexpr unsigned mask = (1u << BITS) - 1u;
  if (BITS <= 4) {
    // the two codes of a register side by side, then the four registers Horner-fashion (integer multiply-adds)
    unsigned f[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const unsigned m = p[j] & (mask | (mask << 16));
      f[j] = (m | (m >> (16 - BITS))) & ((1u << (2 * BITS)) - 1u);
    }
    constexpr unsigned step = 1u << (2 * BITS);
    return ((f[3] * step + f[2]) * step + f[1]) * step + f[0];
  }
  const unsigned lo = (p[0] & mask) | (((p[0] >> 16) & mask) << 8) | ((p[1] & mask) << 16) | (((p[1] >> 16) & mask) << 24);
  const unsigned hi = (p[2] & mask) | (((p[2] >> 16) & mask) << 8) | ((p[3] & mask) << 16) | (((p[3] >> 16) & mask) << 24);
  return ((unsigned long long)hi << 32) | lo;
}

// The chunk's packed bits to their place in the staged row (stage_row = start of the row's packed bytes).
template <int BITS>
__device__ __forceinline__ void stage_chunk(uint8_t* stage_row, int c, unsigned long long v) {
  if (BITS == 8) {
    *reinterpret_cast<uint2*>(stage_row + 8 * c) = make_uint2((unsigned)v, (unsigned)(v >> 32));
  } else if (BITS == 4) {
    *reinterpret_cast<unsigned*>(stage_row + 4 * c) = (unsigned)v;
  } else if (BITS == 3) {
    stage_row[3 * c] = (uint8_t)v;
    stage_row[3 * c + 1] = (uint8_t)(v >> 8);
    stage_row[3 * c + 2] = (uint8_t)(v >> 16);
  } else if (BITS == 2) {
    *reinterpret_cast<unsigned short*>(stage_row + 2 * c) = (unsigned short)v;
  } else {
    stage_row[c] = (uint8_t)v;
  }
}

// The item's staged packed bytes -> global memory, contiguous (the rows of an item are adjacent in the output).
__device__ __forceinline__ void copy_out(const uint8_t* stage, uint8_t* dst, int n_bytes, int lane) {
  if ((n_bytes & 15) == 0) {
    for (int i = lane; i < (n_bytes >> 4); i += 32) reinterpret_cast<uint4*>(dst)[i] = reinterpret_cast<const uint4*>(stage)[i];
  } else {  // a last, shorter item: rows are whole words
    for (int i = lane; i < (n_bytes >> 2); i += 32) reinterpret_cast<unsigned*>(dst)[i] = reinterpret_cast<const unsigned*>(stage)[i];
  }
}

// min(0, min w) and max(0, max w) over the group, compared as fp16 values (exact), two per instruction.
template <int G>
__device__ __forceinline__ void stream_range(const uint8_t* lane_buf, float& mn, float& mx) {
  __half2 lo2, hi2;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint4 v = load_slot(lane_buf, i);
    const unsigned r[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (i == 0 && k == 0) {
        lo2 = sbits_h2(r[0]);
        hi2 = lo2;
      } else {
        lo2 = __hmin2(lo2, sbits_h2(r[k]));
        hi2 = __hmax2(hi2, sbits_h2(r[k]));
      }
    }
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

// Uniform grid with known parameters: fake-quantised weights stored, codes packed and staged.  The centred code
// c = clamp(rne(w / scale), lo, hi) is formed in binary32 exactly as in the fit; being an integer of at most 8
// bits it is exact in fp16, so the stored weight fp16(c * scale) is one half-precision product (scale is an fp16
// value: the product is rounded once either way) and the code c + z comes out of a half-precision add of
// z + 1024, whose low bits are the integer.
template <int G, int BITS>
__device__ __forceinline__ void stream_uniform(const uint8_t* lane_buf, int q, float scale, float zf, float qmax,
                                               __half* wq_row /* NULL: no store */, uint8_t* stage_row) {
  const float inv = __frcp_rn(scale);
  const float2 inv2 = make_float2(inv, inv);
  const float2 magic2 = make_float2(kMagic, kMagic), nmagic2 = make_float2(-kMagic, -kMagic);
  // The clamp is taken on the fp16 copies, two values per instruction.  rne(w / scale) is an integer of magnitude
  // at most 255 * 64 (clip ratios are at least 1/64), far below the fp16 limit; the conversion to fp16 is exact
  // up to 2048 and monotone beyond, and the bounds lo = -z and hi = qmax - z are fp16 integers of magnitude at
  // most 255, so clamp(fp16(x)) = clamp(x) for every such x.
  const __half2 lo2 = __float2half2_rn(__fsub_rn(0.0f, zf)), hi2 = __float2half2_rn(__fsub_rn(qmax, zf));
  const __half2 scale2 = __float2half2_rn(scale);                   // exact
  const __half2 zbias2 = __float2half2_rn(__fadd_rn(zf, 1024.0f));  // exact: an integer below 2048
#pragma unroll
  for (int H = 0; H < 2; ++H) {
    unsigned r[8], wq[8], code[8];
    load_half(lane_buf, H, r);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float2 w = __half22float2(sbits_h2(r[i]));
      const float2 x = add2(fma2(w, inv2, magic2), nmagic2);
      const __half2 c2 = __hmin2(__hmax2(__floats2half2_rn(x.x, x.y), lo2), hi2);
      wq[i] = sh2_bits(__hmul2(c2, scale2));
      code[i] = sh2_bits(__hadd2(c2, zbias2));         // 0x6400 + code in each half
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int c = chunk_of<G>(q, 2 * H + j);
      if (wq_row) *reinterpret_cast<uint4*>(wq_row + 8 * c) = make_uint4(wq[4 * j], wq[4 * j + 1], wq[4 * j + 2], wq[4 * j + 3]);
      stage_chunk<BITS>(stage_row, c, pack_chunk<BITS>(code + 4 * j));
    }
  }
}

// PSUM8 of |w| over the group.  (The sums below walk the lane's chunks half by half in a loop that is NOT
// unrolled, two chunks and their 16 statistics in registers at a time, to stay within the register budget.)
template <int G>
__device__ __forceinline__ float stream_abs_sum(const uint8_t* lane_buf) {
  float t0 = 0.0f, t1 = 0.0f, t2 = 0.0f, t3 = 0.0f;
#pragma unroll 1
  for (int H = 0; H < 2; ++H) {
    unsigned r[8];
    load_half(lane_buf, H, r);
    float leaf[2];
#pragma unroll
    for (int l = 0; l < 2; ++l) {
      float a = 0.0f;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float2 f = __half22float2(__habs2(sbits_h2(r[4 * l + k])));
        a = __fadd_rn(a, f.x);
        a = __fadd_rn(a, f.y);
      }
      leaf[l] = a;
    }
    if (H == 0) { t0 = leaf[0]; t1 = leaf[1]; }
    else { t2 = leaf[0]; t3 = leaf[1]; }
  }
  return slots_tree<G>(t0, t1, t2, t3);
}

// The 1-bit scale of fit_low_bits -- the same operations in the same order -- from the lane's buffer and the
// unit's statistics.  Must be called by all 32 lanes.
template <int G>
__device__ __forceinline__ float stream_binary_scale(const uint8_t* lane_buf, const float* __restrict__ s_unit, int q) {
  float S0 = 0.0f, S1 = 0.0f, S2 = 0.0f, S3 = 0.0f, B0 = 0.0f, B1 = 0.0f, B2 = 0.0f, B3 = 0.0f;
#pragma unroll 1
  for (int H = 0; H < 2; ++H) {
    unsigned r[8];
    load_half(lane_buf, H, r);
    float Sb[2], Bb[2];
#pragma unroll
    for (int l = 0; l < 2; ++l) {
      float sv[8];
      load_stats8(s_unit, chunk_of<G>(q, 2 * H + l), sv);
      float sb = 0.0f, bb = 0.0f;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float2 f = __half22float2(__habs2(sbits_h2(r[4 * l + k])));
        sb = __fadd_rn(sb, sv[2 * k]);
        bb = __fmaf_rn(sv[2 * k], f.x, bb);
        sb = __fadd_rn(sb, sv[2 * k + 1]);
        bb = __fmaf_rn(sv[2 * k + 1], f.y, bb);
      }
      Sb[l] = sb; Bb[l] = bb;
    }
    if (H == 0) { S0 = Sb[0]; S1 = Sb[1]; B0 = Bb[0]; B1 = Bb[1]; }
    else { S2 = Sb[0]; S3 = Sb[1]; B2 = Bb[0]; B3 = Bb[1]; }
  }
  const float sumS = slots_tree<G>(S0, S1, S2, S3), sumB = slots_tree<G>(B0, B1, B2, B3);
  float meanA = 0.0f;
  if (__any_sync(0xffffffffu, sumS == 0.0f)) meanA = __fmul_rn(stream_abs_sum<G>(lane_buf), 1.0f / (float)G);
  return __half2float(__float2half_rn(sumS == 0.0f ? meanA : __fdiv_rn(sumB, sumS)));
}

// The ternary scale for the threshold delta = ratio * mean |w| (0 when the support is empty).
template <int G>
__device__ __forceinline__ float stream_ternary_scale(const uint8_t* lane_buf, const float* __restrict__ s_unit, int q, float ratio,
                                                      float& delta) {
  const float sumA = stream_abs_sum<G>(lane_buf);
  delta = __fmul_rn(ratio, __fmul_rn(sumA, 1.0f / (float)G));
  const float dl = delta;
  float B0 = 0.0f, B1 = 0.0f, B2 = 0.0f, B3 = 0.0f, C0 = 0.0f, C1 = 0.0f, C2 = 0.0f, C3 = 0.0f;
#pragma unroll 1
  for (int H = 0; H < 2; ++H) {
    unsigned r[8];
    load_half(lane_buf, H, r);
    float Bt[2], Ct[2];
#pragma unroll
    for (int l = 0; l < 2; ++l) {
      float sv[8];
      load_stats8(s_unit, chunk_of<G>(q, 2 * H + l), sv);
      float bt = 0.0f, ct = 0.0f;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float2 f = __half22float2(__habs2(sbits_h2(r[4 * l + k])));
        const bool in0 = f.x > dl, in1 = f.y > dl;
        bt = __fmaf_rn(sv[2 * k], in0 ? f.x : 0.0f, bt);
        ct = __fadd_rn(ct, in0 ? sv[2 * k] : 0.0f);
        bt = __fmaf_rn(sv[2 * k + 1], in1 ? f.y : 0.0f, bt);
        ct = __fadd_rn(ct, in1 ? sv[2 * k + 1] : 0.0f);
      }
      Bt[l] = bt; Ct[l] = ct;
    }
    if (H == 0) { B0 = Bt[0]; B1 = Bt[1]; C0 = Ct[0]; C1 = Ct[1]; }
    else { B2 = Bt[0]; B3 = Bt[1]; C2 = Ct[0]; C3 = Ct[1]; }
  }
  float sumBt = slots_tree<G>(B0, B1, B2, B3), sumCt = slots_tree<G>(C0, C1, C2, C3);
  // a weighted sum of zero means no activation weight on the support, or no support at all (a threshold at or
  // above the largest |w|): the unweighted sums decide which, and give the scale in the first case
  const bool some = sumA > 0.0f;
  bool nonempty = some;
  if (__any_sync(0xffffffffu, some && sumCt == 0.0f)) {
    B0 = B1 = B2 = B3 = C0 = C1 = C2 = C3 = 0.0f;
#pragma unroll 1
    for (int H = 0; H < 2; ++H) {
      unsigned r[8];
      load_half(lane_buf, H, r);
      float Bu[2], Cu[2];
#pragma unroll
      for (int l = 0; l < 2; ++l) {
        float bu = 0.0f, cu = 0.0f;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float2 f = __half22float2(__habs2(sbits_h2(r[4 * l + k])));
          bu = __fadd_rn(bu, f.x > dl ? f.x : 0.0f);
          cu = __fadd_rn(cu, f.x > dl ? 1.0f : 0.0f);
          bu = __fadd_rn(bu, f.y > dl ? f.y : 0.0f);
          cu = __fadd_rn(cu, f.y > dl ? 1.0f : 0.0f);
        }
        Bu[l] = bu; Cu[l] = cu;
      }
      if (H == 0) { B0 = Bu[0]; B1 = Bu[1]; C0 = Cu[0]; C1 = Cu[1]; }
      else { B2 = Bu[0]; B3 = Bu[1]; C2 = Cu[0]; C3 = Cu[1]; }
    }
    const float sumBu = slots_tree<G>(B0, B1, B2, B3), sumCu = slots_tree<G>(C0, C1, C2, C3);
    if (sumCt == 0.0f) {
      sumBt = sumBu;
      sumCt = sumCu;
      nonempty = some && sumCu > 0.0f;
    }
  }
  return nonempty ? __half2float(__float2half_rn(__fdiv_rn(sumBt, sumCt))) : 0.0f;
}

template <int G>
__global__ void __launch_bounds__(kStreamWarps * 32, 8)
apply_stream_kernel(const __grid_constant__ StreamArgs args) {
  constexpr int LG = Map<G>::LG, GPW = Map<G>::GPW;
  extern __shared__ uint4 stream_smem[];
  __shared__ uint8_t base3[1024];   // five 2-bit trits (a 10-bit window) -> one base-3 byte
  __shared__ float clip_s[64];
  __shared__ float thr_s[64];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane / LG, q = lane % LG;
  uint8_t* mine = reinterpret_cast<uint8_t*>(stream_smem) + (size_t)warp * kStreamWarpBytes;
  uint8_t* stage = mine + 4096;
  for (int x = threadIdx.x; x < 1024; x += kStreamWarps * 32)
    base3[x] = (uint8_t)((x & 3) + 3 * ((x >> 2) & 3) + 9 * ((x >> 4) & 3) + 27 * ((x >> 6) & 3) + 81 * ((x >> 8) & 3));
  if (threadIdx.x < 64) {
    clip_s[threadIdx.x] = threadIdx.x < args.K ? __ldg(args.clip + threadIdx.x) : 1.0f;
    thr_s[threadIdx.x] = (args.thr_grid && threadIdx.x < args.thr_K) ? __ldg(args.thr_grid + threadIdx.x) : 0.7f;
  }
  __syncthreads();

  // element offsets are 32-bit throughout: the host admits only R * ldw, 4 * U * R below 2^31
  const int R = args.R, U = args.U, rows_blocks = args.rows_blocks, n_plans = args.n_plans, ldw = (int)args.ldw;
  const int n_items = U * rows_blocks;
  const int n_warps = gridDim.x * kStreamWarps;
  int item = blockIdx.x * kStreamWarps + warp;

  // asks for everything item `it` needs from global memory: the lane's four chunks of weights into buffer `buf`
  // (rows past the end repeat the last row) and the metadata, which comes back in registers
  auto prefetch = [&](int it, int u, int rb, int buf) {
    ItemMeta m;
    m.act = 7u; m.off = 0; m.clip = 0u; m.thr = 0u;
    if (it < n_items) {
      const int row = min(rb * GPW + g, R - 1);
      const __half* src = args.W + (unsigned)(row * ldw + u * G);
      uint8_t* dst = mine + buf * 2048 + lane * 16;
#pragma unroll
      for (int i = 0; i < 4; ++i) stream_cp16(dst + 512 * i, src + 8 * chunk_of<G>(q, i));
#pragma unroll
      for (int p = 0; p < kStreamMaxPlans; ++p)
        if (lane == p && p < n_plans) {
          m.act = __ldg(args.plan[p].actions + u);
          m.off = __ldg(args.plan[p].code_offsets + u);
        }
      // bit-width columns b = q, q + LG, ... below 4 (for LG >= 4: lanes q < 4 take b = q)
      for (int b = q; b < 4; b += LG) m.clip |= (unsigned)__ldg(args.clip_idx + (unsigned)((b * U + u) * R + row)) << (8 * b);
      if (args.thr_idx && q == 0) m.thr = __ldg(args.thr_idx + (unsigned)(u * R + row));
    }
    stream_commit();  // one group per call, possibly empty, so that the wait below counts right
    return m;
  };

  // (unit, row block) of an item advance with it: no division in the loop
  const int step_u = n_warps / rows_blocks, step_rb = n_warps - step_u * rows_blocks;
  int u_next = item / rows_blocks, rb_next = item - u_next * rows_blocks;
  ItemMeta next = prefetch(item, u_next, rb_next, 0);
  for (int n = 0; item < n_items; item += n_warps, ++n) {
    const ItemMeta cur = next;
    const int u = u_next, rb = rb_next;
    u_next += step_u;
    rb_next += step_rb;
    if (rb_next >= rows_blocks) {
      rb_next -= rows_blocks;
      ++u_next;
    }
    next = prefetch(item + n_warps, u_next, rb_next, (n + 1) & 1);
    stream_wait_all_but_one();  // this lane's 64 bytes of the current item have arrived
    const uint8_t* lane_buf = mine + (n & 1) * 2048 + lane * 16;
    const int row = rb * GPW + g;
    const bool live = row < R;
    const int rows_here = min(GPW, R - rb * GPW);
    const float* s_unit = args.s + (unsigned)(u * G);
    const unsigned w_off = (unsigned)(row * ldw + u * G);  // of the row's first value, in W and in Wq
    const unsigned sz_off = (unsigned)(u * R + row);       // of the group, in scales and zeros
    float mn = 0.0f, mx = 0.0f;
    bool have_range = false;

#pragma unroll 1
    for (int p = 0; p < n_plans; ++p) {
      const int a = (int)__shfl_sync(0xffffffffu, cur.act, p);
      const long long off = __shfl_sync(0xffffffffu, cur.off, p);
      if (a > 6) continue;  // not an action: the unit's outputs stay as they are
      const StreamPlan& po = args.plan[p];  // the parameter block is addressable (__grid_constant__): no local copy
      const int bpg = group_code_bytes(a, G);
      uint8_t* unit_codes = po.codes + off;
      uint8_t* item_codes = unit_codes + (unsigned)(rb * GPW * bpg);  // the item's rows follow one another
      __half* wq_row = (po.Wq && live) ? po.Wq + w_off : nullptr;      // NULL: this lane stores no weights
      // the unit's last rows also write the zero padding up to the next 16-byte boundary
      if (rb == rows_blocks - 1) {
        const unsigned total = (unsigned)(R * bpg);
        const int pad = (int)(((total + 15u) & ~15u) - total);
        if (lane < pad) unit_codes[total + lane] = 0;
      }
      float scale_store = 0.0f, zero_store = 0.0f;
      if (a == 0) {  // skip: the raw fp16 values are the codes and the reconstruction
        if (live) {
          uint4* dst = reinterpret_cast<uint4*>(item_codes + g * bpg);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint4 v = load_slot(lane_buf, i);
            const int c = chunk_of<G>(q, i);
            dst[c] = v;
            if (wq_row) reinterpret_cast<uint4*>(wq_row)[c] = v;
          }
        }
      } else if (a <= 4) {
        const int bi = a - 1;
        if (!have_range) {
          stream_range<G>(lane_buf, mn, mx);
          have_range = true;
        }
        const unsigned packed = __shfl_sync(0xffffffffu, cur.clip, g * LG + (bi % LG));
        const int k = min((int)((packed >> (8 * bi)) & 0xffu), args.K - 1);
        const UniformSpec us = uniform_spec(bi);
        float scale, zf;
        uniform_scale_zero(mn, __fsub_rn(mx, mn), clip_s[k], us, scale, zf);
        if (args.scale_in) scale = __half2float(args.scale_in[(unsigned)((bi * U + u) * R + min(row, R - 1))]);
        uint8_t* stage_row = stage + g * bpg;
        __syncwarp();  // whoever used the staging area before has read it
        switch (a) {
          case 1: stream_uniform<G, 8>(lane_buf, q, scale, zf, us.qmax, wq_row, stage_row); break;
          case 2: stream_uniform<G, 4>(lane_buf, q, scale, zf, us.qmax, wq_row, stage_row); break;
          case 3: stream_uniform<G, 3>(lane_buf, q, scale, zf, us.qmax, wq_row, stage_row); break;
          default: stream_uniform<G, 2>(lane_buf, q, scale, zf, us.qmax, wq_row, stage_row); break;
        }
        __syncwarp();
        copy_out(stage, item_codes, rows_here * bpg, lane);
        scale_store = scale;
        zero_store = zf;
      } else if (a == 5) {
        const int thr_byte = (int)__shfl_sync(0xffffffffu, cur.thr, g * LG);
        const int kt = args.thr_idx ? min(thr_byte, args.thr_K - 1) : 0;  // an index beyond the grid means the last ratio
        float alpha;
        __half2 delta2;  // |w| > delta, with |w| an fp16 value, is |w| > (delta rounded towards zero to fp16)
        if (args.lowbit && !args.thr_idx) {  // scale and threshold as the fit left them
          const unsigned o = (unsigned)(u * R + min(row, R - 1)), plane = (unsigned)(U * R);
          alpha = __half2float(__ldg(args.lowbit + o));
          delta2 = __half2half2(__ldg(args.lowbit + 2u * plane + o));
        } else {
          float delta;
          alpha = stream_ternary_scale<G>(lane_buf, s_unit, q, thr_s[kt], delta);
          delta2 = __half2half2(__float2half_rz(delta));
        }
        const unsigned alpha2 = sh2_bits(__float2half2_rn(alpha));
        uint8_t* stage_row = stage + g * (G / 4);  // 2-bit fields, one per value
        __syncwarp();  // whoever used the staging area before has read it
#pragma unroll
        for (int H = 0; H < 2; ++H) {
          unsigned r[8], wq[8], code[8];
          load_half(lane_buf, H, r);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const unsigned in = __hgt2_mask(__habs2(sbits_h2(r[i])), delta2);  // 0xffff per value on the support
            wq[i] = ((r[i] & 0x80008000u) | alpha2) & in;                       // +-alpha on the support, +0 elsewhere
            const unsigned neg = (r[i] >> 14) & 0x00020002u;
            code[i] = (in & 0x00020002u & ~neg) | (~in & 0x00010001u);          // trit 2, 0 (negative) or 1 (off the support)
          }
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const int c = chunk_of<G>(q, 2 * H + j);
            if (wq_row) *reinterpret_cast<uint4*>(wq_row + 8 * c) = make_uint4(wq[4 * j], wq[4 * j + 1], wq[4 * j + 2], wq[4 * j + 3]);
            stage_chunk<2>(stage_row, c, pack_chunk<2>(code + 4 * j));
          }
        }
        // an output byte is the base-3 value of five consecutive fields, i.e. of a 10-bit window of the staged
        // row, looked up in the block's table
        __syncwarp();
        for (int B = lane; B < rows_here * bpg; B += 32) {
          const int rl = B / bpg, bj = B - rl * bpg;
          const uint8_t* t = stage + rl * (G / 4) + ((10 * bj) >> 3);
          unsigned x = ((unsigned)t[0] | ((unsigned)t[1] << 8)) >> ((10 * bj) & 7);
          const int valid = min(5, G - 5 * bj);  // the row's last byte holds fewer than five trits
          x &= (1u << (2 * valid)) - 1u;
          item_codes[B] = base3[x];
        }
        scale_store = alpha;
      } else {
        const float alpha = args.lowbit ? __half2float(__ldg(args.lowbit + (unsigned)(U * R) + (unsigned)(u * R + min(row, R - 1))))
                                        : stream_binary_scale<G>(lane_buf, s_unit, q);
        const unsigned alpha2 = sh2_bits(__float2half2_rn(alpha));
        const __half2 zero2 = __float2half2_rn(0.0f);
        uint8_t* stage_row = stage + g * bpg;
        __syncwarp();  // whoever used the staging area before has read it
#pragma unroll
        for (int H = 0; H < 2; ++H) {
          unsigned r[8], wq[8], code[8];
          load_half(lane_buf, H, r);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const unsigned neg = __hlt2_mask(sbits_h2(r[i]), zero2);  // w < 0 (false for -0)
            wq[i] = (neg & 0x80008000u) | alpha2;
            code[i] = ~neg & 0x00010001u;                              // bit = !(w < 0)
          }
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const int c = chunk_of<G>(q, 2 * H + j);
            if (wq_row) *reinterpret_cast<uint4*>(wq_row + 8 * c) = make_uint4(wq[4 * j], wq[4 * j + 1], wq[4 * j + 2], wq[4 * j + 3]);
            stage_chunk<1>(stage_row, c, pack_chunk<1>(code + 4 * j));
          }
        }
        __syncwarp();
        copy_out(stage, item_codes, rows_here * bpg, lane);
        scale_store = alpha;
      }
      if (live && q == 0) {
        po.scales[sz_off] = __float2half_rn(scale_store);
        po.zeros[sz_off] = __float2half_rn(zero_store);
      }
    }
  }
}

template <int G>
static windq_status launch_stream_G(windq_ctx* ctx, StreamArgs& args, cudaStream_t st) {
  constexpr int GPW = Map<G>::GPW;
  const size_t smem = (size_t)kStreamWarps * kStreamWarpBytes;
  const int id = kApplyStreamG32 + g_index(G);
  if (windq_status rc = prepare_kernel(ctx, id, apply_stream_kernel<G>, kStreamWarps * 32, smem, true)) return rc;
  args.rows_blocks = (args.R + GPW - 1) / GPW;
  const int64_t n_items = (int64_t)args.U * args.rows_blocks;
  WINDQ_REQUIRE(ctx, n_items < (1ll << 30) && (int64_t)args.R * args.ldw < (1ll << 31) && 4ll * args.U * args.R < (1ll << 31),  /* clip indices [4][U][R], low-bit table [3][U][R] */
                WINDQ_ERR_SHAPE, "windq_apply_plan: R * ldw must be below 2^31 for one call with clip indices");
  int64_t grid = (int64_t)ctx->sm_count * ctx->occupancy[id];
  const int64_t need = (n_items + kStreamWarps - 1) / kStreamWarps;
  if (grid > need) grid = need;
  apply_stream_kernel<G><<<(unsigned)grid, kStreamWarps * 32, smem, st>>>(args);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

// One matrix, n_plans plans, clip indices supplied.  Arguments have been checked by the caller.
windq_status launch_apply_stream(windq_ctx* ctx, int G, const void* W, int64_t R, int64_t C, int64_t ldw, const float* s,
                                 const float* clip_grid, int K, const uint8_t* clip_idx, const void* scale_in,
                                 const float* thr_grid, int thr_K, const uint8_t* thr_idx, const void* lowbit,
                                 const windq_plan_out* plans, int n_plans, cudaStream_t st) {
  StreamArgs args;
  memset(&args, 0, sizeof(args));
  args.W = (const __half*)W;
  args.s = s;
  args.clip = clip_grid;
  args.clip_idx = clip_idx;
  args.scale_in = (const __half*)scale_in;
  args.thr_grid = thr_grid;
  args.thr_idx = thr_idx;
  args.lowbit = (const __half*)lowbit;
  args.ldw = ldw;
  args.R = (int)R;
  args.U = (int)(C / G);
  args.K = K;
  args.thr_K = thr_K;
  args.n_plans = n_plans;
  for (int p = 0; p < n_plans; ++p) {
    args.plan[p].actions = plans[p].actions;
    args.plan[p].code_offsets = (const long long*)plans[p].code_offsets;
    args.plan[p].codes = plans[p].codes_out;
    args.plan[p].scales = (__half*)plans[p].scales_out;
    args.plan[p].zeros = (__half*)plans[p].zeros_out;
    args.plan[p].Wq = (__half*)plans[p].Wq_out;
  }
  switch (G) {
    case 32: return launch_stream_G<32>(ctx, args, st);
    case 64: return launch_stream_G<64>(ctx, args, st);
    case 128: return launch_stream_G<128>(ctx, args, st);
    case 256: return launch_stream_G<256>(ctx, args, st);
    default: return launch_stream_G<512>(ctx, args, st);
  }
}

// Host-side checks of one plan's pointers.
static windq_status check_plan(windq_ctx* ctx, const char* who, int p, const windq_plan_out& pl, const void* W) {
  WINDQ_REQUIRE(ctx, pl.actions && pl.code_offsets && pl.codes_out && pl.scales_out && pl.zeros_out, WINDQ_ERR_NULL,
                "%s: plan %d: a required pointer is NULL", who, p);
  WINDQ_REQUIRE(ctx, aligned16(pl.codes_out), WINDQ_ERR_ALIGN, "%s: plan %d: codes_out is not 16-byte aligned", who, p);
  WINDQ_REQUIRE(ctx, ((uintptr_t)pl.code_offsets & 7) == 0 && ((uintptr_t)pl.scales_out & 1) == 0 && ((uintptr_t)pl.zeros_out & 1) == 0,
                WINDQ_ERR_ALIGN, "%s: plan %d: code_offsets, scales_out or zeros_out is misaligned", who, p);
  WINDQ_REQUIRE(ctx, pl.Wq_out == nullptr || aligned16(pl.Wq_out), WINDQ_ERR_ALIGN, "%s: plan %d: Wq_out is not 16-byte aligned", who, p);
  WINDQ_REQUIRE(ctx, pl.Wq_out != W, WINDQ_ERR_ARG, "%s: plan %d: Wq_out must not alias W", who, p);
  return WINDQ_OK;
}

}  // namespace windq

extern "C" windq_status windq_apply_plan_multi(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                               const float* s, const float* clip_grid, int K, const uint8_t* clip_idx,
                                               const void* lowbit, const windq_plan_out* plans, int n_plans, void* stream) {
  using namespace windq;
  const char* who = "windq_apply_plan_multi";
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "%s: ctx is NULL", who);
  if (windq_status st = check_matrix(ctx, who, W, R, C, ldw, G)) return st;
  if (windq_status st = check_K(ctx, who, K)) return st;
  WINDQ_REQUIRE(ctx, s && clip_grid && clip_idx && plans, WINDQ_ERR_NULL, "%s: s, clip_grid, clip_idx or plans is NULL", who);
  WINDQ_REQUIRE(ctx, aligned16(s), WINDQ_ERR_ALIGN, "%s: s is not 16-byte aligned", who);
  WINDQ_REQUIRE(ctx, n_plans >= 1 && n_plans <= kStreamMaxPlans, WINDQ_ERR_SHAPE, "%s: n_plans = %d is outside [1, %d]", who,
                n_plans, kStreamMaxPlans);
  for (int p = 0; p < n_plans; ++p) {
    if (windq_status st = check_plan(ctx, who, p, plans[p], W)) return st;
    for (int o = 0; o < p; ++o)
      WINDQ_REQUIRE(ctx, plans[p].codes_out != plans[o].codes_out && plans[p].scales_out != plans[o].scales_out &&
                             plans[p].zeros_out != plans[o].zeros_out && (plans[p].Wq_out == nullptr || plans[p].Wq_out != plans[o].Wq_out),
                    WINDQ_ERR_ARG, "%s: plans %d and %d share an output array", who, o, p);
  }
  WINDQ_REQUIRE(ctx, ((uintptr_t)lowbit & 1) == 0, WINDQ_ERR_ALIGN, "%s: lowbit is misaligned", who);
  DeviceGuard guard(ctx->device);
  return launch_apply_stream(ctx, G, W, R, C, ldw, s, clip_grid, K, clip_idx, nullptr, nullptr, 0, nullptr, lowbit, plans, n_plans,
                             (cudaStream_t)stream);
}

extern "C" windq_status windq_apply_plan_searched(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                                  const float* s, const float* clip_grid, int K, const uint8_t* actions,
                                                  const uint8_t* clip_idx, const float* thr_grid, int thr_K,
                                                  const uint8_t* thr_idx, const int64_t* code_offsets, uint8_t* codes_out,
                                                  void* scales_out, void* zeros_out, void* Wq_out, void* stream) {
  using namespace windq;
  const char* who = "windq_apply_plan_searched";
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "%s: ctx is NULL", who);
  if (windq_status st = check_matrix(ctx, who, W, R, C, ldw, G)) return st;
  if (windq_status st = check_K(ctx, who, K)) return st;
  WINDQ_REQUIRE(ctx, s && clip_grid && clip_idx && thr_grid && thr_idx, WINDQ_ERR_NULL,
                "%s: s, clip_grid, clip_idx, thr_grid or thr_idx is NULL", who);
  WINDQ_REQUIRE(ctx, thr_K >= 1 && thr_K <= 64, WINDQ_ERR_ARG, "%s: thr_K = %d is outside [1, 64]", who, thr_K);
  WINDQ_REQUIRE(ctx, aligned16(s), WINDQ_ERR_ALIGN, "%s: s is not 16-byte aligned", who);
  const windq_plan_out pl = {actions, code_offsets, codes_out, scales_out, zeros_out, Wq_out};
  if (windq_status st = check_plan(ctx, who, 0, pl, W)) return st;
  DeviceGuard guard(ctx->device);
  return launch_apply_stream(ctx, G, W, R, C, ldw, s, clip_grid, K, clip_idx, nullptr, thr_grid, thr_K, thr_idx, nullptr, &pl, 1,
                             (cudaStream_t)stream);
}

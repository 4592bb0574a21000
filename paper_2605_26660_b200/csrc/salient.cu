// windq_salient_select: the top-r fraction of every unit's weights by saliency |w| * a_j
// (App. "Salient Weight Protection"), and windq_effective_bits_protected: Eq. 6 with the protected
// weights counted at 8 bits.
//
// Selection is exact.  The key |w| * sqrt(s_j) is a non-negative binary32 number, so its bit
// pattern orders like its value and the n_p-th largest key of a unit is found by a radix search
// from the top in three levels of 11, 10 and 10 bits: per level one pass over W builds, per unit,
// the histogram of the level's digit over the keys that match the digits already fixed, and a small
// kernel walks it from the top to the bin that holds the wanted rank.  A last pass writes the mask.
// W comes from HBM once and from L2 afterwards when the matrix fits there (2 bytes per weight and
// pass); the histograms live in shared memory (8 KB) and are added to the unit's global histogram
// with integer atomics, so counts are exact and independent of scheduling.
#include "windq_internal.cuh"

namespace windq {

constexpr int kSalThreads = 256;
constexpr int kSalBlocksPerSM = 4;
constexpr int kSalBins = 2048;  // level 0: key >> 20 (bit 31 is zero); levels 1, 2: 1024 of them used

struct SalState {          // per unit, in scratch
  unsigned int prefix;     // digits fixed so far, in place (low bits zero)
  unsigned int pad;
  long long remaining;     // rank still to go inside the chosen bin, counted from the top (>= 1)
  long long above;         // keys in bins above the chosen ones (all levels so far)
};

template <int LEVEL>
__device__ __forceinline__ bool digit_of(unsigned int key, unsigned int prefix, unsigned int& digit) {
  if (LEVEL == 0) { digit = key >> 20; return true; }
  if (LEVEL == 1) { digit = (key >> 10) & 1023u; return (key >> 20) == (prefix >> 20); }
  digit = key & 1023u;
  return (key >> 10) == (prefix >> 10);
}

// The eight keys of a thread's 16 bytes: |w| * a_j, one binary32 product each.
__device__ __forceinline__ void keys8(const uint4& raw, const float (&a)[8], unsigned int (&key)[8]) {
  const __half2* h = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __half22float2(h[i]);
    key[2 * i] = __float_as_uint(__fmul_rn(fabsf(f.x), a[2 * i]));
    key[2 * i + 1] = __float_as_uint(__fmul_rn(fabsf(f.y), a[2 * i + 1]));
  }
}

// a_j = sqrt(s_j), once per call.
__global__ void salient_scale_kernel(const float* __restrict__ s, int C, float* __restrict__ a) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < C) a[j] = __fsqrt_rn(s[j]);
}

// One level of the search: histogram of the level's digit, per unit.  Blocks take equal contiguous
// shares of the U * R (unit, row) pairs, unit-major, and flush their shared-memory histogram when the
// unit changes.
template <int G, int LEVEL>
__global__ void __launch_bounds__(kSalThreads)
salient_hist_kernel(const __half* __restrict__ W, int R, int64_t ldw, const float* __restrict__ scale, long long rows_per_block,
                    long long total_rows, const SalState* __restrict__ state, unsigned int* __restrict__ hist) {
  __shared__ unsigned int sh[kSalBins];
  constexpr int TPR = G / 8;              // threads per row
  constexpr int RPP = kSalThreads / TPR;  // rows per pass
  for (int i = threadIdx.x; i < kSalBins; i += kSalThreads) sh[i] = 0;
  __syncthreads();
  const int tr = threadIdx.x / TPR, tc = threadIdx.x % TPR;
  long long p = (long long)blockIdx.x * rows_per_block;
  const long long p_end = min(p + rows_per_block, total_rows);
  while (p < p_end) {
    const int u = (int)(p / R);
    const int r0 = (int)(p - (long long)u * R);
    const int r1 = (int)min((long long)R, r0 + (p_end - p));
    const unsigned int prefix = LEVEL ? state[u].prefix : 0u;
    float a[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] = scale[(int64_t)u * G + tc * 8 + i];
    const __half* base = W + (int64_t)u * G + tc * 8;
    for (int r = r0 + tr; r < r1; r += 4 * RPP) {
      uint4 raw[4];
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (r + k * RPP < r1) raw[k] = __ldg(reinterpret_cast<const uint4*>(base + (int64_t)(r + k * RPP) * ldw));
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (r + k * RPP < r1) {
          unsigned int key[8];
          keys8(raw[k], a, key);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            unsigned int d;
            if (digit_of<LEVEL>(key[i], prefix, d)) atomicAdd(&sh[d], 1u);
          }
        }
    }
    __syncthreads();
    unsigned int* gh = hist + (int64_t)u * kSalBins;
    for (int i = threadIdx.x; i < kSalBins; i += kSalThreads) {
      const unsigned int c = sh[i];
      if (c) {
        atomicAdd(&gh[i], c);
        sh[i] = 0;
      }
    }
    __syncthreads();
    p += r1 - r0;
  }
}

// One block per unit: walks the level's histogram from the top bin down to the one in which the
// running count reaches the wanted rank, and fixes that digit.  After the last level the key is
// complete: threshold and protected count are written.
template <int LEVEL>
__global__ void __launch_bounds__(kSalThreads)
salient_pick_kernel(const unsigned int* __restrict__ hist, SalState* __restrict__ state, long long n_p,
                    float* __restrict__ thresh_out, long long* __restrict__ count_out) {
  __shared__ long long warp_total[kSalThreads / 32];
  const int u = blockIdx.x, t = threadIdx.x, lane = t & 31, wp = t >> 5;
  constexpr int PER = kSalBins / kSalThreads;  // 8 bins per thread; thread 0 owns the TOP bins
  const unsigned int* h = hist + (int64_t)u * kSalBins;
  const long long want = LEVEL ? state[u].remaining : n_p;
  unsigned int c[PER];
  long long local = 0;
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    c[i] = h[kSalBins - 1 - (t * PER + i)];  // descending bin order
    local += c[i];
  }
  long long incl = local;
#pragma unroll
  for (int m = 1; m < 32; m <<= 1) {
    const long long o = __shfl_up_sync(0xffffffffu, incl, m);
    if (lane >= m) incl += o;
  }
  if (lane == 31) warp_total[wp] = incl;
  __syncthreads();
  long long before_warp = 0;
  for (int i = 0; i < wp; ++i) before_warp += warp_total[i];
  incl += before_warp;
  const long long before = incl - local;
  if (before < want && want <= incl) {  // exactly one thread
    long long run = before;
    int i = 0;
    for (; i < PER - 1; ++i) {
      if (run + c[i] >= want) break;
      run += c[i];
    }
    const unsigned int bin = (unsigned int)(kSalBins - 1 - (t * PER + i));
    SalState st = state[u];
    if (LEVEL == 0) { st.prefix = bin << 20; st.above = 0; }
    if (LEVEL == 1) st.prefix |= bin << 10;
    if (LEVEL == 2) st.prefix |= bin;
    st.above += run;
    st.remaining = want - run;
    state[u] = st;
    if (LEVEL == 2) {
      thresh_out[u] = __uint_as_float(st.prefix);
      count_out[u] = st.above + c[i];  // every key equal to the threshold is in
    }
  }
}

// mask[r][col / 8] bit (col % 8) = key >= threshold of the unit.  A thread owns one byte column
// (8 weights per row) and walks a slice of the rows, four loads in flight; neighbouring threads
// write neighbouring bytes.
template <int G>
__global__ void __launch_bounds__(kSalThreads)
salient_mask_kernel(const __half* __restrict__ W, int R, int C, int64_t ldw, const float* __restrict__ scale,
                    const float* __restrict__ thresh, uint8_t* __restrict__ mask, int rows_per_slice) {
  const int bytes_per_row = C / 8;
  const int cb = blockIdx.x * kSalThreads + threadIdx.x;
  if (cb >= bytes_per_row) return;
  const unsigned int tau = __float_as_uint(thresh[(cb * 8) / G]);
  float a[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) a[i] = scale[cb * 8 + i];
  const int r0 = blockIdx.y * rows_per_slice, r1 = min(r0 + rows_per_slice, R);
  const __half* base = W + cb * 8;
  for (int r = r0; r < r1; r += 4) {
    uint4 raw[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (r + k < r1) raw[k] = __ldg(reinterpret_cast<const uint4*>(base + (int64_t)(r + k) * ldw));
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (r + k < r1) {
        unsigned int key[8];
        keys8(raw[k], a, key);
        unsigned int m = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) m |= (key[i] >= tau ? 1u : 0u) << i;
        mask[(int64_t)(r + k) * bytes_per_row + cb] = (uint8_t)m;
      }
  }
}

__global__ void salient_none_kernel(int U, float* __restrict__ thresh_out, long long* __restrict__ count_out) {
  const int u = blockIdx.x * blockDim.x + threadIdx.x;
  if (u < U) {
    thresh_out[u] = __int_as_float(0x7f800000);
    count_out[u] = 0;
  }
}

template <int G>
windq_status run_salient(windq_ctx* ctx, const __half* W, int R, int C, int64_t ldw, const float* s, long long n_p,
                         float* thresh_out, long long* count_out, uint8_t* mask_out, cudaStream_t st) {
  const int U = C / G;
  unsigned int* hist = (unsigned int*)ctx->scratch;
  SalState* state = (SalState*)((char*)ctx->scratch + (size_t)U * kSalBins * sizeof(unsigned int));
  float* scale = (float*)((char*)state + (size_t)U * sizeof(SalState));
  salient_scale_kernel<<<(unsigned)((C + 255) / 256), 256, 0, st>>>(s, C, scale);
  const long long total = (long long)U * R;
  long long nb = (long long)ctx->sm_count * kSalBlocksPerSM;
  if (nb * 16 > total) nb = (total + 15) / 16;
  const long long rpb = (total + nb - 1) / nb;
  const unsigned grid = (unsigned)((total + rpb - 1) / rpb);
  const size_t hist_bytes = (size_t)U * kSalBins * sizeof(unsigned int);
  WINDQ_CUDA(ctx, cudaMemsetAsync(hist, 0, hist_bytes, st));
  salient_hist_kernel<G, 0><<<grid, kSalThreads, 0, st>>>(W, R, ldw, scale, rpb, total, state, hist);
  salient_pick_kernel<0><<<(unsigned)U, kSalThreads, 0, st>>>(hist, state, n_p, thresh_out, count_out);
  WINDQ_CUDA(ctx, cudaMemsetAsync(hist, 0, hist_bytes, st));
  salient_hist_kernel<G, 1><<<grid, kSalThreads, 0, st>>>(W, R, ldw, scale, rpb, total, state, hist);
  salient_pick_kernel<1><<<(unsigned)U, kSalThreads, 0, st>>>(hist, state, n_p, thresh_out, count_out);
  WINDQ_CUDA(ctx, cudaMemsetAsync(hist, 0, hist_bytes, st));
  salient_hist_kernel<G, 2><<<grid, kSalThreads, 0, st>>>(W, R, ldw, scale, rpb, total, state, hist);
  salient_pick_kernel<2><<<(unsigned)U, kSalThreads, 0, st>>>(hist, state, n_p, thresh_out, count_out);
  WINDQ_CUDA(ctx, cudaGetLastError());
  if (mask_out) {
    const int col_blocks = (C / 8 + kSalThreads - 1) / kSalThreads;
    int slices = (4 * ctx->sm_count + col_blocks - 1) / col_blocks;  // about four blocks per SM
    if (slices > (R + 31) / 32) slices = (R + 31) / 32;
    if (slices > 65535) slices = 65535;
    const int rows_per_slice = (R + slices - 1) / slices;
    salient_mask_kernel<G><<<dim3((unsigned)col_blocks, (unsigned)((R + rows_per_slice - 1) / rows_per_slice)), kSalThreads, 0, st>>>(
        W, R, C, ldw, scale, thresh_out, mask_out, rows_per_slice);
    WINDQ_CUDA(ctx, cudaGetLastError());
  }
  return WINDQ_OK;
}

__global__ void __launch_bounds__(256)
bits_protected_kernel(const uint8_t* __restrict__ actions, const long long* __restrict__ n_protected, long long U,
                      long long R, int G, int scale_bits, int zero_bits, long long* __restrict__ unit_cb,
                      long long* __restrict__ total_cb) {
  __shared__ long long red[8];
  __shared__ int bad_flag;
  const int t = threadIdx.x;
  if (t == 0) bad_flag = 0;
  __syncthreads();
  const long long centi[7] = {1600, 800, 400, 300, 200, 158, 100};
  const long long n = R * G;
  long long sum = 0;
  for (long long u = t; u < U; u += 256) {
    const int a = actions[u];
    const long long np_ = n_protected[u];
    long long cb = -1;
    if (a <= 6 && np_ >= 0 && np_ <= n)
      cb = a == 0 ? 1600 * n : centi[a] * (n - np_) + 800 * np_ + 100 * R * (scale_bits + (a <= 4 ? zero_bits : 0));
    if (cb < 0) bad_flag = 1; else sum += cb;
    if (unit_cb) unit_cb[u] = cb;
  }
#pragma unroll
  for (int m = 16; m > 0; m >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, m);
  if ((t & 31) == 0) red[t >> 5] = sum;
  __syncthreads();
  if (t == 0) {
    long long a = 0;
    for (int i = 0; i < 8; ++i) a += red[i];
    *total_cb = bad_flag ? -1 : a;
  }
}

}  // namespace windq

extern "C" {

int64_t windq_scratch_bytes_salient_select(int64_t R, int64_t C, int G) {
  if (!windq::valid_G(G) || R <= 0 || C <= 0) return 0;
  const int64_t U = C / G;
  // per-unit histograms and search state, then sqrt(s)
  return U * windq::kSalBins * (int64_t)sizeof(unsigned int) + U * (int64_t)sizeof(windq::SalState) + C * (int64_t)sizeof(float);
}

windq_status windq_salient_select(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                                  int64_t rate_ppm, float* thresh_out, int64_t* count_out, uint8_t* mask_out,
                                  void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "windq_salient_select: ctx is NULL");
  if (windq_status st = check_matrix(ctx, "windq_salient_select", W, R, C, ldw, G)) return st;
  WINDQ_REQUIRE(ctx, s && thresh_out && count_out, WINDQ_ERR_NULL, "windq_salient_select: s, thresh_out or count_out is NULL");
  WINDQ_REQUIRE(ctx, rate_ppm >= 0 && rate_ppm <= 1000000, WINDQ_ERR_ARG,
                "windq_salient_select: rate_ppm = %lld is outside [0, 1000000]", (long long)rate_ppm);
  WINDQ_REQUIRE(ctx, ((uintptr_t)count_out & 7) == 0, WINDQ_ERR_ALIGN, "windq_salient_select: count_out is not 8-byte aligned");
  WINDQ_REQUIRE(ctx, R * (int64_t)G < (1ll << 32), WINDQ_ERR_SHAPE, "windq_salient_select: R * G must be below 2^32");
  DeviceGuard guard(ctx->device);
  cudaStream_t st = (cudaStream_t)stream;
  const int U = (int)(C / G);
  const long long n_p = (long long)(((__int128)rate_ppm * (R * (int64_t)G)) / 1000000);
  if (n_p == 0) {
    salient_none_kernel<<<(unsigned)((U + 255) / 256), 256, 0, st>>>(U, thresh_out, (long long*)count_out);
    WINDQ_CUDA(ctx, cudaGetLastError());
    if (mask_out) WINDQ_CUDA(ctx, cudaMemsetAsync(mask_out, 0, (size_t)(R * (C / 8)), st));
    return WINDQ_OK;
  }
  if (windq_status rc = ensure_scratch(ctx, windq_scratch_bytes_salient_select(R, C, G))) return rc;
  const __half* Wh = (const __half*)W;
  long long* cnt = (long long*)count_out;
  switch (G) {
    case 32: return run_salient<32>(ctx, Wh, (int)R, (int)C, ldw, s, n_p, thresh_out, cnt, mask_out, st);
    case 64: return run_salient<64>(ctx, Wh, (int)R, (int)C, ldw, s, n_p, thresh_out, cnt, mask_out, st);
    case 128: return run_salient<128>(ctx, Wh, (int)R, (int)C, ldw, s, n_p, thresh_out, cnt, mask_out, st);
    case 256: return run_salient<256>(ctx, Wh, (int)R, (int)C, ldw, s, n_p, thresh_out, cnt, mask_out, st);
    default: return run_salient<512>(ctx, Wh, (int)R, (int)C, ldw, s, n_p, thresh_out, cnt, mask_out, st);
  }
}

windq_status windq_effective_bits_protected(windq_ctx* ctx, const uint8_t* actions, const int64_t* n_protected, int64_t U,
                                            int64_t R, int G, int scale_bits, int zero_bits, int64_t* unit_centibits_out,
                                            int64_t* total_centibits_out, void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "windq_effective_bits_protected: ctx is NULL");
  WINDQ_REQUIRE(ctx, actions && n_protected && total_centibits_out, WINDQ_ERR_NULL,
                "windq_effective_bits_protected: actions, n_protected or total_centibits_out is NULL");
  WINDQ_REQUIRE(ctx, U > 0 && R > 0 && U < (1ll << 31) && R < (1ll << 31), WINDQ_ERR_SHAPE,
                "windq_effective_bits_protected: U = %lld, R = %lld", (long long)U, (long long)R);
  WINDQ_REQUIRE(ctx, valid_G(G), WINDQ_ERR_ARG, "windq_effective_bits_protected: G = %d is not one of 32, 64, 128, 256, 512", G);
  WINDQ_REQUIRE(ctx, scale_bits >= 0 && scale_bits <= 64 && zero_bits >= 0 && zero_bits <= 64, WINDQ_ERR_ARG,
                "windq_effective_bits_protected: scale_bits = %d, zero_bits = %d must be in [0, 64]", scale_bits, zero_bits);
  WINDQ_REQUIRE(ctx, ((uintptr_t)n_protected & 7) == 0 && ((uintptr_t)unit_centibits_out & 7) == 0 &&
                         ((uintptr_t)total_centibits_out & 7) == 0,
                WINDQ_ERR_ALIGN, "windq_effective_bits_protected: an int64 array is not 8-byte aligned");
  DeviceGuard guard(ctx->device);
  bits_protected_kernel<<<1, 256, 0, (cudaStream_t)stream>>>(actions, (const long long*)n_protected, (long long)U, (long long)R,
                                                           G, scale_bits, zero_bits, (long long*)unit_centibits_out,
                                                           (long long*)total_centibits_out);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

}  // extern "C"

// ---- unit saliency and the fallback rule --------------------------------------------------------
namespace windq {

// Per unit, the sum over its weights of scale_j * |w| ("Comparison with Heuristic Sensitivity
// Allocator": saliency score = mean product of activation scale and weight magnitude).  Same block
// schedule as the histogram passes; a thread adds |w| of its eight columns over its rows in fp32
// (at most a few hundred terms), multiplies by the scales and hands a double to the block sum, which
// goes to the unit's accumulator with one double atomic per (block, unit).
template <int G>
__global__ void __launch_bounds__(kSalThreads)
unit_saliency_kernel(const __half* __restrict__ W, int R, int64_t ldw, const float* __restrict__ s, long long rows_per_block,
                     long long total_rows, double* __restrict__ acc) {
  __shared__ double wsum[kSalThreads / 32];
  constexpr int TPR = G / 8, RPP = kSalThreads / TPR;
  const int tr = threadIdx.x / TPR, tc = threadIdx.x % TPR;
  long long p = (long long)blockIdx.x * rows_per_block;
  const long long p_end = min(p + rows_per_block, total_rows);
  while (p < p_end) {
    const int u = (int)(p / R);
    const int r0 = (int)(p - (long long)u * R);
    const int r1 = (int)min((long long)R, r0 + (p_end - p));
    const __half* base = W + (int64_t)u * G + tc * 8;
    double sum = 0.0;
    float col[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    int n_in_col = 0;
    for (int r = r0 + tr; r < r1; r += 4 * RPP) {
      uint4 raw[4];
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (r + k * RPP < r1) raw[k] = __ldg(reinterpret_cast<const uint4*>(base + (int64_t)(r + k * RPP) * ldw));
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (r + k * RPP < r1) {
          const __half2* h = reinterpret_cast<const __half2*>(&raw[k]);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(h[i]);
            col[2 * i] += fabsf(f.x);
            col[2 * i + 1] += fabsf(f.y);
          }
        }
      if (++n_in_col == 64 || r + 4 * RPP >= r1) {  // at most 256 terms per fp32 column sum
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          sum += (double)col[i] * (double)__fsqrt_rn(__ldg(s + (int64_t)u * G + tc * 8 + i));
          col[i] = 0.0f;
        }
        n_in_col = 0;
      }
    }
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, m);
    if ((threadIdx.x & 31) == 0) wsum[threadIdx.x >> 5] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
      double t = 0.0;
      for (int i = 0; i < kSalThreads / 32; ++i) t += wsum[i];
      atomicAdd(&acc[u], t);
    }
    __syncthreads();
    p += r1 - r0;
  }
}

__global__ void unit_saliency_finish_kernel(const double* __restrict__ acc, int U, double inv_n, float* __restrict__ sal_out) {
  const int u = blockIdx.x * blockDim.x + threadIdx.x;
  if (u < U) sal_out[u] = (float)(acc[u] * inv_n);
}

__global__ void fallback_kernel(const float* __restrict__ err, const float* __restrict__ energy,
                                const uint8_t* __restrict__ actions, long long U, float theta,
                                uint8_t* __restrict__ actions_out, unsigned long long* __restrict__ n_changed) {
  const long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  int changed = 0;
  if (u < U) {
    const int a0 = actions[u];
    int a = a0;
    if (a <= 6) {
      const float limit = __fmul_rn(theta, energy[u]);
      while (a >= 1 && err[u * 6 + (a - 1)] > limit) --a;
    }
    actions_out[u] = (uint8_t)a;
    changed = a != a0;
  }
  const unsigned int votes = __ballot_sync(0xffffffffu, changed);
  if ((threadIdx.x & 31) == 0 && votes && n_changed) atomicAdd(n_changed, (unsigned long long)__popc(votes));
}

template <int G>
windq_status run_saliency(windq_ctx* ctx, const __half* W, int R, int C, int64_t ldw, const float* s, float* sal_out,
                          cudaStream_t st) {
  const int U = C / G;
  double* acc = (double*)ctx->scratch;
  const long long total = (long long)U * R;
  long long nb = (long long)ctx->sm_count * kSalBlocksPerSM;
  if (nb * 16 > total) nb = (total + 15) / 16;
  const long long rpb = (total + nb - 1) / nb;
  WINDQ_CUDA(ctx, cudaMemsetAsync(acc, 0, (size_t)U * sizeof(double), st));
  unit_saliency_kernel<G><<<(unsigned)((total + rpb - 1) / rpb), kSalThreads, 0, st>>>(W, R, ldw, s, rpb, total, acc);
  unit_saliency_finish_kernel<<<(unsigned)((U + 255) / 256), 256, 0, st>>>(acc, U, 1.0 / ((double)R * G), sal_out);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

}  // namespace windq

extern "C" {

windq_status windq_unit_saliency(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                                 float* sal_out, void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "windq_unit_saliency: ctx is NULL");
  if (windq_status st = check_matrix(ctx, "windq_unit_saliency", W, R, C, ldw, G)) return st;
  WINDQ_REQUIRE(ctx, s && sal_out, WINDQ_ERR_NULL, "windq_unit_saliency: s or sal_out is NULL");
  DeviceGuard guard(ctx->device);
  if (windq_status rc = ensure_scratch(ctx, (C / G) * (int64_t)sizeof(double))) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  const __half* Wh = (const __half*)W;
  switch (G) {
    case 32: return run_saliency<32>(ctx, Wh, (int)R, (int)C, ldw, s, sal_out, st);
    case 64: return run_saliency<64>(ctx, Wh, (int)R, (int)C, ldw, s, sal_out, st);
    case 128: return run_saliency<128>(ctx, Wh, (int)R, (int)C, ldw, s, sal_out, st);
    case 256: return run_saliency<256>(ctx, Wh, (int)R, (int)C, ldw, s, sal_out, st);
    default: return run_saliency<512>(ctx, Wh, (int)R, (int)C, ldw, s, sal_out, st);
  }
}

windq_status windq_fallback(windq_ctx* ctx, const float* err, const float* energy, const uint8_t* actions, int64_t U,
                            float theta, uint8_t* actions_out, int64_t* n_changed_out, void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "windq_fallback: ctx is NULL");
  WINDQ_REQUIRE(ctx, err && energy && actions && actions_out, WINDQ_ERR_NULL, "windq_fallback: a required pointer is NULL");
  WINDQ_REQUIRE(ctx, U > 0 && U < (1ll << 31), WINDQ_ERR_SHAPE, "windq_fallback: U = %lld", (long long)U);
  WINDQ_REQUIRE(ctx, theta >= 0.0f, WINDQ_ERR_ARG, "windq_fallback: theta must be a number >= 0");
  WINDQ_REQUIRE(ctx, ((uintptr_t)n_changed_out & 7) == 0, WINDQ_ERR_ALIGN, "windq_fallback: n_changed_out is not 8-byte aligned");
  DeviceGuard guard(ctx->device);
  cudaStream_t st = (cudaStream_t)stream;
  if (n_changed_out) WINDQ_CUDA(ctx, cudaMemsetAsync(n_changed_out, 0, sizeof(int64_t), st));
  fallback_kernel<<<(unsigned)((U + 255) / 256), 256, 0, st>>>(err, energy, actions, (long long)U, theta, actions_out,
                                                               (unsigned long long*)n_changed_out);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

}  // extern "C"

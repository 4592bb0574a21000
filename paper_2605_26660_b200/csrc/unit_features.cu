// windq_unit_features: Table 1 state features (dims 0-4 and 9-11) of every unit.
//
// The magnitude of an fp16 number has 32768 possible bit patterns and their integer order is
// their numeric order, so ONE histogram of |w| per unit gives the nearest-rank P99, the count
// above 0.5 * P99 and the count below 1e-6 exactly, and also sum |w| and sum w^2 exactly up to
// double rounding.  One streaming pass over W (2 bytes per weight, HBM-bound in principle; the
// shared-memory atomics are what limits it in practice):
//   pass 1  blocks = (unit, slice of rows): histogram in shared memory (128 KB), flushed to the
//           unit's histogram in scratch with integer atomics (order-independent, so exact and
//           reproducible); the signed sum of the slice goes to scratch as a double.
//   pass 2  one block per unit scans the histogram and writes the eight features.
#include "windq_internal.cuh"

namespace windq {

constexpr int kBins = 32768;
constexpr int kFeatThreads = 512;

template <int G>
__global__ void __launch_bounds__(kFeatThreads, 1)
feat_hist_kernel(const __half* __restrict__ W, int R, int64_t ldw, int rows_per_slice, unsigned int* __restrict__ hist,
                 double* __restrict__ slice_sum /*[U][slices]*/) {
  extern __shared__ unsigned int sh[];
  __shared__ double wsum[kFeatThreads / 32];
  constexpr int TPR = G / 8;                  // threads per row (8 halves = 16 bytes each)
  constexpr int RPP = kFeatThreads / TPR;     // rows per pass
  const int u = blockIdx.x, slice = blockIdx.y;
  for (int i = threadIdx.x; i < kBins; i += kFeatThreads) sh[i] = 0;
  __syncthreads();
  const int r0 = slice * rows_per_slice, r1 = min(r0 + rows_per_slice, R);
  const int tr = threadIdx.x / TPR, tc = threadIdx.x % TPR;
  const __half* base = W + (int64_t)u * G + tc * 8;
  double sum = 0.0;
  for (int r = r0 + tr; r < r1; r += RPP) {
    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(base + (int64_t)r * ldw));
    const unsigned int v[4] = {raw.x, raw.y, raw.z, raw.w};
    float part = 0.0f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      atomicAdd(&sh[v[i] & 0x7fffu], 1u);
      atomicAdd(&sh[(v[i] >> 16) & 0x7fffu], 1u);
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&v[i]));
      part += f.x + f.y;
    }
    sum += (double)part;
  }
#pragma unroll
  for (int m = 16; m > 0; m >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, m);
  if ((threadIdx.x & 31) == 0) wsum[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int i = 0; i < kFeatThreads / 32; ++i) t += wsum[i];
    slice_sum[(int64_t)u * gridDim.y + slice] = t;
  }
  unsigned int* gh = hist + (int64_t)u * kBins;
  for (int i = threadIdx.x; i < kBins; i += kFeatThreads) {
    const unsigned int c = sh[i];
    if (c) atomicAdd(&gh[i], c);
  }
}

__global__ void __launch_bounds__(1024)
feat_finalize_kernel(const unsigned int* __restrict__ hist, const double* __restrict__ slice_sum, int slices, int R, int G,
                     const float* __restrict__ s, float* __restrict__ feat) {
  __shared__ unsigned long long cnt_scan[1024];
  __shared__ double red[3][32];
  __shared__ unsigned long long redc[2][32];
  __shared__ int p99_bin;
  const int u = blockIdx.x, t = threadIdx.x;
  const unsigned int* h = hist + (int64_t)u * kBins;
  const long long n = (long long)R * G;
  const long long k = (99 * n + 99) / 100;  // rank of P99, 1-indexed

  // each thread owns 32 consecutive bins
  unsigned int c[32];
  unsigned long long local = 0;
#pragma unroll
  for (int i = 0; i < 32; ++i) { c[i] = h[t * 32 + i]; local += c[i]; }
  cnt_scan[t] = local;
  __syncthreads();
  for (int off = 1; off < 1024; off <<= 1) {  // inclusive scan over threads
    unsigned long long v = (t >= off) ? cnt_scan[t - off] : 0;
    __syncthreads();
    cnt_scan[t] += v;
    __syncthreads();
  }
  const unsigned long long before = cnt_scan[t] - local;
  if (before < (unsigned long long)k && (unsigned long long)k <= cnt_scan[t]) {
    unsigned long long run = before;
    for (int i = 0; i < 32; ++i) {
      run += c[i];
      if (run >= (unsigned long long)k) { p99_bin = t * 32 + i; break; }
    }
  }
  __syncthreads();
  const float p99 = __half2float(__ushort_as_half((unsigned short)p99_bin));
  const float thr = 0.5f * p99;

  double sa = 0.0, sq = 0.0;
  unsigned long long n_out = 0, n_tiny = 0;
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    const float v = __half2float(__ushort_as_half((unsigned short)(t * 32 + i)));
    if (c[i] == 0) continue;  // also keeps the Inf / NaN patterns (never counted for finite input) out
    const double dv = (double)v, dc = (double)c[i];
    sa += dc * dv;
    sq += dc * dv * dv;
    if (v > thr) n_out += c[i];
    if (v < 1e-6f) n_tiny += c[i];
  }
  double ss = 0.0;
  for (int i = t; i < slices; i += 1024) ss += slice_sum[(int64_t)u * slices + i];
#pragma unroll
  for (int m = 16; m > 0; m >>= 1) {
    sa += __shfl_xor_sync(0xffffffffu, sa, m);
    sq += __shfl_xor_sync(0xffffffffu, sq, m);
    ss += __shfl_xor_sync(0xffffffffu, ss, m);
    n_out += __shfl_xor_sync(0xffffffffu, n_out, m);
    n_tiny += __shfl_xor_sync(0xffffffffu, n_tiny, m);
  }
  if ((t & 31) == 0) {
    red[0][t >> 5] = sa; red[1][t >> 5] = sq; red[2][t >> 5] = ss;
    redc[0][t >> 5] = n_out; redc[1][t >> 5] = n_tiny;
  }
  __syncthreads();
  if (t == 0) {
    double a = 0, q2 = 0, sg = 0;
    unsigned long long no = 0, nt = 0;
    for (int i = 0; i < 32; ++i) { a += red[0][i]; q2 += red[1][i]; sg += red[2][i]; no += redc[0][i]; nt += redc[1][i]; }
    const double dn = (double)n;
    const double mean = sg / dn;
    double var = q2 / dn - mean * mean;
    if (var < 0.0) var = 0.0;
    double smean = 0.0, smax = (double)s[(int64_t)u * G];
    for (int j = 0; j < G; ++j) { const double v = (double)s[(int64_t)u * G + j]; smean += v; smax = fmax(smax, v); }
    smean /= (double)G;
    double svar = 0.0;
    for (int j = 0; j < G; ++j) { const double d = (double)s[(int64_t)u * G + j] - smean; svar += d * d; }
    svar /= (double)G;
    float* f = feat + (int64_t)u * WINDQ_N_FEATURES;
    f[0] = (float)mean;
    f[1] = (float)sqrt(var);
    f[2] = (float)(a / dn);
    f[3] = (float)((double)nt / dn);
    f[4] = (float)((double)no / dn);
    f[5] = (float)smean;
    f[6] = (float)sqrt(svar);
    f[7] = (float)smax;
  }
}

inline int feat_slices(int sm_count, int64_t R, int U) {
  // about two waves of blocks over the SMs, at least 64 rows per slice
  int64_t want = (2ll * sm_count + U - 1) / U;
  const int64_t max_slices = (R + 63) / 64;
  if (want > max_slices) want = max_slices;
  if (want < 1) want = 1;
  return (int)want;
}

template <int G>
windq_status launch_hist(windq_ctx* ctx, const __half* W, int R, int U, int64_t ldw, int slices, unsigned int* hist,
                         double* slice_sum, cudaStream_t st) {
  static bool configured = false;
  const size_t smem = (size_t)kBins * sizeof(unsigned int);
  if (!configured) {
    WINDQ_CUDA(ctx, cudaFuncSetAttribute(feat_hist_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    configured = true;
  }
  const int rows_per_slice = (R + slices - 1) / slices;
  feat_hist_kernel<G><<<dim3((unsigned)U, (unsigned)slices), kFeatThreads, smem, st>>>(W, R, ldw, rows_per_slice, hist, slice_sum);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

}  // namespace windq

extern "C" {

int64_t windq_scratch_bytes_unit_features(int64_t R, int64_t C, int G) {
  if (!windq::valid_G(G) || R <= 0 || C <= 0) return 0;
  const int64_t U = C / G;
  // histograms + slice sums (at most ceil(R/64) slices per unit)
  return U * windq::kBins * (int64_t)sizeof(unsigned int) + U * ((R + 63) / 64) * (int64_t)sizeof(double);
}

windq_status windq_unit_features(windq_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw, int G,
                                 const float* s, float* feat_out, void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "windq_unit_features: ctx is NULL");
  if (windq_status st = check_matrix(ctx, "windq_unit_features", W, R, C, ldw, G)) return st;
  WINDQ_REQUIRE(ctx, s && feat_out, WINDQ_ERR_NULL, "windq_unit_features: s or feat_out is NULL");
  WINDQ_REQUIRE(ctx, R * (int64_t)G < (1ll << 32), WINDQ_ERR_SHAPE, "windq_unit_features: R * G must be below 2^32");
  DeviceGuard guard(ctx->device);
  if (windq_status st = ensure_scratch(ctx, windq_scratch_bytes_unit_features(R, C, G))) return st;
  const int U = (int)(C / G);
  WINDQ_REQUIRE(ctx, U <= 65535 * 32, WINDQ_ERR_SHAPE, "windq_unit_features: too many units");
  cudaStream_t st = (cudaStream_t)stream;
  unsigned int* hist = (unsigned int*)ctx->scratch;
  double* slice_sum = (double*)((char*)ctx->scratch + (int64_t)U * kBins * sizeof(unsigned int));
  const int slices = feat_slices(ctx->sm_count, R, U);
  WINDQ_CUDA(ctx, cudaMemsetAsync(hist, 0, (size_t)U * kBins * sizeof(unsigned int), st));
  const __half* Wh = (const __half*)W;
  windq_status rc;
  switch (G) {
    case 32: rc = launch_hist<32>(ctx, Wh, (int)R, U, ldw, slices, hist, slice_sum, st); break;
    case 64: rc = launch_hist<64>(ctx, Wh, (int)R, U, ldw, slices, hist, slice_sum, st); break;
    case 128: rc = launch_hist<128>(ctx, Wh, (int)R, U, ldw, slices, hist, slice_sum, st); break;
    case 256: rc = launch_hist<256>(ctx, Wh, (int)R, U, ldw, slices, hist, slice_sum, st); break;
    default: rc = launch_hist<512>(ctx, Wh, (int)R, U, ldw, slices, hist, slice_sum, st); break;
  }
  if (rc != WINDQ_OK) return rc;
  feat_finalize_kernel<<<(unsigned)U, 1024, 0, st>>>(hist, slice_sum, slices, (int)R, G, s, feat_out);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

}  // extern "C"

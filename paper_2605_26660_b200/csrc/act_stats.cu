// windq_act_stats: s_j = mean_t x_tj^2 over a calibration input X[T][C] (fp16).
//
// One streaming pass, bound by HBM: 2 bytes read per element.  A block covers 256 adjacent
// channels (512 contiguous bytes per row, one 128-bit load per thread) and a slice of the
// tokens; its 8 thread rows walk the slice with a stride of 8 rows, each thread adding at most a
// few dozen squares in fp32.  The per-slice sums go to scratch as fp32 and a second kernel adds
// the slices in double and divides by T, so the result does not depend on scheduling.
#include "windq_internal.cuh"

namespace windq {

constexpr int kActCols = 256;   // channels per block
constexpr int kActRowsPar = 8;  // thread rows per block
constexpr int kActMaxRowsPerThread = 8;

__global__ void __launch_bounds__(256)
act_partial_kernel(const __half* __restrict__ X, int64_t T, int C, int64_t ldx, int rows_per_slice,
                   float* __restrict__ partial /*[slices][C]*/) {
  __shared__ float red[kActRowsPar][kActCols + 8];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int col = blockIdx.x * kActCols + tx * 8;
  const int64_t t0 = (int64_t)blockIdx.y * rows_per_slice;
  const int64_t t1 = min(t0 + rows_per_slice, T);
  float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  if (col < C) {
    for (int64_t t = t0 + ty; t < t1; t += kActRowsPar) {
      const uint4 raw = __ldg(reinterpret_cast<const uint4*>(X + t * ldx + col));
      const __half2* h = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(h[i]);
        acc[2 * i] = fmaf(f.x, f.x, acc[2 * i]);
        acc[2 * i + 1] = fmaf(f.y, f.y, acc[2 * i + 1]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) red[ty][tx * 8 + i] = acc[i];
  __syncthreads();
  const int c = threadIdx.x;  // 256 threads, 256 channels
  if (blockIdx.x * kActCols + c < C) {
    float sum = 0.0f;
#pragma unroll
    for (int r = 0; r < kActRowsPar; ++r) sum += red[r][c];
    partial[(int64_t)blockIdx.y * C + blockIdx.x * kActCols + c] = sum;
  }
}

__global__ void __launch_bounds__(256)
act_finalize_kernel(const float* __restrict__ partial, int slices, int C, double inv_T, float* __restrict__ s_out) {
  const int c = blockIdx.x * 256 + threadIdx.x;
  if (c >= C) return;
  double acc = 0.0;
  for (int i = 0; i < slices; ++i) acc += (double)partial[(int64_t)i * C + c];
  s_out[c] = (float)(acc * inv_T);
}

constexpr int64_t kActMaxSlices = 65535;  // grid.y limit

// Token slices of a call (64 rows each), as a 64-bit count: callers compare it with kActMaxSlices
// before they narrow it.
inline int64_t act_slices(int64_t T) {
  const int64_t rows_per_slice = (int64_t)kActRowsPar * kActMaxRowsPerThread;
  return (T + rows_per_slice - 1) / rows_per_slice;
}

}  // namespace windq

extern "C" {

int64_t windq_scratch_bytes_act_stats(int64_t T, int64_t C) {
  if (T <= 0 || C <= 0 || windq::act_slices(T) > windq::kActMaxSlices || C >= (1ll << 31)) return 0;
  return windq::act_slices(T) * C * (int64_t)sizeof(float);
}

windq_status windq_act_stats(windq_ctx* ctx, const void* X, int64_t T, int64_t C, int64_t ldx, float* s_out,
                             void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "windq_act_stats: ctx is NULL");
  WINDQ_REQUIRE(ctx, X && s_out, WINDQ_ERR_NULL, "windq_act_stats: X or s_out is NULL");
  WINDQ_REQUIRE(ctx, T > 0 && C > 0, WINDQ_ERR_SHAPE, "windq_act_stats: T = %lld, C = %lld must be positive",
                (long long)T, (long long)C);
  WINDQ_REQUIRE(ctx, C < (1ll << 31) && T < (1ll << 40), WINDQ_ERR_SHAPE, "windq_act_stats: T or C too large");
  WINDQ_REQUIRE(ctx, C % 8 == 0, WINDQ_ERR_SHAPE, "windq_act_stats: C = %lld is not a multiple of 8", (long long)C);
  WINDQ_REQUIRE(ctx, ldx >= C, WINDQ_ERR_SHAPE, "windq_act_stats: ldx = %lld is below C = %lld", (long long)ldx,
                (long long)C);
  WINDQ_REQUIRE(ctx, ldx % 8 == 0, WINDQ_ERR_ALIGN, "windq_act_stats: ldx = %lld is not a multiple of 8", (long long)ldx);
  WINDQ_REQUIRE(ctx, aligned16(X), WINDQ_ERR_ALIGN, "windq_act_stats: X is not 16-byte aligned");
  WINDQ_REQUIRE(ctx, act_slices(T) <= kActMaxSlices, WINDQ_ERR_SHAPE, "windq_act_stats: T = %lld is too large (at most %lld tokens per call)",
                (long long)T, (long long)(kActMaxSlices * kActRowsPar * kActMaxRowsPerThread));
  const int slices = (int)act_slices(T);
  DeviceGuard guard(ctx->device);
  if (windq_status st = ensure_scratch(ctx, windq_scratch_bytes_act_stats(T, C))) return st;
  const int rows_per_slice = kActRowsPar * kActMaxRowsPerThread;
  cudaStream_t st = (cudaStream_t)stream;
  float* partial = (float*)ctx->scratch;
  dim3 grid((unsigned)((C + kActCols - 1) / kActCols), (unsigned)slices);
  act_partial_kernel<<<grid, 256, 0, st>>>((const __half*)X, T, (int)C, ldx, rows_per_slice, partial);
  WINDQ_CUDA(ctx, cudaGetLastError());
  act_finalize_kernel<<<(unsigned)((C + 255) / 256), 256, 0, st>>>(partial, slices, (int)C, 1.0 / (double)T, s_out);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

}  // extern "C"

// ---- windq_act_stats_noalloc ------------------------------------------------------------------
// Same two kernels as windq_act_stats, with the per-slice partial sums kept in a fixed array in
// device global memory instead of the context's cudaMalloc'ed scratch.  The array is part of the
// library image: every device that loads the library carries WINDQ_NOALLOC_SCRATCH_BYTES of it
// until the process exits, and every call on a device uses the same bytes.
#include <mutex>

namespace windq {

constexpr int64_t kNoallocFloats = WINDQ_NOALLOC_SCRATCH_BYTES / (int64_t)sizeof(float);
static __device__ __align__(256) float g_noalloc_partial[kNoallocFloats];

constexpr int kNoallocMaxDevices = 64;
static std::mutex g_noalloc_mutex;
static float* g_noalloc_ptr[kNoallocMaxDevices];  // device address of the array, per device; NULL until looked up

// Device address of g_noalloc_partial on `device`, which must be the current device.  In host
// code the array's name only stands for the symbol; the address a kernel can use has to be asked
// from the runtime, once per device.
static cudaError_t noalloc_scratch(int device, float** out) {
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (g_noalloc_ptr[device] == nullptr) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_partial);
    if (e != cudaSuccess) return e;
    g_noalloc_ptr[device] = static_cast<float*>(p);
  }
  *out = g_noalloc_ptr[device];
  return cudaSuccess;
}

}  // namespace windq

extern "C" windq_status windq_act_stats_noalloc(windq_ctx* ctx, const void* X, int64_t T, int64_t C, int64_t ldx,
                                                float* s_out, void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "windq_act_stats_noalloc: ctx is NULL");
  WINDQ_REQUIRE(ctx, X && s_out, WINDQ_ERR_NULL, "windq_act_stats_noalloc: X or s_out is NULL");
  WINDQ_REQUIRE(ctx, T > 0 && C > 0, WINDQ_ERR_SHAPE, "windq_act_stats_noalloc: T = %lld, C = %lld must be positive",
                (long long)T, (long long)C);
  WINDQ_REQUIRE(ctx, C < (1ll << 31) && T < (1ll << 40), WINDQ_ERR_SHAPE, "windq_act_stats_noalloc: T or C too large");
  WINDQ_REQUIRE(ctx, C % 8 == 0, WINDQ_ERR_SHAPE, "windq_act_stats_noalloc: C = %lld is not a multiple of 8", (long long)C);
  WINDQ_REQUIRE(ctx, ldx >= C, WINDQ_ERR_SHAPE, "windq_act_stats_noalloc: ldx = %lld is below C = %lld", (long long)ldx,
                (long long)C);
  WINDQ_REQUIRE(ctx, ldx % 8 == 0, WINDQ_ERR_ALIGN, "windq_act_stats_noalloc: ldx = %lld is not a multiple of 8",
                (long long)ldx);
  WINDQ_REQUIRE(ctx, aligned16(X), WINDQ_ERR_ALIGN, "windq_act_stats_noalloc: X is not 16-byte aligned");
  WINDQ_REQUIRE(ctx, act_slices(T) <= kActMaxSlices, WINDQ_ERR_SHAPE, "windq_act_stats_noalloc: T = %lld is too large", (long long)T);
  const int64_t need = windq_scratch_bytes_act_stats(T, C);
  WINDQ_REQUIRE(ctx, need <= (int64_t)WINDQ_NOALLOC_SCRATCH_BYTES, WINDQ_ERR_SCRATCH,
                "windq_act_stats_noalloc: T = %lld, C = %lld needs %lld bytes of scratch, the built-in array has %lld; "
                "use windq_act_stats or split the tokens",
                (long long)T, (long long)C, (long long)need, (long long)WINDQ_NOALLOC_SCRATCH_BYTES);
  WINDQ_REQUIRE(ctx, ctx->device < kNoallocMaxDevices, WINDQ_ERR_UNSUPPORTED,
                "windq_act_stats_noalloc: device %d is beyond the %d devices this entry point keeps addresses for",
                ctx->device, kNoallocMaxDevices);
  const int slices = (int)act_slices(T);
  DeviceGuard guard(ctx->device);
  float* partial = nullptr;
  WINDQ_CUDA(ctx, noalloc_scratch(ctx->device, &partial));
  const int rows_per_slice = kActRowsPar * kActMaxRowsPerThread;
  cudaStream_t st = (cudaStream_t)stream;
  dim3 grid((unsigned)((C + kActCols - 1) / kActCols), (unsigned)slices);
  // every partial[slice][channel] that the second kernel reads is written by the first one, so
  // nothing left in the array by an earlier call is ever read and nothing needs clearing
  act_partial_kernel<<<grid, 256, 0, st>>>((const __half*)X, T, (int)C, ldx, rows_per_slice, partial);
  WINDQ_CUDA(ctx, cudaGetLastError());
  act_finalize_kernel<<<(unsigned)((C + 255) / 256), 256, 0, st>>>(partial, slices, (int)C, 1.0 / (double)T, s_out);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

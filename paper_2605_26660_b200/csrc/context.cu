// Context life cycle, error reporting and the host-side argument checks.
#include <stdarg.h>
#include <string.h>

#include "fit_device.cuh"

namespace {
thread_local char g_create_error[256] = "";

// Every positive finite fp16 value: the fast reciprocal of the fits against IEEE division.
__global__ void selfcheck_reciprocal_kernel(unsigned long long* n_bad) {
  const int h = blockIdx.x * blockDim.x + threadIdx.x;
  if (h < 1 || h >= 0x7c00) return;
  const float x = __half2float(__ushort_as_half((unsigned short)h));
  if (windq::reciprocal_of_half_value(x) != __fdiv_rn(1.0f, x)) atomicAdd(n_bad, 1ull);
}
}

namespace windq {

windq_status fail(windq_ctx* ctx, windq_status st, const char* fmt, ...) {
  char* dst = ctx ? ctx->err : g_create_error;
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(dst, 256, fmt, ap);
  va_end(ap);
  return st;
}

windq_status ensure_scratch(windq_ctx* ctx, int64_t bytes) {
  if (bytes <= ctx->scratch_bytes) return WINDQ_OK;
  const int64_t want = round_up(bytes, 1 << 20);
  void* p = nullptr;
  if (cudaMalloc(&p, (size_t)want) != cudaSuccess) {
    cudaGetLastError();
    return fail(ctx, WINDQ_ERR_SCRATCH, "cannot grow scratch to %lld bytes", (long long)want);
  }
  if (ctx->scratch) {
    // earlier calls may still be using the old buffer on some stream
    cudaDeviceSynchronize();
    cudaFree(ctx->scratch);
  }
  ctx->scratch = p;
  ctx->scratch_bytes = want;
  return WINDQ_OK;
}

windq_status check_matrix(windq_ctx* ctx, const char* who, const void* W, int64_t R, int64_t C, int64_t ldw, int G) {
  WINDQ_REQUIRE(ctx, W != nullptr, WINDQ_ERR_NULL, "%s: W is NULL", who);
  WINDQ_REQUIRE(ctx, valid_G(G), WINDQ_ERR_ARG, "%s: G = %d is not one of 32, 64, 128, 256, 512", who, G);
  WINDQ_REQUIRE(ctx, R > 0 && C > 0, WINDQ_ERR_SHAPE, "%s: R = %lld, C = %lld must be positive", who, (long long)R,
                (long long)C);
  WINDQ_REQUIRE(ctx, R < (1ll << 31) && C < (1ll << 31), WINDQ_ERR_SHAPE, "%s: R and C must be below 2^31", who);
  WINDQ_REQUIRE(ctx, C % G == 0, WINDQ_ERR_SHAPE, "%s: C = %lld is not a multiple of G = %d", who, (long long)C, G);
  WINDQ_REQUIRE(ctx, ldw >= C, WINDQ_ERR_SHAPE, "%s: ldw = %lld is below C = %lld", who, (long long)ldw, (long long)C);
  WINDQ_REQUIRE(ctx, ldw % 8 == 0, WINDQ_ERR_ALIGN, "%s: ldw = %lld is not a multiple of 8", who, (long long)ldw);
  WINDQ_REQUIRE(ctx, aligned16(W), WINDQ_ERR_ALIGN, "%s: W is not 16-byte aligned", who);
  return WINDQ_OK;
}

windq_status check_K(windq_ctx* ctx, const char* who, int K) {
  WINDQ_REQUIRE(ctx, K >= 1 && K <= 64, WINDQ_ERR_ARG, "%s: K = %d is outside [1, 64]", who, K);
  return WINDQ_OK;
}

}  // namespace windq

extern "C" {

windq_status windq_create(windq_ctx** out, int device) {
  if (!out) return windq::fail(nullptr, WINDQ_ERR_NULL, "windq_create: out is NULL");
  *out = nullptr;
  int n = 0;
  if (cudaGetDeviceCount(&n) != cudaSuccess || n == 0) {
    cudaGetLastError();
    return windq::fail(nullptr, WINDQ_ERR_CUDA, "windq_create: no CUDA device");
  }
  if (device < 0 || device >= n)
    return windq::fail(nullptr, WINDQ_ERR_ARG, "windq_create: device %d of %d", device, n);
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) {
    cudaGetLastError();
    return windq::fail(nullptr, WINDQ_ERR_CUDA, "windq_create: cannot query device %d", device);
  }
  if (prop.major != 10)
    return windq::fail(nullptr, WINDQ_ERR_UNSUPPORTED, "windq_create: device %d is sm_%d%d, this library is built for sm_100a",
                       device, prop.major, prop.minor);
  unsigned int* sync = nullptr;
  {
    windq::DeviceGuard guard(device);
    if (cudaMalloc(&sync, windq::kSyncBytes) != cudaSuccess || cudaMemset(sync, 0, windq::kSyncBytes) != cudaSuccess) {
      cudaGetLastError();
      if (sync) cudaFree(sync);
      return windq::fail(nullptr, WINDQ_ERR_CUDA, "windq_create: cannot allocate the arrival counters on device %d", device);
    }
  }
  windq_ctx* ctx = new windq_ctx;
  ctx->device = device;
  ctx->sync = sync;
  ctx->sm_count = prop.multiProcessorCount;
  ctx->scratch = nullptr;
  ctx->scratch_bytes = 0;
  ctx->prepared[0] = ctx->prepared[1] = 0;
  memset(ctx->occupancy, 0, sizeof(ctx->occupancy));
  ctx->err[0] = 0;
  *out = ctx;
  return WINDQ_OK;
}

void windq_destroy(windq_ctx* ctx) {
  if (!ctx) return;
  {
    windq::DeviceGuard guard(ctx->device);
    cudaDeviceSynchronize();
    if (ctx->scratch) cudaFree(ctx->scratch);
    cudaFree(ctx->sync);
  }
  delete ctx;
}

const char* windq_last_error(const windq_ctx* ctx) { return ctx ? ctx->err : g_create_error; }

windq_status windq_selfcheck(windq_ctx* ctx, int64_t* n_failures_out, void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "windq_selfcheck: ctx is NULL");
  WINDQ_REQUIRE(ctx, n_failures_out, WINDQ_ERR_NULL, "windq_selfcheck: n_failures_out is NULL");
  WINDQ_REQUIRE(ctx, ((uintptr_t)n_failures_out & 7) == 0, WINDQ_ERR_ALIGN, "windq_selfcheck: n_failures_out is misaligned");
  DeviceGuard guard(ctx->device);
  cudaStream_t st = (cudaStream_t)stream;
  WINDQ_CUDA(ctx, cudaMemsetAsync(n_failures_out, 0, sizeof(int64_t), st));
  selfcheck_reciprocal_kernel<<<0x7c00 / 256, 256, 0, st>>>((unsigned long long*)n_failures_out);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

windq_status windq_fit_work(windq_ctx* ctx, int64_t* evaluated_out, int64_t* searched_out, int reset) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "windq_fit_work: ctx is NULL");
  WINDQ_REQUIRE(ctx, evaluated_out && searched_out, WINDQ_ERR_NULL, "windq_fit_work: evaluated_out or searched_out is NULL");
  DeviceGuard guard(ctx->device);
  unsigned long long host[2] = {0, 0};
  WINDQ_CUDA(ctx, cudaMemcpy(host, fit_work_counters(ctx), sizeof(host), cudaMemcpyDeviceToHost));
  if (reset) WINDQ_CUDA(ctx, cudaMemset(fit_work_counters(ctx), 0, sizeof(host)));
  *evaluated_out = (int64_t)host[0];
  *searched_out = (int64_t)host[1];
  return WINDQ_OK;
}

windq_status windq_reserve(windq_ctx* ctx, int64_t bytes) {
  if (!ctx) return windq::fail(nullptr, WINDQ_ERR_NULL, "windq_reserve: ctx is NULL");
  WINDQ_REQUIRE(ctx, bytes >= 0, WINDQ_ERR_ARG, "windq_reserve: bytes = %lld", (long long)bytes);
  windq::DeviceGuard guard(ctx->device);
  return windq::ensure_scratch(ctx, bytes);
}

}  // extern "C"

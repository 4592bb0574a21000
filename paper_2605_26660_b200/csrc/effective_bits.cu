// windq_effective_bits: storage cost of a plan (Eq. 6 with no protected weights, plus the scale /
// zero-point overhead of every group) and the byte offsets of the packed blocks.
//
// Integer work on at most a few tens of thousands of units: one block, a running exclusive scan
// over chunks of 1024 units.  All arithmetic is int64, so totals are exact.
#include <string.h>

#include "windq_internal.cuh"

namespace windq {

__device__ __forceinline__ long long unit_cost_centibits(int a, long long R, int G, int scale_bits, int zero_bits) {
  const long long n = R * G;
  const long long sz = 100ll * R * (scale_bits + zero_bits), sc = 100ll * R * scale_bits;
  switch (a) {
    case 0: return 1600 * n;
    case 1: return 800 * n + sz;
    case 2: return 400 * n + sz;
    case 3: return 300 * n + sz;
    case 4: return 200 * n + sz;
    case 5: return 158 * n + sc;
    case 6: return 100 * n + sc;
  }
  return -1;
}

// One plan, by one block of 1024 threads.
__device__ __forceinline__ void effective_bits_block(const uint8_t* __restrict__ actions, long long U, long long R, int G,
                                                     int scale_bits, int zero_bits, long long* __restrict__ unit_cb,
                                                     long long* __restrict__ offsets, long long* __restrict__ total_cb,
                                                     long long* __restrict__ total_bytes) {
  __shared__ long long scan[1024];
  __shared__ long long red[3][32];
  __shared__ int bad_flag;
  const int t = threadIdx.x;
  if (t == 0) bad_flag = 0;
  __syncthreads();
  long long carry = 0, sum_cb = 0, n_params = 0;
  for (long long base = 0; base < U; base += 1024) {
    const long long u = base + t;
    long long bytes = 0;
    if (u < U) {
      const int a = actions[u];
      const long long cb = unit_cost_centibits(a, R, G, scale_bits, zero_bits);
      if (cb < 0) bad_flag = 1;
      else {
        sum_cb += cb;
        bytes = (R * group_code_bytes(a, G) + 15) / 16 * 16;
        n_params += (a >= 1 ? R : 0) + ((a >= 1 && a <= 4) ? R : 0);
      }
      if (unit_cb) unit_cb[u] = cb;
    }
    // inclusive scan of the 1024 byte counts: inside each warp, then over the 32 warp totals
    long long incl = bytes;
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) {
      const long long o = __shfl_up_sync(0xffffffffu, incl, m);
      if ((t & 31) >= m) incl += o;
    }
    if ((t & 31) == 31) scan[t >> 5] = incl;
    __syncthreads();
    if (t < 32) {
      long long w = scan[t];
#pragma unroll
      for (int m = 1; m < 32; m <<= 1) {
        const long long o = __shfl_up_sync(0xffffffffu, w, m);
        if (t >= m) w += o;
      }
      scan[32 + t] = w;
    }
    __syncthreads();
    incl += (t >> 5) ? scan[32 + (t >> 5) - 1] : 0ll;
    const long long chunk_total = scan[63];
    if (u < U && offsets) offsets[u] = carry + incl - bytes;
    carry += chunk_total;
    __syncthreads();
  }
#pragma unroll
  for (int m = 16; m > 0; m >>= 1) {
    sum_cb += __shfl_xor_sync(0xffffffffu, sum_cb, m);
    n_params += __shfl_xor_sync(0xffffffffu, n_params, m);
  }
  if ((t & 31) == 0) { red[0][t >> 5] = sum_cb; red[1][t >> 5] = n_params; }
  __syncthreads();
  if (t == 0) {
    long long a = 0, b = 0;
    for (int i = 0; i < 32; ++i) { a += red[0][i]; b += red[1][i]; }
    if (offsets) offsets[U] = carry;
    *total_cb = bad_flag ? -1 : a;
    if (total_bytes) *total_bytes = bad_flag ? -1 : carry + 2 * b;
  }
}

__global__ void __launch_bounds__(1024)
effective_bits_kernel(const uint8_t* __restrict__ actions, long long U, long long R, int G, int scale_bits, int zero_bits,
                      long long* __restrict__ unit_cb, long long* __restrict__ offsets, long long* __restrict__ total_cb,
                      long long* __restrict__ total_bytes) {
  effective_bits_block(actions, U, R, G, scale_bits, zero_bits, unit_cb, offsets, total_cb, total_bytes);
}

// Several plans in one launch (windq_effective_bits_batch): block j does job j.
constexpr int kBitsMaxJobs = 32;
struct BitsJobs {
  const uint8_t* actions[kBitsMaxJobs];
  long long* unit_cb[kBitsMaxJobs];
  long long* offsets[kBitsMaxJobs];
  long long* total_cb[kBitsMaxJobs];
  long long* total_bytes[kBitsMaxJobs];
  long long U[kBitsMaxJobs];
  long long R[kBitsMaxJobs];
};

__global__ void __launch_bounds__(1024)
effective_bits_batch_kernel(const BitsJobs jobs, int G, int scale_bits, int zero_bits) {
  const int j = blockIdx.x;
  effective_bits_block(jobs.actions[j], jobs.U[j], jobs.R[j], G, scale_bits, zero_bits, jobs.unit_cb[j], jobs.offsets[j],
                       jobs.total_cb[j], jobs.total_bytes[j]);
}

}  // namespace windq

extern "C" windq_status windq_effective_bits(windq_ctx* ctx, const uint8_t* actions, int64_t U, int64_t R, int G,
                                             int scale_bits, int zero_bits, int64_t* unit_centibits_out,
                                             int64_t* code_offsets_out, int64_t* total_centibits_out,
                                             int64_t* total_packed_bytes_out, void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "windq_effective_bits: ctx is NULL");
  WINDQ_REQUIRE(ctx, actions && total_centibits_out, WINDQ_ERR_NULL,
                "windq_effective_bits: actions or total_centibits_out is NULL");
  WINDQ_REQUIRE(ctx, U > 0 && R > 0, WINDQ_ERR_SHAPE, "windq_effective_bits: U = %lld, R = %lld must be positive",
                (long long)U, (long long)R);
  WINDQ_REQUIRE(ctx, U < (1ll << 31) && R < (1ll << 31), WINDQ_ERR_SHAPE, "windq_effective_bits: U and R must be below 2^31");
  WINDQ_REQUIRE(ctx, valid_G(G), WINDQ_ERR_ARG, "windq_effective_bits: G = %d is not one of 32, 64, 128, 256, 512", G);
  WINDQ_REQUIRE(ctx, scale_bits >= 0 && scale_bits <= 64 && zero_bits >= 0 && zero_bits <= 64, WINDQ_ERR_ARG,
                "windq_effective_bits: scale_bits = %d, zero_bits = %d must be in [0, 64]", scale_bits, zero_bits);
  WINDQ_REQUIRE(ctx, ((uintptr_t)unit_centibits_out & 7) == 0 && ((uintptr_t)code_offsets_out & 7) == 0 &&
                         ((uintptr_t)total_centibits_out & 7) == 0 && ((uintptr_t)total_packed_bytes_out & 7) == 0,
                WINDQ_ERR_ALIGN, "windq_effective_bits: an int64 output is not 8-byte aligned");
  DeviceGuard guard(ctx->device);
  effective_bits_kernel<<<1, 1024, 0, (cudaStream_t)stream>>>(
      actions, (long long)U, (long long)R, G, scale_bits, zero_bits, (long long*)unit_centibits_out,
      (long long*)code_offsets_out, (long long*)total_centibits_out, (long long*)total_packed_bytes_out);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

extern "C" windq_status windq_effective_bits_batch(windq_ctx* ctx, const windq_bits_job* jobs, int n_jobs, int G, int scale_bits,
                                                   int zero_bits, void* stream) {
  using namespace windq;
  const char* who = "windq_effective_bits_batch";
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "%s: ctx is NULL", who);
  WINDQ_REQUIRE(ctx, jobs, WINDQ_ERR_NULL, "%s: jobs is NULL", who);
  WINDQ_REQUIRE(ctx, n_jobs >= 1 && n_jobs <= kBitsMaxJobs, WINDQ_ERR_SHAPE, "%s: n_jobs = %d is outside [1, %d]", who, n_jobs,
                kBitsMaxJobs);
  WINDQ_REQUIRE(ctx, valid_G(G), WINDQ_ERR_ARG, "%s: G = %d is not one of 32, 64, 128, 256, 512", who, G);
  WINDQ_REQUIRE(ctx, scale_bits >= 0 && scale_bits <= 64 && zero_bits >= 0 && zero_bits <= 64, WINDQ_ERR_ARG,
                "%s: scale_bits = %d, zero_bits = %d must be in [0, 64]", who, scale_bits, zero_bits);
  BitsJobs bj;
  memset(&bj, 0, sizeof(bj));
  for (int j = 0; j < n_jobs; ++j) {
    const windq_bits_job& b = jobs[j];
    WINDQ_REQUIRE(ctx, b.actions && b.total_centibits_out, WINDQ_ERR_NULL, "%s: job %d: actions or total_centibits_out is NULL", who, j);
    WINDQ_REQUIRE(ctx, b.U > 0 && b.R > 0 && b.U < (1ll << 31) && b.R < (1ll << 31), WINDQ_ERR_SHAPE,
                  "%s: job %d: U = %lld, R = %lld must be positive and below 2^31", who, j, (long long)b.U, (long long)b.R);
    WINDQ_REQUIRE(ctx, ((uintptr_t)b.unit_centibits_out & 7) == 0 && ((uintptr_t)b.code_offsets_out & 7) == 0 &&
                           ((uintptr_t)b.total_centibits_out & 7) == 0 && ((uintptr_t)b.total_packed_bytes_out & 7) == 0,
                  WINDQ_ERR_ALIGN, "%s: job %d: an int64 output is not 8-byte aligned", who, j);
    bj.actions[j] = b.actions;
    bj.unit_cb[j] = (long long*)b.unit_centibits_out;
    bj.offsets[j] = (long long*)b.code_offsets_out;
    bj.total_cb[j] = (long long*)b.total_centibits_out;
    bj.total_bytes[j] = (long long*)b.total_packed_bytes_out;
    bj.U[j] = b.U;
    bj.R[j] = b.R;
  }
  DeviceGuard guard(ctx->device);
  effective_bits_batch_kernel<<<(unsigned)n_jobs, 1024, 0, (cudaStream_t)stream>>>(bj, G, scale_bits, zero_bits);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

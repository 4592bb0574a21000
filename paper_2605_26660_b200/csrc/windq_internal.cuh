// Internal declarations shared by the windq translation units: the context, host-side argument
// checks and small device helpers.  Nothing here is part of the ABI.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "windq.h"

struct windq_ctx {
  int device;
  int sm_count;
  void* scratch;
  int64_t scratch_bytes;
  unsigned int* sync;  // kSyncCounters arrival counters, zero between launches; two 64-bit work counters follow them
  unsigned long long prepared[2];  // kernels whose attributes have been set on this context's device (bit per KernelId)
  int occupancy[128];              // resident blocks per SM of those kernels (0 where not asked)
  char err[256];
};

namespace windq {

constexpr int64_t kSyncCounters = 16384;
constexpr int64_t kSyncBytes = kSyncCounters * (int64_t)sizeof(unsigned int) + 2 * (int64_t)sizeof(unsigned long long);

windq_status fail(windq_ctx* ctx, windq_status st, const char* fmt, ...);
// Where the fits count their clip candidates: [0] those evaluated in full, [1] all of them (see windq_fit_work).
inline unsigned long long* fit_work_counters(windq_ctx* ctx) {
  return reinterpret_cast<unsigned long long*>(ctx->sync + kSyncCounters);
}
// Makes the context's scratch at least `bytes` large (may cudaMalloc).
windq_status ensure_scratch(windq_ctx* ctx, int64_t bytes);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool valid_G(int G) { return G == 32 || G == 64 || G == 128 || G == 256 || G == 512; }
inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }

// Switches to the context's device for the lifetime of the object.
struct DeviceGuard {
  int prev = -1;
  bool switched = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = (cudaSetDevice(dev) == cudaSuccess);
  }
  ~DeviceGuard() {
    if (switched) cudaSetDevice(prev);
  }
};

#define WINDQ_REQUIRE(ctx, cond, st, ...) \
  do {                                    \
    if (!(cond)) return ::windq::fail((ctx), (st), __VA_ARGS__); \
  } while (0)

#define WINDQ_CUDA(ctx, call)                                                                      \
  do {                                                                                             \
    cudaError_t e_ = (call);                                                                       \
    if (e_ != cudaSuccess) return ::windq::fail((ctx), WINDQ_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

// One bit per kernel instantiation that needs a function attribute or an occupancy figure.  Function
// attributes belong to a device, so the record is kept in the context, not in a process-wide static.
enum KernelId { kFitG32 = 0, kApplyG32 = 5, kApplySearchG32 = 10, kHistG32 = 15, kFinalize = 20, kFitProtectG32 = 21, kApplyProtectG32 = 26, kApplyProtectSearchG32 = 31,
                kFitBatchG32 = 41 /* 41..45 whole items, 46..50 in parts */, kApplyBatchG32 = 51 /* 51..55 */, kFitPartsOffset = 36 /* kFitG32 + 36 .. and kFitProtectG32 + 36 ..: the in-parts instantiations (36..40, 57..61) */,
                kApplyStreamG32 = 64 /* 64..68 */, kFitFeatG32 = 79 /* 79..83 whole items, 84..88 in parts */, kTernarySearchG32 = 69 /* 69..73 plain, 74..78 protected */, kFinalize2 = 89, kKernelIds = 128 };
inline int g_index(int G) { return G == 32 ? 0 : G == 64 ? 1 : G == 128 ? 2 : G == 256 ? 3 : 4; }

// Sets the dynamic shared-memory limit of `kernel` once per context and, if asked, records how many
// of its blocks fit on an SM.
template <class K>
windq_status prepare_kernel(windq_ctx* ctx, int id, K kernel, int threads, size_t smem, bool want_occupancy) {
  if (ctx->prepared[id >> 6] & (1ull << (id & 63))) return WINDQ_OK;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    cudaGetLastError();
    return fail(ctx, WINDQ_ERR_CUDA, "cannot reserve %lld bytes of shared memory per block", (long long)smem);
  }
  if (want_occupancy) {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, smem) != cudaSuccess) {
      cudaGetLastError();
      return fail(ctx, WINDQ_ERR_CUDA, "occupancy query failed");
    }
    ctx->occupancy[id] = n > 0 ? n : 1;
  }
  ctx->prepared[id >> 6] |= 1ull << (id & 63);
  return WINDQ_OK;
}

// Checks shared by the calls that take a weight matrix.
windq_status check_matrix(windq_ctx* ctx, const char* who, const void* W, int64_t R, int64_t C, int64_t ldw, int G);
// The clip grid lives on the device and is used as given; only K can be checked on the host.
windq_status check_K(windq_ctx* ctx, const char* who, int K);

// The streaming plan kernel (apply_stream.cu): one matrix, n_plans plans, clip indices supplied; scale_in, thr_grid,
// thr_idx and lowbit may be NULL.  Arguments must have been checked.
windq_status launch_apply_stream(windq_ctx* ctx, int G, const void* W, int64_t R, int64_t C, int64_t ldw, const float* s,
                                 const float* clip_grid, int K, const uint8_t* clip_idx, const void* scale_in,
                                 const float* thr_grid, int thr_K, const uint8_t* thr_idx, const void* lowbit,
                                 const windq_plan_out* plans, int n_plans, cudaStream_t st);

// The state features of every unit of n_jobs matrices from per-unit histograms of |w| bit patterns (32768 bins each,
// units of all jobs in a row) and per-unit sums of w, as the fused fit pass leaves them (unit_features.cu).
windq_status features_from_histograms(windq_ctx* ctx, const unsigned int* hist, const double* unit_wsum, int n_jobs, const int* R,
                                      const int* first_unit, const float* const* s, float* const* feat_out, int G, cudaStream_t st);

// Bytes of one packed group under an action (host and device).
__host__ __device__ inline int group_code_bytes(int action, int G) {
  switch (action) {
    case 0: return 2 * G;
    case 1: return G;
    case 2: return G / 2;
    case 3: return 3 * G / 8;
    case 4: return G / 4;
    case 5: return (G + 4) / 5;
    case 6: return G / 8;
  }
  return 0;
}

}  // namespace windq

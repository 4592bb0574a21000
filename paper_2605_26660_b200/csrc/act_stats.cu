// windq_act_stats: s_j = mean_t x_tj^2 over a calibration input X[T][C] (fp16).
//
// One streaming pass, bound by HBM: 2 bytes read per element.  A block covers 256 adjacent
// channels (512 contiguous bytes per row, one 128-bit load per thread) and a slice of the
// tokens; its 8 thread rows walk the slice with a stride of 8 rows.  Sums of at most 8 squares are formed in
// fp32, everything above them in double and in a fixed order, so the result does not depend on scheduling.
// windq_act_stats and windq_act_stats_batch take ONE launch (act_stats_kernel: slices long enough that a large
// input is one wave of blocks, eight loads in flight per thread, and the block that arrives last at a group of
// 256 channels adds that group's slices).  The two-kernel form before it (64-row slices whose sums a second
// launch adds) serves windq_act_stats_noalloc, and inputs with more channel groups than the context has
// arrival counters.
#include <string.h>

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

// ---- one launch for up to WINDQ_MAX_ACT_JOBS inputs ---------------------------------------------
constexpr int kActRowsPerChunk = kActRowsPar * kActMaxRowsPerThread;  // 64: rows a block reads before it converts to double
constexpr int kActTargetBlocks = 592;  // blocks a large input is cut into: four per SM of a 148-SM part

struct ActJobs {
  const __half* X[WINDQ_MAX_ACT_JOBS];
  float* s_out[WINDQ_MAX_ACT_JOBS];
  int64_t T[WINDQ_MAX_ACT_JOBS], ldx[WINDQ_MAX_ACT_JOBS];
  int64_t partial_at[WINDQ_MAX_ACT_JOBS];  // where the job's [slices][C] partial sums start in the scratch, in floats
  double inv_T[WINDQ_MAX_ACT_JOBS];
  int C[WINDQ_MAX_ACT_JOBS], col_blocks[WINDQ_MAX_ACT_JOBS], slices[WINDQ_MAX_ACT_JOBS], rows_per_slice[WINDQ_MAX_ACT_JOBS];
  int first_counter[WINDQ_MAX_ACT_JOBS];   // the job's first arrival counter (one per block of 256 channels)
  int first_block[WINDQ_MAX_ACT_JOBS + 1]; // blocks are numbered through all jobs; within a job the channel block runs fastest
  int n_jobs;
};

// Rows per token slice of an input: a function of its shape alone, so that an input gives the same bits whatever
// else is in the call.  At least 64 rows; more when that would make more than kActTargetBlocks blocks.
inline int64_t act_rows_per_slice(int64_t T, int64_t C) {
  const int64_t col_blocks = (C + kActCols - 1) / kActCols;
  const int64_t want_slices = col_blocks >= kActTargetBlocks ? 1 : kActTargetBlocks / col_blocks;
  const int64_t rows = round_up((T + want_slices - 1) / want_slices, kActRowsPar);
  return rows < kActRowsPerChunk ? kActRowsPerChunk : rows;
}

// acc + x^2 for the two fp16 values of a word, each product exact in binary32 and added with one rounding: the
// mixed-precision fma of sm_100 takes the fp16 operands as they are (same result as converting first).
__device__ __forceinline__ void add_squares(unsigned int word, float& acc_lo, float& acc_hi) {
  asm("{\n\t"
      ".reg .b16 lo, hi;\n\t"
      "mov.b32 {lo, hi}, %2;\n\t"
      "fma.rn.f32.f16 %0, lo, lo, %0;\n\t"
      "fma.rn.f32.f16 %1, hi, hi, %1;\n\t"
      "}"
      : "+f"(acc_lo), "+f"(acc_hi)
      : "r"(word));
}

// N rows p, p + 8 ldx, ...: all loads first, then the squares of every channel added row after row in fp32, and
// the N-row sums added to the running totals in double.
template <int N>
__device__ __forceinline__ void add_rows(const __half* __restrict__ p, int64_t ldx, double (&total)[8]) {
  uint4 raw[N];
#pragma unroll
  for (int k = 0; k < N; ++k) raw[k] = __ldg(reinterpret_cast<const uint4*>(p + (int64_t)k * kActRowsPar * ldx));
  float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
  for (int k = 0; k < N; ++k) {
    add_squares(raw[k].x, acc[0], acc[1]);
    add_squares(raw[k].y, acc[2], acc[3]);
    add_squares(raw[k].z, acc[4], acc[5]);
    add_squares(raw[k].w, acc[6], acc[7]);
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) total[i] += (double)acc[i];
}

// A block adds the squares of 256 channels over its slice of the tokens: every thread 8 channels, rows ty, ty + 8,
// ...; at most 8 rows in fp32, then on in double.  Its 256 sums go to scratch as fp32; the block that arrives last
// at a group of channels adds the group's slices in double, in a fixed order, and writes the means.  arrivals[]
// holds zeros between launches: the last block to arrive at a counter puts it back.
__global__ void __launch_bounds__(256, 4)
act_stats_kernel(const __grid_constant__ ActJobs jobs, float* __restrict__ scratch, unsigned int* __restrict__ arrivals) {
  __shared__ double red[kActRowsPar][kActCols];
  __shared__ bool last_here;
  int j = 0;
  while (j + 1 < jobs.n_jobs && (int)blockIdx.x >= jobs.first_block[j + 1]) ++j;
  const int local = (int)blockIdx.x - jobs.first_block[j];
  const int cb = local % jobs.col_blocks[j], slice = local / jobs.col_blocks[j];
  const int C = jobs.C[j], slices = jobs.slices[j];
  const int64_t T = jobs.T[j], ldx = jobs.ldx[j];
  float* partial = scratch + jobs.partial_at[j];

  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int col = cb * kActCols + tx * 8;
  const int64_t t0 = (int64_t)slice * jobs.rows_per_slice[j];
  const int64_t t1 = min(t0 + jobs.rows_per_slice[j], T);
  double total[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  const int c = cb * kActCols + threadIdx.x;  // 256 threads, 256 channels
  if (col < C) {
    const int my_rows = (int)((t1 - t0 - ty + kActRowsPar - 1) / kActRowsPar);  // rows t0 + ty + 8 k below t1 (may be 0)
    const __half* p = jobs.X[j] + (t0 + ty) * ldx + col;
    int left = my_rows;
    for (; left >= kActMaxRowsPerThread; left -= kActMaxRowsPerThread, p += (int64_t)kActRowsPerChunk * ldx)
      add_rows<kActMaxRowsPerThread>(p, ldx, total);
    switch (left) {  // the same for all lanes of a warp
      case 7: add_rows<7>(p, ldx, total); break;
      case 6: add_rows<6>(p, ldx, total); break;
      case 5: add_rows<5>(p, ldx, total); break;
      case 4: add_rows<4>(p, ldx, total); break;
      case 3: add_rows<3>(p, ldx, total); break;
      case 2: add_rows<2>(p, ldx, total); break;
      case 1: add_rows<1>(p, ldx, total); break;
      default: break;
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) red[ty][tx * 8 + i] = total[i];
  __syncthreads();
  if (c < C) {
    double sum = 0.0;
#pragma unroll
    for (int r = 0; r < kActRowsPar; ++r) sum += red[r][threadIdx.x];
    partial[(int64_t)slice * C + c] = (float)sum;
  }
  // the last block to arrive at this group of channels adds its slices.  One thread orders the block's stores
  // before its arrival, and the other blocks' stores before this block's loads (the barriers carry both to the
  // rest of the block).
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    unsigned int* a = arrivals + jobs.first_counter[j] + cb;
    last_here = atomicAdd(a, 1u) == (unsigned int)(slices - 1);
    if (last_here) *a = 0u;  // nobody else comes to this counter in this launch
    __threadfence();
  }
  __syncthreads();
  if (!last_here) return;
  // thread row ty adds slices ty, ty + 8, ... (four loads in flight), then the rows' sums are added in order.
  // (The barrier above also says that the block's own sums have been read from red[].)
#pragma unroll
  for (int half = 0; half < 2; ++half) {  // channels col .. col + 3, then col + 4 .. col + 7
    double tot[4] = {0, 0, 0, 0};
    if (col < C) {
      const float* q = partial + col + 4 * half;
      for (int i = ty; i < slices; i += 4 * kActRowsPar) {
        float4 v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int sl = i + k * kActRowsPar;
          v[k] = sl < slices ? __ldcg(reinterpret_cast<const float4*>(q + (int64_t)sl * C)) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          tot[0] += (double)v[k].x; tot[1] += (double)v[k].y; tot[2] += (double)v[k].z; tot[3] += (double)v[k].w;
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) red[ty][tx * 8 + 4 * half + i] = tot[i];
  }
  __syncthreads();
  if (c < C) {
    double sum = 0.0;
#pragma unroll
    for (int r = 0; r < kActRowsPar; ++r) sum += red[r][threadIdx.x];
    jobs.s_out[j][c] = (float)(sum * jobs.inv_T[j]);
  }
}

constexpr int64_t kActMaxSlices = 65535;  // grid.y limit

// Token slices of a call (64 rows each), as a 64-bit count: callers compare it with kActMaxSlices
// before they narrow it.
inline int64_t act_slices(int64_t T) {
  const int64_t rows_per_slice = (int64_t)kActRowsPar * kActMaxRowsPerThread;
  return (T + rows_per_slice - 1) / rows_per_slice;
}

// Argument checks of one input, shared by the single and the batched call.
static windq_status check_act_job(windq_ctx* ctx, const char* who, const windq_act_job& job) {
  const int64_t T = job.T, C = job.C, ldx = job.ldx;
  WINDQ_REQUIRE(ctx, job.X && job.s_out, WINDQ_ERR_NULL, "%s: X or s_out is NULL", who);
  WINDQ_REQUIRE(ctx, T > 0 && C > 0, WINDQ_ERR_SHAPE, "%s: T = %lld, C = %lld must be positive", who, (long long)T, (long long)C);
  WINDQ_REQUIRE(ctx, C < (1ll << 31) && T < (1ll << 40), WINDQ_ERR_SHAPE, "%s: T or C too large", who);
  WINDQ_REQUIRE(ctx, C % 8 == 0, WINDQ_ERR_SHAPE, "%s: C = %lld is not a multiple of 8", who, (long long)C);
  WINDQ_REQUIRE(ctx, ldx >= C, WINDQ_ERR_SHAPE, "%s: ldx = %lld is below C = %lld", who, (long long)ldx, (long long)C);
  WINDQ_REQUIRE(ctx, ldx % 8 == 0, WINDQ_ERR_ALIGN, "%s: ldx = %lld is not a multiple of 8", who, (long long)ldx);
  WINDQ_REQUIRE(ctx, aligned16(job.X), WINDQ_ERR_ALIGN, "%s: X is not 16-byte aligned", who);
  WINDQ_REQUIRE(ctx, act_slices(T) <= kActMaxSlices, WINDQ_ERR_SHAPE, "%s: T = %lld is too large (at most %lld tokens per call)", who,
                (long long)T, (long long)(kActMaxSlices * kActRowsPar * kActMaxRowsPerThread));
  return WINDQ_OK;
}

// One launch for checked jobs whose groups of 256 channels number at most kSyncCounters; the context's device is current.
static windq_status launch_act_jobs(windq_ctx* ctx, const windq_act_job* jobs, int n_jobs, cudaStream_t st) {
  ActJobs a;
  memset(&a, 0, sizeof(a));
  a.n_jobs = n_jobs;
  int64_t floats = 0, blocks = 0;
  int counters = 0;
  for (int j = 0; j < n_jobs; ++j) {
    a.X[j] = (const __half*)jobs[j].X;
    a.s_out[j] = jobs[j].s_out;
    a.T[j] = jobs[j].T;
    a.ldx[j] = jobs[j].ldx;
    a.inv_T[j] = 1.0 / (double)jobs[j].T;
    a.C[j] = (int)jobs[j].C;
    a.col_blocks[j] = (int)((jobs[j].C + kActCols - 1) / kActCols);
    a.rows_per_slice[j] = (int)act_rows_per_slice(jobs[j].T, jobs[j].C);
    a.slices[j] = (int)((jobs[j].T + a.rows_per_slice[j] - 1) / a.rows_per_slice[j]);
    a.partial_at[j] = floats;
    a.first_counter[j] = counters;
    a.first_block[j] = (int)blocks;
    floats += (int64_t)a.slices[j] * jobs[j].C;
    counters += a.col_blocks[j];
    blocks += (int64_t)a.slices[j] * a.col_blocks[j];
    WINDQ_REQUIRE(ctx, blocks < (1ll << 31), WINDQ_ERR_SHAPE, "windq_act_stats: T * C is too large for one call");
  }
  a.first_block[n_jobs] = (int)blocks;
  if (windq_status s = ensure_scratch(ctx, floats * (int64_t)sizeof(float))) return s;
  act_stats_kernel<<<(unsigned)blocks, 256, 0, st>>>(a, (float*)ctx->scratch, ctx->sync);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
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
  const windq_act_job job = {X, T, C, ldx, s_out};
  if (windq_status st = check_act_job(ctx, "windq_act_stats", job)) return st;
  DeviceGuard guard(ctx->device);
  if ((C + kActCols - 1) / kActCols <= kSyncCounters) return launch_act_jobs(ctx, &job, 1, (cudaStream_t)stream);
  // more groups of channels than arrival counters: partial sums, then a second launch that adds them
  const int slices = (int)act_slices(T);
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

int64_t windq_scratch_bytes_act_stats_batch(const windq_act_job* jobs, int n_jobs) {
  if (!jobs || n_jobs < 1 || n_jobs > WINDQ_MAX_ACT_JOBS) return 0;
  int64_t bytes = 0;
  for (int j = 0; j < n_jobs; ++j) {
    const int64_t one = windq_scratch_bytes_act_stats(jobs[j].T, jobs[j].C);
    if (one == 0) return 0;
    bytes += one;
  }
  return bytes;
}

windq_status windq_act_stats_batch(windq_ctx* ctx, const windq_act_job* jobs, int n_jobs, void* stream) {
  using namespace windq;
  const char* who = "windq_act_stats_batch";
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "%s: ctx is NULL", who);
  WINDQ_REQUIRE(ctx, jobs, WINDQ_ERR_NULL, "%s: jobs is NULL", who);
  WINDQ_REQUIRE(ctx, n_jobs >= 1 && n_jobs <= WINDQ_MAX_ACT_JOBS, WINDQ_ERR_ARG, "%s: n_jobs = %d is outside [1, %d]", who, n_jobs,
                WINDQ_MAX_ACT_JOBS);
  int64_t groups = 0;
  for (int j = 0; j < n_jobs; ++j) {
    if (windq_status st = check_act_job(ctx, who, jobs[j])) return st;
    groups += (jobs[j].C + kActCols - 1) / kActCols;
  }
  WINDQ_REQUIRE(ctx, groups <= kSyncCounters, WINDQ_ERR_SHAPE, "%s: %lld channels in all, at most %lld per call", who,
                (long long)(groups * kActCols), (long long)kSyncCounters * kActCols);
  DeviceGuard guard(ctx->device);
  return launch_act_jobs(ctx, jobs, n_jobs, (cudaStream_t)stream);
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

// windq_unit_features: Table 1 state features (dims 0-4 and 9-11) of every unit.
//
// The magnitude of an fp16 number has 32768 possible bit patterns and their integer order is
// their numeric order, so ONE histogram of |w| per unit gives the nearest-rank P99, the count
// above 0.5 * P99 and the count below 1e-6 exactly, and also sum |w| and sum w^2 exactly up to
// double rounding.  One streaming pass over W (2 bytes per weight, bound by HBM):
//   pass 1  one block of 1024 threads per SM.  The U * R (unit, row) pairs, unit-major, are cut
//           into equal contiguous shares, one per block, so a block meets two or three units at
//           most.  It keeps the current unit's histogram in shared memory (128 KB) and, when the
//           unit ends, adds the non-empty bins to the unit's histogram in scratch with integer
//           atomics (order-independent, hence exact and reproducible).  Every thread has four
//           128-bit loads in flight before it touches the histogram: with one block per SM that
//           is what keeps enough bytes on their way from HBM.  The signed sum of every
//           (unit, block) segment goes to its own slot in scratch as a double.
//   pass 2  one block per unit scans the histogram and writes the eight features.
#include <string.h>

#include "windq_internal.cuh"

namespace windq {

constexpr int kBins = 32768;
constexpr int kFeatThreads = 1024;
constexpr int kFeatMaxBlocks = 1024;  // bound on the pass-1 grid that the scratch size assumes
constexpr int kFeatLoads = 4;  // rows in flight per thread

// Several matrices in one pass (windq_unit_features_batch): the (unit, row) pairs are numbered through all
// jobs, job-major; job j owns the pairs [first_pair[j], first_pair[j + 1]) and the units
// [first_unit[j], first_unit[j + 1]) of the histogram and slot arrays.  n = 0: one matrix, described by the
// kernels' scalar parameters.
constexpr int kFeatMaxJobs = 16;
struct FeatJobs {
  const __half* W[kFeatMaxJobs];
  const float* s[kFeatMaxJobs];
  float* feat[kFeatMaxJobs];
  float* feat2[kFeatMaxJobs];  // features of the units of twice the width (pairs of neighbouring units), or NULL
  long long ldw[kFeatMaxJobs];
  long long first_pair[kFeatMaxJobs + 1];
  int R[kFeatMaxJobs];
  int first_unit[kFeatMaxJobs + 1];
  int n;
};

__device__ __forceinline__ void hist_add8(unsigned int* sh, const uint4& raw, float& part) {
  const unsigned int v[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    atomicAdd(&sh[v[i] & 0x7fffu], 1u);
    atomicAdd(&sh[(v[i] >> 16) & 0x7fffu], 1u);
    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&v[i]));
    part += f.x + f.y;
  }
}

// rows_per_block consecutive (unit, row) pairs per block; slot j of unit u belongs to block
// (u * R) / rows_per_block + j.
template <int G>
__global__ void __launch_bounds__(kFeatThreads, 1)  // at most 64 registers per thread
feat_hist_kernel(const __half* __restrict__ W_one, int R_one, int64_t ldw_one, long long rows_per_block, long long total_rows,
                 unsigned int* __restrict__ hist, double* __restrict__ slot_sum, int slots_per_unit, const FeatJobs jobs) {
  extern __shared__ unsigned int sh[];
  __shared__ double wsum[kFeatThreads / 32];
  constexpr int TPR = G / 8;               // threads per row (8 halves = 16 bytes each)
  constexpr int RPP = kFeatThreads / TPR;  // rows per pass
  for (int i = threadIdx.x; i < kBins; i += kFeatThreads) sh[i] = 0;
  __syncthreads();
  const int tr = threadIdx.x / TPR, tc = threadIdx.x % TPR;
  long long p = (long long)blockIdx.x * rows_per_block;
  const long long p_end = min(p + rows_per_block, total_rows);
  while (p < p_end) {
    const __half* W = W_one;
    int R = R_one, unit0 = 0;
    int64_t ldw = ldw_one;
    long long pair0 = 0;
    if (jobs.n) {
      int j = 0;
      while (j + 1 < jobs.n && p >= jobs.first_pair[j + 1]) ++j;
      W = jobs.W[j];
      R = jobs.R[j];
      ldw = jobs.ldw[j];
      unit0 = jobs.first_unit[j];
      pair0 = jobs.first_pair[j];
    }
    const int u = (int)((p - pair0) / R);
    const int r0 = (int)(p - pair0 - (long long)u * R);
    const int r1 = (int)min((long long)R, r0 + (p_end - p));
    const __half* base = W + (int64_t)u * G + tc * 8;
    double sum = 0.0;
    for (int r = r0 + tr; r < r1; r += RPP * kFeatLoads) {
      uint4 raw[kFeatLoads];
#pragma unroll
      for (int k = 0; k < kFeatLoads; ++k)
        if (r + k * RPP < r1) raw[k] = __ldg(reinterpret_cast<const uint4*>(base + (int64_t)(r + k * RPP) * ldw));
      float part = 0.0f;
#pragma unroll
      for (int k = 0; k < kFeatLoads; ++k)
        if (r + k * RPP < r1) hist_add8(sh, raw[k], part);
      sum += (double)part;
    }
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, m);
    if ((threadIdx.x & 31) == 0) wsum[threadIdx.x >> 5] = sum;
    __syncthreads();  // also: every histogram update of this segment is done
    if (threadIdx.x == 0) {
      double t = 0.0;
      for (int i = 0; i < kFeatThreads / 32; ++i) t += wsum[i];
      const long long first_block = (pair0 + (long long)u * R) / rows_per_block;
      slot_sum[(int64_t)(unit0 + u) * slots_per_unit + (blockIdx.x - first_block)] = t;
    }
    unsigned int* gh = hist + (int64_t)(unit0 + u) * kBins;
    for (int i = threadIdx.x; i < kBins; i += kFeatThreads) {
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

// One block per unit.  The unit's histogram is first copied to shared memory with coalesced 128-bit
// loads; thread t then owns the 32 consecutive bins 32 t .. 32 t + 31 and walks them from shared
// memory starting at bin t mod 32, so that the lanes of a warp stay on different banks.
// MERGE = 2: the block forms the features of a unit of width 2G from the histograms and sums of the two units of width
// G it consists of (a histogram of a union is the sum of the histograms), for jobs that ask for both widths.
template <int MERGE>
__global__ void __launch_bounds__(1024)
feat_finalize_kernel(const unsigned int* __restrict__ hist, const double* __restrict__ slot_sum, int slots_per_unit,
                     long long rows_per_block, int R_one, int G, const float* __restrict__ s_one, float* __restrict__ feat_one,
                     const FeatJobs jobs) {
  extern __shared__ unsigned int sh[];  // kBins counts
  __shared__ unsigned long long warp_total[32];
  __shared__ double red[3][32];
  __shared__ unsigned long long redc[2][32];
  __shared__ double s_stat[3];
  __shared__ int p99_bin;
  const int t = threadIdx.x, lane = t & 31, wp = t >> 5;
  int ug = blockIdx.x * MERGE;  // the (first) unit's place in hist and slot_sum
  int u = ug, R = R_one;
  const float* s = s_one;
  float* feat = feat_one;
  long long pair0 = 0;
  if (jobs.n) {
    int j = 0;
    while (j + 1 < jobs.n && ug >= jobs.first_unit[j + 1]) ++j;  // every job has a multiple of MERGE units
    u = ug - jobs.first_unit[j];
    R = jobs.R[j];
    s = jobs.s[j];
    feat = MERGE == 1 ? jobs.feat[j] : jobs.feat2[j];
    pair0 = jobs.first_pair[j];
    if (MERGE > 1 && feat == nullptr) return;  // this job did not ask for the wider units
  }
  const int GW = G * MERGE;                // width of the unit whose features are formed
  const long long n = (long long)R * GW;
  const unsigned long long k = (unsigned long long)((99 * n + 99) / 100);  // rank of P99, 1-indexed
  {
    const uint4* src = reinterpret_cast<const uint4*>(hist + (int64_t)ug * kBins);
    uint4* dst = reinterpret_cast<uint4*>(sh);
#pragma unroll
    for (int i = 0; i < kBins / 4 / 1024; ++i) {
      uint4 v = src[i * 1024 + t];
      if (MERGE > 1) {
        const uint4 w2 = src[kBins / 4 + i * 1024 + t];  // the neighbouring unit's histogram follows
        v.x += w2.x; v.y += w2.y; v.z += w2.z; v.w += w2.w;
      }
      dst[i * 1024 + t] = v;
    }
  }
  __syncthreads();
  const unsigned int* mine = sh + t * 32;
  unsigned long long local = 0;
#pragma unroll
  for (int i = 0; i < 32; ++i) local += mine[(i + lane) & 31];
  // inclusive scan of the per-thread counts: inside the warp, then over the warp totals
  unsigned long long incl = local;
#pragma unroll
  for (int m = 1; m < 32; m <<= 1) {
    const unsigned long long o = __shfl_up_sync(0xffffffffu, incl, m);
    if (lane >= m) incl += o;
  }
  if (lane == 31) warp_total[wp] = incl;
  __syncthreads();
  if (wp == 0) {
    unsigned long long w = warp_total[lane];
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) {
      const unsigned long long o = __shfl_up_sync(0xffffffffu, w, m);
      if (lane >= m) w += o;
    }
    warp_total[lane] = w;  // inclusive over warps
  }
  // statistics of s over the unit's G channels: warp 1, in double
  if (wp == 1) {
    const float* su = s + (int64_t)u * G;  // u counts units of width G: the wider unit starts at the same channel
    double sm = 0.0, mx = (double)su[0];
    for (int j = lane; j < GW; j += 32) { const double v = (double)su[j]; sm += v; mx = fmax(mx, v); }
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) {
      sm += __shfl_xor_sync(0xffffffffu, sm, m);
      mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, m));
    }
    const double mean = sm / (double)GW;
    double var = 0.0;
    for (int j = lane; j < GW; j += 32) { const double d = (double)su[j] - mean; var += d * d; }
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) var += __shfl_xor_sync(0xffffffffu, var, m);
    if (lane == 0) { s_stat[0] = mean; s_stat[1] = sqrt(var / (double)GW); s_stat[2] = mx; }
  }
  __syncthreads();
  incl += wp ? warp_total[wp - 1] : 0ull;
  const unsigned long long before = incl - local;
  if (before < k && k <= incl) {  // exactly one thread: the rank-k value is in its bins
    unsigned long long run = before;
    int i = 0;
    for (; i < 31; ++i) {
      run += mine[i];
      if (run >= k) break;
    }
    p99_bin = t * 32 + i;
  }
  __syncthreads();
  const float p99 = __half2float(__ushort_as_half((unsigned short)p99_bin));
  const float thr = 0.5f * p99;

  double sa = 0.0, sq = 0.0;
  unsigned long long n_out = 0, n_tiny = 0;
  if (local) {
#pragma unroll 4
    for (int i = 0; i < 32; ++i) {
      const int b = (i + lane) & 31;
      const unsigned int c = mine[b];
      if (c == 0) continue;  // also keeps the Inf / NaN patterns (never counted for finite input) out
      const float x = __half2float(__ushort_as_half((unsigned short)(t * 32 + b)));
      const double dv = (double)x, dc = (double)c;
      sa += dc * dv;
      sq += dc * dv * dv;
      if (x > thr) n_out += c;
      if (x < 1e-6f) n_tiny += c;
    }
  }
  double ss = 0.0;
#pragma unroll
  for (int h = 0; h < MERGE; ++h) {
    const long long first = (pair0 + (long long)(u + h) * R) / rows_per_block;
    const long long last = (pair0 + (long long)(u + h + 1) * R - 1) / rows_per_block;
    const int cnt = (int)(last - first + 1);
    for (int i = t; i < cnt; i += 1024) ss += slot_sum[(int64_t)(ug + h) * slots_per_unit + i];
  }
#pragma unroll
  for (int m = 16; m > 0; m >>= 1) {
    sa += __shfl_xor_sync(0xffffffffu, sa, m);
    sq += __shfl_xor_sync(0xffffffffu, sq, m);
    ss += __shfl_xor_sync(0xffffffffu, ss, m);
    n_out += __shfl_xor_sync(0xffffffffu, n_out, m);
    n_tiny += __shfl_xor_sync(0xffffffffu, n_tiny, m);
  }
  if (lane == 0) {
    red[0][wp] = sa; red[1][wp] = sq; red[2][wp] = ss;
    redc[0][wp] = n_out; redc[1][wp] = n_tiny;
  }
  __syncthreads();
  if (wp == 0) {
    double a = red[0][lane], q2 = red[1][lane], sg = red[2][lane];
    unsigned long long no = redc[0][lane], nt = redc[1][lane];
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) {
      a += __shfl_xor_sync(0xffffffffu, a, m);
      q2 += __shfl_xor_sync(0xffffffffu, q2, m);
      sg += __shfl_xor_sync(0xffffffffu, sg, m);
      no += __shfl_xor_sync(0xffffffffu, no, m);
      nt += __shfl_xor_sync(0xffffffffu, nt, m);
    }
    if (lane == 0) {
      const double dn = (double)n;
      const double mean = sg / dn;
      double var = q2 / dn - mean * mean;
      if (var < 0.0) var = 0.0;
      float* f = feat + (int64_t)(u / MERGE) * WINDQ_N_FEATURES;
      f[0] = (float)mean;
      f[1] = (float)sqrt(var);
      f[2] = (float)(a / dn);
      f[3] = (float)((double)nt / dn);
      f[4] = (float)((double)no / dn);
      f[5] = (float)s_stat[0];
      f[6] = (float)s_stat[1];
      f[7] = (float)s_stat[2];
    }
  }
}

// Pass-1 geometry: blocks and (unit, row) pairs per block.
struct FeatGrid {
  int blocks;
  long long rows_per_block;
  int slots_per_unit;
};
inline FeatGrid feat_grid(int sm_count, int64_t R, int64_t U, long long total_pairs = 0) {  // R: the largest row count
  FeatGrid g;
  const long long total = total_pairs ? total_pairs : (long long)U * R;
  int nb = sm_count < kFeatMaxBlocks ? sm_count : kFeatMaxBlocks;
  const long long min_rows = 16;  // a block should see at least a few rows
  if ((long long)nb * min_rows > total) nb = (int)((total + min_rows - 1) / min_rows);
  g.rows_per_block = (total + nb - 1) / nb;
  g.blocks = (int)((total + g.rows_per_block - 1) / g.rows_per_block);
  g.slots_per_unit = (int)(R / g.rows_per_block) + 2;
  return g;
}

template <int G>
windq_status launch_hist(windq_ctx* ctx, const __half* W, int R, int U, int64_t ldw, const FeatGrid& fg,
                         unsigned int* hist, double* slot_sum, cudaStream_t st, const FeatJobs& jobs = FeatJobs(),
                         long long total_pairs = 0) {
  const size_t smem = (size_t)kBins * sizeof(unsigned int);
  if (windq_status rc = prepare_kernel(ctx, kHistG32 + g_index(G), feat_hist_kernel<G>, kFeatThreads, smem, false)) return rc;
  feat_hist_kernel<G><<<(unsigned)fg.blocks, kFeatThreads, smem, st>>>(
      W, R, ldw, fg.rows_per_block, total_pairs ? total_pairs : (long long)U * R, hist, slot_sum, fg.slots_per_unit, jobs);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

windq_status features_from_histograms(windq_ctx* ctx, const unsigned int* hist, const double* unit_wsum, int n_jobs, const int* R,
                                      const int* first_unit, const float* const* s, float* const* feat_out, int G, cudaStream_t st) {
  FeatJobs fj;
  memset(&fj, 0, sizeof(fj));
  fj.n = n_jobs;
  for (int j = 0; j < n_jobs; ++j) {
    fj.s[j] = s[j];
    fj.feat[j] = feat_out[j];
    fj.R[j] = R[j];
    fj.first_unit[j] = first_unit[j];
  }
  fj.first_unit[n_jobs] = first_unit[n_jobs];
  if (windq_status rc = prepare_kernel(ctx, kFinalize, feat_finalize_kernel<1>, 1024, kBins * sizeof(unsigned int), false)) return rc;
  // one sum per unit (slots_per_unit = 1); a "rows per block" beyond every pair count makes the kernel read exactly that one
  feat_finalize_kernel<1><<<(unsigned)first_unit[n_jobs], 1024, kBins * sizeof(unsigned int), st>>>(hist, unit_wsum, 1, 1ll << 62, 0, G,
                                                                                               nullptr, nullptr, fj);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

}  // namespace windq

extern "C" {

int64_t windq_scratch_bytes_unit_features(int64_t R, int64_t C, int G) {
  if (!windq::valid_G(G) || R <= 0 || C <= 0) return 0;
  const int64_t U = C / G;
  // histograms + one double per (unit, block that holds rows of it): a unit meets at most
  // blocks / U + 2 blocks, and the grid has at most kFeatMaxBlocks blocks
  return U * windq::kBins * (int64_t)sizeof(unsigned int) + (windq::kFeatMaxBlocks + 2 * U) * (int64_t)sizeof(double);
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
  double* slot_sum = (double*)((char*)ctx->scratch + (int64_t)U * kBins * sizeof(unsigned int));
  const FeatGrid fg = feat_grid(ctx->sm_count, R, U);
  WINDQ_CUDA(ctx, cudaMemsetAsync(hist, 0, (size_t)U * kBins * sizeof(unsigned int), st));
  const __half* Wh = (const __half*)W;
  windq_status rc;
  switch (G) {
    case 32: rc = launch_hist<32>(ctx, Wh, (int)R, U, ldw, fg, hist, slot_sum, st); break;
    case 64: rc = launch_hist<64>(ctx, Wh, (int)R, U, ldw, fg, hist, slot_sum, st); break;
    case 128: rc = launch_hist<128>(ctx, Wh, (int)R, U, ldw, fg, hist, slot_sum, st); break;
    case 256: rc = launch_hist<256>(ctx, Wh, (int)R, U, ldw, fg, hist, slot_sum, st); break;
    default: rc = launch_hist<512>(ctx, Wh, (int)R, U, ldw, fg, hist, slot_sum, st); break;
  }
  if (rc != WINDQ_OK) return rc;
  if (windq_status st2 = prepare_kernel(ctx, kFinalize, feat_finalize_kernel<1>, 1024, kBins * sizeof(unsigned int), false)) return st2;
  feat_finalize_kernel<1><<<(unsigned)U, 1024, kBins * sizeof(unsigned int), st>>>(hist, slot_sum, fg.slots_per_unit, fg.rows_per_block, (int)R, G, s, feat_out, FeatJobs());
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

int64_t windq_scratch_bytes_unit_features_batch(const windq_feat_job* jobs, int n_jobs, int G) {
  if (!jobs || n_jobs <= 0 || !windq::valid_G(G)) return 0;
  int64_t U = 0, pairs = 0, max_R = 0;
  for (int j = 0; j < n_jobs; ++j) {
    if (jobs[j].R <= 0 || jobs[j].C <= 0) return 0;
    U += jobs[j].C / G;
    pairs += (jobs[j].C / G) * jobs[j].R;
    max_R = jobs[j].R > max_R ? jobs[j].R : max_R;
  }
  if (pairs <= 0) return 0;
  // histograms + one double per (unit, block that can hold rows of it): a block has at least
  // pairs / kFeatMaxBlocks pairs, so a unit of at most max_R rows meets at most the number of blocks below
  const int64_t slots = max_R * windq::kFeatMaxBlocks / pairs + 3;
  return U * windq::kBins * (int64_t)sizeof(unsigned int) + U * slots * (int64_t)sizeof(double);
}

static windq_status unit_features_batch_any(windq_ctx* ctx, const char* who, const windq_feat_job* jobs, float* const* feat2, int n_jobs,
                                            int G, void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "%s: ctx is NULL", who);
  WINDQ_REQUIRE(ctx, jobs, WINDQ_ERR_NULL, "%s: jobs is NULL", who);
  WINDQ_REQUIRE(ctx, n_jobs >= 1 && n_jobs <= kFeatMaxJobs, WINDQ_ERR_SHAPE, "%s: n_jobs = %d is outside [1, %d]", who, n_jobs,
                kFeatMaxJobs);
  FeatJobs fj;
  memset(&fj, 0, sizeof(fj));
  fj.n = n_jobs;
  long long pairs = 0;
  int64_t units = 0, max_R = 0;
  bool any_wide = false;
  for (int j = 0; j < n_jobs; ++j) {
    const windq_feat_job& b = jobs[j];
    if (windq_status st = check_matrix(ctx, who, b.W, b.R, b.C, b.ldw, G)) return st;
    WINDQ_REQUIRE(ctx, b.s && b.feat_out, WINDQ_ERR_NULL, "%s: job %d: s or feat_out is NULL", who, j);
    WINDQ_REQUIRE(ctx, b.R * (int64_t)G < (1ll << 32), WINDQ_ERR_SHAPE, "%s: job %d: R * G must be below 2^32", who, j);
    fj.W[j] = (const __half*)b.W;
    fj.s[j] = b.s;
    fj.feat[j] = b.feat_out;
    fj.feat2[j] = feat2 ? feat2[j] : nullptr;
    if (fj.feat2[j]) {
      any_wide = true;
      WINDQ_REQUIRE(ctx, b.C % (2 * (int64_t)G) == 0, WINDQ_ERR_SHAPE, "%s: job %d: C = %lld is not a multiple of 2 G = %d", who, j,
                    (long long)b.C, 2 * G);
      WINDQ_REQUIRE(ctx, b.R * 2 * (int64_t)G < (1ll << 32), WINDQ_ERR_SHAPE, "%s: job %d: R * 2 G must be below 2^32", who, j);
    }
    fj.ldw[j] = b.ldw;
    fj.R[j] = (int)b.R;
    fj.first_pair[j] = pairs;
    fj.first_unit[j] = (int)units;
    pairs += (b.C / G) * b.R;
    units += b.C / G;
    max_R = b.R > max_R ? b.R : max_R;
  }
  fj.first_pair[n_jobs] = pairs;
  fj.first_unit[n_jobs] = (int)units;
  WINDQ_REQUIRE(ctx, units <= 65535 * 32, WINDQ_ERR_SHAPE, "%s: too many units", who);
  if (any_wide)
    for (int j = 0; j < n_jobs; ++j)
      WINDQ_REQUIRE(ctx, jobs[j].C % (2 * (int64_t)G) == 0, WINDQ_ERR_SHAPE,
                    "%s: job %d: with features at width 2 G every job needs an even number of units", who, j);
  DeviceGuard guard(ctx->device);
  if (windq_status st = ensure_scratch(ctx, windq_scratch_bytes_unit_features_batch(jobs, n_jobs, G))) return st;
  cudaStream_t st = (cudaStream_t)stream;
  unsigned int* hist = (unsigned int*)ctx->scratch;
  double* slot_sum = (double*)((char*)ctx->scratch + units * kBins * (int64_t)sizeof(unsigned int));
  const FeatGrid fg = feat_grid(ctx->sm_count, max_R, units, pairs);
  WINDQ_CUDA(ctx, cudaMemsetAsync(hist, 0, (size_t)units * kBins * sizeof(unsigned int), st));
  windq_status rc;
  switch (G) {
    case 32: rc = launch_hist<32>(ctx, nullptr, 0, 0, 0, fg, hist, slot_sum, st, fj, pairs); break;
    case 64: rc = launch_hist<64>(ctx, nullptr, 0, 0, 0, fg, hist, slot_sum, st, fj, pairs); break;
    case 128: rc = launch_hist<128>(ctx, nullptr, 0, 0, 0, fg, hist, slot_sum, st, fj, pairs); break;
    case 256: rc = launch_hist<256>(ctx, nullptr, 0, 0, 0, fg, hist, slot_sum, st, fj, pairs); break;
    default: rc = launch_hist<512>(ctx, nullptr, 0, 0, 0, fg, hist, slot_sum, st, fj, pairs); break;
  }
  if (rc != WINDQ_OK) return rc;
  if (windq_status st2 = prepare_kernel(ctx, kFinalize, feat_finalize_kernel<1>, 1024, kBins * sizeof(unsigned int), false)) return st2;
  feat_finalize_kernel<1><<<(unsigned)units, 1024, kBins * sizeof(unsigned int), st>>>(hist, slot_sum, fg.slots_per_unit,
                                                                                       fg.rows_per_block, 0, G, nullptr, nullptr, fj);
  WINDQ_CUDA(ctx, cudaGetLastError());
  if (any_wide) {
    if (windq_status st2 = prepare_kernel(ctx, kFinalize2, feat_finalize_kernel<2>, 1024, kBins * sizeof(unsigned int), false)) return st2;
    feat_finalize_kernel<2><<<(unsigned)(units / 2), 1024, kBins * sizeof(unsigned int), st>>>(hist, slot_sum, fg.slots_per_unit,
                                                                                              fg.rows_per_block, 0, G, nullptr, nullptr, fj);
    WINDQ_CUDA(ctx, cudaGetLastError());
  }
  return WINDQ_OK;
}

windq_status windq_unit_features_batch(windq_ctx* ctx, const windq_feat_job* jobs, int n_jobs, int G, void* stream) {
  return unit_features_batch_any(ctx, "windq_unit_features_batch", jobs, nullptr, n_jobs, G, stream);
}

windq_status windq_unit_features_batch2(windq_ctx* ctx, const windq_feat_job* jobs, float* const* feat_out_2G, int n_jobs, int G,
                                        void* stream) {
  const char* who = "windq_unit_features_batch2";
  if (!ctx) return windq::fail(nullptr, WINDQ_ERR_NULL, "%s: ctx is NULL", who);
  if (!feat_out_2G) return windq::fail(ctx, WINDQ_ERR_NULL, "%s: feat_out_2G is NULL", who);
  if (G == 512) return windq::fail(ctx, WINDQ_ERR_ARG, "%s: G = 512 has no supported width 2 G", who);
  return unit_features_batch_any(ctx, who, jobs, feat_out_2G, n_jobs, G, stream);
}

}  // extern "C"

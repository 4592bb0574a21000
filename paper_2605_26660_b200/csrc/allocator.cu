// windq_greedy_allocate: the deterministic rule of the heuristic sensitivity allocator ("Comparison
// with Heuristic Sensitivity Allocator"): rank the units by saliency, start all at 2 bit, push the
// least sensitive to 1.58 / 1 bit until enough budget is free, promote the most sensitive to 4 / 3 bit
// while the budget permits.  Costs are Eq. 6 in centibits, all arithmetic int64.
//
// Ranking is by counting: a unit's rank is the number of units that come before it under (score
// descending, index ascending), which is exact, stable and needs no sort.  To keep that from costing
// U^2 comparisons the units are first spread over buckets by score (a linear map of the score's
// order-preserving bit pattern between the smallest and the largest one, so equal scores share a bucket
// and a lower bucket holds strictly larger scores); a unit then counts inside its own bucket only and
// adds the sizes of the buckets before it.  If all scores are equal that is the U^2 count again, which
// the limit on U bounds.  The rule itself runs in one block:
// the two sweeps of step 2 are prefix sums (a unit moves while the running total is above the floor,
// and the savings are never negative, so the moved units are a prefix of the sweep), step 3 is serial by
// nature and runs in one warp, 32 units at a time, over counts gathered in rank order beforehand, with
// two shortcuts for chunks that take all or nothing.
#include "windq_internal.cuh"

namespace windq {

constexpr int kMaxBuckets = 65536;

// comp as above, and the smallest and largest key.
__global__ void alloc_key_range_kernel(const float* __restrict__ sal, int U, unsigned long long* __restrict__ comp,
                                       unsigned int* __restrict__ key_min_max) {
  const int u = blockIdx.x * blockDim.x + threadIdx.x;
  unsigned lo = 0xffffffffu, hi = 0u;
  if (u < U) {
    const unsigned b = __float_as_uint(sal[u]);
    const unsigned key = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
    comp[u] = ((unsigned long long)key << 32) | (unsigned long long)(0xffffffffu - (unsigned)u);
    lo = hi = key;
  }
#pragma unroll
  for (int m = 16; m; m >>= 1) {
    lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, m));
    hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, m));
  }
  if ((threadIdx.x & 31) == 0) {
    atomicMin(key_min_max, lo);
    atomicMax(key_min_max + 1, hi);
  }
}

// Bucket of a key: 0 for the largest key, growing as keys fall; monotone, equal keys share a bucket.
__device__ __forceinline__ int alloc_bucket(unsigned key, unsigned kmin, unsigned kmax, int n_buckets) {
  const unsigned long long span = (unsigned long long)(kmax - kmin) + 1ull;
  return (int)(((unsigned long long)(kmax - key) * (unsigned long long)n_buckets) / span);
}

__global__ void alloc_hist_kernel(const unsigned long long* __restrict__ comp, int U, const unsigned int* __restrict__ key_min_max,
                                  int n_buckets, unsigned int* __restrict__ hist) {
  const int u = blockIdx.x * blockDim.x + threadIdx.x;
  if (u >= U) return;
  atomicAdd(hist + alloc_bucket((unsigned)(comp[u] >> 32), key_min_max[0], key_min_max[1], n_buckets), 1u);
}

// start[b] = number of units in the buckets before b (one block; n_buckets is a multiple of 1024 or below it).
__global__ void __launch_bounds__(1024)
alloc_scan_kernel(const unsigned int* __restrict__ hist, int n_buckets, unsigned int* __restrict__ start,
                  unsigned int* __restrict__ cursor) {
  __shared__ unsigned int warp_tot[32];
  const int t = threadIdx.x, per = (n_buckets + 1023) / 1024;
  unsigned int mine = 0;
  for (int i = 0; i < per; ++i) {
    const int b = t * per + i;
    if (b < n_buckets) mine += hist[b];
  }
  unsigned int incl = mine;
#pragma unroll
  for (int m = 1; m < 32; m <<= 1) {
    const unsigned int o = __shfl_up_sync(0xffffffffu, incl, m);
    if ((t & 31) >= m) incl += o;
  }
  if ((t & 31) == 31) warp_tot[t >> 5] = incl;
  __syncthreads();
  unsigned int before = incl - mine;
  for (int w = 0; w < (t >> 5); ++w) before += warp_tot[w];
  for (int i = 0; i < per; ++i) {
    const int b = t * per + i;
    if (b < n_buckets) {
      start[b] = before;
      cursor[b] = before;
      before += hist[b];
    }
  }
}

// Units into their buckets, in whatever order the atomics give: the count below does not depend on it.
__global__ void alloc_scatter_kernel(const unsigned long long* __restrict__ comp, int U,
                                     const unsigned int* __restrict__ key_min_max, int n_buckets,
                                     unsigned int* __restrict__ cursor, unsigned long long* __restrict__ members) {
  const int u = blockIdx.x * blockDim.x + threadIdx.x;
  if (u >= U) return;
  const unsigned long long c = comp[u];
  const int b = alloc_bucket((unsigned)(c >> 32), key_min_max[0], key_min_max[1], n_buckets);
  members[atomicAdd(cursor + b, 1u)] = c;
}

__global__ void alloc_rank_kernel(const unsigned long long* __restrict__ comp, int U, const unsigned int* __restrict__ key_min_max,
                                  int n_buckets, const unsigned int* __restrict__ start, const unsigned int* __restrict__ hist,
                                  const unsigned long long* __restrict__ members, int* __restrict__ order,
                                  long long* __restrict__ order64) {
  const int u = blockIdx.x * blockDim.x + threadIdx.x;
  if (u >= U) return;
  const unsigned long long mine = comp[u];
  const int b = alloc_bucket((unsigned)(mine >> 32), key_min_max[0], key_min_max[1], n_buckets);
  const unsigned int first = start[b], n = hist[b];
  unsigned int before = first;
  for (unsigned int i = 0; i < n; ++i) before += members[first + i] > mine;
  order[before] = u;
  if (order64) order64[before] = u;
}

struct AllocArgs {
  const long long* n_weights;
  const long long* n_protected;  // nullable
  const long long* n_groups;
  int U;
  long long target_cb, headroom_cb;
  int scale_bits, zero_bits;
};

__device__ __forceinline__ long long alloc_cost(int a, long long q, long long p, long long g, int scale_bits, int zero_bits) {
  const long long centi = a == 2 ? 400 : a == 3 ? 300 : a == 4 ? 200 : a == 5 ? 158 : 100;
  return centi * q + 800 * p + 100 * g * (scale_bits + (a <= 4 ? zero_bits : 0));
}

__device__ __forceinline__ long long warp_sum(long long v) {
#pragma unroll
  for (int m = 16; m; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
  return v;
}

// Sum over the block (1024 threads); every thread gets the result.
__device__ __forceinline__ long long block_sum(long long v, long long* red) {
  v = warp_sum(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  long long w = red[threadIdx.x & 31];
  return warp_sum(w);
}

__global__ void __launch_bounds__(1024)
alloc_greedy_kernel(AllocArgs a, const int* __restrict__ order, long long* __restrict__ walk, uint8_t* actions,
                    long long* __restrict__ total_out) {
  __shared__ long long red[32];
  __shared__ long long warp_incl[32];
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int U = a.U;

  // step 1: everything at 2 bit
  long long sum_n = 0, sum_c = 0;
  int bad = 0;
  for (int u = t; u < U; u += 1024) {
    const long long n = a.n_weights[u], p = a.n_protected ? a.n_protected[u] : 0, g = a.n_groups[u];
    if (n < 0 || p < 0 || p > n || g < 0) bad = 1;
    sum_n += n;
    sum_c += alloc_cost(4, n - p, p, g, a.scale_bits, a.zero_bits);
    actions[u] = 4;
  }
  bad = __syncthreads_or(bad);
  if (bad) {
    if (t == 0) *total_out = -1;
    return;
  }
  const long long N = block_sum(sum_n, red);
  long long total = block_sum(sum_c, red);
  const long long budget = a.target_cb * N, floor_cb = budget - a.headroom_cb * N;

  // step 2: two sweeps from the least sensitive unit upwards
  bool freed = false;
  for (int down = 5; down <= 6 && !freed; ++down) {
    for (int top = U - 1; top >= 0; top -= 1024) {
      const int r = top - t;
      int u = -1;
      long long saving = 0;
      if (r >= 0) {
        u = order[r];
        const long long n = a.n_weights[u], p = a.n_protected ? a.n_protected[u] : 0, g = a.n_groups[u];
        saving = alloc_cost(down - 1, n - p, p, g, a.scale_bits, a.zero_bits) - alloc_cost(down, n - p, p, g, a.scale_bits, a.zero_bits);
      }
      long long incl = saving;
#pragma unroll
      for (int m = 1; m < 32; m <<= 1) {
        const long long o = __shfl_up_sync(0xffffffffu, incl, m);
        if (lane >= m) incl += o;
      }
      __syncthreads();
      if (lane == 31) warp_incl[warp] = incl;
      __syncthreads();
      long long before_warp = 0;
      for (int w = 0; w < warp; ++w) before_warp += warp_incl[w];
      const long long before = total - (before_warp + incl - saving);  // the total when the sweep reaches this unit
      const bool moves = r >= 0 && before > floor_cb;
      if (moves) actions[u] = (uint8_t)down;
      total -= block_sum(moves ? saving : 0, red);
      if (__syncthreads_or(r >= 0 && !moves)) {
        freed = true;
        break;
      }
    }
  }
  __syncthreads();  // the actions written above are read below

  // step 3: most sensitive first, only units still at 2 bit (those moved down are the tail of the
  // ranking).  All warps first gather, in rank order, what the walk needs -- the unit's quantised
  // weight count, or a mark for a unit that was moved down -- so that the one warp that walks reads
  // consecutive words instead of chasing order[] -> counts through memory one chunk at a time.
  for (int r = t; r < U; r += 1024) {
    const int u = order[r];
    walk[r] = actions[u] == 4 ? a.n_weights[u] - (a.n_protected ? a.n_protected[u] : 0) : -1;
  }
  __syncthreads();
  if (warp != 0) return;
  long long q_next = lane < U ? walk[lane] : -1;
  for (int base = 0; base < U; base += 32) {
    const int r = base + lane;
    const long long q = q_next;
    q_next = r + 32 < U ? walk[r + 32] : -1;  // in flight while this chunk is decided
    const bool cand = r < U && q >= 0;
    const unsigned cands = __ballot_sync(0xffffffffu, cand);
    const bool tail = __any_sync(0xffffffffu, r < U && q < 0);
    if (cands) {
      const long long all4 = warp_sum(cand ? 200 * q : 0);
      long long qmin = cand ? q : 0x7fffffffffffffffll;
#pragma unroll
      for (int m = 16; m; m >>= 1) qmin = min(qmin, __shfl_xor_sync(0xffffffffu, qmin, m));
      int choice = 4;
      if (total + all4 <= budget) {  // the whole chunk takes 4 bit
        total += all4;
        choice = 2;
      } else if (total + 100 * qmin > budget) {  // not even the cheapest move fits
      } else {
        for (int i = 0; i < 32; ++i) {
          const long long qi = __shfl_sync(0xffffffffu, q, i);
          if (!((cands >> i) & 1u)) continue;
          int c = 4;
          if (total + 200 * qi <= budget) {
            total += 200 * qi;
            c = 2;
          } else if (total + 100 * qi <= budget) {
            total += 100 * qi;
            c = 3;
          }
          if (i == lane) choice = c;
        }
      }
      if (cand && choice != 4) actions[order[r]] = (uint8_t)choice;
    }
    if (tail) break;
  }
  if (lane == 0) *total_out = total;
}

}  // namespace windq

extern "C" {

int64_t windq_scratch_bytes_greedy_allocate(int64_t U) {
  if (U <= 0) return 0;
  // composite keys, bucket members, walk array (8 bytes per unit each), order (4), three bucket tables, key range
  return 3 * windq::round_up(U * 8, 256) + windq::round_up(U * 4, 256) + 3 * (int64_t)windq::kMaxBuckets * 4 + 256;
}

windq_status windq_greedy_allocate(windq_ctx* ctx, const float* saliency, const int64_t* n_weights, const int64_t* n_protected,
                                   const int64_t* n_groups, int64_t U, int64_t target_cb, int64_t headroom_cb, int scale_bits,
                                   int zero_bits, uint8_t* actions_out, int64_t* order_out, int64_t* total_centibits_out,
                                   void* stream) {
  using namespace windq;
  if (!ctx) return fail(nullptr, WINDQ_ERR_NULL, "windq_greedy_allocate: ctx is NULL");
  WINDQ_REQUIRE(ctx, saliency && n_weights && n_groups && actions_out && total_centibits_out, WINDQ_ERR_NULL,
                "windq_greedy_allocate: a required pointer is NULL");
  WINDQ_REQUIRE(ctx, U > 0 && U <= WINDQ_MAX_ALLOC_UNITS, WINDQ_ERR_SHAPE, "windq_greedy_allocate: U = %lld is outside [1, %d]",
                (long long)U, WINDQ_MAX_ALLOC_UNITS);
  WINDQ_REQUIRE(ctx, target_cb >= 0 && target_cb <= 1600 && headroom_cb >= 0 && headroom_cb <= 1600, WINDQ_ERR_SHAPE,
                "windq_greedy_allocate: target %lld or headroom %lld centibits is outside [0, 1600]", (long long)target_cb,
                (long long)headroom_cb);
  WINDQ_REQUIRE(ctx, scale_bits >= 0 && zero_bits >= 0 && scale_bits <= 64 && zero_bits <= 64, WINDQ_ERR_SHAPE,
                "windq_greedy_allocate: scale_bits / zero_bits outside [0, 64]");
  DeviceGuard guard(ctx->device);
  if (windq_status rc = ensure_scratch(ctx, windq_scratch_bytes_greedy_allocate(U))) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  char* base = (char*)ctx->scratch;
  unsigned long long* comp = (unsigned long long*)base;
  unsigned long long* members = (unsigned long long*)(base + round_up(U * 8, 256));
  long long* walk = (long long*)(base + 2 * round_up(U * 8, 256));
  int* order = (int*)(base + 3 * round_up(U * 8, 256));
  unsigned int* hist = (unsigned int*)(base + 3 * round_up(U * 8, 256) + round_up(U * 4, 256));
  unsigned int* start = hist + kMaxBuckets;
  unsigned int* cursor = start + kMaxBuckets;
  unsigned int* key_min_max = cursor + kMaxBuckets;
  int n_buckets = 256;  // about four units per bucket
  while (n_buckets < kMaxBuckets && (int64_t)n_buckets * 4 < U) n_buckets *= 2;
  const unsigned blocks = (unsigned)((U + 255) / 256);
  WINDQ_CUDA(ctx, cudaMemsetAsync(hist, 0, (size_t)n_buckets * sizeof(unsigned int), st));
  WINDQ_CUDA(ctx, cudaMemsetAsync(key_min_max, 0xff, sizeof(unsigned int), st));
  WINDQ_CUDA(ctx, cudaMemsetAsync(key_min_max + 1, 0, sizeof(unsigned int), st));
  alloc_key_range_kernel<<<blocks, 256, 0, st>>>(saliency, (int)U, comp, key_min_max);
  alloc_hist_kernel<<<blocks, 256, 0, st>>>(comp, (int)U, key_min_max, n_buckets, hist);
  alloc_scan_kernel<<<1, 1024, 0, st>>>(hist, n_buckets, start, cursor);
  alloc_scatter_kernel<<<blocks, 256, 0, st>>>(comp, (int)U, key_min_max, n_buckets, cursor, members);
  alloc_rank_kernel<<<blocks, 256, 0, st>>>(comp, (int)U, key_min_max, n_buckets, start, hist, members, order,
                                            (long long*)order_out);
  AllocArgs a{(const long long*)n_weights, (const long long*)n_protected, (const long long*)n_groups, (int)U,
              target_cb, headroom_cb, scale_bits, zero_bits};
  alloc_greedy_kernel<<<1, 1024, 0, st>>>(a, order, walk, actions_out, (long long*)total_centibits_out);
  WINDQ_CUDA(ctx, cudaGetLastError());
  return WINDQ_OK;
}

}  // extern "C"

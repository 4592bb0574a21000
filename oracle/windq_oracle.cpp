// windq oracle -- TEST INFRASTRUCTURE, not the product.
//
// A plain, slow, single-threaded C++17 restatement of the scoring / fitting hot
// path of WINDQuant's allocation loop: activation statistics, per-unit state
// features, per-group quantizer fits under all six bit-widths, plan
// application (codes, packing, fake-quantised weights) and effective-bit
// accounting.  It shares no code with the CUDA library and neither includes
// the other.  Only the tests, the smoke check and the benchmark's CPU-baseline
// leg may call it.  Build: g++ -O2 -ffp-contract=off (no fast-math, no
// -march): every float operation below is one IEEE-754 binary32 operation,
// rounded to nearest even, in exactly the order written.
//
// What the paper fixes and what it leaves open
//   * Units are column chunks of a linear weight matrix; every unit gets one of
//     seven actions {16, 8, 4, 3, 2, 1.58, 1} (Eq. 3, "Action Space").
//   * State features 0-4 and 9-11 are those of Table 1.
//   * The engine fits a local scale per group (group = one row of one chunk,
//     App. "Per-unit Scale Optimization") and scores it by reconstruction error
//     (Sec. 3.5 "Quantization Engine and Bit Accounting").
//   * Storage is counted in effective bits, b_bar = sum B_i / sum n_i (Eq. 6).
//   The paper gives no formula for its quantizers.  The ones used here are the
//   closed-form / grid-search readings listed beside each function; every such
//   reading is marked "READING".
//
// Arithmetic model (READING; the paper is silent).  Every quantity that feeds
// an integer code, a clip index or a stored fp16 value is a fixed sequence of
// binary32 operations.  A sum over the G elements of a row-group is PSUM8:
// leaves of 8 consecutive elements, each accumulated left to right from +0,
// then combined by a balanced binary tree that adds adjacent leaves first.
// Sums over rows (unit level) are taken in double and compared with tolerance.
//
// Pins (see tests/test_oracle_*.py): fp16 conversion against all 65536
// patterns; PSUM8 order against hand-worked cancellation cases; 8-bit round
// trip on grid values; brute-force clip search in float64 on tiny chunks;
// ternary / binary closed forms and stationarity; scale invariance by powers of
// two; degenerate groups; monotone error in bit-width; Eq. 6 bit arithmetic;
// pack/unpack identity with an independent unpacker; nearest-rank P99 against a
// full sort; salient selection against a full sort, its count arithmetic and
// Eq. 6 with protected weights against the paper's formula; the ternary
// threshold search against a hand-worked case, against the exhaustive optimum
// over all 3^8 codes of toy groups, and against its reduction to the 0.7 rule;
// the 1-bit fit against the exhaustive optimum over all 2^8 sign patterns.
// Parity unpinned: that these fits resemble the paper's Adam-fitted operators
// -- not claimed.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

namespace {

// ---------------------------------------------------------------- fp16 <-> fp32
inline uint32_t f32_bits(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }
inline float bits_f32(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }

// binary16 -> binary32, exact.
float half_to_float(uint16_t h) {
  const uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
  const uint32_t e = (h >> 10) & 31u;
  const uint32_t m = h & 0x3ffu;
  if (e == 0) {                                  // zero or subnormal: m * 2^-24
    float v = (float)m * 5.9604644775390625e-08f;
    return bits_f32(f32_bits(v) | sign);
  }
  if (e == 31) return bits_f32(sign | 0x7f800000u | (m << 13));
  return bits_f32(sign | ((e + 112u) << 23) | (m << 13));
}

// binary32 -> binary16, round to nearest even, overflow to infinity.
uint16_t float_to_half(float f) {
  uint32_t x = f32_bits(f);
  const uint16_t sign = (uint16_t)((x >> 16) & 0x8000u);
  x &= 0x7fffffffu;
  if (x > 0x7f800000u) return (uint16_t)(sign | 0x7e00u);            // NaN
  if (x >= 0x477ff000u) return (uint16_t)(sign | 0x7c00u);           // >= 65520 -> inf
  if (x < 0x38800000u) {                                              // below 2^-14
    const float a = bits_f32(x) * 16777216.0f;                        // exact: units of 2^-24
    const uint32_t m = (uint32_t)std::nearbyintf(a);                  // 0..1024, RNE
    return (uint16_t)(sign | m);
  }
  const uint32_t odd = (x >> 13) & 1u;
  x += 0xfffu + odd;
  x -= 0x38000000u;
  return (uint16_t)(sign | (x >> 13));
}

inline float round_through_half(float f) { return half_to_float(float_to_half(f)); }

// ---------------------------------------------------------------- PSUM8
// leaf(l) must return the left-to-right accumulation, from +0.0f, over the
// elements 8l .. 8l+7.  G is 8 * 2^m.
template <class Leaf>
float psum8(int G, Leaf leaf) {
  float node[64] = {0.0f};
  const int nleaf = G / 8;
  for (int l = 0; l < nleaf; ++l) node[l] = leaf(l);
  for (int n = nleaf; n > 1; n /= 2)
    for (int i = 0; i < n / 2; ++i) node[i] = node[2 * i] + node[2 * i + 1];
  return node[0];
}

bool valid_group_width(int G) {
  return G == 8 || G == 16 || G == 32 || G == 64 || G == 128 || G == 256 || G == 512;
}

// ---------------------------------------------------------------- constants
const float kMagic = 12582912.0f;            // 1.5 * 2^23: adding it rounds to an integer (RNE)
const int kUniformBits[4] = {8, 4, 3, 2};    // order of the bit-width columns 0..3
// columns of every per-bit-width table: 0:8  1:4  2:3  3:2  4:1.58 (ternary)  5:1 (binary)
// action codes (Eq. 3 order): 0 skip(16)  1:8  2:4  3:3  4:2  5:1.58  6:1

// ---------------------------------------------------------------- one row-group
struct Group {
  int G;
  const float* w;   // G weights of one row inside one unit, converted from fp16
  const float* s;   // G activation statistics of the unit's input channels
};

struct UniformParams {
  float scale;      // value of the stored fp16 scale (1.0 if it rounded to zero)
  float inv;        // 1 / scale, IEEE division
  float zf;         // integer zero point as a float, in [0, qmax]
  float qmaxf;
};

// READING: asymmetric uniform grid over [p*mn, p*mx] with zero forced into the
// range (mn <= 0 <= mx), scale rounded to fp16 before it is used, integer
// zero point.
UniformParams uniform_params(float mn, float rng, float p, int bits) {
  UniformParams u;
  const int qmax = (1 << bits) - 1;
  u.qmaxf = (float)qmax;
  const float rq = (float)(1.0 / (double)qmax);
  const float scale32 = (p * rng) * rq;
  u.scale = round_through_half(scale32);
  if (u.scale == 0.0f) u.scale = 1.0f;
  u.inv = 1.0f / u.scale;
  float z = std::nearbyintf(std::fabs(p * mn) * u.inv);   // mn <= 0: |p*mn| = -(p*mn), and never -0
  if (z < 0.0f) z = 0.0f;
  if (z > u.qmaxf) z = u.qmaxf;
  u.zf = z;
  return u;
}

// c = q - z, the zero-centred integer code as a float.
inline float centred_code(float w, const UniformParams& u) {
  const float r = std::fmaf(w, u.inv, kMagic);   // nearest-even integer of the exact product
  float c = r - kMagic;
  const float lo = 0.0f - u.zf, hi = u.qmaxf - u.zf;    // 0 - 0 = +0: no negative zero codes
  if (c < lo) c = lo;
  if (c > hi) c = hi;
  return c;
}

// s-weighted squared reconstruction error of one uniform candidate.
float uniform_error(const Group& g, const UniformParams& u) {
  return psum8(g.G, [&](int l) {
    float acc = 0.0f;
    for (int j = 8 * l; j < 8 * l + 8; ++j) {
      const float c = centred_code(g.w[j], u);
      const float d = std::fmaf(c, u.scale, -g.w[j]);
      const float t = g.s[j] * d;
      acc = std::fmaf(t, d, acc);
    }
    return acc;
  });
}

void group_range(const Group& g, float* mn, float* rng) {
  float lo = 0.0f, hi = 0.0f;
  for (int j = 0; j < g.G; ++j) {
    if (g.w[j] < lo) lo = g.w[j];
    if (g.w[j] > hi) hi = g.w[j];
  }
  *mn = lo;
  *rng = hi - lo;
}

// Clip search for one bit-width: smallest k with minimal error (strict '<').
void search_uniform(const Group& g, float mn, float rng, int bits, const float* clip, int K,
                    int* best_k, float* best_e) {
  int bk = 0;
  float be = 0.0f;
  for (int k = 0; k < K; ++k) {
    const UniformParams u = uniform_params(mn, rng, clip[k], bits);
    const float e = uniform_error(g, u);
    if (k == 0 || e < be) { be = e; bk = k; }
  }
  *best_k = bk;
  *best_e = be;
}

float sum_abs(const Group& g) {
  return psum8(g.G, [&](int l) {
    float acc = 0.0f;
    for (int j = 8 * l; j < 8 * l + 8; ++j) acc = acc + std::fabs(g.w[j]);
    return acc;
  });
}

float error_against(const Group& g, const float* what) {   // what[j] = reconstructed weight
  return psum8(g.G, [&](int l) {
    float acc = 0.0f;
    for (int j = 8 * l; j < 8 * l + 8; ++j) {
      const float d = what[j] - g.w[j];
      const float t = g.s[j] * d;
      acc = std::fmaf(t, d, acc);
    }
    return acc;
  });
}

// READING: ternary = threshold rho * mean|w|, one scale alpha = s-weighted mean
// of |w| on the support, stored in fp16.  trit[j] in {0,1,2} = 1 + sign(w_j) on
// the support, 1 elsewhere.  A = PSUM8 of |w| over the group.
float fit_ternary_at(const Group& g, float A, float rho, uint8_t* trit /*nullable*/, float* what /*nullable*/) {
  const int G = g.G;
  const float delta = rho * (A * (1.0f / (float)G));
  bool any = false;
  std::vector<uint8_t> in(G);
  for (int j = 0; j < G; ++j) { in[j] = std::fabs(g.w[j]) > delta; any = any || in[j]; }
  float B = psum8(G, [&](int l) {
    float acc = 0.0f;
    for (int j = 8 * l; j < 8 * l + 8; ++j) acc = std::fmaf(g.s[j], in[j] ? std::fabs(g.w[j]) : 0.0f, acc);
    return acc;
  });
  float Cs = psum8(G, [&](int l) {
    float acc = 0.0f;
    for (int j = 8 * l; j < 8 * l + 8; ++j) acc = acc + (in[j] ? g.s[j] : 0.0f);
    return acc;
  });
  if (Cs == 0.0f) {               // no activation weight on the support: fit with s == 1
    B = psum8(G, [&](int l) {
      float acc = 0.0f;
      for (int j = 8 * l; j < 8 * l + 8; ++j) acc = std::fmaf(1.0f, in[j] ? std::fabs(g.w[j]) : 0.0f, acc);
      return acc;
    });
    Cs = psum8(G, [&](int l) {
      float acc = 0.0f;
      for (int j = 8 * l; j < 8 * l + 8; ++j) acc = acc + (in[j] ? 1.0f : 0.0f);
      return acc;
    });
  }
  const float alpha = any ? round_through_half(B / Cs) : 0.0f;
  for (int j = 0; j < G; ++j) {
    const int t = in[j] ? (g.w[j] < 0.0f ? 0 : 2) : 1;
    if (trit) trit[j] = (uint8_t)t;
    if (what) what[j] = (float)(t - 1) * alpha;
  }
  return alpha;
}

// The fit of windq_fit_eval: rho = 0.7 (textbook ternary weights).
float fit_ternary(const Group& g, float A, uint8_t* trit /*nullable*/, float* what /*nullable*/) {
  return fit_ternary_at(g, A, 0.7f, trit, what);
}

// READING: binary = sign(w) * alpha, alpha = s-weighted mean |w| in fp16;
// sign(0) = +.  bit[j] = !(w_j < 0).
float fit_binary(const Group& g, float A, uint8_t* bit /*nullable*/, float* what /*nullable*/) {
  const int G = g.G;
  const float B = psum8(G, [&](int l) {
    float acc = 0.0f;
    for (int j = 8 * l; j < 8 * l + 8; ++j) acc = std::fmaf(g.s[j], std::fabs(g.w[j]), acc);
    return acc;
  });
  const float Cs = psum8(G, [&](int l) {
    float acc = 0.0f;
    for (int j = 8 * l; j < 8 * l + 8; ++j) acc = acc + g.s[j];
    return acc;
  });
  const float alpha = round_through_half(Cs == 0.0f ? A * (1.0f / (float)G) : B / Cs);
  for (int j = 0; j < G; ++j) {
    const int b = !(g.w[j] < 0.0f);
    if (bit) bit[j] = (uint8_t)b;
    if (what) what[j] = b ? alpha : -alpha;
  }
  return alpha;
}

void load_group(const uint16_t* W, int64_t ldw, int64_t r, int64_t u, int G, float* w) {
  const uint16_t* p = W + r * ldw + u * (int64_t)G;
  for (int j = 0; j < G; ++j) w[j] = half_to_float(p[j]);
}

// ---------------------------------------------------------------- packing
int64_t group_code_bytes(int action, int G) {
  switch (action) {
    case 0: return 2 * (int64_t)G;
    case 1: return G;
    case 2: return G / 2;
    case 3: return 3 * (int64_t)G / 8;
    case 4: return G / 4;
    case 5: return (G + 4) / 5;
    case 6: return G / 8;
  }
  return -1;
}

int64_t round_up16(int64_t x) { return (x + 15) / 16 * 16; }

// codes[j] -> bytes of one row-group.  Little-endian inside a byte.
void pack_group(int action, int G, const uint8_t* q, uint8_t* out) {
  const int64_t nb = group_code_bytes(action, G);
  std::memset(out, 0, (size_t)nb);
  switch (action) {
    case 1: for (int j = 0; j < G; ++j) out[j] = q[j]; break;
    case 2: for (int j = 0; j < G; ++j) out[j / 2] |= (uint8_t)(q[j] << (4 * (j % 2))); break;
    case 3:
      for (int j = 0; j < G; ++j)
        for (int t = 0; t < 3; ++t)
          if ((q[j] >> t) & 1) { const int pos = 3 * j + t; out[pos / 8] |= (uint8_t)(1u << (pos % 8)); }
      break;
    case 4: for (int j = 0; j < G; ++j) out[j / 4] |= (uint8_t)(q[j] << (2 * (j % 4))); break;
    case 5: {
      const int pow3[5] = {1, 3, 9, 27, 81};
      for (int j = 0; j < G; ++j) out[j / 5] = (uint8_t)(out[j / 5] + q[j] * pow3[j % 5]);
      break;
    }
    case 6: for (int j = 0; j < G; ++j) out[j / 8] |= (uint8_t)(q[j] << (j % 8)); break;
  }
}

int64_t unit_centibits(int action, int64_t R, int G, int scale_bits, int zero_bits) {
  const int64_t n = R * (int64_t)G;
  switch (action) {
    case 0: return 1600 * n;
    case 1: return 800 * n + R * 100 * (int64_t)(scale_bits + zero_bits);
    case 2: return 400 * n + R * 100 * (int64_t)(scale_bits + zero_bits);
    case 3: return 300 * n + R * 100 * (int64_t)(scale_bits + zero_bits);
    case 4: return 200 * n + R * 100 * (int64_t)(scale_bits + zero_bits);
    case 5: return 158 * n + R * 100 * (int64_t)scale_bits;
    case 6: return 100 * n + R * 100 * (int64_t)scale_bits;
  }
  return -1;
}

}  // namespace

extern "C" {

// ---- helpers exported only so that the tests can pin them -------------------
float oracle_half_to_float(uint16_t h) { return half_to_float(h); }
uint16_t oracle_float_to_half(float f) { return float_to_half(f); }
// PSUM8 of x[0..G) with plain addition in the leaves.
float oracle_psum8(const float* x, int G) {
  if (!valid_group_width(G)) return NAN;
  return psum8(G, [&](int l) {
    float acc = 0.0f;
    for (int j = 8 * l; j < 8 * l + 8; ++j) acc = acc + x[j];
    return acc;
  });
}
// One uniform candidate on one group: scale, zero, error, codes (for the pins).
int oracle_uniform_candidate(const float* w, const float* s, int G, int bits, float p,
                             float* scale, float* zero, float* err, uint8_t* codes /*nullable*/) {
  if (!valid_group_width(G) || bits < 1 || bits > 8) return 1;
  Group g{G, w, s};
  float mn, rng;
  group_range(g, &mn, &rng);
  const UniformParams u = uniform_params(mn, rng, p, bits);
  *scale = u.scale;
  *zero = u.zf;
  *err = uniform_error(g, u);
  if (codes) for (int j = 0; j < G; ++j) codes[j] = (uint8_t)(int)(centred_code(w[j], u) + u.zf);
  return 0;
}

// ---- a1: activation statistics (calibration forward pass, App. "Salient Weight
// Protection": per-channel activation scale).  READING: s_j = mean_t x_tj^2.
int oracle_act_stats(const uint16_t* X, int64_t T, int64_t C, int64_t ldx, float* s_out) {
  if (!X || !s_out || T <= 0 || C <= 0 || ldx < C) return 1;
  for (int64_t j = 0; j < C; ++j) {
    double acc = 0.0;
    for (int64_t t = 0; t < T; ++t) {
      const double x = (double)half_to_float(X[t * ldx + j]);
      acc += x * x;
    }
    s_out[j] = (float)(acc / (double)T);
  }
  return 0;
}

// ---- a2: Table 1, dims 0-4 and 9-11, for every unit.
// feat[u] = {mean, std, abs_mean, sparsity, outlier_frac, s_mean, s_std, s_max}.
// READING: population std; nearest-rank P99 (k = ceil(0.99 n), 1-indexed).
int oracle_unit_features(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                         float* feat_out) {
  if (!W || !s || !feat_out || R <= 0 || C <= 0 || G <= 0 || C % G != 0 || ldw < C) return 1;
  const int64_t U = C / G;
  const int64_t n = R * (int64_t)G;
  std::vector<float> a((size_t)n);
  for (int64_t u = 0; u < U; ++u) {
    double sum = 0.0, sum_abs_w = 0.0;
    int64_t tiny = 0;
    for (int64_t r = 0; r < R; ++r)
      for (int j = 0; j < G; ++j) {
        const float w = half_to_float(W[r * ldw + u * G + j]);
        const float aw = std::fabs(w);
        a[(size_t)(r * G + j)] = aw;
        sum += (double)w;
        sum_abs_w += (double)aw;
        if (aw < 1e-6f) ++tiny;
      }
    const double mean = sum / (double)n;
    double var = 0.0;
    for (int64_t r = 0; r < R; ++r)
      for (int j = 0; j < G; ++j) {
        const double d = (double)half_to_float(W[r * ldw + u * G + j]) - mean;
        var += d * d;
      }
    var /= (double)n;
    const int64_t k = (99 * n + 99) / 100;                       // ceil(0.99 n)
    std::vector<float> sorted(a);
    std::sort(sorted.begin(), sorted.end());
    const float p99 = sorted[(size_t)(k - 1)];
    const float thr = 0.5f * p99;
    int64_t outl = 0;
    for (int64_t i = 0; i < n; ++i) if (a[(size_t)i] > thr) ++outl;

    double ssum = 0.0, smax = (double)s[u * G];
    for (int j = 0; j < G; ++j) { ssum += (double)s[u * G + j]; smax = std::max(smax, (double)s[u * G + j]); }
    const double smean = ssum / (double)G;
    double svar = 0.0;
    for (int j = 0; j < G; ++j) { const double d = (double)s[u * G + j] - smean; svar += d * d; }
    svar /= (double)G;

    float* f = feat_out + u * 8;
    f[0] = (float)mean;
    f[1] = (float)std::sqrt(var);
    f[2] = (float)(sum_abs_w / (double)n);
    f[3] = (float)((double)tiny / (double)n);
    f[4] = (float)((double)outl / (double)n);
    f[5] = (float)smean;
    f[6] = (float)std::sqrt(svar);
    f[7] = (float)smax;
  }
  return 0;
}

// ---- a3: fit every row-group of units [u_begin, u_end) under all six bit-widths.
// err_out[U][6], energy_out[U] (nullable), clip_idx_out[4][U][R] (nullable),
// group_err_out[6][U][R] (nullable).  Only rows of the requested units are written.
// thresh == NULL: the fit of every group as it is.  thresh != NULL (one saliency threshold per unit,
// from oracle_salient_select): READING -- a protected weight (key |w| * sqrt(s_j) >= thresh[u]) is
// stored apart in INT8, so it is taken out of its group's fit: inside the group it counts as a zero
// weight with zero activation weight (its position and the group size stay), which removes it from
// the range, from every sum and from every error; the error of its INT8 copy is not part of err.
static int fit_eval_impl(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                         const float* clip_grid, int K, int64_t u_begin, int64_t u_end, const float* thresh,
                         float* err_out, float* energy_out, uint8_t* clip_idx_out, float* group_err_out) {
  if (!W || !s || !clip_grid || !err_out || R <= 0 || C <= 0 || !valid_group_width(G) || C % G != 0 ||
      ldw < C || K < 1 || K > 64)
    return 1;
  const int64_t U = C / G;
  if (u_begin < 0 || u_end > U || u_begin > u_end) return 1;
  std::vector<float> w((size_t)G), what((size_t)G), sm((size_t)G);
  for (int64_t u = u_begin; u < u_end; ++u) {
    double tot[6] = {0, 0, 0, 0, 0, 0};
    double energy = 0.0;
    const float* su = s + u * G;
    for (int64_t r = 0; r < R; ++r) {
      load_group(W, ldw, r, u, G, w.data());
      if (thresh) {
        for (int j = 0; j < G; ++j) {
          const bool prot = std::fabs(w[(size_t)j]) * std::sqrt(s[u * G + j]) >= thresh[u];
          sm[(size_t)j] = prot ? 0.0f : s[u * G + j];
          if (prot) w[(size_t)j] = 0.0f;
        }
        su = sm.data();
      }
      Group g{G, w.data(), su};
      float e[6];
      float mn, rng;
      group_range(g, &mn, &rng);
      for (int bi = 0; bi < 4; ++bi) {
        int bk;
        search_uniform(g, mn, rng, kUniformBits[bi], clip_grid, K, &bk, &e[bi]);
        if (clip_idx_out) clip_idx_out[((int64_t)bi * U + u) * R + r] = (uint8_t)bk;
      }
      const float A = sum_abs(g);
      fit_ternary(g, A, nullptr, what.data());
      e[4] = error_against(g, what.data());
      fit_binary(g, A, nullptr, what.data());
      e[5] = error_against(g, what.data());
      for (int b = 0; b < 6; ++b) {
        tot[b] += (double)e[b];
        if (group_err_out) group_err_out[((int64_t)b * U + u) * R + r] = e[b];
      }
      for (int j = 0; j < G; ++j) energy += (double)su[j] * (double)w[j] * (double)w[j];
    }
    for (int b = 0; b < 6; ++b) err_out[u * 6 + b] = (float)tot[b];
    if (energy_out) energy_out[u] = (float)energy;
  }
  return 0;
}

int oracle_fit_eval(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                    const float* clip_grid, int K, int64_t u_begin, int64_t u_end, float* err_out,
                    float* energy_out, uint8_t* clip_idx_out, float* group_err_out) {
  return fit_eval_impl(W, R, C, ldw, G, s, clip_grid, K, u_begin, u_end, nullptr, err_out, energy_out, clip_idx_out,
                       group_err_out);
}

int oracle_fit_eval_protected(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                              const float* clip_grid, int K, int64_t u_begin, int64_t u_end, const float* thresh,
                              float* err_out, float* energy_out, uint8_t* clip_idx_out, float* group_err_out) {
  if (!thresh) return 1;
  return fit_eval_impl(W, R, C, ldw, G, s, clip_grid, K, u_begin, u_end, thresh, err_out, energy_out, clip_idx_out,
                       group_err_out);
}

// ---- a5: effective bits (Eq. 6 with no protected weights, extended by the
// per-group scale / zero-point overhead) in integer centibits, plus the byte
// offset of every unit's packed block (each rounded up to 16 bytes).
int oracle_effective_bits(const uint8_t* actions, int64_t U, int64_t R, int G, int scale_bits,
                          int zero_bits, int64_t* unit_centibits_out, int64_t* code_offsets_out,
                          int64_t* total_centibits_out, int64_t* total_packed_bytes_out) {
  if (!actions || U <= 0 || R <= 0 || G <= 0 || scale_bits < 0 || zero_bits < 0) return 1;
  int64_t total = 0, off = 0, n_scales = 0, n_zeros = 0;
  for (int64_t u = 0; u < U; ++u) {
    const int a = actions[u];
    if (a > 6) return 1;
    const int64_t cb = unit_centibits(a, R, G, scale_bits, zero_bits);
    if (unit_centibits_out) unit_centibits_out[u] = cb;
    total += cb;
    if (code_offsets_out) code_offsets_out[u] = off;
    off += round_up16(R * group_code_bytes(a, G));
    if (a >= 1) n_scales += R;
    if (a >= 1 && a <= 4) n_zeros += R;
  }
  if (code_offsets_out) code_offsets_out[U] = off;
  if (total_centibits_out) *total_centibits_out = total;
  if (total_packed_bytes_out) *total_packed_bytes_out = off + 2 * (n_scales + n_zeros);
  return 0;
}

// ---- a4: apply a plan.  codes_out must hold code_offsets[U] bytes and is fully
// written (padding = 0); scales_out / zeros_out are fp16 [U][R]; Wq_out is
// fp16 [R][ldw] (nullable).  clip_idx [4][U][R] may be null: the clip search is
// then repeated for the chosen bit-width.
// thresh == NULL: the plan applied to every weight.  thresh != NULL: salient-weight protection.
// READING (the paper says no more than that protected weights are kept in INT8): in every unit that is
// not skipped, a weight whose key |w| * sqrt(s_j) reaches thresh[u] is protected.  Inside its group it
// counts as a zero weight with zero activation weight (as in the protected fit), so the group's
// parameters and the codes of the other weights are those of the masked group, and its own slot in the
// packed stream holds the code of the value 0 (a reader skips it by the mask).  The protected weights
// of a unit share one symmetric INT8 grid: scale sigma_u = fp16(max |w| over them / 127) (1 if that is
// zero), code clamp(rne(w / sigma_u), -127, 127), rounding as in the uniform fit; their fake-quantised
// value is fp16(code * sigma_u).  The INT8 codes of a unit are listed in row-major order of the unit
// (rows, then columns) starting at prot_offsets_out[u]; a skipped unit protects nothing.
static int apply_plan_impl(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                           const float* clip_grid, int K, const uint8_t* actions, const uint8_t* clip_idx,
                           const int64_t* code_offsets, const float* thresh, uint8_t* codes_out, uint16_t* scales_out,
                           uint16_t* zeros_out, uint16_t* Wq_out, uint16_t* prot_scale_out, int64_t* prot_offsets_out,
                           int8_t* prot_q_out, const uint16_t* scale_in = nullptr, const float* thr_grid = nullptr,
                           int Kt = 0, const uint8_t* thr_idx = nullptr) {
  if (thresh && (!prot_scale_out || !prot_offsets_out || !prot_q_out)) return 1;
  if (thr_idx && (!thr_grid || Kt < 1 || Kt > 64)) return 1;
  if (!W || !s || !clip_grid || !actions || !code_offsets || !codes_out || !scales_out || !zeros_out ||
      R <= 0 || C <= 0 || !valid_group_width(G) || C % G != 0 || ldw < C || K < 1 || K > 64)
    return 1;
  const int64_t U = C / G;
  std::memset(codes_out, 0, (size_t)code_offsets[U]);
  std::vector<float> w((size_t)G), what((size_t)G), worig((size_t)G), sm((size_t)G);
  std::vector<uint8_t> q((size_t)G), prot((size_t)G);
  int64_t n_prot = 0;
  for (int64_t u = 0; u < U; ++u) {
    const int a = actions[u];
    if (a > 6) return 1;
    const float* su = s + u * G;
    const int64_t gb = group_code_bytes(a, G);
    const bool protect = thresh && a != 0;
    float sigma = 1.0f, inv8 = 1.0f;
    if (thresh) {
      prot_offsets_out[u] = n_prot;
      float m = 0.0f;
      if (protect)
        for (int64_t r = 0; r < R; ++r)
          for (int j = 0; j < G; ++j) {
            const float aw = std::fabs(half_to_float(W[r * ldw + u * G + j]));
            if (aw * std::sqrt(s[u * G + j]) >= thresh[u] && aw > m) m = aw;
          }
      sigma = round_through_half(m / 127.0f);
      if (sigma == 0.0f) sigma = 1.0f;
      inv8 = 1.0f / sigma;
      prot_scale_out[u] = protect ? float_to_half(sigma) : (uint16_t)0;
    }
    for (int64_t r = 0; r < R; ++r) {
      uint8_t* dst = codes_out + code_offsets[u] + r * gb;
      uint16_t scale_h = 0, zero_h = 0;
      if (a == 0) {
        std::memcpy(dst, W + r * ldw + u * G, (size_t)(2 * G));
        if (Wq_out) std::memcpy(Wq_out + r * ldw + u * G, W + r * ldw + u * G, (size_t)(2 * G));
      } else {
        load_group(W, ldw, r, u, G, w.data());
        if (protect) {
          for (int j = 0; j < G; ++j) {
            worig[(size_t)j] = w[(size_t)j];
            prot[(size_t)j] = std::fabs(w[(size_t)j]) * std::sqrt(s[u * G + j]) >= thresh[u];
            sm[(size_t)j] = prot[(size_t)j] ? 0.0f : s[u * G + j];
            if (prot[(size_t)j]) w[(size_t)j] = 0.0f;
          }
          su = sm.data();
        }
        Group g{G, w.data(), su};
        if (a <= 4) {
          const int bi = a - 1, bits = kUniformBits[bi];
          float mn, rng;
          group_range(g, &mn, &rng);
          int k;
          if (clip_idx) {
            k = clip_idx[((int64_t)bi * U + u) * R + r];
            if (k >= K) k = K - 1;  // the interface treats an index beyond the grid as the last ratio
          } else {
            float e;
            search_uniform(g, mn, rng, bits, clip_grid, K, &k, &e);
          }
          UniformParams p = uniform_params(mn, rng, clip_grid[k], bits);
          if (scale_in) {  // a refined step size replaces the clip-grid scale; the zero point stays
            p.scale = half_to_float(scale_in[((int64_t)bi * U + u) * R + r]);
            p.inv = 1.0f / p.scale;
          }
          for (int j = 0; j < G; ++j) {
            const float c = centred_code(w[j], p);
            q[j] = (uint8_t)(int)(c + p.zf);
            what[j] = c * p.scale;
          }
          scale_h = float_to_half(p.scale);
          zero_h = float_to_half(p.zf);
        } else {
          const float A = sum_abs(g);
          float rho = 0.7f;
          if (thr_idx) {  // the threshold ratio the search chose for this group (an index beyond the grid = the last)
            int kt = thr_idx[u * R + r];
            if (kt >= Kt) kt = Kt - 1;
            rho = thr_grid[kt];
          }
          const float alpha = (a == 5) ? fit_ternary_at(g, A, rho, q.data(), what.data())
                                       : fit_binary(g, A, q.data(), what.data());
          scale_h = float_to_half(alpha);
        }
        pack_group(a, G, q.data(), dst);
        if (protect)
          for (int j = 0; j < G; ++j)
            if (prot[(size_t)j]) {
              float c = std::fmaf(worig[(size_t)j], inv8, kMagic) - kMagic;   // rne(w / sigma), one rounding
              c = std::min(std::max(c, -127.0f), 127.0f);
              what[(size_t)j] = c * sigma;
              prot_q_out[n_prot++] = (int8_t)(int)c;
            }
        if (Wq_out)
          for (int j = 0; j < G; ++j) Wq_out[r * ldw + u * G + j] = float_to_half(what[j]);
      }
      scales_out[u * R + r] = scale_h;
      zeros_out[u * R + r] = zero_h;
    }
  }
  if (thresh) prot_offsets_out[U] = n_prot;
  return 0;
}

int oracle_apply_plan(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                      const float* clip_grid, int K, const uint8_t* actions, const uint8_t* clip_idx,
                      const int64_t* code_offsets, uint8_t* codes_out, uint16_t* scales_out,
                      uint16_t* zeros_out, uint16_t* Wq_out) {
  return apply_plan_impl(W, R, C, ldw, G, s, clip_grid, K, actions, clip_idx, code_offsets, nullptr, codes_out,
                         scales_out, zeros_out, Wq_out, nullptr, nullptr, nullptr);
}

int oracle_apply_plan_protected(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                                const float* clip_grid, int K, const uint8_t* actions, const uint8_t* clip_idx,
                                const int64_t* code_offsets, const float* thresh, uint8_t* codes_out,
                                uint16_t* scales_out, uint16_t* zeros_out, uint16_t* Wq_out, uint16_t* prot_scale_out,
                                int64_t* prot_offsets_out, int8_t* prot_q_out) {
  if (!thresh) return 1;
  return apply_plan_impl(W, R, C, ldw, G, s, clip_grid, K, actions, clip_idx, code_offsets, thresh, codes_out,
                         scales_out, zeros_out, Wq_out, prot_scale_out, prot_offsets_out, prot_q_out);
}

// Protection and refined step sizes together (scale_in from oracle_fit_refine_protected; needs clip_idx).
int oracle_apply_plan_protected_refined(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                                        const float* clip_grid, int K, const uint8_t* actions, const uint8_t* clip_idx,
                                        const uint16_t* scale_in, const int64_t* code_offsets, const float* thresh,
                                        uint8_t* codes_out, uint16_t* scales_out, uint16_t* zeros_out, uint16_t* Wq_out,
                                        uint16_t* prot_scale_out, int64_t* prot_offsets_out, int8_t* prot_q_out) {
  if (!thresh || !clip_idx || !scale_in) return 1;
  return apply_plan_impl(W, R, C, ldw, G, s, clip_grid, K, actions, clip_idx, code_offsets, thresh, codes_out,
                         scales_out, zeros_out, Wq_out, prot_scale_out, prot_offsets_out, prot_q_out, scale_in);
}

// ---- search over the ternary assignment (App. "Per-unit Scale Optimization": the low-bit operators
// fit their assignment and a per-group scale; Sec. 3.5) ------------------------------------------------
// The paper prints no formula for its low-bit operators.  READING: for a fixed scale alpha the best
// ternary code of w_j is sign(w_j) when |w_j| > alpha / 2 and 0 otherwise, whatever s_j is, so the best
// support is always a threshold set {|w| > tau}; and for a fixed support the best scale is the
// s-weighted mean of |w| on it.  The search therefore tries Kt thresholds tau_k = thr_grid[k] * mean|w|
// (ratios supplied by the caller, like the clip ratios), fits each exactly as fit_ternary_at does, scores
// it by the s-weighted squared error in PSUM8 order, and keeps the smallest k with the least error.
// With thr_grid = {0.7} the result is the ternary column of oracle_fit_eval, bit for bit.
// The 1-bit operator needs no search: with the two levels +-alpha the code sign(w_j) is the best one for
// every alpha > 0, and alpha has its closed form (fit_binary).
// thresh (nullable): salient weights are taken out of the group as in the protected fit.
//   err_out fp32 [U] (double accumulation over rows), thr_idx_out u8 [U][R], alpha_out fp16 bits [U][R],
//   group_err_out fp32 [U][R] (nullable)
int oracle_fit_ternary_search(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                              const float* thr_grid, int Kt, int64_t u_begin, int64_t u_end, const float* thresh,
                              float* err_out, uint8_t* thr_idx_out, uint16_t* alpha_out, float* group_err_out) {
  if (!W || !s || !thr_grid || !err_out || !thr_idx_out || !alpha_out || R <= 0 || C <= 0 || !valid_group_width(G) ||
      C % G != 0 || ldw < C || Kt < 1 || Kt > 64)
    return 1;
  const int64_t U = C / G;
  if (u_begin < 0 || u_end > U || u_begin > u_end) return 1;
  std::vector<float> w((size_t)G), what((size_t)G), sm((size_t)G);
  for (int64_t u = u_begin; u < u_end; ++u) {
    double tot = 0.0;
    const float* su = s + u * G;
    for (int64_t r = 0; r < R; ++r) {
      load_group(W, ldw, r, u, G, w.data());
      if (thresh) {
        for (int j = 0; j < G; ++j) {
          const bool prot = std::fabs(w[(size_t)j]) * std::sqrt(s[u * G + j]) >= thresh[u];
          sm[(size_t)j] = prot ? 0.0f : s[u * G + j];
          if (prot) w[(size_t)j] = 0.0f;
        }
        su = sm.data();
      }
      Group g{G, w.data(), su};
      const float A = sum_abs(g);
      int bk = 0;
      float be = 0.0f, balpha = 0.0f;
      for (int k = 0; k < Kt; ++k) {
        const float alpha = fit_ternary_at(g, A, thr_grid[k], nullptr, what.data());
        const float e = error_against(g, what.data());
        if (k == 0 || e < be) { be = e; bk = k; balpha = alpha; }
      }
      thr_idx_out[u * R + r] = (uint8_t)bk;
      alpha_out[u * R + r] = float_to_half(balpha);
      if (group_err_out) group_err_out[u * R + r] = be;
      tot += (double)be;
    }
    err_out[u] = (float)tot;
  }
  return 0;
}

// One threshold ratio on one group (exported so that the tests can pin it): scale, error, trits.
int oracle_ternary_candidate(const float* w, const float* s, int G, float rho, float* alpha_out, float* err_out,
                             uint8_t* trits_out /*nullable*/) {
  if (!w || !s || !valid_group_width(G) || !alpha_out || !err_out) return 1;
  Group g{G, w, s};
  std::vector<float> what((size_t)G);
  *alpha_out = fit_ternary_at(g, sum_abs(g), rho, trits_out, what.data());
  *err_out = error_against(g, what.data());
  return 0;
}

// One group under the 1-bit fit (exported for the pins): scale, error, bits.
int oracle_binary_candidate(const float* w, const float* s, int G, float* alpha_out, float* err_out, uint8_t* bits_out /*nullable*/) {
  if (!w || !s || !valid_group_width(G) || !alpha_out || !err_out) return 1;
  Group g{G, w, s};
  std::vector<float> what((size_t)G);
  *alpha_out = fit_binary(g, sum_abs(g), bits_out, what.data());
  *err_out = error_against(g, what.data());
  return 0;
}

// oracle_apply_plan with the thresholds the search chose for the 1.58-bit units (thr_idx u8 [U][R]).
int oracle_apply_plan_searched(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                               const float* clip_grid, int K, const uint8_t* actions, const uint8_t* clip_idx,
                               const float* thr_grid, int Kt, const uint8_t* thr_idx, const int64_t* code_offsets,
                               uint8_t* codes_out, uint16_t* scales_out, uint16_t* zeros_out, uint16_t* Wq_out) {
  if (!thr_grid || !thr_idx) return 1;
  return apply_plan_impl(W, R, C, ldw, G, s, clip_grid, K, actions, clip_idx, code_offsets, nullptr, codes_out,
                         scales_out, zeros_out, Wq_out, nullptr, nullptr, nullptr, nullptr, thr_grid, Kt, thr_idx);
}

// ---- salient-weight selection (App. "Salient Weight Protection") -----------------------------
// The saliency of a weight is the product of its magnitude and the activation scale of its input
// channel; the top-r fraction of a unit's weights by saliency is kept in INT8.
// READING: the activation scale of channel j is a_j = sqrt(s_j), the root of the mean square that
// act_stats returns (binary32 square root, then one binary32 product |w| * a_j: two IEEE
// operations, so the key is reproducible).  n_p = floor(rate_ppm * n / 10^6) weights are asked
// for; the threshold is the n_p-th largest key of the unit and every weight whose key reaches it
// is protected, so equal keys at the threshold are all in (the protected count can exceed n_p,
// and it is the count that Eq. 6 uses).  n_p = 0 protects nothing (threshold +infinity).
int oracle_salient_select(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                          int64_t rate_ppm, float* thresh_out, int64_t* count_out, uint8_t* mask_out) {
  if (!W || !s || !thresh_out || !count_out || R <= 0 || C <= 0 || G <= 0 || C % G || ldw < C) return 1;
  if (rate_ppm < 0 || rate_ppm > 1000000) return 1;
  const int64_t U = C / G, n = R * G;
  const int64_t n_p = (int64_t)(((__int128)rate_ppm * n) / 1000000);
  if (mask_out) std::memset(mask_out, 0, (size_t)(R * (C / 8)));
  std::vector<float> key((size_t)n);
  for (int64_t u = 0; u < U; ++u) {
    for (int64_t r = 0; r < R; ++r)
      for (int j = 0; j < G; ++j) {
        const float a = std::sqrt(s[u * G + j]);
        key[(size_t)(r * G + j)] = std::fabs(half_to_float(W[r * ldw + u * G + j])) * a;
      }
    float tau = std::numeric_limits<float>::infinity();
    int64_t count = 0;
    if (n_p > 0) {
      std::vector<float> sorted(key);
      std::nth_element(sorted.begin(), sorted.begin() + (n - n_p), sorted.end());
      tau = sorted[(size_t)(n - n_p)];   // (n - n_p + 1)-th smallest = n_p-th largest
      for (int64_t i = 0; i < n; ++i) count += key[(size_t)i] >= tau;
    }
    thresh_out[u] = tau;
    count_out[u] = count;
    if (mask_out && n_p > 0)
      for (int64_t r = 0; r < R; ++r)
        for (int j = 0; j < G; ++j)
          if (key[(size_t)(r * G + j)] >= tau) {
            const int64_t col = u * G + j;
            mask_out[r * (C / 8) + col / 8] |= (uint8_t)(1u << (col % 8));
          }
  }
  return 0;
}

// Eq. 6 in full: B_i = 16 n_i for skip, else b_i (n_i - n_i^(p)) + 8 n_i^(p), in centibits, plus
// the per-group scale / zero-point overhead of the quantised part as in oracle_effective_bits.
// A skipped unit protects nothing (its weights stay fp16).
int oracle_effective_bits_protected(const uint8_t* actions, const int64_t* n_protected, int64_t U, int64_t R, int G,
                                    int scale_bits, int zero_bits, int64_t* unit_centibits_out,
                                    int64_t* total_centibits_out) {
  if (!actions || !n_protected || U <= 0 || R <= 0 || G <= 0 || scale_bits < 0 || zero_bits < 0) return 1;
  static const int64_t centi[7] = {1600, 800, 400, 300, 200, 158, 100};
  int64_t total = 0;
  for (int64_t u = 0; u < U; ++u) {
    const int a = actions[u];
    const int64_t n = R * G, np_ = n_protected[u];
    if (a > 6 || np_ < 0 || np_ > n) return 1;
    int64_t cb;
    if (a == 0) cb = 1600 * n;
    else cb = centi[a] * (n - np_) + 800 * np_ + 100 * R * (scale_bits + ((a <= 4) ? zero_bits : 0));
    if (unit_centibits_out) unit_centibits_out[u] = cb;
    total += cb;
  }
  if (total_centibits_out) *total_centibits_out = total;
  return 0;
}

// ---- heuristic allocator inputs ("Comparison with Heuristic Sensitivity Allocator") and fallback ----
// Saliency score of a unit: the mean, over the unit's weights, of activation scale times weight
// magnitude, with the activation scale a_j = sqrt(s_j) as in oracle_salient_select.  Products and
// the sum are taken in double (tolerance output).
int oracle_unit_saliency(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s, float* sal_out) {
  if (!W || !s || !sal_out || R <= 0 || C <= 0 || G <= 0 || C % G || ldw < C) return 1;
  for (int64_t u = 0; u < C / G; ++u) {
    double acc = 0.0;
    for (int64_t r = 0; r < R; ++r)
      for (int j = 0; j < G; ++j)
        acc += (double)std::sqrt(s[u * G + j]) * (double)std::fabs(half_to_float(W[r * ldw + u * G + j]));
    sal_out[u] = (float)(acc / (double)(R * G));
  }
  return 0;
}

// The engine's fallback (Sec. 3.5): an operator whose reconstruction error turns out too large is
// replaced by one of higher precision.  READING (the paper gives neither the measure nor the
// threshold): the error of action a is excessive when err[u][a] > theta * energy[u], both binary32,
// one binary32 product on the right; the unit then moves to the next higher precision (1 -> 1.58 -> 2
// -> 3 -> 4 -> 8 -> skip) until the test passes; skip has no error and always passes.
int oracle_fallback(const float* err, const float* energy, const uint8_t* actions, int64_t U, float theta,
                    uint8_t* actions_out, int64_t* n_changed_out) {
  if (!err || !energy || !actions || !actions_out || U <= 0 || !(theta >= 0.0f)) return 1;
  int64_t changed = 0;
  for (int64_t u = 0; u < U; ++u) {
    int a = actions[u];
    const float limit = theta * energy[u];
    while (a >= 1 && a <= 6 && err[u * 6 + (a - 1)] > limit) --a;   // codes above 6 are not actions: copied as they are
    actions_out[u] = (uint8_t)a;
    changed += a != actions[u];
  }
  if (n_changed_out) *n_changed_out = changed;
  return 0;
}

// The deterministic rule of the heuristic sensitivity allocator ("Comparison with Heuristic
// Sensitivity Allocator"): units are ranked by saliency, all start at 2 bit, the least sensitive are
// pushed to 1.58 or 1 bit to free budget and the most sensitive are promoted to 3 or 4 bit while the
// budget permits.  READING (the paper fixes neither the order of the moves nor how much is freed):
//   cost(u, a) = Eq. 6 of unit u under action a, in centibits, with the per-group parameter bits
//                counted as in oracle_effective_bits_protected
//   budget     = target_cb * N,   floor = budget - headroom_cb * N,   N = sum of n_weights
//   rank       : saliency descending under the total order of the binary32 bit patterns (sign and
//                magnitude; -0 below +0), equal scores by ascending unit index
//   1. every unit takes the 2-bit action; total = sum of cost(u, 2 bit)
//   2. two sweeps from the least sensitive unit upwards, the first to 1.58 bit, the second to 1 bit:
//      a unit is moved down while total > floor; the first unit met with total <= floor ends step 2
//   3. one pass from the most sensitive unit downwards over the units still at 2 bit: the unit takes
//      4 bit if total stays <= budget, else 3 bit if total stays <= budget, else it stays
// order_out (nullable) receives the ranking, total_out the final total.
static uint32_t saliency_key(float x) {
  uint32_t b;
  std::memcpy(&b, &x, 4);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

static int64_t unit_cost(int a, int64_t n, int64_t np_, int64_t groups, int scale_bits, int zero_bits) {
  static const int64_t centi[7] = {1600, 800, 400, 300, 200, 158, 100};
  if (a == 0) return 1600 * n;
  return centi[a] * (n - np_) + 800 * np_ + 100 * groups * (scale_bits + ((a <= 4) ? zero_bits : 0));
}

int oracle_greedy_allocate(const float* saliency, const int64_t* n_weights, const int64_t* n_protected,
                           const int64_t* n_groups, int64_t U, int64_t target_cb, int64_t headroom_cb, int scale_bits,
                           int zero_bits, uint8_t* actions_out, int64_t* order_out, int64_t* total_out) {
  if (!saliency || !n_weights || !n_groups || !actions_out || U <= 0 || target_cb < 0 || headroom_cb < 0 ||
      scale_bits < 0 || zero_bits < 0)
    return 1;
  int64_t N = 0;
  for (int64_t u = 0; u < U; ++u) {
    const int64_t np_ = n_protected ? n_protected[u] : 0;
    if (n_weights[u] < 0 || n_groups[u] < 0 || np_ < 0 || np_ > n_weights[u]) return 1;
    N += n_weights[u];
  }
  std::vector<int64_t> order((size_t)U);
  for (int64_t u = 0; u < U; ++u) order[(size_t)u] = u;
  std::sort(order.begin(), order.end(), [&](int64_t a, int64_t b) {
    const uint32_t ka = saliency_key(saliency[a]), kb = saliency_key(saliency[b]);
    return ka != kb ? ka > kb : a < b;
  });
  auto cost = [&](int64_t u, int a) {
    return unit_cost(a, n_weights[u], n_protected ? n_protected[u] : 0, n_groups[u], scale_bits, zero_bits);
  };
  const int64_t budget = target_cb * N, floor_ = budget - headroom_cb * N;
  int64_t total = 0;
  for (int64_t u = 0; u < U; ++u) {
    actions_out[u] = 4;
    total += cost(u, 4);
  }
  bool freed = false;
  for (int down = 5; down <= 6 && !freed; ++down)
    for (int64_t r = U - 1; r >= 0; --r) {
      if (total <= floor_) {
        freed = true;
        break;
      }
      const int64_t u = order[(size_t)r];
      total += cost(u, down) - cost(u, actions_out[u]);
      actions_out[u] = (uint8_t)down;
    }
  for (int64_t r = 0; r < U; ++r) {
    const int64_t u = order[(size_t)r];
    if (actions_out[u] != 4) continue;
    for (int up = 2; up <= 3; ++up) {
      const int64_t with = total + cost(u, up) - cost(u, 4);
      if (with <= budget) {
        total = with;
        actions_out[u] = (uint8_t)up;
        break;
      }
    }
  }
  if (order_out)
    for (int64_t r = 0; r < U; ++r) order_out[r] = order[(size_t)r];
  if (total_out) *total_out = total;
  return 0;
}

// oracle_apply_plan with the scales of the uniform groups taken from oracle_fit_refine (scale_in fp16 bits
// [4][U][R]); zero points are those of the clip-grid fit that clip_idx names.
int oracle_apply_plan_refined(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                              const float* clip_grid, int K, const uint8_t* actions, const uint8_t* clip_idx,
                              const uint16_t* scale_in, const int64_t* code_offsets, uint8_t* codes_out,
                              uint16_t* scales_out, uint16_t* zeros_out, uint16_t* Wq_out) {
  if (!clip_idx || !scale_in) return 1;
  return apply_plan_impl(W, R, C, ldw, G, s, clip_grid, K, actions, clip_idx, code_offsets, nullptr, codes_out,
                         scales_out, zeros_out, Wq_out, nullptr, nullptr, nullptr, scale_in);
}

// ---- iterative step-size refinement (App. "Per-unit Scale Optimization") -------------------------
// The paper's operators fit their scale by a small local optimisation, typically 10 Adam steps on
// the reconstruction loss of the current chunk, and the 3/4/8-bit ones treat the step size as a learned
// parameter, with the rounding passed straight through (the LSQ rule, Esser et al. 2020).  It prints no
// formulas.  READING, for the four uniform bit-widths, per group, all in binary32:
//   warm start   the clip-grid fit: Delta_0 = its stored fp16 scale, zero point z fixed at its value
//   iterate t    Delta_h = fp16(Delta_t) is the step actually used (a scale is stored in fp16);
//                c_j = clamp(rne(w_j / Delta_h), -z, qmax - z), d_j = c_j Delta_h - w_j,
//                loss e_t = sum s_j d_j^2            (the operations of uniform_error, same order)
//                psi_j = rne(w_j / Delta_h) - w_j / Delta_h inside the range, c_j where clipped
//                g_t = sum (s_j d_j) psi_j           (half the LSQ gradient; PSUM8 order)
//   Adam         beta1 0.9, beta2 0.999, eps 1e-8, bias-corrected, learning rate lr * Delta_0:
//                m = 0.9 m + 0.1 g;  v = 0.999 v + 0.001 g^2;
//                Delta_{t+1} = Delta_t - (lr Delta_0) * (m c1_t) / (sqrt(v c2_t) + eps),
//                c1_t = 1 / (1 - 0.9^t), c2_t = 1 / (1 - 0.999^t) rounded to binary32
//   result       the iterate with the least loss among t = 0..T (first one on ties), so the refined
//                error never exceeds the clip-grid error; the iteration stops early when fp16(Delta)
//                is not a positive finite number.
struct RefineStep {
  float scale;  // Delta_h
  float loss;
  float grad;
};

static void refine_eval(const Group& g, float scale, float zf, float qmaxf, float* loss, float* grad) {
  UniformParams u;
  u.scale = scale;
  u.inv = 1.0f / scale;
  u.zf = zf;
  u.qmaxf = qmaxf;
  *loss = uniform_error(g, u);
  *grad = psum8(g.G, [&](int l) {
    float acc = 0.0f;
    for (int j = 8 * l; j < 8 * l + 8; ++j) {
      const float r = std::fmaf(g.w[j], u.inv, kMagic) - kMagic;
      const float c = centred_code(g.w[j], u);
      const float x = g.w[j] * u.inv;
      const float psi = (c == r) ? r - x : c;
      const float d = std::fmaf(c, u.scale, -g.w[j]);
      const float t = g.s[j] * d;
      acc = std::fmaf(t, psi, acc);
    }
    return acc;
  });
}

static void adam_corrections(int T, float* c1, float* c2) {  // c[t-1] for t = 1..T
  double p1 = 1.0, p2 = 1.0;
  for (int t = 1; t <= T; ++t) {
    p1 *= 0.9;
    p2 *= 0.999;
    c1[t - 1] = (float)(1.0 / (1.0 - p1));
    c2[t - 1] = (float)(1.0 / (1.0 - p2));
  }
}

// Runs the iteration on one group; trace (nullable) receives every iterate that was evaluated.
// Returns the number of iterates evaluated (1..T+1).
static int refine_group(const Group& g, float scale0, float zf, float qmaxf, int T, float lr, float* best_scale,
                        float* best_loss, RefineStep* trace) {
  float c1[32], c2[32];
  adam_corrections(T, c1, c2);
  const float step = lr * scale0;
  float delta = scale0, m = 0.0f, v = 0.0f;
  int n = 0;
  for (int t = 0; t <= T; ++t) {
    const float sh = round_through_half(delta);
    if (!(sh > 0.0f) || std::isinf(sh)) break;
    float loss, grad;
    refine_eval(g, sh, zf, qmaxf, &loss, &grad);
    if (trace) trace[n] = RefineStep{sh, loss, grad};
    if (n == 0 || loss < *best_loss) {
      *best_loss = loss;
      *best_scale = sh;
    }
    ++n;
    if (t == T) break;
    m = std::fmaf(0.9f, m, 0.1f * grad);
    v = std::fmaf(0.999f, v, 0.001f * (grad * grad));
    const float mhat = m * c1[t], vhat = v * c2[t];
    const float upd = mhat / (std::sqrt(vhat) + 1e-8f);
    delta = std::fmaf(-step, upd, delta);
  }
  return n;
}

// One group, for the pins: w, s of length G; scale0 and zf as a clip-grid fit would give them.
// scales / losses / grads receive T+1 entries (unused ones untouched); returns the number evaluated.
int oracle_refine_trace(const float* w, const float* s, int G, int bits, float scale0, float zf, int T, float lr,
                        float* scales, float* losses, float* grads) {
  if (!w || !s || !valid_group_width(G) || T < 0 || T > 32) return -1;
  RefineStep tr[33];
  float bs = 0.0f, bl = 0.0f;
  Group g{G, w, s};
  const int n = refine_group(g, scale0, zf, (float)((1 << bits) - 1), T, lr, &bs, &bl, tr);
  for (int i = 0; i < n; ++i) {
    if (scales) scales[i] = tr[i].scale;
    if (losses) losses[i] = tr[i].loss;
    if (grads) grads[i] = tr[i].grad;
  }
  return n;
}

// Refinement of every group's step size for the four uniform bit-widths, warm-started from the clip
// indices of oracle_fit_eval.  err_out [U][4] (unit sums in double, rows ascending), scale_out fp16
// bits [4][U][R], group_err_out [4][U][R] (nullable).
static int fit_refine_impl(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                           const float* clip_grid, int K, const uint8_t* clip_idx, const float* thresh, int T, float lr,
                           float* err_out, uint16_t* scale_out, float* group_err_out) {
  if (!W || !s || !clip_grid || !clip_idx || !err_out || !scale_out || R <= 0 || C <= 0 || !valid_group_width(G) ||
      C % G != 0 || ldw < C || K < 1 || K > 64 || T < 0 || T > 32 || !(lr >= 0.0f))
    return 1;
  const int64_t U = C / G;
  std::vector<float> w((size_t)G), sm((size_t)G);
  for (int64_t u = 0; u < U; ++u) {
    double tot[4] = {0, 0, 0, 0};
    for (int64_t r = 0; r < R; ++r) {
      load_group(W, ldw, r, u, G, w.data());
      const float* su = s + u * G;
      if (thresh) {  // protected weights leave the group as in the protected fit: zero weight, zero activation weight
        for (int j = 0; j < G; ++j) {
          const bool prot = std::fabs(w[(size_t)j]) * std::sqrt(s[u * G + j]) >= thresh[u];
          sm[(size_t)j] = prot ? 0.0f : s[u * G + j];
          if (prot) w[(size_t)j] = 0.0f;
        }
        su = sm.data();
      }
      Group g{G, w.data(), su};
      float mn, rng;
      group_range(g, &mn, &rng);
      for (int bi = 0; bi < 4; ++bi) {
        const int64_t o = ((int64_t)bi * U + u) * R + r;
        int k = clip_idx[o];
        if (k >= K) k = K - 1;
        const UniformParams p = uniform_params(mn, rng, clip_grid[k], kUniformBits[bi]);
        float bs = 0.0f, bl = 0.0f;
        const int n = refine_group(g, p.scale, p.zf, p.qmaxf, T, lr, &bs, &bl, nullptr);
        if (n == 0) return 2;  // cannot happen: the warm-start scale is a positive finite fp16 value
        tot[bi] += (double)bl;
        scale_out[o] = float_to_half(bs);
        if (group_err_out) group_err_out[o] = bl;
      }
    }
    for (int bi = 0; bi < 4; ++bi) err_out[u * 4 + bi] = (float)tot[bi];
  }
  return 0;
}

int oracle_fit_refine(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                      const float* clip_grid, int K, const uint8_t* clip_idx, int T, float lr, float* err_out,
                      uint16_t* scale_out, float* group_err_out) {
  return fit_refine_impl(W, R, C, ldw, G, s, clip_grid, K, clip_idx, nullptr, T, lr, err_out, scale_out, group_err_out);
}

// The refinement with the salient weights taken out of the groups (thresh [U] from oracle_salient_select,
// clip_idx from oracle_fit_eval_protected with the same thresholds).
int oracle_fit_refine_protected(const uint16_t* W, int64_t R, int64_t C, int64_t ldw, int G, const float* s,
                                const float* clip_grid, int K, const uint8_t* clip_idx, const float* thresh, int T,
                                float lr, float* err_out, uint16_t* scale_out, float* group_err_out) {
  if (!thresh) return 1;
  return fit_refine_impl(W, R, C, ldw, G, s, clip_grid, K, clip_idx, thresh, T, lr, err_out, scale_out, group_err_out);
}

}  // extern "C"

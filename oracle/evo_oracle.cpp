// Reference oracle for the candidate-evaluation step (TEST INFRASTRUCTURE ONLY).
//
// A plain, slow, single-threaded CPU statement of what the evaluation step of
// the EvoEngineer method computes: seeded trial inputs, the functional-
// correctness constraint g(p) (paper Section 3.1, Eq. 1; Section 4.3 "Modular
// Architecture Design", functional testing: outputs are compared against the
// reference implementation over the test cases) and the runtime objective f(p)
// (Section 4.3: times collected over repeated runs; Section 5.1 "Evaluation
// Metric": speedup over the baseline kernel).
//
// This file is used by the tests, by the smoke check and by the benchmark's CPU
// baseline leg only.  It shares no code, header, table or constant generator
// with the CUDA library and the product never calls it.
//
// Build: g++ -std=c++17 -O2 -ffp-contract=off -fno-fast-math (see build.py).
// Contraction must stay off: the closeness rule is defined on individually
// rounded binary32 operations.
//
// Pins (tests/test_oracle_*.py): Philox known-answer vectors; Box-Muller against
// 50-digit evaluation, distribution tests and closed-form invariants; narrowing
// against numpy/torch conversions; the closeness rule against a table of
// hand-worked cases, torch.isclose, an exhaustive 16-bit sweep evaluated through
// double, and brute force; medians against the statistics module.
// No function here is "parity unpinned".

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

namespace {

// ---------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy
// as 1, 2, 3", SC'11).  The paper only says that the test inputs are random
// (Section 4.3: five test cases; Appendix A.8.1 "Evaluation Method": five
// random inputs); the generator is fixed by this library's interface.
// ---------------------------------------------------------------------------
constexpr uint32_t kMul0 = 0xD2511F53u;  // multiplier applied to counter word 0
constexpr uint32_t kMul1 = 0xCD9E8D57u;  // multiplier applied to counter word 2
constexpr uint32_t kWeyl0 = 0x9E3779B9u; // key word 0 increment per round
constexpr uint32_t kWeyl1 = 0xBB67AE85u; // key word 1 increment per round

void philox_round(uint32_t c[4], const uint32_t k[2]) {
    const uint64_t p0 = static_cast<uint64_t>(kMul0) * c[0];
    const uint64_t p1 = static_cast<uint64_t>(kMul1) * c[2];
    const uint32_t hi0 = static_cast<uint32_t>(p0 >> 32), lo0 = static_cast<uint32_t>(p0);
    const uint32_t hi1 = static_cast<uint32_t>(p1 >> 32), lo1 = static_cast<uint32_t>(p1);
    const uint32_t n0 = hi1 ^ c[1] ^ k[0];
    const uint32_t n1 = lo1;
    const uint32_t n2 = hi0 ^ c[3] ^ k[1];
    const uint32_t n3 = lo0;
    c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
}

void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c[4] = {ctr[0], ctr[1], ctr[2], ctr[3]};
    uint32_t k[2] = {key[0], key[1]};
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k[0] += kWeyl0; k[1] += kWeyl1; }
        philox_round(c, k);
    }
    for (int i = 0; i < 4; ++i) out[i] = c[i];
}

// Stream layout: element g of the stream of `seed` is word (g mod 4) of the
// Philox block whose counter is (lo32(g/4), hi32(g/4), 0, 0) under the key
// (lo32(seed), hi32(seed)).
uint32_t stream_word(uint64_t seed, uint64_t g) {
    const uint64_t b = g >> 2;
    const uint32_t ctr[4] = {static_cast<uint32_t>(b), static_cast<uint32_t>(b >> 32), 0u, 0u};
    const uint32_t key[2] = {static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32)};
    uint32_t out[4];
    philox4x32_10(ctr, key, out);
    return out[g & 3];
}

// ---------------------------------------------------------------------------
// Box-Muller.  Words pair up inside a block: (x0,x1) -> (z0,z1), (x2,x3) ->
// (z2,z3).  u1 = ((xa >> 8) + 1) / 2^24 in (0, 1];  u2 = (xb >> 8) / 2^24 in
// [0, 1).  z_even = sqrt(-2 ln u1) cos(2 pi u2), z_odd = sqrt(-2 ln u1)
// sin(2 pi u2).  Evaluated in double; the angle is reduced by quadrant on the
// integer so that the exact zeros of sin/cos at multiples of pi/2 stay exact.
// ---------------------------------------------------------------------------
void box_muller(uint32_t xa, uint32_t xb, double* z_cos, double* z_sin) {
    const double u1 = (static_cast<double>(xa >> 8) + 1.0) / 16777216.0;
    const uint32_t k = xb >> 8;                 // angle = 2 pi k / 2^24
    const uint32_t quadrant = k >> 22;          // 0..3
    const uint32_t m = k & ((1u << 22) - 1u);   // position inside the quadrant
    const double half_pi = 1.57079632679489661923132169163975144;
    // Inside the quadrant measure the angle from the nearer axis, so that the
    // value next to a zero crossing keeps full relative accuracy.
    double s, c;
    if (m <= (1u << 21)) {
        const double phi = half_pi * (static_cast<double>(m) / 4194304.0);
        s = std::sin(phi); c = std::cos(phi);
    } else {
        const double psi = half_pi * (static_cast<double>((1u << 22) - m) / 4194304.0);
        s = std::cos(psi); c = std::sin(psi);
    }
    double cosv, sinv;
    switch (quadrant) {
        case 0: cosv = c;  sinv = s;  break;
        case 1: cosv = -s; sinv = c;  break;
        case 2: cosv = -c; sinv = -s; break;
        default: cosv = s; sinv = -c; break;
    }
    const double rho = std::sqrt(-2.0 * std::log(u1));
    *z_cos = rho * cosv;
    *z_sin = rho * sinv;
}

double normal_f64(uint64_t seed, uint64_t g) {
    const uint64_t pair_first = g & ~static_cast<uint64_t>(1);
    const uint32_t xa = stream_word(seed, pair_first);
    const uint32_t xb = stream_word(seed, pair_first + 1);
    double zc, zs;
    box_muller(xa, xb, &zc, &zs);
    return (g & 1) ? zs : zc;
}

// ---------------------------------------------------------------------------
// Storage formats.  Widening is exact; narrowing is round-to-nearest-even.
// ---------------------------------------------------------------------------
uint32_t f32_bits(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }
float bits_f32(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }

float widen_bf16(uint16_t h) { return bits_f32(static_cast<uint32_t>(h) << 16); }

float widen_f16(uint16_t h) {
    const uint32_t sign = (h & 0x8000u) ? 0x80000000u : 0u;
    const int e = (h >> 10) & 0x1f;
    const uint32_t frac = h & 0x3ffu;
    if (e == 0x1f) return bits_f32(sign | 0x7f800000u | (frac << 13));       // Inf / NaN
    if (e == 0) {                                                             // zero / subnormal
        const float mag = std::ldexp(static_cast<float>(frac), -24);          // exact
        return sign ? -mag : mag;
    }
    return bits_f32(sign | (static_cast<uint32_t>(e - 15 + 127) << 23) | (frac << 13));
}

uint16_t narrow_bf16(float f) {
    const uint32_t u = f32_bits(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return static_cast<uint16_t>((u >> 16) | 0x0040u);  // NaN stays NaN
    const uint32_t lower = u & 0xffffu;
    uint32_t upper = u >> 16;
    if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u))) upper += 1;   // carry into exponent is correct
    return static_cast<uint16_t>(upper);
}

uint16_t narrow_f16(float f) {
    const uint32_t u = f32_bits(f);
    const uint16_t sign = static_cast<uint16_t>((u >> 16) & 0x8000u);
    const uint32_t absu = u & 0x7fffffffu;
    if (absu > 0x7f800000u) return static_cast<uint16_t>(sign | 0x7e00u);     // NaN
    if (absu == 0x7f800000u) return static_cast<uint16_t>(sign | 0x7c00u);    // Inf
    const double mag = std::fabs(static_cast<double>(f));
    if (mag == 0.0) return sign;
    // Scale so that one unit is the spacing of the target format at this
    // magnitude, round to nearest even on the integer, rebuild.
    int e;
    std::frexp(mag, &e);                       // mag = m * 2^e, m in [0.5, 1)
    int exp_unbiased = e - 1;                  // mag in [2^exp, 2^(exp+1))
    if (exp_unbiased < -14) exp_unbiased = -14;  // subnormal spacing is fixed at 2^-24
    const double spacing = std::ldexp(1.0, exp_unbiased - 10);
    const double scaled = mag / spacing;       // exact (power-of-two scaling)
    double r = std::floor(scaled);
    const double rem = scaled - r;
    if (rem > 0.5 || (rem == 0.5 && std::fmod(r, 2.0) == 1.0)) r += 1.0;
    const double rounded = r * spacing;
    if (rounded >= 65520.0) return static_cast<uint16_t>(sign | 0x7c00u);     // overflows to Inf
    if (rounded < std::ldexp(1.0, -14)) {                                     // subnormal or zero
        return static_cast<uint16_t>(sign | static_cast<uint16_t>(rounded / std::ldexp(1.0, -24)));
    }
    int e2;
    const double m2 = std::frexp(rounded, &e2);   // rounded = m2 * 2^e2, m2 in [0.5,1)
    const int biased = (e2 - 1) + 15;
    const uint32_t frac = static_cast<uint32_t>((m2 * 2.0 - 1.0) * 1024.0);
    return static_cast<uint16_t>(sign | (static_cast<uint32_t>(biased) << 10) | frac);
}

enum { DT_U32 = 0, DT_F32 = 1, DT_F16 = 2, DT_BF16 = 3 };

float load_widened(const void* p, uint64_t i, int dtype) {
    switch (dtype) {
        case DT_F32:  return static_cast<const float*>(p)[i];
        case DT_F16:  return widen_f16(static_cast<const uint16_t*>(p)[i]);
        default:      return widen_bf16(static_cast<const uint16_t*>(p)[i]);
    }
}

}  // namespace

extern "C" {

struct oracle_result {
    uint64_t n_mismatch;
    uint64_t n_nonfinite;
    double sse;
    float max_abs;
    float max_rel;
    uint32_t flags;   // 1 cand NaN, 2 cand +Inf, 4 cand -Inf, 8 ref NaN, 16 ref +-Inf
    uint32_t pass;
};

struct oracle_fit {
    float median_ms;
    float speedup;
    uint32_t valid;
    uint32_t status;  // 0 ok, 1 a candidate time is not finite and positive, 2 same for a baseline time
};

void oracle_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
    philox4x32_10(ctr, key, out);
}

// The transform alone: two words -> (z_even, z_odd), unrounded.
void oracle_box_muller(uint32_t xa, uint32_t xb, double* out2) { box_muller(xa, xb, &out2[0], &out2[1]); }

void oracle_gen_u32(uint64_t seed, uint64_t offset, uint64_t n, uint32_t* out) {
    for (uint64_t i = 0; i < n; ++i) out[i] = stream_word(seed, offset + i);
}

// Unrounded (double) normals, for ulp measurements.
void oracle_gen_normal_f64(uint64_t seed, uint64_t offset, uint64_t n, double* out) {
    for (uint64_t i = 0; i < n; ++i) out[i] = normal_f64(seed, offset + i);
}

// dtype 0: raw words; 1: fp32 normals (one rounding from double); 2/3: the
// fp32 value narrowed once more to fp16 / bf16.
int oracle_gen_inputs(uint64_t seed, uint64_t offset, int dtype, uint64_t n, void* out) {
    if (dtype == DT_U32) { oracle_gen_u32(seed, offset, n, static_cast<uint32_t*>(out)); return 0; }
    if (dtype != DT_F32 && dtype != DT_F16 && dtype != DT_BF16) return -3;
    for (uint64_t i = 0; i < n; ++i) {
        const float z = static_cast<float>(normal_f64(seed, offset + i));
        if (dtype == DT_F32) static_cast<float*>(out)[i] = z;
        else if (dtype == DT_F16) static_cast<uint16_t*>(out)[i] = narrow_f16(z);
        else static_cast<uint16_t*>(out)[i] = narrow_bf16(z);
    }
    return 0;
}

void oracle_narrow(int dtype, const float* in, uint64_t n, uint16_t* out) {
    for (uint64_t i = 0; i < n; ++i) out[i] = (dtype == DT_F16) ? narrow_f16(in[i]) : narrow_bf16(in[i]);
}

void oracle_widen(int dtype, const uint16_t* in, uint64_t n, float* out) {
    for (uint64_t i = 0; i < n; ++i) out[i] = (dtype == DT_F16) ? widen_f16(in[i]) : widen_bf16(in[i]);
}

// Closeness rule for one element, every operation a single binary32 rounding:
//   d = |c - r|;  tol = atol + rtol * |r|;  close = (c == r) or (d finite and d <= tol).
// Returns 1 when the element is a mismatch.
int oracle_element_mismatch(float c, float r, float atol, float rtol) {
    const float diff = c - r;
    const float d = std::fabs(diff);
    const float t = rtol * std::fabs(r);
    const float tol = atol + t;
    const bool close = (c == r) || (std::isfinite(d) && d <= tol);
    return close ? 0 : 1;
}

// The correctness constraint over one tensor (Section 3.1 Eq. 1, g(p); Section
// 4.3 functional testing), plus the error statistics reported with it.
// Elements where c or r is NaN/Inf are counted and flagged, judged by the rule
// above, and left out of max_abs, max_rel and sse.  max_rel skips r == 0.
int oracle_validate(const void* cand, const void* ref, uint64_t n, int dtype,
                    float atol, float rtol, oracle_result* out) {
    if (dtype != DT_F32 && dtype != DT_F16 && dtype != DT_BF16) return -3;
    oracle_result res{};
    res.max_abs = 0.0f;
    res.max_rel = 0.0f;
    double sse = 0.0;
    for (uint64_t i = 0; i < n; ++i) {
        const float c = load_widened(cand, i, dtype);
        const float r = load_widened(ref, i, dtype);
        res.n_mismatch += static_cast<uint64_t>(oracle_element_mismatch(c, r, atol, rtol));
        bool nonfinite = false;
        if (std::isnan(c)) { res.flags |= 1u; nonfinite = true; }
        if (std::isinf(c)) { res.flags |= (c > 0.0f) ? 2u : 4u; nonfinite = true; }
        if (std::isnan(r)) { res.flags |= 8u; nonfinite = true; }
        if (std::isinf(r)) { res.flags |= 16u; nonfinite = true; }
        if (nonfinite) { res.n_nonfinite += 1; continue; }
        const float d = std::fabs(c - r);
        if (d > res.max_abs) res.max_abs = d;
        if (r != 0.0f) {
            const float q = d / std::fabs(r);
            if (q > res.max_rel) res.max_rel = q;
        }
        sse += static_cast<double>(d) * static_cast<double>(d);
    }
    res.sse = sse;
    res.pass = (res.n_mismatch == 0) ? 1u : 0u;
    *out = res;
    return 0;
}

// A candidate is valid when every one of its output tensors / test cases
// passes: AND over the descriptors carrying the same group id.
void oracle_group_pass(const oracle_result* results, const uint32_t* group, uint64_t n_desc,
                       uint32_t* group_pass, uint64_t n_group) {
    for (uint64_t g = 0; g < n_group; ++g) group_pass[g] = 1u;
    for (uint64_t i = 0; i < n_desc; ++i)
        if (group[i] < n_group && !results[i].pass) group_pass[group[i]] = 0u;
}

// Median of a row of run times: the middle order statistic, or the mean of the
// two middle ones (each operation one binary32 rounding).  Returns false when a
// time is not finite and positive.
static bool row_median(const float* row, uint32_t trials, float* median) {
    std::vector<float> v(row, row + trials);
    for (float x : v) if (!(std::isfinite(x) && x > 0.0f)) return false;
    std::sort(v.begin(), v.end());
    if (trials & 1u) { *median = v[trials / 2]; return true; }
    const float s = v[trials / 2 - 1] + v[trials / 2];
    *median = 0.5f * s;
    return true;
}

// Objective f(p): speedup of the candidate over the baseline kernel from the
// medians of their run times (Section 4.3 timing protocol; Appendix A.7.1
// "Limitations and Threats to Validity" states that the median of the runs is
// taken; Section 5.1 "Evaluation Metric": speedup over the baseline).  A
// candidate that failed the constraint gets valid = 0 and speedup 0.
int oracle_fitness(const float* times, uint64_t n_cand, uint32_t trials,
                   const float* base_times, uint32_t base_trials,
                   const uint32_t* pass, oracle_fit* out) {
    if (trials == 0 || base_trials == 0) return -1;
    float base_median = 0.0f;
    const bool base_ok = row_median(base_times, base_trials, &base_median);
    for (uint64_t i = 0; i < n_cand; ++i) {
        oracle_fit f{};
        float med = 0.0f;
        const bool ok = row_median(times + i * static_cast<uint64_t>(trials), trials, &med);
        if (!ok) { f.status = 1u; }
        else if (!base_ok) { f.status = 2u; f.median_ms = med; }
        else {
            f.median_ms = med;
            const bool passed = (pass == nullptr) || (pass[i] != 0u);
            if (passed) { f.valid = 1u; f.speedup = base_median / med; }
        }
        out[i] = f;
    }
    return 0;
}

}  // extern "C"

// ---------------------------------------------------------------------------
// Other run-time statistics.  Section 4.3 says the run times over the repeated
// runs are averaged, Appendix A.7.1 that their median is taken; both are
// offered, with the minimum and a trimmed mean, and with the option to leave
// out the first `warmup` runs.  Definitions (binary32 in, binary32 out):
//   mean          sum of the kept runs, accumulated in binary64 in run order,
//                 divided by their count in binary64, rounded once to binary32
//   min           the smallest kept run
//   trimmed mean  the kept runs sorted ascending, `trim` dropped at each end,
//                 the rest summed in binary64 in ascending order, divided by
//                 their count, rounded once to binary32
// Speedup = baseline statistic / candidate statistic (one binary32 division),
// the baseline's statistic being of the same kind.
// ---------------------------------------------------------------------------
enum { STAT_MEDIAN = 0, STAT_MEAN = 1, STAT_MIN = 2, STAT_TRIMMED_MEAN = 3 };

static bool row_statistic(const float* row, uint32_t trials, int stat, uint32_t warmup, uint32_t trim, float* value) {
    if (warmup >= trials) return false;
    std::vector<float> v(row + warmup, row + trials);
    for (float x : v) if (!(std::isfinite(x) && x > 0.0f)) return false;
    const size_t m = v.size();
    switch (stat) {
        case STAT_MEDIAN: return row_median(v.data(), static_cast<uint32_t>(m), value);
        case STAT_MEAN: {
            double sum = 0.0;
            for (float x : v) sum += static_cast<double>(x);
            *value = static_cast<float>(sum / static_cast<double>(m));
            return true;
        }
        case STAT_MIN: {
            float lo = v[0];
            for (float x : v) if (x < lo) lo = x;
            *value = lo;
            return true;
        }
        case STAT_TRIMMED_MEAN: {
            if (2ull * trim >= m) return false;
            std::sort(v.begin(), v.end());
            double sum = 0.0;
            for (size_t i = trim; i < m - trim; ++i) sum += static_cast<double>(v[i]);
            *value = static_cast<float>(sum / static_cast<double>(m - 2ull * trim));
            return true;
        }
        default: return false;
    }
}

extern "C" int oracle_fitness_ex(const float* times, uint64_t n_cand, uint32_t trials, const float* base_times,
                                 uint32_t base_trials, const uint32_t* pass, int stat, uint32_t warmup, uint32_t trim,
                                 oracle_fit* out) {
    if (trials == 0 || base_trials == 0 || stat < 0 || stat > 3) return -1;
    if (warmup >= trials || warmup >= base_trials) return -1;
    if (stat == STAT_TRIMMED_MEAN && (2ull * trim >= trials - warmup || 2ull * trim >= base_trials - warmup)) return -1;
    float base_value = 0.0f;
    const bool base_ok = row_statistic(base_times, base_trials, stat, warmup, trim, &base_value);
    for (uint64_t i = 0; i < n_cand; ++i) {
        oracle_fit f{};
        float val = 0.0f;
        const bool ok = row_statistic(times + i * static_cast<uint64_t>(trials), trials, stat, warmup, trim, &val);
        if (!ok) { f.status = 1u; }
        else if (!base_ok) { f.status = 2u; f.median_ms = val; }
        else {
            f.median_ms = val;
            const bool passed = (pass == nullptr) || (pass[i] != 0u);
            if (passed) { f.valid = 1u; f.speedup = base_value / val; }
        }
        out[i] = f;
    }
    return 0;
}

// ---------------------------------------------------------------------------
// Population summary: the paper's reporting metrics (Section 5.1 "Evaluation
// Metric"; the speedup-range table of Appendix A.5) from the per-candidate
// fitness records of one or several independent runs.
//   best[r][k]   largest speedup among the valid candidates of kernel k in run
//                r (0 if none is valid)
//   per run      median over the kernels of max(best, 1.0): a kernel without a
//                candidate that beats the baseline counts as 1.0
//   median_speedup  mean of the per-run medians (binary64 sum in run order,
//                one rounding to binary32): "averaged over three runs"
//   validity     valid candidates / candidates (Pass@1), binary32 division of
//                the two counts converted to binary64 and rounded once
//   speedup_count   kernels whose best over all runs exceeds 1.0
//   hist[5]      kernels by their best over all runs: < 1, [1, 2), [2, 5),
//                [5, 10), >= 10 (the table prints "<1.0, 1.0~2.0, 2.0~5.0,
//                5.0~10.0, >10.0"; which side the boundaries fall is this
//                library's reading)
// ---------------------------------------------------------------------------
struct oracle_summary_rec {
    float median_speedup;
    float validity;
    uint32_t n_valid;
    uint32_t n_cand;
    uint32_t speedup_count;
    uint32_t hist[5];
    uint32_t n_kernel;
    uint32_t n_run;
};

extern "C" int oracle_summary(const oracle_fit* fits, const uint32_t* kernel_of, const uint32_t* run_of, uint64_t n_cand,
                              uint32_t n_kernel, uint32_t n_run, oracle_summary_rec* out, float* best /* n_run*n_kernel */,
                              float* run_median /* n_run */) {
    if (n_kernel == 0 || n_run == 0) return -1;
    std::vector<float> b(static_cast<size_t>(n_run) * n_kernel, 0.0f);
    uint32_t n_valid = 0;
    for (uint64_t i = 0; i < n_cand; ++i) {
        const uint32_t k = kernel_of[i], r = run_of ? run_of[i] : 0u;
        if (k >= n_kernel || r >= n_run) return -1;
        if (!fits[i].valid) continue;
        ++n_valid;
        float& slot = b[static_cast<size_t>(r) * n_kernel + k];
        if (fits[i].speedup > slot) slot = fits[i].speedup;
    }
    double sum = 0.0;
    for (uint32_t r = 0; r < n_run; ++r) {
        std::vector<float> v(n_kernel);
        for (uint32_t k = 0; k < n_kernel; ++k) {
            const float x = b[static_cast<size_t>(r) * n_kernel + k];
            v[k] = x > 1.0f ? x : 1.0f;
        }
        std::sort(v.begin(), v.end());
        float med;
        if (n_kernel & 1u) med = v[n_kernel / 2];
        else { const float s = v[n_kernel / 2 - 1] + v[n_kernel / 2]; med = 0.5f * s; }
        if (run_median) run_median[r] = med;
        sum += static_cast<double>(med);
    }
    oracle_summary_rec s{};
    s.median_speedup = static_cast<float>(sum / static_cast<double>(n_run));
    s.n_valid = n_valid;
    s.n_cand = static_cast<uint32_t>(n_cand);
    s.validity = n_cand ? static_cast<float>(static_cast<double>(n_valid) / static_cast<double>(n_cand)) : 0.0f;
    s.n_kernel = n_kernel;
    s.n_run = n_run;
    for (uint32_t k = 0; k < n_kernel; ++k) {
        float top = 0.0f;
        for (uint32_t r = 0; r < n_run; ++r) top = std::max(top, b[static_cast<size_t>(r) * n_kernel + k]);
        if (top > 1.0f) ++s.speedup_count;
        const int bin = top < 1.0f ? 0 : top < 2.0f ? 1 : top < 5.0f ? 2 : top < 10.0f ? 3 : 4;
        ++s.hist[bin];
    }
    if (best) std::memcpy(best, b.data(), b.size() * sizeof(float));
    *out = s;
    return 0;
}

// ---------------------------------------------------------------------------
// Elite selection (Section 4.2 "Population Management": the single-solution
// strategy keeps the current best solution, elite preservation keeps a small
// set of high-performing ones).  The k valid candidates with the largest
// speedup, best first; equal speedups in order of their index.  Writes
// min(k, number of valid candidates) indices, fills the rest with 0xffffffff.
// ---------------------------------------------------------------------------
extern "C" int oracle_select_elite(const oracle_fit* fits, uint64_t n_cand, uint32_t k, uint32_t* idx, uint32_t* count) {
    std::vector<uint32_t> order;
    for (uint64_t i = 0; i < n_cand; ++i) if (fits[i].valid) order.push_back(static_cast<uint32_t>(i));
    std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return fits[a].speedup > fits[b].speedup; });
    const uint32_t m = static_cast<uint32_t>(std::min<size_t>(k, order.size()));
    for (uint32_t i = 0; i < k; ++i) idx[i] = i < m ? order[i] : 0xffffffffu;
    *count = m;
    return 0;
}

// ---------------------------------------------------------------------------
// Feedback on a failing candidate (Section 4.3: the system's third step is
// feedback collection for the next round of generation): where it is wrong.
// The first `max_out` elements, in index order, that violate the closeness
// rule, each with its index and the two values widened to binary32; and the
// total number of violations.
// ---------------------------------------------------------------------------
struct oracle_offender { uint64_t index; float cand; float ref; };

extern "C" int oracle_mismatch_sample(const void* cand, const void* ref, uint64_t n, int dtype, float atol, float rtol,
                                      uint64_t max_out, oracle_offender* out, uint64_t* n_found) {
    if (dtype < 1 || dtype > 3) return -1;
    uint64_t found = 0;
    for (uint64_t i = 0; i < n; ++i) {
        const float c = load_widened(cand, i, dtype), r = load_widened(ref, i, dtype);
        if (!oracle_element_mismatch(c, r, atol, rtol)) continue;
        if (found < max_out) { out[found].index = i; out[found].cand = c; out[found].ref = r; }
        ++found;
    }
    *n_found = found;
    return 0;
}

// ---------------------------------------------------------------------------
// Integer and boolean outputs (index results such as an argmax, masks, counts).
// The paper's constraint is that the output matches the reference (Section 3.1,
// Eq. 1; Section 4.3); for these types that is read as equality, element by
// element.  Reports the number of unequal elements and the largest |c - r|,
// exactly, as an unsigned 64-bit integer.  dtype: 5 = int32, 6 = int64,
// 7 = uint8 (also bool).
// ---------------------------------------------------------------------------
struct oracle_result_exact { uint64_t n_mismatch; uint64_t max_abs_diff; uint32_t pass; uint32_t pad; };

extern "C" int oracle_validate_exact(const void* cand, const void* ref, uint64_t n, int dtype, oracle_result_exact* out) {
    oracle_result_exact res{};
    for (uint64_t i = 0; i < n; ++i) {
        uint64_t diff;
        if (dtype == 5) {
            const int64_t c = static_cast<const int32_t*>(cand)[i], r = static_cast<const int32_t*>(ref)[i];
            diff = static_cast<uint64_t>(c > r ? c - r : r - c);
        } else if (dtype == 6) {
            const int64_t c = static_cast<const int64_t*>(cand)[i], r = static_cast<const int64_t*>(ref)[i];
            // the true difference may not fit int64: subtract as unsigned (exact modulo 2^64, and below 2^64)
            diff = c > r ? static_cast<uint64_t>(c) - static_cast<uint64_t>(r) : static_cast<uint64_t>(r) - static_cast<uint64_t>(c);
        } else if (dtype == 7) {
            const int c = static_cast<const uint8_t*>(cand)[i], r = static_cast<const uint8_t*>(ref)[i];
            diff = static_cast<uint64_t>(c > r ? c - r : r - c);
        } else {
            return -1;
        }
        if (diff != 0) ++res.n_mismatch;
        if (diff > res.max_abs_diff) res.max_abs_diff = diff;
    }
    res.pass = res.n_mismatch == 0 ? 1u : 0u;
    *out = res;
    return 0;
}

extern "C" void oracle_group_pass_exact(const oracle_result_exact* results, const uint32_t* group, uint64_t n_desc,
                                        uint32_t* group_pass, uint64_t n_group) {
    for (uint64_t g = 0; g < n_group; ++g) group_pass[g] = 1u;
    for (uint64_t i = 0; i < n_desc; ++i)
        if (group[i] < n_group && !results[i].pass) group_pass[group[i]] = 0u;
}

// ---------------------------------------------------------------------------
// binary64 outputs: the same rule and statistics as oracle_validate, with every
// operation an individually rounded binary64 operation (no fused multiply-add):
// d = |c - r|, tol = atol + rtol*|r|, close = (c == r) or (d finite and d <= tol);
// NaN/Inf elements are counted and flagged and stay out of max_abs, max_rel and
// sse.  The square is one more individually rounded binary64 operation (a square
// below the binary64 range is lost, one in its subnormal range keeps only the bits
// that fit); the rounded squares are then accumulated in extended precision (long
// double) so that the oracle's own summation error stays far below the comparison
// bar.
// ---------------------------------------------------------------------------
struct oracle_result64 {
    uint64_t n_mismatch, n_nonfinite;
    double sse, max_abs, max_rel;
    uint32_t flags, pass;
};

extern "C" int oracle_validate_f64(const double* cand, const double* ref, uint64_t n, double atol, double rtol,
                                   oracle_result64* out) {
    oracle_result64 res{};
    long double sse = 0.0L;
    for (uint64_t i = 0; i < n; ++i) {
        const double c = cand[i], r = ref[i];
        const double d = std::fabs(c - r);
        const double t = rtol * std::fabs(r);
        const double tol = atol + t;
        const bool close = (c == r) || (std::isfinite(d) && d <= tol);
        if (!close) ++res.n_mismatch;
        uint32_t f = 0;
        if (std::isnan(c)) f |= 1u;
        if (std::isinf(c)) f |= (c > 0 ? 2u : 4u);
        if (std::isnan(r)) f |= 8u;
        if (std::isinf(r)) f |= 16u;
        if (f) { ++res.n_nonfinite; res.flags |= f; continue; }
        if (d > res.max_abs) res.max_abs = d;
        if (r != 0.0) { const double q = d / std::fabs(r); if (q > res.max_rel) res.max_rel = q; }
        const double sq = d * d;                      // rounded once to binary64
        sse += static_cast<long double>(sq);
    }
    res.sse = static_cast<double>(sse);
    res.pass = res.n_mismatch == 0 ? 1u : 0u;
    *out = res;
    return 0;
}

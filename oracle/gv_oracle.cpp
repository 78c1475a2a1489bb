// gv_oracle.cpp -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
//
// Plain, slow, single-threaded CPU statement of what the batched output verifier computes:
// the paper's Section 3.1 (TritonBench-revised, second bullet) has test outputs compared tensor
// against tensor within tolerances rather than as printed text; here that comparison is applied to
// one candidate output against one reference output, as the inner step of the Evaluator's functionality test
// (Section 4.1) whose outcome feeds Execution Accuracy (Section 3.3: a kernel passes when it
// satisfies all unit tests, i.e. n_mismatch == 0 for every test tensor).
//
// The paper states the comparison in one phrase and prints no formula. The rule below is the
// torch.isclose rule (reference inside the relative term), evaluated element by element in
// IEEE binary32 after exact widening, with every rounding written out. It shares no code,
// header, table or constant generator with the CUDA library and is only ever used by tests/,
// the smoke check and the CPU-baseline leg of the benchmark.
//
// Build: g++ -std=c++17 -O2 -ffp-contract=off -fno-fast-math -fPIC -shared
//        (no -march flags, no -ffast-math / -Ofast: those would fuse, reassociate or flush
//         subnormals to zero and change results).
//
// Every function here is pinned by tests/test_oracle_*.py against values fixed outside this
// file (published SplitMix64 outputs, a hand-derived truth table, torch.isclose / numpy on the
// host, closed forms and by-construction counts; the grouping by a hand-worked example, its
// degenerate cases and a dictionary of byte strings; the accuracies by the fractions the paper's
// result tables print; the memory efficiency by a hand-worked example and exact rationals).

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

// ---- element types ---------------------------------------------------------------------
enum Dtype { F32 = 0, BF16 = 1, F16 = 2, I32 = 3, I64 = 4 };

inline int elem_size(int dt) {
    switch (dt) {
        case F32: return 4;
        case BF16: return 2;
        case F16: return 2;
        case I32: return 4;
        case I64: return 8;
        default: return 0;
    }
}

inline float bits_to_float(uint32_t b) {
    float f;
    std::memcpy(&f, &b, 4);
    return f;
}
inline uint32_t float_to_bits(float f) {
    uint32_t b;
    std::memcpy(&b, &f, 4);
    return b;
}

// Exact widening of a bfloat16 bit pattern: bf16 is the top half of a binary32.
inline float widen_bf16(uint16_t h) { return bits_to_float(static_cast<uint32_t>(h) << 16); }

// Exact widening of an IEEE binary16 bit pattern (1 sign, 5 exponent, 10 fraction bits).
inline float widen_f16(uint16_t h) {
    const uint32_t sign = static_cast<uint32_t>(h >> 15) << 31;
    const uint32_t e = (h >> 10) & 0x1Fu;
    const uint32_t m = h & 0x3FFu;
    if (e == 0x1Fu) {                      // Inf (m == 0) or NaN (payload kept, moved up)
        return bits_to_float(sign | 0x7F800000u | (m << 13));
    }
    if (e == 0) {
        if (m == 0) return bits_to_float(sign);           // +-0
        // subnormal half: value = m * 2^-24, exactly representable as a normal binary32
        float v = static_cast<float>(m) * bits_to_float(0x33800000u);  // 2^-24, exact product
        return sign ? -v : v;
    }
    // normal: rebias exponent 15 -> 127
    return bits_to_float(sign | ((e + 112u) << 23) | (m << 13));
}

inline bool is_nan(float f) { return (float_to_bits(f) & 0x7FFFFFFFu) > 0x7F800000u; }
inline int inf_class(float f) {
    const uint32_t b = float_to_bits(f);
    if ((b & 0x7FFFFFFFu) != 0x7F800000u) return 0;
    return (b >> 31) ? -1 : +1;
}
inline bool is_finite(float f) { return (float_to_bits(f) & 0x7F800000u) != 0x7F800000u; }
inline float f_abs(float f) { return bits_to_float(float_to_bits(f) & 0x7FFFFFFFu); }

}  // namespace

extern "C" {

// 64-byte result record, one per candidate. Field meaning as in the library's public header,
// restated here because the two sides share no header.
struct gvo_result {
    uint64_t n_mismatch;        // elements that are not close
    uint64_t first_mismatch;    // smallest such index, all-ones when there is none
    uint64_t n_nan_disagree;    // isnan(c) != isnan(r)
    uint64_t n_inf_disagree;    // infclass(c) != infclass(r)
    uint64_t hash;              // content hash of the candidate's bytes
    uint64_t max_abs_diff_int;  // integer dtypes: max |c - r|, exact
    float max_abs_err;          // float dtypes: max |fl(c - r)| over finite pairs
    float max_rel_err;          // float dtypes: max fl(|d| / |r|) over finite pairs with r != 0
    uint64_t reserved;          // 0
};

// SplitMix64 output function (Steele, Lea, Flood 2014; public domain reference by Vigna):
// add the golden-gamma, two xor-shift-multiply rounds, final xor-shift. All mod 2^64.
uint64_t gvo_splitmix64(uint64_t x) {
    uint64_t z = x + 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// Order-independent content hash: the byte image, zero-padded to a multiple of 8, is read as
// little-endian 64-bit words W_k; hash = sum over k of splitmix64(k xor W_k), wrapping.
// ("index" = word index, "raw bits" = the word; the length is not mixed in.)
uint64_t gvo_hash(const void* buf, uint64_t nbytes) {
    const unsigned char* p = static_cast<const unsigned char*>(buf);
    const uint64_t nwords = (nbytes + 7) / 8;
    uint64_t h = 0;
    for (uint64_t k = 0; k < nwords; ++k) {
        uint64_t w = 0;
        for (int b = 0; b < 8; ++b) {
            const uint64_t pos = 8 * k + static_cast<uint64_t>(b);
            if (pos < nbytes) w |= static_cast<uint64_t>(p[pos]) << (8 * b);
        }
        h += gvo_splitmix64(k ^ w);
    }
    return h;
}

// Second hash lane, for callers that want a stronger duplicate key than the one in the records: the
// same sum with the word index multiplied by the odd constant 0x9E3779B97F4A7C15 (mod 2^64) before the
// xor: hash2 = sum over k of splitmix64((k * gamma) xor W_k). Buffers that collide in the first lane
// because their sets {k xor W_k} coincide (e.g. int64 [0, 0] and [1, 1]) do not collide here.
uint64_t gvo_hash2(const void* buf, uint64_t nbytes) {
    const unsigned char* p = static_cast<const unsigned char*>(buf);
    const uint64_t nwords = (nbytes + 7) / 8;
    uint64_t h = 0;
    for (uint64_t k = 0; k < nwords; ++k) {
        uint64_t w = 0;
        for (int b = 0; b < 8; ++b) {
            const uint64_t pos = 8 * k + static_cast<uint64_t>(b);
            if (pos < nbytes) w |= static_cast<uint64_t>(p[pos]) << (8 * b);
        }
        h += gvo_splitmix64((k * 0x9E3779B97F4A7C15ull) ^ w);
    }
    return h;
}

// Widening used by the compare; exported so a test can check it against numpy for all 2^16
// patterns of both 16-bit types. Returns the binary32 bit pattern.
uint32_t gvo_widen_bits(int dtype, uint32_t raw) {
    if (dtype == BF16) return float_to_bits(widen_bf16(static_cast<uint16_t>(raw)));
    if (dtype == F16) return float_to_bits(widen_f16(static_cast<uint16_t>(raw)));
    return raw;
}

// One candidate against one reference. Returns 0, or 1 for an unknown dtype.
// Float dtypes: atol and rtol are converted once to binary32 (round to nearest); integer
// dtypes ignore them and compare exactly.
int gvo_verify(const void* ref, const void* cand, uint64_t n, int dtype, double atol, double rtol,
               int equal_nan, gvo_result* out) {
    const int esz = elem_size(dtype);
    if (esz == 0) return 1;

    gvo_result res;
    res.n_mismatch = 0;
    res.first_mismatch = ~0ull;
    res.n_nan_disagree = 0;
    res.n_inf_disagree = 0;
    res.hash = gvo_hash(cand, n * static_cast<uint64_t>(esz));
    res.max_abs_diff_int = 0;
    res.max_abs_err = 0.0f;
    res.max_rel_err = 0.0f;
    res.reserved = 0;

    if (dtype == I32 || dtype == I64) {
        for (uint64_t i = 0; i < n; ++i) {
            int64_t c, r;
            if (dtype == I32) {
                int32_t c32, r32;
                std::memcpy(&c32, static_cast<const char*>(cand) + 4 * i, 4);
                std::memcpy(&r32, static_cast<const char*>(ref) + 4 * i, 4);
                c = c32;
                r = r32;
            } else {
                std::memcpy(&c, static_cast<const char*>(cand) + 8 * i, 8);
                std::memcpy(&r, static_cast<const char*>(ref) + 8 * i, 8);
            }
            if (c != r) {
                res.n_mismatch += 1;
                if (i < res.first_mismatch) res.first_mismatch = i;
                // |c - r| in unsigned arithmetic: exact even at the int64 extremes
                const uint64_t diff = (c > r) ? static_cast<uint64_t>(c) - static_cast<uint64_t>(r)
                                              : static_cast<uint64_t>(r) - static_cast<uint64_t>(c);
                if (diff > res.max_abs_diff_int) res.max_abs_diff_int = diff;
            }
        }
        *out = res;
        return 0;
    }

    const float atol_f = static_cast<float>(atol);
    const float rtol_f = static_cast<float>(rtol);
    const float pos_inf = bits_to_float(0x7F800000u);

    for (uint64_t i = 0; i < n; ++i) {
        float c, r;
        if (dtype == F32) {
            std::memcpy(&c, static_cast<const char*>(cand) + 4 * i, 4);
            std::memcpy(&r, static_cast<const char*>(ref) + 4 * i, 4);
        } else {
            uint16_t cb, rb;
            std::memcpy(&cb, static_cast<const char*>(cand) + 2 * i, 2);
            std::memcpy(&rb, static_cast<const char*>(ref) + 2 * i, 2);
            c = (dtype == BF16) ? widen_bf16(cb) : widen_f16(cb);
            r = (dtype == BF16) ? widen_bf16(rb) : widen_f16(rb);
        }

        const float d = c - r;                 // one rounding
        const float ad = f_abs(d);             // NaN stays NaN
        const float prod = rtol_f * f_abs(r);  // one rounding
        const float tol = atol_f + prod;       // a second rounding: never a fused multiply-add

        const bool c_nan = is_nan(c), r_nan = is_nan(r);
        bool close = (c == r);                                    // IEEE ==: +0 == -0, Inf == Inf
        if (equal_nan && c_nan && r_nan) close = true;
        if (ad < pos_inf && ad <= tol) close = true;              // false for NaN or infinite ad

        if (!close) {
            res.n_mismatch += 1;
            if (i < res.first_mismatch) res.first_mismatch = i;
        }
        if (c_nan != r_nan) res.n_nan_disagree += 1;
        if (inf_class(c) != inf_class(r)) res.n_inf_disagree += 1;

        if (is_finite(c) && is_finite(r)) {
            if (ad > res.max_abs_err) res.max_abs_err = ad;       // ad in [0, +Inf]
            if (r != 0.0f) {
                const float rel = ad / f_abs(r);                  // IEEE division
                if (rel > res.max_rel_err) res.max_rel_err = rel;
            }
        }
    }
    *out = res;
    return 0;
}

// Ragged batch: T tensors, each with N candidates. Tensor t starts at ref_base + ref_off[t], has
// element size given by dtypes[t] and n_elems[t] elements (when n_elems is null the tensors are
// packed back to back and the count is (ref_off[t+1] - ref_off[t]) / element size); candidate
// (t, j) starts at cand_base + cand_off[t*N + j]. results is tensor-major (t*N + j);
// first_mismatch is relative to the tensor's own start. Nothing but a double loop over gvo_verify.
int gvo_verify_ragged(const void* ref_base, const int64_t* ref_off, const void* cand_base,
                      const int64_t* cand_off, const uint8_t* dtypes, const int64_t* n_elems,
                      int64_t T, int32_t N, double atol, double rtol, int equal_nan,
                      gvo_result* results) {
    for (int64_t t = 0; t < T; ++t) {
        const int esz = elem_size(dtypes[t]);
        if (esz == 0) return 1;
        const uint64_t n = n_elems ? static_cast<uint64_t>(n_elems[t])
                                   : static_cast<uint64_t>(ref_off[t + 1] - ref_off[t]) / static_cast<uint64_t>(esz);
        for (int32_t j = 0; j < N; ++j) {
            const int rc = gvo_verify(static_cast<const char*>(ref_base) + ref_off[t],
                                      static_cast<const char*>(cand_base) + cand_off[t * N + j], n,
                                      dtypes[t], atol, rtol, equal_nan, &results[t * N + j]);
            if (rc) return rc;
        }
    }
    return 0;
}

// Grouping of duplicate candidates (the use the content hash is computed for: parallel sampling
// of many generation runs per reference, Section 4.2 "parallel scaling", yields identical
// candidates, which need to be examined only once). Two candidates belong to one group exactly
// when their 64-byte records are identical byte for byte -- same content hash and same statistics.
//   group_id[j]    = the smallest index i whose record equals record j (so the representative of a
//                    group is its first member, and group_id[j] == j marks representatives)
//   group_count[j] = number of members of the group when j is its representative, else 0
//   *n_groups      = number of representatives
// Written as the definition: a double loop over whole records.
int gvo_group(const gvo_result* results, int64_t N, int32_t* group_id, int32_t* group_count,
              int32_t* n_groups) {
    int32_t groups = 0;
    for (int64_t j = 0; j < N; ++j) group_count[j] = 0;
    for (int64_t j = 0; j < N; ++j) {
        int64_t first = j;
        for (int64_t i = 0; i < j; ++i) {
            if (std::memcmp(&results[i], &results[j], sizeof(gvo_result)) == 0) { first = i; break; }
        }
        group_id[j] = static_cast<int32_t>(first);
        group_count[first] += 1;
        if (first == j) ++groups;
    }
    *n_groups = groups;
    return 0;
}

// Error profile of ONE candidate against the reference: the richer "error trace" an Evaluator can
// hand to the Reflector when the functionality test fails (Section 4.1: the trace of a failing run
// is fed back; Section 4.2, Reflexion) -- where the errors are and how large, not just that there
// are some. The paper does not define such a profile; this is the reading used here, written out
// element by element with the same close rule as gvo_verify:
//   ulp_hist[b]   all n elements, by the distance between candidate and reference in units of the
//                 dtype's own spacing: float dtypes order their bit patterns (negative values
//                 mirrored, so -0 and +0 coincide and the distance counts representable values
//                 in between); integer dtypes use |c - r|. b = 0: distance 0; b = 1 + floor(log2
//                 distance) for distance >= 1 (b <= 64); b = 65: a NaN is involved.
//   n_mismatch    elements that are not close (same as the record's)
//   worst_*       the mismatching element with the largest error, ties to the smallest index.
//                 Error of a float element: |fl(c - r)|, with NaN ranking above everything (bit
//                 patterns compared as unsigned, NaN taken as all ones); of an integer: |c - r|.
//   first_*       the (up to) 8 mismatching elements of smallest index, in order
//   *_raw         the element's own bits, zero-extended
//   rows          optional: mismatches per row of row_len elements (row i = elements
//                 [i*row_len, (i+1)*row_len)), ceil(n / row_len) counters
struct gvo_profile {
    uint64_t ulp_hist[66];
    uint64_t n_mismatch;
    uint64_t worst_index;
    uint64_t worst_c_raw, worst_r_raw;
    uint64_t n_first;
    uint64_t first_index[8];
    uint64_t first_c_raw[8];
    uint64_t first_r_raw[8];
};

int gvo_profile_pair(const void* ref, const void* cand, uint64_t n, int dtype, double atol, double rtol,
                     int equal_nan, uint64_t row_len, gvo_profile* out, uint32_t* rows) {
    const int esz = elem_size(dtype);
    if (esz == 0) return 1;
    gvo_profile p;
    std::memset(&p, 0, sizeof(p));
    p.worst_index = ~0ull;
    for (int i = 0; i < 8; ++i) p.first_index[i] = ~0ull;
    if (rows && row_len)
        for (uint64_t i = 0; i < (n + row_len - 1) / row_len; ++i) rows[i] = 0;
    const float atol_f = static_cast<float>(atol), rtol_f = static_cast<float>(rtol);
    const float pos_inf = bits_to_float(0x7F800000u);
    uint64_t worst_key = 0;
    bool have_worst = false;

    for (uint64_t i = 0; i < n; ++i) {
        uint64_t c_raw = 0, r_raw = 0;
        std::memcpy(&c_raw, static_cast<const char*>(cand) + esz * i, esz);      // little-endian host
        std::memcpy(&r_raw, static_cast<const char*>(ref) + esz * i, esz);
        bool close;
        uint64_t key;        // error used to rank mismatches
        int bucket;
        if (dtype == I32 || dtype == I64) {
            const int64_t c = dtype == I32 ? static_cast<int64_t>(static_cast<int32_t>(c_raw)) : static_cast<int64_t>(c_raw);
            const int64_t r = dtype == I32 ? static_cast<int64_t>(static_cast<int32_t>(r_raw)) : static_cast<int64_t>(r_raw);
            const uint64_t diff = (c > r) ? static_cast<uint64_t>(c) - static_cast<uint64_t>(r)
                                          : static_cast<uint64_t>(r) - static_cast<uint64_t>(c);
            close = (c == r);
            key = diff;
            bucket = 0;
            for (uint64_t d = diff; d; d >>= 1) ++bucket;                          // 1 + floor(log2 diff)
        } else {
            float c, r;
            const int width = esz * 8;
            if (dtype == F32) { c = bits_to_float(static_cast<uint32_t>(c_raw)); r = bits_to_float(static_cast<uint32_t>(r_raw)); }
            else if (dtype == BF16) { c = widen_bf16(static_cast<uint16_t>(c_raw)); r = widen_bf16(static_cast<uint16_t>(r_raw)); }
            else { c = widen_f16(static_cast<uint16_t>(c_raw)); r = widen_f16(static_cast<uint16_t>(r_raw)); }
            const float d = c - r;
            const float ad = f_abs(d);
            const float prod = rtol_f * f_abs(r);
            const float tol = atol_f + prod;
            const bool c_nan = is_nan(c), r_nan = is_nan(r);
            close = (c == r);
            if (equal_nan && c_nan && r_nan) close = true;
            if (ad < pos_inf && ad <= tol) close = true;
            key = is_nan(ad) ? 0xFFFFFFFFull : static_cast<uint64_t>(float_to_bits(ad));
            if (c_nan || r_nan) {
                bucket = 65;
            } else {
                const uint64_t sign_bit = 1ull << (width - 1);
                const int64_t oc = (c_raw & sign_bit) ? -static_cast<int64_t>(c_raw & (sign_bit - 1)) : static_cast<int64_t>(c_raw);
                const int64_t orf = (r_raw & sign_bit) ? -static_cast<int64_t>(r_raw & (sign_bit - 1)) : static_cast<int64_t>(r_raw);
                const uint64_t dist = static_cast<uint64_t>(oc > orf ? oc - orf : orf - oc);
                bucket = 0;
                for (uint64_t dd = dist; dd; dd >>= 1) ++bucket;
            }
        }
        p.ulp_hist[bucket] += 1;
        if (!close) {
            if (p.n_first < 8) {
                p.first_index[p.n_first] = i;
                p.first_c_raw[p.n_first] = c_raw;
                p.first_r_raw[p.n_first] = r_raw;
                p.n_first += 1;
            }
            p.n_mismatch += 1;
            if (!have_worst || key > worst_key) {
                have_worst = true;
                worst_key = key;
                p.worst_index = i;
                p.worst_c_raw = c_raw;
                p.worst_r_raw = r_raw;
            }
            if (rows && row_len) rows[i / row_len] += 1;
        }
    }
    *out = p;
    return 0;
}

// Pass/fail summary of one kernel's candidates and the pass@k estimate (Section 3.3: a generated
// kernel counts as correct when it satisfies ALL unit tests -- Execution Accuracy; Section 4.2:
// accuracy under parallel sampling is estimated with the pass@k metric).
// results is tensor-major, T unit-test tensors x N candidates (results[t*N + j], the layout the
// ragged verifier writes). pass[j] = 1 when candidate j has n_mismatch == 0 on every one of the T
// tensors (with T == 0 every candidate passes vacuously). c = number of passing candidates.
// pass_at_k[k-1], k = 1..kmax, is the standard unbiased estimator 1 - C(N-c, k) / C(N, k), evaluated
// in binary64 as 1 - prod_{i=0}^{k-1} (N-c-i)/(N-i), factors multiplied left to right, each factor one
// division; it is exactly 1 when N - c < k, and k > N is not allowed.
int gvo_exec_summary(const gvo_result* results, int64_t T, int32_t N, int32_t kmax, uint8_t* pass,
                     int32_t* n_pass, double* pass_at_k) {
    if (T < 0 || N < 0 || kmax < 0 || kmax > N) return 1;
    int32_t c = 0;
    for (int32_t j = 0; j < N; ++j) {
        bool ok = true;
        for (int64_t t = 0; t < T; ++t) ok = ok && results[t * N + j].n_mismatch == 0;
        pass[j] = ok ? 1 : 0;
        c += ok ? 1 : 0;
    }
    *n_pass = c;
    for (int32_t k = 1; k <= kmax; ++k) {
        if (N - c < k) { pass_at_k[k - 1] = 1.0; continue; }
        double prod = 1.0;
        for (int32_t i = 0; i < k; ++i) prod = prod * (static_cast<double>(N - c - i) / static_cast<double>(N - i));
        pass_at_k[k - 1] = 1.0 - prod;
    }
    return 0;
}

// Speedup of a generated kernel over the reference kernel (Section 3.3: the expectation, over the
// unit tests, of the ratio of the median reference latency to the generated kernel's latency;
// computed only for kernels that pass). ref_lat is T x S_ref, gen_lat T x S_gen latency samples
// (binary32, row per unit test). Reading: both latencies are summarised by their medians (the
// evaluator times each kernel several times); median of an even count = fl32((a + b) / 2) of the two
// middle values, computed as fl32(fl32(a + b) * 0.5); ratio[t] = fl32(median_ref[t] / median_gen[t]);
// speedup = (sum over t of ratio[t], accumulated in binary64 in index order) / T. NaN samples are not
// allowed. T == 0 gives speedup 0.
int gvo_speedup(const float* ref_lat, const float* gen_lat, int64_t T, int32_t S_ref, int32_t S_gen,
                float* median_ref, float* median_gen, float* ratio, double* speedup) {
    if (T < 0 || S_ref < 1 || S_gen < 1) return 1;
    double sum = 0.0;
    for (int64_t t = 0; t < T; ++t) {
        float med[2];
        for (int which = 0; which < 2; ++which) {
            const float* row = which == 0 ? ref_lat + t * S_ref : gen_lat + t * S_gen;
            const int32_t S = which == 0 ? S_ref : S_gen;
            // the definition: sort a copy of the row, take the middle value (odd count) or the two middle
            // values (even count). A middle value that is a zero is taken as +0 (-0 and +0 compare equal, so
            // their order after sorting is arbitrary).
            std::vector<float> sorted(row, row + S);
            std::sort(sorted.begin(), sorted.end());
            float picked[2] = {sorted[(S - 1) / 2], sorted[S / 2]};
            for (int w = 0; w < 2; ++w)
                if (picked[w] == 0.0f) picked[w] = 0.0f;
            const float s2 = picked[0] + picked[1];
            med[which] = (S & 1) ? picked[0] : s2 * 0.5f;
        }
        median_ref[t] = med[0];
        median_gen[t] = med[1];
        ratio[t] = med[0] / med[1];
        sum += static_cast<double>(ratio[t]);
    }
    *speedup = T ? sum / static_cast<double>(T) : 0.0;
    return 0;
}

// Memory efficiency of a generated kernel from latency samples. Section 4.1 says that, for code that
// passed the functionality test, the Evaluator assesses "latency and memory efficiency" and gives no
// formula; the case study of Appendix A argues in bytes moved (one read and one write of the data
// against two). Reading: per unit test, the bandwidth a kernel achieved on the bytes the test HAS to
// move (inputs read once, outputs written once -- supplied by the caller), as a fraction of the
// device's peak bandwidth; the latency of a test is summarised by the median of its samples, as for
// Speedup (even count: fl32(fl32(a + b) * 0.5) of the two middle values; a zero median is +0).
//   median[t]     binary32, from lat[t][0..S)
//   bandwidth[t]  = (double)bytes[t] / (double)median[t]          one binary64 division
//   efficiency[t] = bandwidth[t] / peak                           one binary64 division
//   mean_eff      = (sum over t of efficiency[t], accumulated in binary64 in index order) / T; 0 for T == 0
// peak is in bytes per unit of the latency samples (bytes per millisecond when the samples are in ms)
// and must be finite and > 0. Samples are finite and > 0.
int gvo_mem_efficiency(const float* lat, const uint64_t* bytes, int64_t T, int32_t S, double peak, float* median,
                       double* bandwidth, double* efficiency, double* mean_eff) {
    if (T < 0 || S < 1 || !(peak > 0.0) || !(peak <= 1.7976931348623157e308)) return 1;
    double sum = 0.0;
    for (int64_t t = 0; t < T; ++t) {
        std::vector<float> sorted(lat + t * S, lat + (t + 1) * S);
        std::sort(sorted.begin(), sorted.end());
        float lo = sorted[(S - 1) / 2], hi = sorted[S / 2];
        if (lo == 0.0f) lo = 0.0f;
        if (hi == 0.0f) hi = 0.0f;
        const float s2 = lo + hi;
        median[t] = (S & 1) ? lo : s2 * 0.5f;
        bandwidth[t] = static_cast<double>(bytes[t]) / static_cast<double>(median[t]);
        efficiency[t] = bandwidth[t] / peak;
        sum += efficiency[t];
    }
    *mean_eff = T ? sum / static_cast<double>(T) : 0.0;
    return 0;
}

// Call accuracy and execution accuracy over a (kernel x run) matrix (Section 3.3: Call Accuracy is the
// fraction of generated kernels that compile and run without error, Execution Accuracy the fraction
// that satisfy all unit tests, counted only for kernels that compiled; Section 4.2 / Section 5.2: with R
// independent runs per kernel both are reported as pass@k over the runs, k = 1..R). The denominator
// is the number of kernels in the benchmark (the result tables divide the correctly generated kernels by
// the total kernels in the dataset: 101 of 184 is printed as 54.89 %).
// status[q*R + r], kernel q, run r: bit 0 = the run's kernel compiled and ran, bit 1 = it satisfied all
// unit tests (the pass flag of gvo_exec_summary). A run counts for execution accuracy only with both.
//   n_call[q], n_exec[q]   numbers of such runs of kernel q
//   call_acc[k-1], exec_acc[k-1], k = 1..kmax <= R: (sum over q, in index order, in binary64, of
//       pass@k(R, c_q)) / K with pass@k(R, c) = 1 - prod_{i<k} (R-c-i)/(R-i), factors multiplied left to
//       right, each one division; exactly 1 when R - c < k. As fractions, not per cent. K == 0 gives 0.
int gvo_accuracy_matrix(const uint8_t* status, int64_t K, int32_t R, int32_t kmax, int32_t* n_call, int32_t* n_exec,
                        double* call_acc, double* exec_acc) {
    if (K < 0 || R < 0 || kmax < 0 || kmax > R) return 1;
    for (int64_t q = 0; q < K; ++q) {
        int32_t a = 0, b = 0;
        for (int32_t r = 0; r < R; ++r) {
            const uint8_t s = status[q * R + r];
            a += (s & 1) ? 1 : 0;
            b += ((s & 3) == 3) ? 1 : 0;
        }
        n_call[q] = a;
        n_exec[q] = b;
    }
    for (int32_t k = 1; k <= kmax; ++k) {
        double sums[2] = {0.0, 0.0};
        for (int64_t q = 0; q < K; ++q) {
            const int32_t c[2] = {n_call[q], n_exec[q]};
            for (int w = 0; w < 2; ++w) {
                double pass_k = 1.0;
                if (R - c[w] >= k) {
                    double prod = 1.0;
                    for (int32_t i = 0; i < k; ++i)
                        prod = prod * (static_cast<double>(R - c[w] - i) / static_cast<double>(R - i));
                    pass_k = 1.0 - prod;
                }
                sums[w] += pass_k;
            }
        }
        call_acc[k - 1] = K ? sums[0] / static_cast<double>(K) : 0.0;
        exec_acc[k - 1] = K ? sums[1] / static_cast<double>(K) : 0.0;
    }
    return 0;
}


}  // extern "C"

/* gv.h -- C ABI of the batched candidate-vs-reference output verifier (NVIDIA B200, sm_100a).
 *
 * What it computes. The GEAK paper's Evaluator runs a "functionality test" on every generated
 * kernel (Section 4.1): the candidate's unit-test outputs are checked against the reference
 * kernel's tensor against tensor within tolerances, not as printed text (Section 3.1), and a
 * kernel counts towards Execution Accuracy when all its tests pass (Section 3.3). Parallel and
 * sequential scaling (Section 4.2, Section 5.2) produce many candidates per reference output;
 * this library verifies N candidates against one reference in a single pass over the data.
 *
 * Per candidate it returns a 64-byte record: number of elements that are not close, the first
 * such index, NaN / Inf disagreement counts, maximum absolute and relative error, an exact
 * maximum difference for integer outputs, and an order-independent 64-bit content hash of the
 * candidate's bytes (for de-duplicating identical candidates).
 *
 * Per-element rule (float dtypes; c = candidate, r = reference, both widened exactly to
 * binary32; fl() = one round-to-nearest-even binary32 operation; subnormals are preserved):
 *     d = fl(c - r), ad = |d|, tol = fl(atol_f + fl(rtol_f * |r|))        (two roundings, no FMA)
 *     close = (c == r) or (equal_nan and isnan(c) and isnan(r)) or (ad < +Inf and ad <= tol)
 *     n_nan_disagree counts isnan(c) != isnan(r); n_inf_disagree counts infclass(c) != infclass(r)
 *     over pairs with c and r both finite: max_abs_err = max ad;  where also r != 0:
 *     max_rel_err = max fl(ad / |r|)                                       (IEEE division)
 *   atol_f = (float)atol, rtol_f = (float)rtol. torch.allclose(c.float(), r.float(), rtol, atol,
 *   equal_nan) is true exactly when n_mismatch == 0.
 * Integer dtypes are always compared exactly (tolerances ignored): close = (c == r),
 *   max_abs_diff_int = max |c - r| computed without overflow.
 * Content hash: the tensor's byte image, zero-padded to a multiple of 8 bytes, read as
 *   little-endian 64-bit words W_k; hash = sum_k splitmix64(k xor W_k) mod 2^64. The length is
 *   not mixed in. Equal hashes indicate *candidate* duplicates (k xor W_k is a weak combiner: e.g.
 *   int64 [0,0] and [1,1] collide); confirm with the other fields or a byte compare.
 * Every field has exactly one correct value; all reductions are integer sums / minima / maxima,
 * so results do not depend on scheduling.
 *
 * Conventions for every entry point below.
 *  - Pointers marked "device" must be device-accessible memory of the current CUDA device;
 *    "host" pointers are ordinary host memory. The library allocates and frees no memory.
 *  - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*; NULL = default stream)
 *    and return without synchronising. Outputs are valid once the stream reaches that point.
 *    Host arrays passed in (the candidate pointer list) are consumed before the call returns.
 *  - Errors are reported by return code only. When a call returns anything but GV_OK because of
 *    its arguments, nothing was enqueued and no output was touched.
 *  - Inputs are read-only. Tensors are contiguous. Base addresses must be multiples of the
 *    element size; 16-byte aligned bases take the fast path, others a slower path with the same
 *    results.
 */
#ifndef GV_H_
#define GV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum gv_dtype { GV_F32 = 0, GV_BF16 = 1, GV_F16 = 2, GV_I32 = 3, GV_I64 = 4 } gv_dtype;

typedef enum gv_status {
    GV_OK = 0,
    GV_ERR_INVALID_ARG = 1,    /* null pointer, negative count, negative tolerance or one above FLT_MAX */
    GV_ERR_UNSUPPORTED = 2,    /* dtype code out of range                                       */
    GV_ERR_MISALIGNED = 3,     /* a base address is not a multiple of the element size          */
    GV_ERR_WORKSPACE = 4,      /* workspace missing, misaligned or smaller than gv_workspace_bytes */
    GV_ERR_CUDA = 5,           /* a CUDA runtime call failed; see gv_last_cuda_error()           */
    GV_ERR_DEVICE_TIMEOUT = 6, /* a bounded device-side wait expired (reported by gv_check)      */
    GV_ERR_BAD_TABLE = 7       /* ragged tables inconsistent (reported by gv_check)              */
} gv_status;

#define GV_NO_INDEX 0xFFFFFFFFFFFFFFFFull

/* One record per candidate. 64 bytes, little-endian, comparable with memcmp. */
typedef struct gv_result {
    uint64_t n_mismatch;       /* elements that are not close                                   */
    uint64_t first_mismatch;   /* smallest flat index that is not close, else GV_NO_INDEX        */
    uint64_t n_nan_disagree;   /* float dtypes; 0 for integer dtypes                             */
    uint64_t n_inf_disagree;   /* float dtypes; 0 for integer dtypes                             */
    uint64_t hash;             /* content hash of the candidate's bytes                          */
    uint64_t max_abs_diff_int; /* integer dtypes: exact max |c - r|; float dtypes: 0             */
    float max_abs_err;         /* float dtypes; integer dtypes: 0. Never NaN, never -0           */
    float max_rel_err;         /* float dtypes; integer dtypes: 0. Never NaN, never -0           */
    uint64_t reserved;         /* 0                                                              */
} gv_result;

/* Tolerances of the comparison (Section 3.1 names them without values; callers choose). */
typedef struct gv_tol {
    double atol;       /* >= 0 and at most FLT_MAX: it is used as a finite binary32 value */
    double rtol;       /* the same */
    int32_t equal_nan; /* nonzero: NaN in both c and r counts as close */
    int32_t reserved;  /* 0 */
} gv_tol;

/* Dense batch: N candidates, each n_elems elements of dtype dt, against one reference
 * (the Evaluator's functionality test of Section 4.1 applied to one unit-test output).
 *   ref        device, n_elems elements.
 *   cands      HOST array of N device pointers (copied before return).
 *   tol        host; ignored (may be NULL) for integer dtypes.
 *   results    device, N records, fully overwritten (see gv_check for the one case in which they are
 *              incomplete).
 *   ref_hash   device, one uint64, receives the reference's content hash; may be NULL.
 *   workspace  device, >= gv_workspace_bytes(0, N) bytes, 16-byte aligned; must stay untouched
 *              until the stream has passed this call. It carries a status word for gv_check() and
 *              one byte per candidate for the pass that samples each candidate and decides which
 *              of the kernel's loops handles it (a matter of speed only: records do not depend on it).
 * Enqueues up to three kernels per 256 candidates (record initialisation once, sampling pass, verify).
 * N == 0 or n_elems == 0 is legal (no records / zero records: all fields 0, first_mismatch
 * GV_NO_INDEX, hash 0). The paper notes that an earlier harness silently compared empty outputs
 * (Section 3.1); deciding that an empty test output is an error is left to the caller, who can
 * see it from n_elems. */
gv_status gv_verify_batch(const void* ref, const void* const* cands, int32_t N, uint64_t n_elems,
                          gv_dtype dt, const gv_tol* tol, gv_result* results, uint64_t* ref_hash,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Ragged batch: T test tensors of mixed dtype and size packed into one reference buffer, each
 * with N candidates packed into one candidate buffer (many small unit-test outputs, cf. the
 * handful of unit tests per kernel noted in the paper's Appendix B).
 *   ref_off    device, int64[T+1]: byte offset of tensor t in ref_base; entry T is the end of the
 *              last tensor.
 *   cand_off   device, int64[T*N], tensor-major: byte offset of candidate (t, j) in cand_base.
 *   dtypes     device, uint8[T]: gv_dtype code of tensor t.
 *   n_elems    device, int64[T]: element count of tensor t; may be NULL when tensors are packed
 *              back to back, in which case it is (ref_off[t+1] - ref_off[t]) / element size.
 *   T          at most 2^31 - 1 tensors; a table entry describing more than 2^40 bytes is a bad entry.
 *   results    device, T*N records, tensor-major; first_mismatch is relative to the tensor.
 *   workspace  device, >= gv_workspace_bytes(T, N) bytes, 16-byte aligned.
 * Offsets must be multiples of the tensor's element size. The tables live on the device and are
 * checked there: a bad entry (negative or absurd size, misaligned offset, unknown dtype) makes that
 * tensor's records stay zero records and sets GV_ERR_BAD_TABLE in the status word read by gv_check().
 * The library cannot check offsets against the buffers' sizes (they are not arguments): a table that
 * points outside ref_base / cand_base is the caller's error.
 * Enqueues three kernels (record initialisation, table pre-pass, verify). Tensors whose bases are 16-byte
 * aligned are streamed at full speed; unaligned ones, the last partial tile of each tensor and tensors of
 * 32 GiB or more take a slower path with the same results (such giants belong in gv_verify_batch). */
gv_status gv_verify_ragged(const void* ref_base, const int64_t* ref_off, const void* cand_base,
                           const int64_t* cand_off, const uint8_t* dtypes, const int64_t* n_elems,
                           int64_t T, int32_t N, const gv_tol* tol, gv_result* results,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Ragged verification without any caller-provided scratch. (The paper has no counterpart to this
 * entry point; it exists for a class of callers, not for a passage of the text.)
 *
 * Who needs it: host programs that are not allowed to obtain device memory themselves -- for example a
 * plug-in running inside a framework or server that has handed the whole device to its own pool and
 * forbids foreign cudaMalloc/cudaFree calls, or a control loop that cannot accept the device-wide
 * synchronisation an allocation may cause -- and that therefore cannot produce the `workspace` buffer
 * gv_verify_ragged asks for. Here the scratch (a status word and the tile-prefix table the pre-pass
 * builds) lives in a fixed array inside the library's device image: 256 + 8 * (GV_NOALLOC_MAX_TENSORS + 1)
 * bytes (about 0.5 MiB), held on every GPU that loads the library until the process exits. The call
 * itself allocates and frees nothing, on the host or on the device, and calls no allocating routine.
 *
 * Arguments are those of gv_verify_ragged minus the workspace, plus
 *   status_out  device, one uint32, nullable: receives the status bits that gv_check() would report
 *               for a workspace (0 = fine, bit 0 = device-side wait expired, bit 1 = inconsistent
 *               tables); valid once the stream has passed the call. With NULL the bits are not
 *               retrievable.
 * Limits and rules:
 *   - T <= GV_NOALLOC_MAX_TENSORS, otherwise GV_ERR_WORKSPACE is returned, nothing is enqueued and
 *     gv_last_cuda_error() explains the limit. N is not limited.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current) and sets kernel attributes. Make that first call outside any stream
 *     capture.
 *   - All calls on a device share the one array, and it keeps the previous call's contents. The call
 *     rewrites everything it later reads, so calls that follow one another on a stream are
 *     independent; calls whose kernels overlap on the GPU (different streams, no ordering between
 *     them) race on the array and give undefined records. Order them, or use gv_verify_ragged with
 *     separate workspaces.
 * Results are byte-identical to gv_verify_ragged's. */
#define GV_NOALLOC_MAX_TENSORS 65536
gv_status gv_verify_ragged_noalloc(const void* ref_base, const int64_t* ref_off, const void* cand_base,
                                   const int64_t* cand_off, const uint8_t* dtypes, const int64_t* n_elems,
                                   int64_t T, int32_t N, const gv_tol* tol, gv_result* results,
                                   uint32_t* status_out, void* cuda_stream);

/* Content hash of nbytes bytes at buf (device) into *out (device). buf needs no alignment.
 * The same function the verifier applies to each candidate (used to de-duplicate candidates). */
gv_status gv_hash(const void* buf, uint64_t nbytes, uint64_t* out, void* cuda_stream);

/* Second hash lane, same arguments: sum over the 64-bit words W_k of splitmix64((k * 0x9E3779B97F4A7C15)
 * xor W_k). Buffers whose first-lane hashes collide because their sets {k xor W_k} coincide (int64 [0, 0]
 * and [1, 1]) differ here. It is not part of the verify pass or of the records (it would double the hash
 * work of data that differs); call it on the few candidates whose records fall into one duplicate group
 * when a stronger key than the record's hash is wanted. */
gv_status gv_hash2(const void* buf, uint64_t nbytes, uint64_t* out, void* cuda_stream);

/* Groups of duplicate candidates (what the content hash is for: the paper's parallel scaling,
 * Section 4.2, samples many generation runs per reference, and identical candidates need to be
 * examined only once). Candidates i and j are duplicates exactly when their 64-byte records are
 * identical byte for byte: same content hash and same statistics against the reference.
 *   results      device, N records as a verify call wrote them (read only, 16-byte aligned).
 *   group_id     device, int32[N]: the smallest index whose record equals record j. Representatives
 *                are the j with group_id[j] == j.
 *   group_count  device, int32[N], nullable: size of the group at its representative's index, 0
 *                elsewhere.
 *   n_groups     device, int32[1], nullable: number of groups.
 *   workspace    device, >= gv_group_workspace_bytes(N) bytes, 16-byte aligned; carries a status word
 *                for gv_check() (GV_ERR_DEVICE_TIMEOUT would mean a bounded table probe gave up, which
 *                the table's load factor of at most 1/2 rules out).
 * N == 0 is legal (n_groups = 0). N > GV_GROUP_MAX returns GV_ERR_UNSUPPORTED and enqueues nothing.
 * Up to 2048 records are grouped by one launch with the table in shared memory; beyond that the
 * table lives in the workspace and the call enqueues three launches. The outputs do not depend on
 * thread scheduling. Enqueue it on the stream of the verify call that writes `results`. */
#define GV_GROUP_MAX (1ll << 28)
size_t gv_group_workspace_bytes(int64_t N);
gv_status gv_group_candidates(const gv_result* results, int64_t N, int32_t* group_id, int32_t* group_count,
                              int32_t* n_groups, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Error profile of ONE candidate against the reference: a richer error trace for a candidate that
 * failed the functionality test (the paper feeds the trace of a failing run back to the Reflector,
 * Sections 4.1 and 4.2; it does not define such a profile -- this is this library's reading). Meant to be
 * called on demand for the few failing candidates; the verify calls carry none of its cost.
 *   ulp_hist[b]   every element, by the distance between candidate and reference in units of the dtype's
 *                 own spacing: float dtypes order their bit patterns (negative values mirrored, so -0 and
 *                 +0 coincide); integer dtypes use |c - r|. b = 0: distance 0; b = 1 + floor(log2
 *                 distance) otherwise (b <= 64); b = 65: a NaN is involved. The buckets sum to n_elems.
 *   n_mismatch    elements that are not close (the verify record's count, same rule, same tolerances).
 *   worst_*       the mismatching element with the largest error, ties to the smallest index; error of a
 *                 float element = bits of |fl(c - r)| with NaN above everything, of an integer = |c - r|.
 *                 worst_index = GV_NO_INDEX (raw values 0) when nothing mismatches.
 *   first_*       the n_first <= 8 mismatching elements of smallest index, ascending; unused entries have
 *                 index GV_NO_INDEX and raw values 0.
 *   *_raw         the element's own bits, zero-extended to 64.
 *   row_mismatch  device, uint32[ceil(n_elems / row_len)], mismatches per row of row_len consecutive
 *                 elements; pass row_len = 0 and NULL to skip.
 *   out           device, one gv_profile, fully overwritten.   tol as in gv_verify_batch.
 *   workspace     device, >= gv_profile_workspace_bytes() bytes, 16-byte aligned.
 * Bases must be multiples of the element size (16-byte aligned bases take 128-bit loads). n_elems == 0
 * is legal (all zero, indices GV_NO_INDEX). Enqueues one kernel (a cooperative launch: the device must
 * support cudaLaunchCooperativeKernel, as every sm_100 part does). */
#define GV_PROFILE_BUCKETS 66
#define GV_PROFILE_LIST 8
typedef struct gv_profile {
    uint64_t ulp_hist[GV_PROFILE_BUCKETS];
    uint64_t n_mismatch;
    uint64_t worst_index;
    uint64_t worst_c_raw, worst_r_raw;
    uint64_t n_first;
    uint64_t first_index[GV_PROFILE_LIST];
    uint64_t first_c_raw[GV_PROFILE_LIST];
    uint64_t first_r_raw[GV_PROFILE_LIST];
} gv_profile;
size_t gv_profile_workspace_bytes(void);
gv_status gv_error_profile(const void* ref, const void* cand, uint64_t n_elems, gv_dtype dt, const gv_tol* tol,
                           uint64_t row_len, gv_profile* out, uint32_t* row_mismatch, void* workspace,
                           size_t workspace_bytes, void* cuda_stream);

/* Pass/fail summary of one kernel's candidates and the pass@k estimate (paper Section 3.3: a generated
 * kernel is correct when it satisfies all unit tests; Section 4.2: accuracy under parallel sampling is
 * estimated with pass@k).
 *   results     device, T x N records, tensor-major (results[t*N + j]: unit-test tensor t, candidate j --
 *               the layout gv_verify_ragged writes; a dense call's N records are the case T = 1).
 *   pass        device, uint8[N]: 1 when candidate j has n_mismatch == 0 on all T tensors (T == 0: all 1).
 *   n_pass      device, int32[1]: c, the number of passing candidates.
 *   pass_at_k   device, double[kmax]: entry k-1 = 1 - C(N-c, k) / C(N, k), evaluated in binary64 as
 *               1 - prod_{i<k} (N-c-i)/(N-i) (factors multiplied left to right); exactly 1 when N-c < k.
 * 0 <= kmax <= N and kmax <= GV_PASSK_MAX, else GV_ERR_INVALID_ARG. One launch. */
#define GV_PASSK_MAX 65536
gv_status gv_exec_summary(const gv_result* results, int64_t T, int32_t N, int32_t kmax, uint8_t* pass,
                          int32_t* n_pass, double* pass_at_k, void* cuda_stream);

/* Speedup of a generated kernel over the reference kernel from latency samples (paper Section 3.3: the
 * expectation over the unit tests of the ratio of the median reference latency to the generated kernel's
 * latency; meaningful only for kernels that pass). Reading: both latencies are summarised by medians.
 *   ref_lat     device, float[T][S_ref]; gen_lat device, float[T][S_gen]: samples per unit test (no NaNs;
 *               a median that falls on a zero is reported as +0 whatever the zeros' signs).
 *   median_ref, median_gen, ratio   device, float[T]: medians (even count: fl((a + b) * 0.5) of the two
 *               middle values, the sum rounded first) and ratio[t] = fl(median_ref[t] / median_gen[t]).
 *   speedup     device, double[1]: the mean of ratio[] accumulated in binary64 in index order; 0 for T == 0.
 * 1 <= S_ref, S_gen <= GV_SAMPLES_MAX. Two launches (one CTA per unit test, then one thread for the mean). */
#define GV_SAMPLES_MAX 4096
gv_status gv_speedup(const float* ref_lat, const float* gen_lat, int64_t T, int32_t S_ref, int32_t S_gen,
                     float* median_ref, float* median_gen, float* ratio, double* speedup, void* cuda_stream);

/* Memory efficiency of a generated kernel from latency samples. Paper Section 4.1: for code that passed
 * the functionality test the Evaluator assesses latency and memory efficiency; no formula is given, and
 * the case study of Appendix A argues in bytes moved (one read and one write of the data against two).
 * Reading: per unit test, the bandwidth achieved on the bytes the test HAS to move (inputs read once,
 * outputs written once; the caller supplies them) as a fraction of the device's peak bandwidth, the
 * latency summarised by the median of its samples exactly as in gv_speedup.
 *   lat         device, float[T][S] latency samples (finite, > 0);  bytes  device, uint64[T].
 *   peak        peak bandwidth in bytes per unit of the samples (bytes per ms for samples in ms); finite, > 0.
 *   median      device, float[T];  bandwidth device, double[T] = (double)bytes[t] / (double)median[t];
 *   efficiency  device, double[T] = bandwidth[t] / peak (each one correctly rounded binary64 division).
 *   mean_efficiency  device, double[1]: mean of efficiency[] accumulated in index order; 0 for T == 0.
 * 1 <= S <= GV_SAMPLES_MAX. Two launches. */
gv_status gv_mem_efficiency(const float* lat, const uint64_t* bytes, int64_t T, int32_t S, double peak, float* median,
                            double* bandwidth, double* efficiency, double* mean_efficiency, void* cuda_stream);

/* Call accuracy and execution accuracy over a (kernel x run) matrix (paper Section 3.3: the fraction of
 * generated kernels that compile and run, and the fraction that satisfy all unit tests, the latter counted
 * only for kernels that compiled; Sections 4.2 and 5.2: with R independent runs per kernel both are
 * reported as pass@k over the runs). The denominator is the number of kernels of the benchmark, as in the
 * paper's result tables (correctly generated kernels / total kernels in the dataset).
 *   status      device, uint8[K][R]: bit 0 = run r of kernel q compiled and ran, bit 1 = it satisfied all
 *               unit tests (the pass flag gv_exec_summary produces). A run counts as correct only with both.
 *   n_call, n_exec   device, int32[K]: such runs per kernel.
 *   call_acc, exec_acc   device, double[kmax]: entry k-1 = (sum over the kernels, in index order, of
 *               pass@k(R, count)) / K with pass@k as in gv_exec_summary; fractions, not per cent; 0 for K == 0.
 * 0 <= kmax <= R <= GV_RUNS_MAX. Two launches. */
#define GV_RUNS_MAX 1024
gv_status gv_accuracy_matrix(const uint8_t* status, int64_t K, int32_t R, int32_t kmax, int32_t* n_call, int32_t* n_exec,
                             double* call_acc, double* exec_acc, void* cuda_stream);

/* Host-buffer convenience for callers whose outputs live in host memory: copies the reference and
 * the candidates host->device in slabs through `staging` (device, staging_bytes), verifies them and
 * copies the N records (and the reference hash) back to host memory. Copies and kernels are
 * enqueued on cuda_stream; the call returns after synchronising that stream, so results are valid
 * on return. Same computation as gv_verify_batch.
 *   ref_host, cands_host[j]   host memory (pinned memory makes the copies fast)
 *   results_host              host, N records;  ref_hash_host host, may be NULL
 *   staging                   device, 256-byte aligned, >= gv_host_staging_bytes(n_elems, dt, 1) */
gv_status gv_verify_batch_host(const void* ref_host, const void* const* cands_host, int32_t N,
                               uint64_t n_elems, gv_dtype dt, const gv_tol* tol,
                               gv_result* results_host, uint64_t* ref_hash_host, void* staging,
                               size_t staging_bytes, void* cuda_stream);

/* Bytes of staging needed by gv_verify_batch_host to hold the reference plus `slab` candidates
 * (slab >= 1; larger slabs amortise launches), including records and workspace. */
size_t gv_host_staging_bytes(uint64_t n_elems, gv_dtype dt, int32_t slab);

/* Upper bound on the workspace either verify call needs (T = 0 for the dense call). */
size_t gv_workspace_bytes(int64_t T, int32_t N);

/* Synchronises cuda_stream, reads the status word of `workspace` and returns GV_OK,
 * GV_ERR_DEVICE_TIMEOUT or GV_ERR_BAD_TABLE (or GV_ERR_CUDA). Optional, with one exception of
 * meaning: every wait inside the kernels is bounded, and a warp whose wait expires stops working on
 * its share of the data, so when gv_check reports GV_ERR_DEVICE_TIMEOUT the records (and ref_hash) of
 * that call are INCOMPLETE AND MUST NOT BE USED -- they look like ordinary records. A caller that needs
 * to rule this out calls gv_check; on healthy hardware the waits (tens of milliseconds of patience for
 * a 512-byte copy) do not expire. GV_ERR_BAD_TABLE leaves the records of the well-formed tensors valid. */
gv_status gv_check(const void* workspace, void* cuda_stream);

/* Diagnostic for the path above (no counterpart in the paper): enqueues one warp that waits, through
 * the kernels' own bounded wait with a limit of a few milliseconds, on a transfer that is never
 * started, records the expiry in the status word of `workspace` (>= 256 bytes, 16-byte aligned; the
 * word is overwritten) and returns by itself. gv_check(workspace) afterwards reports
 * GV_ERR_DEVICE_TIMEOUT; the device and the workspace remain usable. */
gv_status gv_selftest_wait_expiry(void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Diagnostic (no counterpart in the paper): the wrapping sum, modulo 2^64, of all little-endian 32-bit
 * words of a device buffer, computed by a kernel that does nothing but stream the buffer with 128-bit
 * loads. Timed on a buffer much larger than L2 it gives the read-only bandwidth of the device, the
 * ceiling of the verify kernels (which only read), beside the read+write copy figure usually quoted.
 *   buf  device, 16-byte aligned;  nbytes a multiple of 16;  out device, one uint64. Memset + one launch. */
gv_status gv_selftest_read_sum(const void* buf, uint64_t nbytes, uint64_t* out, void* cuda_stream);

const char* gv_status_string(gv_status s);
const char* gv_last_cuda_error(void); /* text of the last CUDA error seen by this thread, or "" */
uint32_t gv_version(void);            /* major << 16 | minor << 8 | patch */

#ifdef __cplusplus
}
#endif
#endif /* GV_H_ */

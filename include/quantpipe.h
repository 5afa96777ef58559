/*
 * quantpipe.h -- C ABI of the activation-quantization path of QuantPipe (arXiv 2211.04515)
 * for NVIDIA B200 (sm_100a).
 *
 * The path (paper Sec. 3, "System Design and Implementation"):
 *   sender    qp_stats -> [qp_dsaciq_search] -> qp_aciq_alpha / qp_aciq_qparams_device
 *             -> qp_quantize_pack
 *   receiver  qp_unpack_dequantize
 *   control   qp_select_bits (bit-width from the measured link bandwidth)
 *
 * Conventions
 *   - Plain C.  No exceptions cross the boundary.  Every call returns a qp_status value:
 *     0 = QP_OK, negative = error (outputs undefined), positive = warning (outputs defined).
 *   - "d_" arguments are DEVICE pointers, "h_" arguments are HOST pointers; the caller owns
 *     every buffer it passes.  The library owns only the qp_ctx (a few MB of device
 *     scratch: block partials, histogram, candidate table, counters, status word).
 *   - Device-taking calls enqueue work on `stream` (a cudaStream_t passed as void*; NULL is
 *     the legacy default stream) and return without synchronising.  One qp_ctx may be used
 *     from one stream at a time.  Inputs and outputs must not overlap.
 *   - dtype: QP_F32 (0) or QP_BF16 (1).  Tensors are contiguous; n is the element count.
 *   - bits: 1..8 or 16 for quantize/pack and unpack/dequantize; 32 ("send raw fp32") is only
 *     a possible result of qp_select_bits.
 *   - Non-finite inputs: NaN quantizes to code 0, +-Inf clamps to the clip range; the
 *     statistics and the search skip and count them.
 */
#ifndef QUANTPIPE_H
#define QUANTPIPE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct qp_ctx qp_ctx;

enum {
    QP_OK = 0,
    QP_ERR_INVALID_ARG = -1,
    QP_ERR_UNSUPPORTED_BITS = -2,
    QP_ERR_UNSUPPORTED_DTYPE = -3,
    QP_ERR_BUFFER_TOO_SMALL = -4,
    QP_ERR_ALIGNMENT = -5,
    QP_ERR_CUDA = -6,
    QP_ERR_TIMEOUT = -7,
    QP_ERR_TOO_LARGE = -8,    /* size beyond a stated maximum of the entry point          */
    QP_WARN_INFEASIBLE = 1,   /* qp_select_bits: nothing fits, smallest width returned   */
    QP_WARN_DEGENERATE = 2,   /* empty clip range (constant tensor): all codes are 0     */
    QP_WARN_NONFINITE = 3     /* reported by qp_get_status: NaN/Inf were seen and skipped */
};

enum { QP_F32 = 0, QP_BF16 = 1 };
enum { QP_DIST_LAPLACE = 0, QP_DIST_GAUSS = 1 };
enum { QP_B_MAD = 0 /* sum|x-mean|/N */, QP_B_MEAN_ABS = 1 /* sum|x|/N, the formula as printed */ };
#define QP_B_MIDRISE 0x10  /* qp_dsaciq_search: bmode | QP_B_MIDRISE scores every candidate on the mid-rise grid */
#define QP_B_GAUSS 0x20    /* qp_dsaciq_search: QP_B_MAD | QP_B_GAUSS searches under the normal model (see there) */
#define QP_B_HIST_IN_STATS 0x40  /* qp_dsaciq_search: the caller vouches that d_stats carries this histogram (see there) */

#define QP_DEFAULT_STEPS 100      /* search steps t (Sec. 3, directed search) */
#define QP_DEFAULT_HIST_BINS 100
#define QP_MAX_STEPS 1023
#define QP_MAX_HIST_BINS 16384

/* bits of the device status word returned by qp_get_status */
#define QP_DEV_BITS_MISMATCH 1u   /* a device-resident qp_qparams_t had other bits than the call */
#define QP_DEV_DEGENERATE 2u
#define QP_DEV_NONFINITE 4u
#define QP_DEV_STREAM_TIMEOUT 8u  /* a bounded wait for a tile copy ran out; results of that call are invalid */
#define QP_DEV_HIST_MISSING 16u   /* a search was promised a histogram in the statistics (QP_B_HIST_IN_STATS) that is not there */
#define QP_DEV_INDEX_RANGE 32u    /* debug build only: an index into a shared-memory or scratch table was out of range (redirected to entry 0) */

/* Per-tensor statistics (Sec. 3: min/max of naive PTQ; mean and Laplace scale b of ACIQ;
 * b_E of the directed search).  All fields but n are over the finite elements. */
typedef struct {
    uint64_t n;          /* elements given                                   */
    uint64_t nonfinite;  /* NaN or +-Inf among them                          */
    double mean;
    double mean_abs;     /* sum|x| / N      (b_E exactly as the paper prints it) */
    double mad;          /* sum|x - mean| / N  (Laplace scale about the mean)    */
    double var;          /* sum (x - mean)^2 / N                              */
    double min, max;
    uint64_t hist_peak;  /* largest bin count of the hist_bins-bin histogram over [min, max] */
    int32_t hist_bins;   /* bins of that histogram; 0 = qp_stats did not compute one          */
    int32_t reserved;
} qp_stats_t;            /* 80 bytes */

/* Uniform quantizer over the clip range [lo, hi] with L = 2^bits levels, both ends included. */
typedef struct {
    float lo, hi;
    float scale;         /* (hi - lo) / (L - 1) */
    float inv_scale;     /* (L - 1) / (hi - lo) */
    int32_t bits;
    int32_t flags;       /* bit 0: degenerate range, scale = inv_scale = 0 */
} qp_qparams_t;          /* 24 bytes */

/* Outcome of the directed search (Sec. 3, Eq. 1). */
typedef struct {
    double b_e;          /* scale estimated from the data                    */
    double b_r;          /* search boundary 1 / (2 * peak of the histogram density) */
    double b_star;       /* chosen scale                                      */
    double alpha_e;      /* F(q) * b_e                                        */
    double alpha_star;   /* F(q) * b_star                                     */
    double mse_e;        /* quantization MSE at b_e                           */
    double mse_star;     /* quantization MSE at b_star (<= mse_e)             */
    int32_t k_star;      /* chosen step, 0 = b_e kept                         */
    int32_t steps, hist_bins, bits;
} qp_ds_result_t;        /* 72 bytes */

/* ---- context -------------------------------------------------------------------------
 * qp_create allocates the scratch on `device` (cudaMalloc; call it outside stream capture).
 * qp_destroy frees it.  Errors: QP_ERR_INVALID_ARG, QP_ERR_CUDA. */
int32_t qp_create(int device, qp_ctx** out);
int32_t qp_destroy(qp_ctx* ctx);
/* Waits for `stream`, then returns and clears the device status word (QP_DEV_* bits), or a
 * negative qp_status: QP_ERR_CUDA if a CUDA error is pending, QP_ERR_TIMEOUT if the word
 * carries QP_DEV_STREAM_TIMEOUT (a bounded wait inside a kernel ran out: the results of the
 * calls since the last qp_get_status are invalid; the call also puts the scratch of the
 * cooperative kernels back to its initial state, so the context can be used again at once;
 * qp_last_error gives the whole word). */
int32_t qp_get_status(qp_ctx* ctx, void* stream);
/* Test hook for the time-out paths (no counterpart in the paper; not for production use).
 * Every wait inside the kernels is bounded: a wait for a tile copy by a number of clock
 * cycles, a wait at a grid-wide barrier by a number of polls.  This call replaces the limits
 * of later launches on this context: tile_wait_cycles < 0 and barrier_polls = 0 restore the
 * defaults (about two seconds; a quarter of a second at least); tile_wait_cycles = 0 makes a
 * wait give up at the first attempt that finds the copy still in flight.  (The second wait that
 * a block which gave up grants its own copies in flight before it leaves always keeps the
 * default.)  barrier_extra_arrivals = 1 makes every grid barrier wait for one arrival more
 * than there are blocks, so that it can only end by running out.  A wait that runs out
 * raises QP_DEV_STREAM_TIMEOUT, the kernel leaves without output, and nothing faults.
 * Drops the stored graphs (they carry the old limits).  Errors: QP_ERR_INVALID_ARG. */
int32_t qp_set_wait_limit_for_testing(qp_ctx* ctx, long long tile_wait_cycles, uint32_t barrier_polls,
                                      int barrier_extra_arrivals);
/* Text of the last error recorded on this context (never NULL). */
const char* qp_last_error(qp_ctx* ctx);
const char* qp_status_string(int32_t status);
/* 1 if the library was built with index checks (-DQP_CHECK_BOUNDS; `python -m paper_2211_04515_b200.build
 * --check` writes libquantpipe_check.so): every index into the kernels' shared-memory tables and scratch
 * rows is then range-checked, an index out of range is redirected to entry 0 (nothing traps or faults) and
 * qp_get_status reports QP_DEV_INDEX_RANGE.  The stand-in, on this library's own tables, for a memory
 * checker where none can be run.  0 for the ordinary build. */
int32_t qp_built_with_index_checks(void);
/* Number of kernels this context has launched since qp_create (host-side count). */
uint64_t qp_launch_count(qp_ctx* ctx);

/* ---- sizes and parameters (host, pure) ------------------------------------------------*/

/* Bytes of the packed stream: ceil(n*bits/8) rounded up to a multiple of 16.
 * 8-bit codes take a quarter of the fp32 tensor (Sec. 3).  Returns 0 for bits outside
 * 1..8, 16. */
uint64_t qp_packed_bytes(uint64_t n, int bits);

/* ACIQ multiplier F(q) with alpha = F(q) * b (Sec. 3).  Laplace: the minimiser of
 * 2 b^2 exp(-alpha/b) + alpha^2 / (3 * 4^q), i.e. F = W0(3 * 4^q).  Gauss: the minimiser
 * of the corresponding normal-tail model.  Returns 0 for unsupported bits/dist. */
double qp_aciq_F(int bits, int dist);

/* Fills a quantizer for the clip range [lo, hi]: ends rounded to fp32, scale and
 * inv_scale derived in fp64 from the rounded ends and rounded once.
 * Returns QP_OK, QP_WARN_DEGENERATE (hi <= lo after rounding), QP_ERR_UNSUPPORTED_BITS,
 * QP_ERR_INVALID_ARG (NaN/Inf ends, NULL). */
int32_t qp_make_qparams(double lo, double hi, int bits, qp_qparams_t* h_out);

/* ---- a1 (+ a2): statistics (Sec. 3) ----------------------------------------------------
 * One call fills *d_out (device memory, 80 bytes, 8-byte aligned) from the n elements at
 * d_x.  Two passes over x (sums/min/max, then deviations about the mean), fp64 merges in a
 * fixed order: results are bit-reproducible run to run.  n = 0 gives all-zero statistics.
 * For 16-byte aligned tensors of at least 128 KB both passes run in one cooperative launch
 * (the second pass starts on the tiles that the first one left in shared memory), see
 * qp_set_stats_path.
 * hist_bins > 0 asks the second pass to carry the directed search's histogram along
 * (hist_bins equal bins over [min, max]; only its peak count is kept, in hist_peak): a later
 * qp_dsaciq_search with the same hist_bins then skips its own histogram pass.  The fusion is
 * done for 16-byte aligned tensors of at least 128 KB and hist_bins <= 4096; otherwise, and
 * for hist_bins = 0, d_out->hist_bins is 0 and the search counts for itself.
 * d_x must be aligned to its element size.
 * Errors: QP_ERR_INVALID_ARG (NULL, hist_bins outside 0..QP_MAX_HIST_BINS),
 * QP_ERR_UNSUPPORTED_DTYPE, QP_ERR_ALIGNMENT, QP_ERR_CUDA. */
int32_t qp_stats(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, int hist_bins, qp_stats_t* d_out,
                 void* stream);
/* 1 if qp_stats with these arguments carries the histogram along (so that d_out->hist_bins
 * will equal hist_bins), else 0.  Host, pure: it depends only on the pointer's alignment, the
 * size and hist_bins. */
int qp_stats_carries_histogram(const void* d_x, int dtype, uint64_t n, int hist_bins);
/* How qp_stats runs its two passes on 16-byte aligned tensors of at least 128 KB (an execution
 * option without a counterpart in the paper; min, max, the counts and the histogram's peak are
 * identical on both paths, the other fields agree to ~1e-8 relative):
 *   QP_STATS_TWO_KERNELS  one kernel per pass
 *   QP_STATS_FUSED        one cooperative launch for both (one block per SM; every block keeps the
 *                         last tiles of its first pass in shared memory and starts the second pass,
 *                         which walks backwards, on them).  Falls back to two kernels on a device
 *                         that cannot hold it.
 *   QP_STATS_AUTO         the cooperative launch for hist_bins = 0, the two kernels when the histogram
 *                         rides along (default: the faster of the two inside the sender chain; called
 *                         alone the cooperative launch is the faster with the histogram too)
 * A grid barrier or tile wait of the cooperative launch that runs out sets QP_DEV_STREAM_TIMEOUT
 * and the launch ends without output. */
enum { QP_STATS_AUTO = 0, QP_STATS_TWO_KERNELS = 1, QP_STATS_FUSED = 2 };
int32_t qp_set_stats_path(qp_ctx* ctx, int path);

/* Statistics for callers that cannot allocate device memory (no counterpart in the paper;
 * same results as qp_stats).  Some code may not call cudaMalloc or any allocating routine:
 * it runs while the framework's memory pool is frozen, or all device memory was handed out
 * before this library came in.  This entry point takes no qp_ctx and allocates nothing: its
 * scratch (block partials, tickets, status word; 49,408 bytes) is a fixed array inside the
 * library image, resident on every GPU that loads the library until the process exits.
 * It works on the calling thread's current device and enqueues on `stream`.
 *   - The first call on each device looks up the array's device address (a set-up step that
 *     talks to the driver): make that first call before starting any stream capture.
 *   - n may not exceed QP_STATS_STATIC_MAX_N; larger tensors return QP_ERR_TOO_LARGE and
 *     nothing is enqueued (use qp_stats, whose context has room for them).
 *   - All calls on a device share the one array, which keeps the previous call's contents
 *     (the counters that must start at zero are cleared on `stream` first).  Two calls
 *     that overlap on the GPU (different streams, no ordering between them) race on it and
 *     give wrong statistics: order them.
 *   - There is no context, hence no status word to read: NaN and +-Inf among the input are
 *     reported through d_out->nonfinite only.
 * Errors: QP_ERR_INVALID_ARG (NULL), QP_ERR_UNSUPPORTED_DTYPE, QP_ERR_ALIGNMENT,
 * QP_ERR_TOO_LARGE, QP_ERR_CUDA. */
#define QP_STATS_STATIC_MAX_N (1ull << 31)
int32_t qp_stats_static(const void* d_x, int dtype, uint64_t n, qp_stats_t* d_out, void* stream);

/* ---- a3: ACIQ clip (Sec. 3: alpha = F(q) * b under L(mu, b)) ---------------------------
 * Host form: from statistics already copied to the host.  b is h_stats->mad (bmode
 * QP_B_MAD), h_stats->mean_abs (QP_B_MEAN_ABS), sqrt(var) for QP_DIST_GAUSS, or b_override
 * when b_override > 0.  Writes alpha (optional) and the quantizer for
 * [mean - alpha, mean + alpha] (optional).  Returns as qp_make_qparams. */
int32_t qp_aciq_alpha(const qp_stats_t* h_stats, int bits, int dist, int bmode, double b_override,
                      double* h_alpha_out, qp_qparams_t* h_qp_out);
/* Device form: same arithmetic in a one-thread kernel reading *d_stats and writing
 * *d_qp_out, so that stats -> clip -> quantize needs no host round trip. */
int32_t qp_aciq_qparams_device(qp_ctx* ctx, const qp_stats_t* d_stats, int bits, int dist, int bmode,
                               qp_qparams_t* d_qp_out, void* stream);
/* Clip range by method (Sec. 3, "Naive PTQ and ACIQ"):
 *   QP_CLIP_ACIQ    [mean - alpha, mean + alpha], alpha = F(q) b (as qp_aciq_alpha)
 *   QP_CLIP_DSACIQ  ACIQ refined by the directed search (qp_dsaciq_search / qp_sender_*; not a
 *                   closed form of the statistics, so not accepted by the two calls below)
 *   QP_CLIP_MINMAX  naive PTQ: the tensor's own [min, max]
 * QP_CLIP_ACIQ | QP_CLIP_INTERSECT cuts the ACIQ range back to the data's range,
 * [max(mean - alpha, min), min(mean + alpha, max)]: no element lies outside [min, max], so
 * the clipping error is unchanged and the step shrinks whenever alpha reaches past the data
 * (a variant of this library; the paper clips at mean -/+ alpha only).
 * ... | QP_CLIP_MIDRISE (any method) puts the mid-rise grid on the range: 2^bits equal bins,
 * every element reconstructed at the centre of its bin (the other reading of Sec. 3's "equal
 * intervals", and the grid the ACIQ noise term alpha^2 / (3 * 4^q) models).  The bin centres
 * are the levels of the ordinary quantizer on the range pulled in by half a bin on each side,
 * [lo + w/2, hi - w/2] with w = (hi - lo) / 2^bits, and its rounding boundaries are the bin
 * edges: the flag changes the clip range and nothing else (qp_midrise_range does just that),
 * so packing and the receiver are the same.
 * qp_clip_range: host form, writes the ends (optional) and the quantizer (optional).
 * qp_clip_qparams_device: one-thread kernel from device-resident statistics.
 * Errors: QP_ERR_INVALID_ARG (NULL, unknown method, dist, bmode), QP_ERR_UNSUPPORTED_BITS;
 * QP_WARN_DEGENERATE as qp_make_qparams (host form; status word on the device). */
enum { QP_CLIP_ACIQ = 0, QP_CLIP_DSACIQ = 1, QP_CLIP_MINMAX = 2 };
#define QP_CLIP_INTERSECT 0x10
#define QP_CLIP_MIDRISE 0x20
int32_t qp_midrise_range(double lo, double hi, int bits, double* h_lo_out, double* h_hi_out);
int32_t qp_clip_range(const qp_stats_t* h_stats, int bits, int method, int dist, int bmode, double* h_lo_out,
                      double* h_hi_out, qp_qparams_t* h_qp_out);
int32_t qp_clip_qparams_device(qp_ctx* ctx, const qp_stats_t* d_stats, int bits, int method, int dist, int bmode,
                               qp_qparams_t* d_qp_out, void* stream);

/* ---- a2 + a4: directed search DS-ACIQ (Sec. 3 "Directed Search", Eq. 1) -----------------
 * Histogram of x with hist_bins equal bins over [min, max]; b_R = 1 / (2 * peak density);
 * candidates b_k = b_E + k (b_R - b_E) / steps, k = 0..steps; each is scored by the
 * quantization MSE of x under the clip F(bits) * b_k about the mean; the smallest k with
 * the lowest MSE wins (k = 0 keeps b_E).  d_stats must hold the statistics of the same x.
 * Writes *d_out (optional) and the winning quantizer *d_qp_out (optional); both device
 * memory.  bits 1..8; 1 <= steps <= QP_MAX_STEPS; 1 <= hist_bins <= QP_MAX_HIST_BINS;
 * bmode QP_B_MAD or QP_B_MEAN_ABS, optionally | QP_B_MIDRISE.
 * QP_B_MAD | QP_B_GAUSS (optionally | QP_B_MIDRISE) runs the same search under the normal
 * model that ACIQ also offers (the paper searches under the Laplace model only): the scale is
 * the standard deviation, sigma_E = sqrt(var); a normal density peaks at 1 / (sigma sqrt(2 pi)),
 * so sigma_R = 1 / (sqrt(2 pi) * peak density); the clip is F_gauss(bits) * sigma_k.  The
 * result's b_e, b_r, b_star then hold sigma_E, sigma_R, sigma*.
 * The call first checks on the device whether d_stats already carries the peak of this
 * histogram (qp_stats with the same hist_bins) and counts for itself if not; that check is a
 * memset and a kernel launch.  bmode | QP_B_HIST_IN_STATS skips them: the caller vouches that
 * d_stats came from qp_stats(x, hist_bins) with qp_stats_carries_histogram() = 1.  If it did
 * not, QP_DEV_HIST_MISSING is raised in the status word and the search keeps b_E (k* = 0).
 * Errors: as qp_stats, plus QP_ERR_UNSUPPORTED_BITS. */
int32_t qp_dsaciq_search(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, const qp_stats_t* d_stats,
                         int bits, int bmode, int steps, int hist_bins,
                         qp_ds_result_t* d_out, qp_qparams_t* d_qp_out, void* stream);
/* How qp_dsaciq_search scores the candidates.  Both ways give the same MSE per candidate
 * (to ~1e-8 relative) and the same winner.
 *   QP_SEARCH_CANDIDATES  every element is quantized under every candidate (any bits/steps)
 *   QP_SEARCH_INTERVALS   one pass gathers moments per interval between the candidates'
 *                         decision thresholds; used where (steps+1)*(2^bits-1) <= 2048 and
 *                         n < ~1.8e9, otherwise the call falls back to the first way
 *   QP_SEARCH_AUTO        intervals for n >= 2^20 where they apply (default)
 * The pass over x that gathers the moments has two forms with identical results: the plain one
 * (every element looks its interval up), and one that adds elements of grid cells without a
 * threshold straight into per-cell, per-lane sums and looks up only the others; the second is
 * used up to ~150 M elements, QP_SEARCH_INTERVALS_PLAIN forces the first.  Around the pass, two small
 * kernels build the tables (candidates and thresholds; their sorted order and the cell table) and two
 * finish (the blocks' partials added up; every candidate scored and the winner picked). */
enum { QP_SEARCH_AUTO = 0, QP_SEARCH_CANDIDATES = 1, QP_SEARCH_INTERVALS = 2, QP_SEARCH_INTERVALS_PLAIN = 3 };
int32_t qp_set_search_path(qp_ctx* ctx, int path);
/* Graph replay of the multi-kernel calls (an execution option; the paper has no counterpart,
 * results are unchanged).  With on = 1, qp_stats, qp_dsaciq_search and qp_sender_device
 * record their kernels into a CUDA graph the first time they see an argument set (all
 * pointers, sizes and options; not the stream) and launch the stored graph on later calls
 * with the same arguments, which removes most of the gaps between the small kernels.  Up to
 * 64 graphs are kept per context, the least recently used one is dropped.  A call on the
 * legacy default stream (NULL), or on a stream the caller is capturing, is enqueued directly.
 * The buffers of a recorded call must stay valid while it may be replayed; on = 0 drops all
 * stored graphs.  Default off.  qp_graph_replays counts the calls served by a stored graph.
 * Errors: QP_ERR_INVALID_ARG. */
int32_t qp_set_graph_replay(qp_ctx* ctx, int on);
uint64_t qp_graph_replays(qp_ctx* ctx);
/* Copies the MSE of every candidate of the last search on this context (steps+1 values)
 * to host memory after waiting for `stream`.  Diagnostic. */
int32_t qp_dsaciq_curve(qp_ctx* ctx, double* h_curve, int capacity, void* stream);
/* Copies the quantizer of every candidate of the last search on this context (steps+1 entries:
 * the clip range [mean - F b_k, mean + F b_k] as the kernels rounded it to fp32, its scale and
 * reciprocal, bits; flags bit 0 marks an empty range, which is also what a step that is not a
 * candidate looks like) to host memory after waiting for `stream`.  Diagnostic: with it a
 * candidate's error can be recomputed for exactly the quantizer that the library scored.
 * Errors: QP_ERR_INVALID_ARG (NULL, no search yet), QP_ERR_BUFFER_TOO_SMALL, QP_ERR_CUDA. */
int32_t qp_dsaciq_candidates(qp_ctx* ctx, qp_qparams_t* h_out, int capacity, void* stream);
/* Policy of the paper's evaluation (Sec. 3): the search is switched on at 4 bits and below. */
int32_t qp_policy_use_ds(int bits);

/* ---- a5: clamp, quantize, bit-pack (Sec. 3: uniform quantization of the clipped tensor) -
 * code_i = round_half_even((clamp(x_i, lo, hi) - lo) * inv_scale), each fp32 operation
 * rounded on its own.  Element i occupies stream bits [i*bits, (i+1)*bits), least
 * significant bit first; stream bit j is bit (j mod 8) of byte (j div 8); bits = 16 is one
 * little-endian uint16 per element.  All qp_packed_bytes(n, bits) bytes are written, pad
 * bits zero.  `qp` is a host pointer (qp_on_device = 0, read before returning) or a
 * device pointer (qp_on_device = 1, read by the kernel; its bits must equal `bits`,
 * otherwise QP_DEV_BITS_MISMATCH is raised in the status word).
 * d_packed must be 16-byte aligned; d_x aligned to its element size.  Only a 16-byte aligned d_x
 * takes the warp-tile kernel; an x that is merely element-aligned (a view that starts at an odd
 * element) sends the WHOLE tensor through the scalar kernel (a thread per 32 elements, 4-byte
 * loads): the same bytes, about 5x the time (129 MB tensor on B200: 153-162 us against 33-35 us).
 * Copy such a view to an aligned buffer first if speed matters.  The same holds for d_y of
 * qp_unpack_dequantize (179 us against 31-34 us); qp_stats loses less (66 us against 46 us).
 * Errors: QP_ERR_INVALID_ARG, QP_ERR_UNSUPPORTED_BITS, QP_ERR_UNSUPPORTED_DTYPE,
 * QP_ERR_BUFFER_TOO_SMALL (packed_capacity < qp_packed_bytes), QP_ERR_ALIGNMENT, QP_ERR_CUDA. */
int32_t qp_quantize_pack(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, int bits,
                         const qp_qparams_t* qp, int qp_on_device,
                         void* d_packed, uint64_t packed_capacity, void* stream);

/* ---- a6: unpack, dequantize (the receiver's side of Sec. 3) -----------------------------
 * y_i = fma(code_i, scale, lo) in fp32 (one rounding), written as out_dtype (QP_F32, or
 * QP_BF16 rounded to nearest even).  d_packed as written by qp_quantize_pack (16-byte
 * aligned, qp_packed_bytes long); d_y aligned to its element size.
 * Errors: as qp_quantize_pack. */
int32_t qp_unpack_dequantize(qp_ctx* ctx, const void* d_packed, uint64_t n, int bits,
                             const qp_qparams_t* qp, int qp_on_device,
                             void* d_y, int out_dtype, void* stream);

/* ---- a7: bit-width from bandwidth (Sec. 1, Sec. 3 "Adaptive PDA", Eq. 2) ----------------
 * Widest allowed width whose payload fits the budget:
 * 8 * (ceil(n_elems*q/8) + overhead_bytes) <= bandwidth_bps * budget_s; q = 32 is the raw
 * fp32 tensor.  h_allowed: n_allowed widths in 1..32, any order; NULL selects the widths of
 * the paper's Table 1, {32,16,8,6,4,2}.  Nothing fits: smallest allowed and
 * QP_WARN_INFEASIBLE. */
int32_t qp_select_bits(double bandwidth_bps, double budget_s, uint64_t n_elems, uint64_t overhead_bytes,
                       const int32_t* h_allowed, int n_allowed, int32_t* h_bits_out);
/* Eq. 2 as printed: q' = 32 / 2^ceil(log2((V*32/q) / ((S/R) * B))), V bytes at the current
 * width q, B bit/s, S images per microbatch, R target images/s; clamped to [1, 32]. */
int32_t qp_select_bits_eq2(double v_bytes, int q_t, double s_images, double r_images_per_s,
                           double bandwidth_bps, int32_t* h_bits_out);

/* ---- adaptive controller (Sec. 3 "Adaptive PDA", Sec. 4.2) -------------------------------
 * Host-only state machine of the paper's runtime loop: the monitor reports every
 * microbatch's transfer (bytes put on the link, seconds it took); the averages are taken
 * over a window of microbatches (50 in the paper); at the end of a window the link
 * bandwidth is 8 * sum(bytes) / sum(seconds), and if it differs from the bandwidth of the
 * last decision by more than rel_change (relative; 0 = decide at every window) the
 * bit-width is chosen anew for the budget S / R seconds per microbatch:
 *   QP_CTRL_FIT  widest allowed width whose payload fits (qp_select_bits)
 *   QP_CTRL_EQ2  Eq. 2 as printed (qp_select_bits_eq2), from the current width and payload
 * The struct is plain data owned by the caller (copy it to snapshot the controller). */
enum { QP_CTRL_FIT = 0, QP_CTRL_EQ2 = 1 };
#define QP_CTRL_MAX_ALLOWED 8
typedef struct {
    int32_t window, count;            /* microbatches per decision; seen so far in this window   */
    int32_t bits, mode;               /* width in force (32 = raw fp32); QP_CTRL_FIT / QP_CTRL_EQ2 */
    double s_images, r_images_per_s;  /* microbatch size S and target rate R                      */
    uint64_t n_elems, overhead_bytes; /* tensor elements per microbatch; header bytes per transfer */
    double rel_change;
    double sum_bytes, sum_seconds;    /* of the current window                                    */
    double ref_bandwidth_bps;         /* window bandwidth at the last decision; 0 before the first */
    int32_t n_allowed;
    int32_t allowed[QP_CTRL_MAX_ALLOWED];
} qp_controller_t;
/* h_allowed NULL selects the widths of the paper's Table 1, {32,16,8,6,4,2}.
 * Errors: QP_ERR_INVALID_ARG (NULL, window < 1, S or R not positive, widths outside 1..32,
 * more than QP_CTRL_MAX_ALLOWED widths, unknown mode, rel_change < 0). */
int32_t qp_controller_init(qp_controller_t* h_c, int window, double s_images, double r_images_per_s,
                           uint64_t n_elems, uint64_t overhead_bytes, const int32_t* h_allowed, int n_allowed,
                           int mode, double rel_change, int initial_bits);
/* One microbatch's transfer.  *h_bits_out = width to use from now on; *h_decided_out = 1 when
 * this call closed a window and chose the width anew.  Returns QP_OK, QP_WARN_INFEASIBLE (the
 * smallest width does not fit either; it is chosen) or QP_ERR_INVALID_ARG. */
int32_t qp_controller_observe(qp_controller_t* h_c, double bytes_sent, double seconds, int32_t* h_bits_out,
                              int32_t* h_decided_out);
/* Payload of one microbatch at `bits` (32 = raw fp32): ceil(n_elems*bits/8) + overhead_bytes. */
uint64_t qp_controller_payload_bytes(const qp_controller_t* h_c, int bits);

/* ---- channel-wise variant (the paper, Sec. 3, clips per tensor; this is the per-channel form
 * that its cited PTQ work uses for activations with outlier channels) ----------------------
 * The tensor is [rows, channels], row-major: element i belongs to channel i mod channels.
 * Every channel gets the statistics, clip range and quantizer that the per-tensor calls give
 * for its column alone; bit-width and packed layout (qp_packed_bytes(rows * channels, bits))
 * are shared, so the receiver needs the `channels` quantizers (24 bytes each) with the stream.
 *   qp_stats_channels                fills d_out[0..channels) (hist fields 0).  Keeps its block
 *                                    partials in the context, allocated on the first call and
 *                                    when a larger tensor comes (cudaMalloc: not during capture).
 *   qp_clip_qparams_channels_device  d_qp_out[c] from d_stats[c]; method, dist, bmode as
 *                                    qp_clip_qparams_device.
 *   qp_quantize_pack_channels        code of element i with d_qp[i mod channels].
 *   qp_unpack_dequantize_channels    the inverse, fp32 or bf16 out.
 *   qp_sender_channels_device        the three sender calls in one: statistics -> clip by `method`
 *                                    (Laplace model; QP_CLIP_DSACIQ runs qp_dsaciq_search_channels with
 *                                    QP_DEFAULT_STEPS and QP_DEFAULT_HIST_BINS) -> quantize+pack; writes the packed stream,
 *                                    d_qp_out[0..channels) and, if d_stats_out is not NULL, the
 *                                    statistics (otherwise they stay in a buffer of the context,
 *                                    allocated on first use).
 * d_stats, d_qp: device arrays of `channels` entries.  1 <= channels <= QP_MAX_CHANNELS.
 * Errors: as the per-tensor calls, plus QP_ERR_INVALID_ARG for channels out of range. */
#define QP_MAX_CHANNELS 4096
int32_t qp_stats_channels(qp_ctx* ctx, const void* d_x, int dtype, uint64_t rows, uint32_t channels,
                          qp_stats_t* d_out, void* stream);
int32_t qp_clip_qparams_channels_device(qp_ctx* ctx, const qp_stats_t* d_stats, uint32_t channels, int bits,
                                        int method, int dist, int bmode, qp_qparams_t* d_qp_out, void* stream);
int32_t qp_quantize_pack_channels(qp_ctx* ctx, const void* d_x, int dtype, uint64_t rows, uint32_t channels,
                                  int bits, const qp_qparams_t* d_qp, void* d_packed, uint64_t packed_capacity,
                                  void* stream);
int32_t qp_unpack_dequantize_channels(qp_ctx* ctx, const void* d_packed, uint64_t rows, uint32_t channels, int bits,
                                      const qp_qparams_t* d_qp, void* d_y, int out_dtype, void* stream);
int32_t qp_sender_channels_device(qp_ctx* ctx, const void* d_x, int dtype, uint64_t rows, uint32_t channels, int bits,
                                  int method, int bmode, void* d_packed, uint64_t packed_capacity,
                                  qp_qparams_t* d_qp_out, qp_stats_t* d_stats_out, void* stream);

/* Channel-wise directed search (the search of Sec. 3 / Eq. 1 applied to each column of the
 * [rows, channels] tensor; the paper searches per tensor): channel c gets the histogram,
 * b_R, candidates, MSE curve and winner that qp_dsaciq_search gives for its column alone with
 * d_stats[c] (from qp_stats_channels).  Writes d_qp_out[0..channels) and, if not NULL,
 * d_out[0..channels).  Two ways, same winner: where (steps + 1) * (2^bits - 1) <= 2048 and
 * rows <= 65535, one pass over the tensor gathers count and sum per interval between the
 * candidates' decision thresholds of every channel and every candidate is evaluated from prefix
 * sums (the default); otherwise, and under qp_set_search_path(QP_SEARCH_CANDIDATES), every
 * candidate is scored on every element ((steps + 1) * 9 fp32 instructions per element).
 * bits 1..8; 1 <= steps <= QP_CH_MAX_STEPS; 1 <= hist_bins <= QP_CH_MAX_HIST_BINS; bmode as for
 * qp_dsaciq_search (QP_B_HIST_IN_STATS has no meaning here and is rejected).  Scratch
 * (histograms, candidates, sums; for the first way also thresholds, positions and interval sums:
 * about 18 (steps + 1) (2^bits - 1) bytes per channel) is allocated by the context on first use
 * (cudaMalloc: not during capture) and kept.
 * qp_dsaciq_curve_channels copies the MSE curve of one channel of the last such search to
 * host memory (steps + 1 doubles) and synchronizes the stream.
 * Errors: as qp_dsaciq_search, plus QP_ERR_INVALID_ARG for channels out of range. */
#define QP_CH_MAX_STEPS 127
#define QP_CH_MAX_HIST_BINS 256
int32_t qp_dsaciq_search_channels(qp_ctx* ctx, const void* d_x, int dtype, uint64_t rows, uint32_t channels,
                                  const qp_stats_t* d_stats, int bits, int bmode, int steps, int hist_bins,
                                  qp_ds_result_t* d_out, qp_qparams_t* d_qp_out, void* stream);
int32_t qp_dsaciq_curve_channels(qp_ctx* ctx, uint32_t channel, double* h_curve, int capacity, void* stream);
/* The candidates' quantizers of the last channel-wise search, as qp_dsaciq_candidates:
 * h_out[c * (steps + 1) + k] for channel c and step k; capacity in entries.  Diagnostic. */
int32_t qp_dsaciq_candidates_channels(qp_ctx* ctx, qp_qparams_t* h_out, uint64_t capacity, void* stream);

/* ---- token-wise variant (the other axis of the channel-wise variant above; the paper clips per
 * tensor) -------------------------------------------------------------------------------------
 * The tensor is [tokens, channels], row-major: token t is the row of `channels` contiguous elements
 * t * channels .. (t + 1) * channels - 1 (one position of a ViT sequence).  Every token gets the
 * statistics, clip range and quantizer that the per-tensor calls give for its row alone; bit-width
 * and packed layout (qp_packed_bytes(tokens * channels, bits)) are shared, so the receiver needs the
 * `tokens` quantizers (24 bytes each) with the stream.
 *   qp_stats_tokens                fills d_out[0..tokens) (hist fields 0); a warp per token, the
 *                                  tensor is read from HBM once
 *   qp_clip_qparams_tokens_device  d_qp_out[t] from d_stats[t]; method, dist, bmode as
 *                                  qp_clip_qparams_device (closed-form clips only: no search per token)
 *   qp_quantize_pack_tokens        code of element i with d_qp[i / channels]
 *   qp_unpack_dequantize_tokens    the inverse, fp32 or bf16 out
 *   qp_sender_tokens_device        the three sender calls in one; d_stats_work is the caller's device
 *                                  memory for `tokens` statistics
 * The fast kernels need a 16-byte aligned tensor, `channels` a multiple of 4 (fp32) or 8 (bf16) and
 * bits <= 8; other shapes, and 16 bits, take a scalar kernel (one thread per 32 elements).
 * d_stats, d_qp: device arrays of `tokens` entries; channels >= 1.
 * Errors: as the per-tensor calls. */
int32_t qp_stats_tokens(qp_ctx* ctx, const void* d_x, int dtype, uint64_t tokens, uint32_t channels, qp_stats_t* d_out,
                        void* stream);
int32_t qp_clip_qparams_tokens_device(qp_ctx* ctx, const qp_stats_t* d_stats, uint64_t tokens, int bits, int method,
                                      int dist, int bmode, qp_qparams_t* d_qp_out, void* stream);
int32_t qp_quantize_pack_tokens(qp_ctx* ctx, const void* d_x, int dtype, uint64_t tokens, uint32_t channels, int bits,
                                const qp_qparams_t* d_qp, void* d_packed, uint64_t packed_capacity, void* stream);
int32_t qp_unpack_dequantize_tokens(qp_ctx* ctx, const void* d_packed, uint64_t tokens, uint32_t channels, int bits,
                                    const qp_qparams_t* d_qp, void* d_y, int out_dtype, void* stream);
int32_t qp_sender_tokens_device(qp_ctx* ctx, const void* d_x, int dtype, uint64_t tokens, uint32_t channels, int bits,
                                int method, int bmode, void* d_packed, uint64_t packed_capacity, qp_qparams_t* d_qp_out,
                                qp_stats_t* d_stats_work, void* stream);

/* ---- whole sender / receiver on HOST buffers (Sec. 3: the module sits between a stage's
 * output and the link, and between the link and the next stage's input) -------------------
 * qp_sender_host: copies the n elements at h_x to d_x_work, runs statistics, the clip
 * by `method` (as qp_sender_device), quantize+pack
 * into d_packed_work, and copies the packed stream to h_packed and the quantizer to
 * *h_qp_out.  qp_receiver_host: copies h_packed to d_packed_work, unpacks+dequantizes into
 * d_y_work and copies the tensor to h_y.  Everything is enqueued on `stream`; host outputs
 * are valid after the caller has synchronised the stream.  Host buffers should be
 * page-locked for the copies to be asynchronous.  The caller owns all six buffers:
 * d_x_work >= n elements of dtype, d_packed_work and h_packed >= qp_packed_bytes(n, bits)
 * (d_packed_work 16-byte aligned), d_y_work and h_y >= n elements of out_dtype.
 * Errors: as the calls they are made of. */
/* qp_sender_device: the sender's whole chain on DEVICE buffers in one call, nothing read back
 * to the host: statistics (carrying the histogram along for the search), the clip by
 * `method` (QP_CLIP_ACIQ = 0, optionally | QP_CLIP_INTERSECT; QP_CLIP_DSACIQ = 1, bits <= 8;
 * QP_CLIP_MINMAX = 2; each optionally | QP_CLIP_MIDRISE; Laplace model), quantize+pack.
 * Writes the packed stream to d_packed, the quantizer to *d_qp_out (what the receiver needs)
 * and, if d_stats_out is not NULL, the statistics.  Equivalent to qp_stats +
 * qp_dsaciq_search / qp_aciq_qparams_device + qp_quantize_pack with the same arguments.
 *
 * How the chain runs (qp_set_sender_path; the paper has no counterpart):
 *   QP_SENDER_CHAIN  the kernels of the separate calls, one after the other; the outputs are
 *                    bit for bit those of the separate calls
 *   QP_SENDER_FUSED  one cooperative launch: every SM keeps its slice of x in shared memory, the
 *                    tensor-wide steps are separated by grid barriers.  Applies to 0 < n <= 2^20
 *                    with the search (and steps <= 127, hist_bins <= 4096) and to n <= 6.5e6
 *                    with a closed-form clip (less where the GPU's shared memory holds less);
 *                    other arguments fall back to the chain.  Same arithmetic per element, but
 *                    the sums are merged in another order: statistics agree with the chain to
 *                    ~1e-15 relative, the error curve to ~1e-6, so the clip range can differ in
 *                    its last fp32 bit or, where two steps of the search tie, by one step.
 *   QP_SENDER_AUTO   fused where it is the faster of the two on a B200: n <= 2^20 with the
 *                    search, n <= 2^21 otherwise (default)
 * A grid barrier that does not complete within about a quarter of a second sets
 * QP_DEV_STREAM_TIMEOUT in the status word and the launch ends without output
 * (qp_get_status then returns QP_ERR_TIMEOUT). */
enum { QP_SENDER_AUTO = 0, QP_SENDER_CHAIN = 1, QP_SENDER_FUSED = 2 };
int32_t qp_set_sender_path(qp_ctx* ctx, int path);
int32_t qp_sender_device(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, int bits, int method, int bmode,
                         int steps, int hist_bins, void* d_packed, uint64_t packed_capacity,
                         qp_qparams_t* d_qp_out, qp_stats_t* d_stats_out, void* stream);
int32_t qp_sender_host(qp_ctx* ctx, const void* h_x, int dtype, uint64_t n, int bits, int method, int bmode,
                       int steps, int hist_bins, void* d_x_work, void* d_packed_work, void* h_packed,
                       uint64_t packed_capacity, qp_qparams_t* h_qp_out, void* stream);
int32_t qp_receiver_host(qp_ctx* ctx, const void* h_packed, uint64_t n, int bits, const qp_qparams_t* h_qp,
                         void* d_packed_work, void* d_y_work, void* h_y, int out_dtype, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* QUANTPIPE_H */

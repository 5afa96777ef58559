// Host side of the C ABI: context, argument checks, the O(1) host functions.
#include <math.h>
#include <string.h>

#include <new>

#include "qp_internal.cuh"

// ------------------------------------------------------------------ errors

int32_t qp_fail(qp_ctx* ctx, int32_t status, const char* what)
{
    if (ctx) snprintf(ctx->err, sizeof ctx->err, "%s: %s", qp_status_string(status), what);
    return status;
}

int32_t qp_check_launch(qp_ctx* ctx, const char* what)
{
    const cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) return QP_OK;
    if (ctx) snprintf(ctx->err, sizeof ctx->err, "CUDA error in %s: %s", what, cudaGetErrorString(e));
    return QP_ERR_CUDA;
}

extern "C" const char* qp_status_string(int32_t s)
{
    switch (s) {
        case QP_OK: return "ok";
        case QP_ERR_INVALID_ARG: return "invalid argument";
        case QP_ERR_UNSUPPORTED_BITS: return "unsupported bit-width";
        case QP_ERR_UNSUPPORTED_DTYPE: return "unsupported dtype";
        case QP_ERR_BUFFER_TOO_SMALL: return "buffer too small";
        case QP_ERR_ALIGNMENT: return "misaligned pointer";
        case QP_ERR_CUDA: return "CUDA error";
        case QP_ERR_TIMEOUT: return "device wait timed out";
        case QP_ERR_TOO_LARGE: return "size exceeds the maximum this entry point supports";
        case QP_WARN_INFEASIBLE: return "warning: no allowed bit-width fits the budget";
        case QP_WARN_DEGENERATE: return "warning: degenerate clip range";
        case QP_WARN_NONFINITE: return "warning: non-finite inputs were skipped";
        default: return "unknown status";
    }
}

extern "C" const char* qp_last_error(qp_ctx* ctx) { return ctx ? ctx->err : "no context"; }

// ----------------------------------------------------------------- index checks of the debug build

#ifdef QP_CHECK_BOUNDS
static qp_ck_unit* g_ck_units = nullptr;
void qp_ck_register(qp_ck_unit* u)
{
    u->next = g_ck_units;
    g_ck_units = u;
}
static unsigned qp_ck_collect()
{
    unsigned any = 0;
    for (qp_ck_unit* u = g_ck_units; u; u = u->next) any |= u->read_and_clear();
    return any;
}
#endif

extern "C" int32_t qp_built_with_index_checks(void)
{
#ifdef QP_CHECK_BOUNDS
    return 1;
#else
    return 0;
#endif
}

// ----------------------------------------------------------------- context

static void qp_drop_graphs(qp_ctx* ctx);

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

extern "C" int32_t qp_create(int device, qp_ctx** out)
{
    if (!out) return QP_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess) { cudaGetLastError(); return QP_ERR_CUDA; }
    if (device < 0 || device >= count) return QP_ERR_INVALID_ARG;
    qp_device_guard guard(device);
    if (!guard.ok) return QP_ERR_CUDA;

    qp_ctx* c = new (std::nothrow) qp_ctx();
    if (!c) return QP_ERR_CUDA;
    memset(c, 0, sizeof *c);
    c->device = device;
    strcpy(c->err, "ok");
    c->wait_cycles = QP_WAIT_CYCLES_DEFAULT;
    c->spin_limit = QP_SPIN_LIMIT_DEFAULT;
    if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
        delete c;
        return QP_ERR_CUDA;
    }

    size_t off = 0;
    const size_t o_part = off;   off = align_up(off + sizeof(qp_stats_partial) * QP_MAX_BLOCKS, 256);
    const size_t o_hist = off;   off = align_up(off + sizeof(unsigned long long) * QP_MAX_HIST_BINS, 256);
    const size_t o_cand = off;   off = align_up(off + sizeof(float4) * (QP_MAX_STEPS + 1), 256);
    const size_t o_valid = off;  off = align_up(off + sizeof(int) * (QP_MAX_STEPS + 1), 256);
    const size_t o_sums = off;   off = align_up(off + sizeof(double) * QP_MAX_BLOCKS * QP_EVAL_K, 256);
    const size_t o_curve = off;  off = align_up(off + sizeof(double) * (QP_MAX_STEPS + 1), 256);
    const size_t o_setup = off;  off = align_up(off + sizeof(qp_ds_setup), 256);
    const size_t o_ticket = off; off = align_up(off + sizeof(unsigned) * 4, 256);
    const size_t o_status = off; off = align_up(off + sizeof(unsigned), 256);
    c->iv_blocks = c->sm_count * QP_IV_BLOCKS_PER_SM;
    const size_t o_ivbnd = off;  off = align_up(off + sizeof(float) * QP_IV_MAXB, 256);
    const size_t o_ivbb = off;   off = align_up(off + sizeof(float) * (QP_IV_MAXB + 1), 256);
    const size_t o_ivedge = off; off = align_up(off + sizeof(float) * (QP_IV_CELLS + 1), 256);
    const size_t o_ivfirst = off; off = align_up(off + sizeof(unsigned) * (QP_IV_CELLS + 8), 256);
    const size_t o_ivpart = off; off = align_up(off + sizeof(unsigned long long) * (size_t)c->iv_blocks * (QP_IV_MAXB + 1), 256);
    const size_t o_ivouter = off; off = align_up(off + sizeof(double) * 8 * (c->iv_blocks + 1), 256);
    const size_t o_ivtot = off;  off = align_up(off + sizeof(qp_iv_total) * (QP_IV_MAXB + 1), 256);
    const size_t o_tstats = off; off = align_up(off + sizeof(qp_stats_t), 256);
    const size_t o_tqp = off;    off = align_up(off + sizeof(qp_qparams_t), 256);
    const size_t o_fused = off;  off = align_up(off + QP_FUSED_BYTES, 256);

    if (cudaMalloc(&c->d_base, off) != cudaSuccess || cudaMemset(c->d_base, 0, off) != cudaSuccess) {
        cudaGetLastError();
        if (c->d_base) cudaFree(c->d_base);
        delete c;
        return QP_ERR_CUDA;
    }
    char* b = static_cast<char*>(c->d_base);
    c->d_part = reinterpret_cast<qp_stats_partial*>(b + o_part);
    c->d_hist = reinterpret_cast<unsigned long long*>(b + o_hist);
    c->d_cand = reinterpret_cast<float4*>(b + o_cand);
    c->d_valid = reinterpret_cast<int*>(b + o_valid);
    c->d_sums = reinterpret_cast<double*>(b + o_sums);
    c->d_curve = reinterpret_cast<double*>(b + o_curve);
    c->d_setup = reinterpret_cast<qp_ds_setup*>(b + o_setup);
    c->d_ticket = reinterpret_cast<unsigned*>(b + o_ticket);
    c->d_status = reinterpret_cast<unsigned*>(b + o_status);
    c->d_iv_bnd = reinterpret_cast<float*>(b + o_ivbnd);
    c->d_iv_bb = reinterpret_cast<float*>(b + o_ivbb);
    c->d_iv_edges = reinterpret_cast<float*>(b + o_ivedge);
    c->d_iv_first = reinterpret_cast<unsigned*>(b + o_ivfirst);
    c->d_iv_part = reinterpret_cast<unsigned long long*>(b + o_ivpart);
    c->d_iv_outer = reinterpret_cast<double*>(b + o_ivouter);
    c->d_iv_tot = reinterpret_cast<qp_iv_total*>(b + o_ivtot);
    c->d_tmp_stats = reinterpret_cast<qp_stats_t*>(b + o_tstats);
    c->d_tmp_qp = reinterpret_cast<qp_qparams_t*>(b + o_tqp);
    c->d_fused = b + o_fused;
    *out = c;
    return QP_OK;
}

extern "C" int32_t qp_destroy(qp_ctx* ctx)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    qp_device_guard guard(ctx->device);
    qp_drop_graphs(ctx);
    if (ctx->d_ch_part) cudaFree(ctx->d_ch_part);
    if (ctx->d_ch_stats) cudaFree(ctx->d_ch_stats);
    if (ctx->d_ch_search) cudaFree(ctx->d_ch_search);
    const cudaError_t e = cudaFree(ctx->d_base);
    delete ctx;
    return e == cudaSuccess ? QP_OK : QP_ERR_CUDA;
}

extern "C" int32_t qp_get_status(qp_ctx* ctx, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    qp_device_guard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, ctx->d_status, sizeof word, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_status, 0, sizeof word, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) {
        snprintf(ctx->err, sizeof ctx->err, "CUDA error in qp_get_status: %s", cudaGetErrorString(e));
        return QP_ERR_CUDA;
    }
#ifdef QP_CHECK_BOUNDS
    if (qp_ck_collect()) word |= QP_DEV_INDEX_RANGE;         // (the flags are per translation unit, not per context)
#endif
    if (word & QP_DEV_STREAM_TIMEOUT) {
        // a cooperative launch that gave up may have left its arrival counters and histogram mid-way
        e = cudaMemsetAsync(ctx->d_fused, 0, QP_FUSED_BYTES, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) {
            snprintf(ctx->err, sizeof ctx->err, "CUDA error in qp_get_status: %s", cudaGetErrorString(e));
            return QP_ERR_CUDA;
        }
        snprintf(ctx->err, sizeof ctx->err, "%s: a bounded wait on the device ran out (status word 0x%x); "
                 "the results of the calls since the last qp_get_status are invalid", qp_status_string(QP_ERR_TIMEOUT), word);
        return QP_ERR_TIMEOUT;
    }
    return (int32_t)word;
}

extern "C" uint64_t qp_launch_count(qp_ctx* ctx) { return ctx ? ctx->launches : 0; }

extern "C" int32_t qp_set_search_path(qp_ctx* ctx, int path)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (path < QP_SEARCH_AUTO || path > QP_SEARCH_INTERVALS_PLAIN) return qp_fail(ctx, QP_ERR_INVALID_ARG, "search path");
    ctx->moments_form = path == QP_SEARCH_INTERVALS_PLAIN ? 1 : 0;
    ctx->search_path = path >= QP_SEARCH_INTERVALS_PLAIN ? QP_SEARCH_INTERVALS : path;
    return QP_OK;
}

extern "C" int32_t qp_set_wait_limit_for_testing(qp_ctx* ctx, long long tile_wait_cycles, uint32_t barrier_polls,
                                                 int barrier_extra_arrivals)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (barrier_extra_arrivals < 0 || barrier_extra_arrivals > 1) return qp_fail(ctx, QP_ERR_INVALID_ARG, "barrier_extra_arrivals");
    ctx->wait_cycles = tile_wait_cycles < 0 ? QP_WAIT_CYCLES_DEFAULT : tile_wait_cycles;
    ctx->spin_limit = barrier_polls == 0 ? QP_SPIN_LIMIT_DEFAULT : barrier_polls;
    ctx->bar_extra = barrier_extra_arrivals;
    qp_device_guard guard(ctx->device);
    qp_drop_graphs(ctx);                      // recorded launches carry the old limits
    return QP_OK;
}

extern "C" int32_t qp_set_stats_path(qp_ctx* ctx, int path)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (path < QP_STATS_AUTO || path > QP_STATS_FUSED) return qp_fail(ctx, QP_ERR_INVALID_ARG, "statistics path");
    ctx->stats_path = path;
    return QP_OK;
}

extern "C" int32_t qp_set_sender_path(qp_ctx* ctx, int path)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (path < QP_SENDER_AUTO || path > QP_SENDER_FUSED) return qp_fail(ctx, QP_ERR_INVALID_ARG, "sender path");
    ctx->sender_path = path;
    return QP_OK;
}

// ------------------------------------------------------ host, pure functions

extern "C" uint64_t qp_packed_bytes(uint64_t n, int bits)
{
    if (!qp_bits_ok(bits)) return 0;
    const uint64_t raw = (n * (uint64_t)bits + 7u) / 8u;
    return (raw + 15u) / 16u * 16u;
}

// Laplace: F = W0(3 * 4^q) by Halley's iteration on w e^w = z.
static double lambert_w0(double z)
{
    double w = z < 3.0 ? 0.5 : log(z) - log(log(z));
    for (int it = 0; it < 64; ++it) {
        const double e = exp(w);
        const double f = w * e - z;
        const double d = e * (w + 1.0) - (w + 2.0) * f / (2.0 * w + 2.0);
        const double step = f / d;
        w -= step;
        if (fabs(step) <= 4e-16 * fabs(w)) break;
    }
    return w;
}

// Gauss: root of 4 [a (1 - Phi(a)) - phi(a)] + 2a / (3 * 4^q) by Newton from above
// (the function is increasing and concave on a > 0), guarded by bisection bounds.
static double gauss_F(int bits)
{
    const double c = 2.0 / (3.0 * pow(4.0, (double)bits));
    double lo = 0.0, hi = 64.0, a = 1.0 + 0.45 * bits;
    for (int it = 0; it < 200; ++it) {
        const double tail = 0.5 * erfc(a * M_SQRT1_2);
        const double pdf = exp(-0.5 * a * a) * 0.3989422804014327;
        const double g = 4.0 * (a * tail - pdf) + c * a;
        if (g < 0.0) lo = a; else hi = a;
        const double dg = 4.0 * tail + c;
        double next = a - g / dg;
        if (!(next > lo && next < hi)) next = 0.5 * (lo + hi);
        if (fabs(next - a) <= 1e-15 * fabs(a)) { a = next; break; }
        a = next;
    }
    return a;
}

double qp_host_aciq_F(int bits, int dist)
{
    if (!qp_bits_ok(bits)) return 0.0;
    if (dist == QP_DIST_LAPLACE) return lambert_w0(3.0 * pow(4.0, (double)bits));
    if (dist == QP_DIST_GAUSS) return gauss_F(bits);
    return 0.0;
}

extern "C" double qp_aciq_F(int bits, int dist) { return qp_host_aciq_F(bits, dist); }

extern "C" int32_t qp_make_qparams(double lo, double hi, int bits, qp_qparams_t* h_out)
{
    if (!h_out) return QP_ERR_INVALID_ARG;
    if (!qp_bits_ok(bits)) return QP_ERR_UNSUPPORTED_BITS;
    if (!isfinite(lo) || !isfinite(hi)) return QP_ERR_INVALID_ARG;
    return qp_fill_qparams(lo, hi, bits, h_out);
}

extern "C" int32_t qp_aciq_alpha(const qp_stats_t* h_stats, int bits, int dist, int bmode, double b_override,
                                 double* h_alpha_out, qp_qparams_t* h_qp_out)
{
    if (!h_stats) return QP_ERR_INVALID_ARG;
    if (!qp_bits_ok(bits)) return QP_ERR_UNSUPPORTED_BITS;
    if ((dist != QP_DIST_LAPLACE && dist != QP_DIST_GAUSS) || (bmode != QP_B_MAD && bmode != QP_B_MEAN_ABS))
        return QP_ERR_INVALID_ARG;
    const double b = b_override > 0.0       ? b_override
                     : dist == QP_DIST_GAUSS ? sqrt(h_stats->var)
                     : bmode == QP_B_MEAN_ABS ? h_stats->mean_abs
                                              : h_stats->mad;
    const double alpha = qp_host_aciq_F(bits, dist) * b;
    if (h_alpha_out) *h_alpha_out = alpha;
    if (!h_qp_out) return QP_OK;
    const double lo = h_stats->mean - alpha, hi = h_stats->mean + alpha;
    if (!isfinite(lo) || !isfinite(hi)) return QP_ERR_INVALID_ARG;
    return qp_fill_qparams(lo, hi, bits, h_qp_out);
}

bool qp_clip_method_closed_form(int method)
{
    const int base = method & 0xF, flags = method & ~0xF;
    if (flags & ~(QP_CLIP_INTERSECT | QP_CLIP_MIDRISE)) return false;
    if (base == QP_CLIP_ACIQ) return true;
    return base == QP_CLIP_MINMAX && !(flags & QP_CLIP_INTERSECT);
}
static bool clip_method_closed_form(int method) { return qp_clip_method_closed_form(method); }

extern "C" int32_t qp_midrise_range(double lo, double hi, int bits, double* h_lo_out, double* h_hi_out)
{
    if (!qp_bits_ok(bits)) return QP_ERR_UNSUPPORTED_BITS;
    if (!h_lo_out || !h_hi_out || !isfinite(lo) || !isfinite(hi)) return QP_ERR_INVALID_ARG;
    qp_midrise_ends(bits, lo, hi);
    *h_lo_out = lo;
    *h_hi_out = hi;
    return QP_OK;
}

extern "C" int32_t qp_clip_range(const qp_stats_t* h_stats, int bits, int method, int dist, int bmode, double* h_lo_out,
                                 double* h_hi_out, qp_qparams_t* h_qp_out)
{
    if (!h_stats) return QP_ERR_INVALID_ARG;
    if (!qp_bits_ok(bits)) return QP_ERR_UNSUPPORTED_BITS;
    if (!clip_method_closed_form(method)) return QP_ERR_INVALID_ARG;
    if ((dist != QP_DIST_LAPLACE && dist != QP_DIST_GAUSS) || (bmode != QP_B_MAD && bmode != QP_B_MEAN_ABS))
        return QP_ERR_INVALID_ARG;
    double lo, hi;
    qp_clip_ends(*h_stats, method, dist, bmode, bits, qp_host_aciq_F(bits, dist), lo, hi);
    if (h_lo_out) *h_lo_out = lo;
    if (h_hi_out) *h_hi_out = hi;
    if (!h_qp_out) return QP_OK;
    if (!isfinite(lo) || !isfinite(hi)) return QP_ERR_INVALID_ARG;
    return qp_fill_qparams(lo, hi, bits, h_qp_out);
}

extern "C" int32_t qp_policy_use_ds(int bits) { return bits >= 1 && bits <= 4 ? 1 : 0; }

extern "C" int32_t qp_select_bits(double bandwidth_bps, double budget_s, uint64_t n_elems, uint64_t overhead_bytes,
                                  const int32_t* h_allowed, int n_allowed, int32_t* h_bits_out)
{
    static const int32_t table1[6] = {32, 16, 8, 6, 4, 2};
    if (!h_bits_out || !(bandwidth_bps >= 0.0) || !(budget_s >= 0.0)) return QP_ERR_INVALID_ARG;
    if (!h_allowed) { h_allowed = table1; n_allowed = 6; }
    if (n_allowed < 1) return QP_ERR_INVALID_ARG;
    const double capacity = bandwidth_bps * budget_s;
    int best = 0, smallest = 33;
    for (int i = 0; i < n_allowed; ++i) {
        const int q = h_allowed[i];
        if (q < 1 || q > 32) return QP_ERR_INVALID_ARG;
        smallest = q < smallest ? q : smallest;
        const uint64_t payload = (n_elems * (uint64_t)q + 7u) / 8u;
        const double need = 8.0 * ((double)payload + (double)overhead_bytes);
        if (need <= capacity && q > best) best = q;
    }
    if (best == 0) { *h_bits_out = smallest; return QP_WARN_INFEASIBLE; }
    *h_bits_out = best;
    return QP_OK;
}

extern "C" int32_t qp_select_bits_eq2(double v_bytes, int q_t, double s_images, double r_images_per_s,
                                      double bandwidth_bps, int32_t* h_bits_out)
{
    if (!h_bits_out || !(v_bytes > 0.0) || q_t < 1 || q_t > 32 || !(s_images > 0.0) || !(r_images_per_s > 0.0) ||
        !(bandwidth_bps > 0.0))
        return QP_ERR_INVALID_ARG;
    const double fp32_bits = v_bytes * 8.0 * 32.0 / (double)q_t;
    const double ratio = fp32_bits / ((s_images / r_images_per_s) * bandwidth_bps);
    double e = ceil(log2(ratio));
    if (!(e > 0.0)) e = 0.0;
    if (e > 5.0) e = 5.0;
    *h_bits_out = 32 >> (int)e;
    return QP_OK;
}

// ------------------------------------------------------- adaptive controller

extern "C" uint64_t qp_controller_payload_bytes(const qp_controller_t* c, int bits)
{
    if (!c || bits < 1 || bits > 32) return 0;
    return (c->n_elems * (uint64_t)bits + 7u) / 8u + c->overhead_bytes;
}

extern "C" int32_t qp_controller_init(qp_controller_t* c, int window, double s_images, double r_images_per_s,
                                      uint64_t n_elems, uint64_t overhead_bytes, const int32_t* h_allowed,
                                      int n_allowed, int mode, double rel_change, int initial_bits)
{
    static const int32_t table1[6] = {32, 16, 8, 6, 4, 2};
    if (!c || window < 1 || !(s_images > 0.0) || !(r_images_per_s > 0.0) || !(rel_change >= 0.0)) return QP_ERR_INVALID_ARG;
    if (mode != QP_CTRL_FIT && mode != QP_CTRL_EQ2) return QP_ERR_INVALID_ARG;
    if (initial_bits < 1 || initial_bits > 32) return QP_ERR_INVALID_ARG;
    if (!h_allowed) { h_allowed = table1; n_allowed = 6; }
    if (n_allowed < 1 || n_allowed > QP_CTRL_MAX_ALLOWED) return QP_ERR_INVALID_ARG;
    memset(c, 0, sizeof *c);
    for (int i = 0; i < n_allowed; ++i) {
        if (h_allowed[i] < 1 || h_allowed[i] > 32) return QP_ERR_INVALID_ARG;
        c->allowed[i] = h_allowed[i];
    }
    c->n_allowed = n_allowed;
    c->window = window;
    c->bits = initial_bits;
    c->mode = mode;
    c->s_images = s_images;
    c->r_images_per_s = r_images_per_s;
    c->n_elems = n_elems;
    c->overhead_bytes = overhead_bytes;
    c->rel_change = rel_change;
    return QP_OK;
}

extern "C" int32_t qp_controller_observe(qp_controller_t* c, double bytes_sent, double seconds, int32_t* h_bits_out,
                                         int32_t* h_decided_out)
{
    if (!c || !h_bits_out || !(bytes_sent >= 0.0) || !(seconds >= 0.0) || c->window < 1) return QP_ERR_INVALID_ARG;
    if (h_decided_out) *h_decided_out = 0;
    c->sum_bytes += bytes_sent;
    c->sum_seconds += seconds;
    c->count += 1;
    *h_bits_out = c->bits;
    if (c->count < c->window) return QP_OK;
    // window closed: average bandwidth of the window
    const double bw = c->sum_seconds > 0.0 ? 8.0 * c->sum_bytes / c->sum_seconds : 0.0;
    c->count = 0;
    c->sum_bytes = 0.0;
    c->sum_seconds = 0.0;
    if (!(bw > 0.0)) return QP_OK;                               // nothing was measured
    if (c->ref_bandwidth_bps > 0.0 && fabs(bw - c->ref_bandwidth_bps) <= c->rel_change * c->ref_bandwidth_bps)
        return QP_OK;                                            // no significant change
    int32_t rc, q = c->bits;
    if (c->mode == QP_CTRL_EQ2) {
        rc = qp_select_bits_eq2((double)qp_controller_payload_bytes(c, c->bits), c->bits, c->s_images,
                                c->r_images_per_s, bw, &q);
    } else {
        rc = qp_select_bits(bw, c->s_images / c->r_images_per_s, c->n_elems, c->overhead_bytes, c->allowed,
                            c->n_allowed, &q);
    }
    if (rc < 0) return rc;
    c->ref_bandwidth_bps = bw;
    c->bits = q;
    *h_bits_out = q;
    if (h_decided_out) *h_decided_out = 1;
    return rc;
}

// ------------------------------------------------ device-taking entry points

static int32_t check_x(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (dtype != QP_F32 && dtype != QP_BF16) return qp_fail(ctx, QP_ERR_UNSUPPORTED_DTYPE, "dtype must be QP_F32 or QP_BF16");
    if (n > 0 && !d_x) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null tensor");
    const uintptr_t a = dtype == QP_F32 ? 3u : 1u;
    if ((uintptr_t)d_x & a) return qp_fail(ctx, QP_ERR_ALIGNMENT, "tensor not aligned to its element size");
    if (n >= (1ull << 40)) return qp_fail(ctx, QP_ERR_INVALID_ARG, "n too large");
    return QP_OK;
}

// ------------------------------------------- optional graph replay of the multi-kernel calls
//
// A call such as qp_dsaciq_search enqueues up to nine small kernels; at the sizes of the
// paper's micro-batches the gaps between them are a visible share of its time.  With replay
// switched on, the first call with a given argument set records its kernels into a CUDA graph
// (stream capture on the caller's stream), and every later call with the same arguments
// launches the stored graph instead.  Calls on the legacy default stream, or on a stream the
// caller is itself capturing, are enqueued directly as before.
template <typename F>
static int32_t qp_graphed(qp_ctx* ctx, cudaStream_t stream, const unsigned long long (&key)[QP_GRAPH_KEY_WORDS], F&& enqueue)
{
    if (!ctx->graphs_on || stream == nullptr || stream == cudaStreamLegacy || stream == cudaStreamPerThread)
        return enqueue();
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) {
        cudaGetLastError();
        return enqueue();
    }
    ++ctx->graph_clock;
    for (int i = 0; i < ctx->n_graphs; ++i) {
        qp_graph_entry& e = ctx->graphs[i];
        if (memcmp(e.key, key, sizeof key) != 0) continue;
        if (cudaGraphLaunch(e.exec, stream) != cudaSuccess) return qp_check_launch(ctx, "graph replay");
        e.used = ctx->graph_clock;
        ctx->launches += e.launches;
        ++ctx->graph_hits;
        return e.rc;
    }
    if (cudaStreamBeginCapture(stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
        cudaGetLastError();
        return enqueue();
    }
    const unsigned long long before = ctx->launches;
    const int32_t rc = enqueue();
    cudaGraph_t graph = nullptr;
    const cudaError_t ce = cudaStreamEndCapture(stream, &graph);
    const unsigned recorded = (unsigned)(ctx->launches - before);
    ctx->launches = before;                                  // nothing has run yet
    if (rc < 0) {                                            // the call refused its arguments: nothing is enqueued
        if (graph) cudaGraphDestroy(graph);
        cudaGetLastError();
        return rc;
    }
    cudaGraphExec_t exec = nullptr;
    if (ce != cudaSuccess || !graph || cudaGraphInstantiate(&exec, graph, 0) != cudaSuccess) {
        if (graph) cudaGraphDestroy(graph);
        cudaGetLastError();
        return enqueue();                                    // recording failed: run the call the plain way
    }
    cudaGraphDestroy(graph);
    int slot = ctx->n_graphs;
    if (slot == QP_GRAPH_SLOTS) {                            // full: drop the entry unused for longest
        slot = 0;
        for (int i = 1; i < QP_GRAPH_SLOTS; ++i)
            if (ctx->graphs[i].used < ctx->graphs[slot].used) slot = i;
        cudaGraphExecDestroy(ctx->graphs[slot].exec);
    } else {
        ++ctx->n_graphs;
    }
    qp_graph_entry& e = ctx->graphs[slot];
    memcpy(e.key, key, sizeof key);
    e.exec = exec;
    e.launches = recorded;
    e.rc = rc;
    e.used = ctx->graph_clock;
    if (cudaGraphLaunch(exec, stream) != cudaSuccess) return qp_check_launch(ctx, "graph launch");
    ctx->launches += recorded;
    return rc;
}

static void qp_drop_graphs(qp_ctx* ctx)
{
    for (int i = 0; i < ctx->n_graphs; ++i) cudaGraphExecDestroy(ctx->graphs[i].exec);
    ctx->n_graphs = 0;
}

extern "C" int32_t qp_set_graph_replay(qp_ctx* ctx, int on)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (on != 0 && on != 1) return qp_fail(ctx, QP_ERR_INVALID_ARG, "on must be 0 or 1");
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    if (!on) qp_drop_graphs(ctx);
    ctx->graphs_on = on;
    return QP_OK;
}

extern "C" uint64_t qp_graph_replays(qp_ctx* ctx) { return ctx ? ctx->graph_hits : 0; }

extern "C" int32_t qp_stats(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, int hist_bins, qp_stats_t* d_out,
                            void* stream)
{
    int32_t rc = check_x(ctx, d_x, dtype, n);
    if (rc) return rc;
    if (hist_bins < 0 || hist_bins > QP_MAX_HIST_BINS) return qp_fail(ctx, QP_ERR_INVALID_ARG, "hist_bins out of range");
    if (!d_out) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null d_out");
    if ((uintptr_t)d_out & 7u) return qp_fail(ctx, QP_ERR_ALIGNMENT, "d_out must be 8-byte aligned");
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // one word per argument: no two argument sets share a key
    const unsigned long long key[QP_GRAPH_KEY_WORDS] = {1, (unsigned long long)(uintptr_t)d_x, (unsigned long long)dtype, n,
                                                        (unsigned long long)hist_bins, (unsigned long long)(uintptr_t)d_out,
                                                        (unsigned long long)ctx->stats_path};
    ctx->last_x = d_x;                    // the second pass walks backwards (the plain kernels for small tensors do not,
    ctx->last_x_end = 0;                  // but those tensors sit in L2 whole)
    return qp_graphed(ctx, s, key, [&] { return qp_launch_stats(ctx, d_x, dtype, n, hist_bins, d_out, s); });
}

extern "C" int32_t qp_aciq_qparams_device(qp_ctx* ctx, const qp_stats_t* d_stats, int bits, int dist, int bmode,
                                          qp_qparams_t* d_qp_out, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (!d_stats || !d_qp_out) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null pointer");
    if (!qp_bits_ok(bits)) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "bits must be 1..8 or 16");
    if ((dist != QP_DIST_LAPLACE && dist != QP_DIST_GAUSS) || (bmode != QP_B_MAD && bmode != QP_B_MEAN_ABS))
        return qp_fail(ctx, QP_ERR_INVALID_ARG, "dist/bmode");
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    return qp_launch_aciq_device(ctx, d_stats, bits, QP_CLIP_ACIQ, dist, bmode, qp_host_aciq_F(bits, dist), d_qp_out,
                                 static_cast<cudaStream_t>(stream));
}

extern "C" int32_t qp_clip_qparams_device(qp_ctx* ctx, const qp_stats_t* d_stats, int bits, int method, int dist,
                                          int bmode, qp_qparams_t* d_qp_out, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (!d_stats || !d_qp_out) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null pointer");
    if (!qp_bits_ok(bits)) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "bits must be 1..8 or 16");
    if (!clip_method_closed_form(method)) return qp_fail(ctx, QP_ERR_INVALID_ARG, "method must be ACIQ (| INTERSECT) or MINMAX");
    if ((dist != QP_DIST_LAPLACE && dist != QP_DIST_GAUSS) || (bmode != QP_B_MAD && bmode != QP_B_MEAN_ABS))
        return qp_fail(ctx, QP_ERR_INVALID_ARG, "dist/bmode");
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    return qp_launch_aciq_device(ctx, d_stats, bits, method, dist, bmode, qp_host_aciq_F(bits, dist), d_qp_out,
                                 static_cast<cudaStream_t>(stream));
}

extern "C" int32_t qp_dsaciq_search(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, const qp_stats_t* d_stats,
                                    int bits, int bmode, int steps, int hist_bins, qp_ds_result_t* d_out,
                                    qp_qparams_t* d_qp_out, void* stream)
{
    int32_t rc = check_x(ctx, d_x, dtype, n);
    if (rc) return rc;
    if (!d_stats) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null d_stats");
    if (bits < 1 || bits > 8) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "the search supports 1..8 bits");
    {
        const int base = bmode & ~(QP_B_MIDRISE | QP_B_GAUSS | QP_B_HIST_IN_STATS);
        if ((base != QP_B_MAD && base != QP_B_MEAN_ABS) || ((bmode & QP_B_GAUSS) && base != QP_B_MAD))
            return qp_fail(ctx, QP_ERR_INVALID_ARG, "bmode");
    }
    if (steps < 1 || steps > QP_MAX_STEPS) return qp_fail(ctx, QP_ERR_INVALID_ARG, "steps out of range");
    if (hist_bins < 1 || hist_bins > QP_MAX_HIST_BINS) return qp_fail(ctx, QP_ERR_INVALID_ARG, "hist_bins out of range");
    if (((uintptr_t)d_out & 7u) || ((uintptr_t)d_qp_out & 3u)) return qp_fail(ctx, QP_ERR_ALIGNMENT, "result pointers");
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const unsigned long long key[QP_GRAPH_KEY_WORDS] = {
        2, (unsigned long long)(uintptr_t)d_x, n, (unsigned long long)(uintptr_t)d_stats,
        (unsigned long long)(uintptr_t)d_out, (unsigned long long)(uintptr_t)d_qp_out,
        (unsigned long long)dtype | (unsigned long long)bits << 8 | (unsigned long long)ctx->search_path << 16 |
            (unsigned long long)ctx->moments_form << 24,
        (unsigned long long)(unsigned)bmode, (unsigned long long)steps, (unsigned long long)hist_bins};
    rc = qp_graphed(ctx, s, key, [&] {
        return qp_launch_search(ctx, d_x, dtype, n, d_stats, bits, bmode, steps, hist_bins,
                                qp_host_aciq_F(bits, (bmode & QP_B_GAUSS) ? QP_DIST_GAUSS : QP_DIST_LAPLACE), d_out,
                                d_qp_out, s);
    });
    if (rc == QP_OK) { ctx->last_steps = steps; ctx->last_bits = bits; }
    ctx->last_x = d_x;                    // both scoring paths walk x forwards
    ctx->last_x_end = 1;
    return rc;
}

extern "C" int32_t qp_dsaciq_curve(qp_ctx* ctx, double* h_curve, int capacity, void* stream)
{
    if (!ctx || !h_curve) return QP_ERR_INVALID_ARG;
    if (ctx->last_steps < 1) return qp_fail(ctx, QP_ERR_INVALID_ARG, "no search has run on this context");
    if (capacity < ctx->last_steps + 1) return qp_fail(ctx, QP_ERR_BUFFER_TOO_SMALL, "curve buffer");
    qp_device_guard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(h_curve, ctx->d_curve, sizeof(double) * (ctx->last_steps + 1),
                                    cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) {
        snprintf(ctx->err, sizeof ctx->err, "CUDA error in qp_dsaciq_curve: %s", cudaGetErrorString(e));
        return QP_ERR_CUDA;
    }
    return QP_OK;
}

extern "C" int32_t qp_dsaciq_candidates(qp_ctx* ctx, qp_qparams_t* h_out, int capacity, void* stream)
{
    if (!ctx || !h_out) return QP_ERR_INVALID_ARG;
    if (ctx->last_steps < 1) return qp_fail(ctx, QP_ERR_INVALID_ARG, "no search has run on this context");
    const int ncand = ctx->last_steps + 1;
    if (capacity < ncand) return qp_fail(ctx, QP_ERR_BUFFER_TOO_SMALL, "candidate buffer");
    qp_device_guard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    float4* tmp = new (std::nothrow) float4[ncand];
    if (!tmp) return qp_fail(ctx, QP_ERR_CUDA, "out of host memory");
    cudaError_t e = cudaMemcpyAsync(tmp, ctx->d_cand, sizeof(float4) * ncand, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) {
        delete[] tmp;
        snprintf(ctx->err, sizeof ctx->err, "CUDA error in qp_dsaciq_candidates: %s", cudaGetErrorString(e));
        return QP_ERR_CUDA;
    }
    for (int k = 0; k < ncand; ++k) {
        h_out[k].lo = tmp[k].x; h_out[k].hi = tmp[k].y; h_out[k].scale = tmp[k].z; h_out[k].inv_scale = tmp[k].w;
        h_out[k].bits = ctx->last_bits;
        h_out[k].flags = tmp[k].y > tmp[k].x ? 0 : 1;
    }
    delete[] tmp;
    return QP_OK;
}

static int32_t resolve_qp(qp_ctx* ctx, const qp_qparams_t* qp, int qp_on_device, int bits, const qp_qparams_t** d_qp,
                          qp_qparams_t* h_qp)
{
    if (!qp) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null qparams");
    memset(h_qp, 0, sizeof *h_qp);
    if (qp_on_device) {
        if ((uintptr_t)qp & 3u) return qp_fail(ctx, QP_ERR_ALIGNMENT, "device qparams");
        *d_qp = qp;
    } else {
        *d_qp = nullptr;
        *h_qp = *qp;
        if (h_qp->bits != bits) return qp_fail(ctx, QP_ERR_INVALID_ARG, "qparams were made for another bit-width");
    }
    return QP_OK;
}

extern "C" int32_t qp_quantize_pack(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, int bits,
                                    const qp_qparams_t* qp, int qp_on_device, void* d_packed,
                                    uint64_t packed_capacity, void* stream)
{
    int32_t rc = check_x(ctx, d_x, dtype, n);
    if (rc) return rc;
    if (!qp_bits_ok(bits)) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "bits must be 1..8 or 16");
    const uint64_t need = qp_packed_bytes(n, bits);
    if (packed_capacity < need) return qp_fail(ctx, QP_ERR_BUFFER_TOO_SMALL, "packed_capacity < qp_packed_bytes(n, bits)");
    if (need > 0 && !d_packed) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null d_packed");
    if ((uintptr_t)d_packed & 15u) return qp_fail(ctx, QP_ERR_ALIGNMENT, "d_packed must be 16-byte aligned");
    const qp_qparams_t* d_qp;
    qp_qparams_t h_qp;
    rc = resolve_qp(ctx, qp, qp_on_device, bits, &d_qp, &h_qp);
    if (rc) return rc;
    if (n == 0) return QP_OK;
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    return qp_launch_pack(ctx, d_x, dtype, n, bits, d_qp, h_qp, d_packed, static_cast<cudaStream_t>(stream));
}

extern "C" int32_t qp_unpack_dequantize(qp_ctx* ctx, const void* d_packed, uint64_t n, int bits,
                                        const qp_qparams_t* qp, int qp_on_device, void* d_y, int out_dtype,
                                        void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (out_dtype != QP_F32 && out_dtype != QP_BF16) return qp_fail(ctx, QP_ERR_UNSUPPORTED_DTYPE, "out_dtype");
    if (!qp_bits_ok(bits)) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "bits must be 1..8 or 16");
    if (n >= (1ull << 40)) return qp_fail(ctx, QP_ERR_INVALID_ARG, "n too large");
    if (n > 0 && (!d_packed || !d_y)) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null buffer");
    if ((uintptr_t)d_packed & 15u) return qp_fail(ctx, QP_ERR_ALIGNMENT, "d_packed must be 16-byte aligned");
    if ((uintptr_t)d_y & (out_dtype == QP_F32 ? 3u : 1u)) return qp_fail(ctx, QP_ERR_ALIGNMENT, "d_y");
    const qp_qparams_t* d_qp;
    qp_qparams_t h_qp;
    int32_t rc = resolve_qp(ctx, qp, qp_on_device, bits, &d_qp, &h_qp);
    if (rc) return rc;
    if (n == 0) return QP_OK;
    qp_device_guard guard(ctx->device);
    if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
    return qp_launch_unpack(ctx, d_packed, n, bits, d_qp, h_qp, d_y, out_dtype, static_cast<cudaStream_t>(stream));
}

// ------------------------------------------- whole sender on device buffers

// statistics -> clip -> quantize+pack on device buffers: one cooperative launch where that
// applies (small tensors), the kernel chain of the separate calls otherwise
static int32_t sender_on_device(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, int bits, int method, int bmode,
                                int steps, int hist_bins, void* d_packed, uint64_t packed_capacity,
                                qp_qparams_t* d_qp_out, qp_stats_t* st, void* stream)
{
    int32_t rc;
    const int use_ds = (method & 0xF) == QP_CLIP_DSACIQ;
    const int search_mode = bmode | ((method & QP_CLIP_MIDRISE) ? QP_B_MIDRISE : 0);
    if (ctx->sender_path != QP_SENDER_CHAIN &&
        qp_sender_fused_applies(n, use_ds, steps, hist_bins, ctx->sender_path == QP_SENDER_FUSED)) {
        // the checks of the separate calls
        rc = check_x(ctx, d_x, dtype, n);
        if (rc) return rc;
        if (bmode != QP_B_MAD && bmode != QP_B_MEAN_ABS) return qp_fail(ctx, QP_ERR_INVALID_ARG, "bmode");
        if (use_ds && (steps < 1 || hist_bins < 1)) return qp_fail(ctx, QP_ERR_INVALID_ARG, "steps / hist_bins out of range");
        if (!d_packed) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null d_packed");
        if ((uintptr_t)d_packed & 15u) return qp_fail(ctx, QP_ERR_ALIGNMENT, "d_packed must be 16-byte aligned");
        if (((uintptr_t)st & 7u) || ((uintptr_t)d_qp_out & 3u)) return qp_fail(ctx, QP_ERR_ALIGNMENT, "result pointers");
        qp_device_guard guard(ctx->device);
        if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
        rc = qp_launch_sender_fused(ctx, d_x, dtype, n, bits, method, bmode, steps, hist_bins,
                                    qp_host_aciq_F(bits, QP_DIST_LAPLACE), d_packed, d_qp_out, st,
                                    static_cast<cudaStream_t>(stream));
        if (rc == QP_OK && use_ds) { ctx->last_steps = steps; ctx->last_bits = bits; }
        if (rc != QP_WARN_INFEASIBLE) return rc;               // else: this device cannot hold the grid
    }
    rc = qp_stats(ctx, d_x, dtype, n, use_ds ? hist_bins : 0, st, stream);
    if (rc < 0) return rc;
    // the statistics above carry the histogram whenever they can: then the search need not look
    const int in_stats = (use_ds && qp_stats_carries_histogram(d_x, dtype, n, hist_bins)) ? QP_B_HIST_IN_STATS : 0;
    if (use_ds) rc = qp_dsaciq_search(ctx, d_x, dtype, n, st, bits, search_mode | in_stats, steps, hist_bins, nullptr, d_qp_out, stream);
    else        rc = qp_clip_qparams_device(ctx, st, bits, method, QP_DIST_LAPLACE, bmode, d_qp_out, stream);
    if (rc < 0) return rc;
    return qp_quantize_pack(ctx, d_x, dtype, n, bits, d_qp_out, 1, d_packed, packed_capacity, stream);
}

extern "C" int32_t qp_sender_device(qp_ctx* ctx, const void* d_x, int dtype, uint64_t n, int bits, int method, int bmode,
                                    int steps, int hist_bins, void* d_packed, uint64_t packed_capacity,
                                    qp_qparams_t* d_qp_out, qp_stats_t* d_stats_out, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (!d_qp_out) return qp_fail(ctx, QP_ERR_INVALID_ARG, "null d_qp_out");
    if (!qp_bits_ok(bits)) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "bits must be 1..8 or 16");
    if ((method & ~QP_CLIP_MIDRISE) != QP_CLIP_DSACIQ && !clip_method_closed_form(method))
        return qp_fail(ctx, QP_ERR_INVALID_ARG, "clip method");
    if ((method & 0xF) == QP_CLIP_DSACIQ && bits > 8) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "the search supports 1..8 bits");
    if (packed_capacity < qp_packed_bytes(n, bits))
        return qp_fail(ctx, QP_ERR_BUFFER_TOO_SMALL, "packed_capacity < qp_packed_bytes(n, bits)");
    qp_stats_t* st = d_stats_out ? d_stats_out : ctx->d_tmp_stats;
    // The inner calls see a capturing stream while this one records, and enqueue directly into it.
    // Every argument and every context option that the recorded kernels depend on has a word (or a
    // byte of a word whose fields are each below 256) of its own, so that two different calls can
    // never share a key.
    const unsigned long long key[QP_GRAPH_KEY_WORDS] = {
        3, (unsigned long long)(uintptr_t)d_x, n, (unsigned long long)(uintptr_t)d_packed, packed_capacity,
        (unsigned long long)(uintptr_t)d_qp_out, (unsigned long long)(uintptr_t)st,
        (unsigned long long)dtype | (unsigned long long)bits << 8 | (unsigned long long)ctx->search_path << 16 |
            (unsigned long long)ctx->moments_form << 24 | (unsigned long long)ctx->sender_path << 32 |
            (unsigned long long)ctx->stats_path << 40,
        (unsigned long long)(unsigned)method, (unsigned long long)(unsigned)bmode, (unsigned long long)steps,
        (unsigned long long)hist_bins};
    const int32_t rc = qp_graphed(ctx, static_cast<cudaStream_t>(stream), key, [&]() -> int32_t {
        return sender_on_device(ctx, d_x, dtype, n, bits, method, bmode, steps, hist_bins, d_packed, packed_capacity,
                                d_qp_out, st, stream);
    });
    if (rc >= 0 && (method & 0xF) == QP_CLIP_DSACIQ) { ctx->last_steps = steps; ctx->last_bits = bits; }   // also after a replay
    return rc;
}

// ------------------------------------------- host-buffer sender and receiver

extern "C" int32_t qp_sender_host(qp_ctx* ctx, const void* h_x, int dtype, uint64_t n, int bits, int method, int bmode,
                                  int steps, int hist_bins, void* d_x_work, void* d_packed_work, void* h_packed,
                                  uint64_t packed_capacity, qp_qparams_t* h_qp_out, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (dtype != QP_F32 && dtype != QP_BF16) return qp_fail(ctx, QP_ERR_UNSUPPORTED_DTYPE, "dtype");
    if (!qp_bits_ok(bits)) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "bits must be 1..8 or 16");
    if ((method & ~QP_CLIP_MIDRISE) != QP_CLIP_DSACIQ && !clip_method_closed_form(method))
        return qp_fail(ctx, QP_ERR_INVALID_ARG, "clip method");
    if ((method & 0xF) == QP_CLIP_DSACIQ && bits > 8) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "the search supports 1..8 bits");
    if (!h_qp_out || (n > 0 && (!h_x || !d_x_work || !d_packed_work || !h_packed)))
        return qp_fail(ctx, QP_ERR_INVALID_ARG, "null buffer");
    const uint64_t need = qp_packed_bytes(n, bits);
    if (packed_capacity < need) return qp_fail(ctx, QP_ERR_BUFFER_TOO_SMALL, "packed_capacity < qp_packed_bytes(n, bits)");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t esz = dtype == QP_F32 ? 4 : 2;
    {
        qp_device_guard guard(ctx->device);
        if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
        if (n && cudaMemcpyAsync(d_x_work, h_x, n * esz, cudaMemcpyHostToDevice, s) != cudaSuccess)
            return qp_check_launch(ctx, "qp_sender_host (copy in)");
    }
    int32_t rc = sender_on_device(ctx, d_x_work, dtype, n, bits, method, bmode, steps, hist_bins, d_packed_work, need,
                                  ctx->d_tmp_qp, ctx->d_tmp_stats, stream);
    if (rc < 0) return rc;
    qp_device_guard guard(ctx->device);
    cudaError_t e = cudaSuccess;
    if (need) e = cudaMemcpyAsync(h_packed, d_packed_work, need, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h_qp_out, ctx->d_tmp_qp, sizeof(qp_qparams_t), cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return qp_check_launch(ctx, "qp_sender_host (copy out)");
    return QP_OK;
}

extern "C" int32_t qp_receiver_host(qp_ctx* ctx, const void* h_packed, uint64_t n, int bits, const qp_qparams_t* h_qp,
                                    void* d_packed_work, void* d_y_work, void* h_y, int out_dtype, void* stream)
{
    if (!ctx) return QP_ERR_INVALID_ARG;
    if (out_dtype != QP_F32 && out_dtype != QP_BF16) return qp_fail(ctx, QP_ERR_UNSUPPORTED_DTYPE, "out_dtype");
    if (!qp_bits_ok(bits)) return qp_fail(ctx, QP_ERR_UNSUPPORTED_BITS, "bits must be 1..8 or 16");
    if (!h_qp || (n > 0 && (!h_packed || !d_packed_work || !d_y_work || !h_y)))
        return qp_fail(ctx, QP_ERR_INVALID_ARG, "null buffer");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const uint64_t need = qp_packed_bytes(n, bits);
    {
        qp_device_guard guard(ctx->device);
        if (!guard.ok) return qp_fail(ctx, QP_ERR_CUDA, "cannot select device");
        if (need && cudaMemcpyAsync(d_packed_work, h_packed, need, cudaMemcpyHostToDevice, s) != cudaSuccess)
            return qp_check_launch(ctx, "qp_receiver_host (copy in)");
    }
    const int32_t rc = qp_unpack_dequantize(ctx, d_packed_work, n, bits, h_qp, 0, d_y_work, out_dtype, stream);
    if (rc < 0) return rc;
    qp_device_guard guard(ctx->device);
    const size_t esz = out_dtype == QP_F32 ? 4 : 2;
    if (n && cudaMemcpyAsync(h_y, d_y_work, n * esz, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return qp_check_launch(ctx, "qp_receiver_host (copy out)");
    return QP_OK;
}

// Host-side plumbing of the C ABI: status strings, thread-local error text,
// argument helpers, the batch-norm fold.
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <atomic>
#include <climits>
#include <cstdlib>
#include "qnn_internal.cuh"

namespace qnn {

static thread_local char g_err[512] = "";
static std::atomic<uint64_t> g_launches{0};

int fail(int code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

void clear_error() { g_err[0] = 0; }

void note(const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

bool pdl_enabled()
{
    static const bool on = [] { const char *e = getenv("QNN_PDL"); return !(e && e[0] == '0'); }();
    return on;
}
void profile_arm(cudaEvent_t a, cudaEvent_t b, int skip);

int check_launch(const char *what)
{
    g_launches.fetch_add(1, std::memory_order_relaxed);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(QNN_ERR_CUDA, "%s: launch failed: %s", what, cudaGetErrorString(e));
    return QNN_OK;
}

static thread_local cudaEvent_t g_ev_start = nullptr, g_ev_stop = nullptr;
static thread_local int g_ev_skip = 0;          // product kernels to let pass before the armed one

void profile_before(cudaStream_t st)
{
    if (g_ev_start && g_ev_skip == 0) cudaEventRecord(g_ev_start, st);
}
void profile_after(cudaStream_t st)
{
    if (!g_ev_start) return;
    if (g_ev_skip > 0) { --g_ev_skip; return; }
    if (g_ev_stop) cudaEventRecord(g_ev_stop, st);
    g_ev_start = g_ev_stop = nullptr;
}
void profile_arm(cudaEvent_t a, cudaEvent_t b, int skip) { g_ev_start = a; g_ev_stop = b; g_ev_skip = skip; }

int sm_count()
{
    static thread_local int cached_dev = -1;
    static thread_local int cached = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (dev != cached_dev) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached = n;
        cached_dev = dev;
    }
    return cached;
}

}  // namespace qnn

extern "C" {

int qnn_version(void) { return QNN_VERSION; }

int qnn_set_kernel_events(void *start, void *stop)
{
    QNN_REQUIRE((start == nullptr) == (stop == nullptr), QNN_ERR_INVALID_ARG, "qnn_set_kernel_events: pass both events or neither");
    qnn::profile_arm(static_cast<cudaEvent_t>(start), static_cast<cudaEvent_t>(stop), 0);
    return QNN_OK;
}

int qnn_set_kernel_events_nth(void *start, void *stop, int nth)
{
    QNN_REQUIRE((start == nullptr) == (stop == nullptr), QNN_ERR_INVALID_ARG, "qnn_set_kernel_events_nth: pass both events or neither");
    QNN_REQUIRE(nth >= 0, QNN_ERR_INVALID_ARG, "qnn_set_kernel_events_nth: nth is negative");
    qnn::profile_arm(static_cast<cudaEvent_t>(start), static_cast<cudaEvent_t>(stop), nth);
    return QNN_OK;
}

const char *qnn_status_string(int status)
{
    switch (status) {
        case QNN_OK: return "ok";
        case QNN_ERR_INVALID_ARG: return "invalid argument";
        case QNN_ERR_ALIGNMENT: return "misaligned pointer or leading dimension";
        case QNN_ERR_UNSUPPORTED: return "unsupported request";
        case QNN_ERR_OVERFLOW: return "result may overflow int32";
        case QNN_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case QNN_ERR_CUDA: return "CUDA runtime error";
        case QNN_ERR_TIMEOUT: return "bounded device-side wait ran out";
        default: return "unknown status";
    }
}

const char *qnn_last_error(void) { return qnn::g_err; }

uint64_t qnn_launch_count(void) { return qnn::g_launches.load(std::memory_order_relaxed); }

int qnn_fold_bn(const double *gamma, const double *beta, const double *mean, const double *var,
                double eps, int64_t N, int32_t *thr_host, uint8_t *flip_host)
{
    QNN_REQUIRE(gamma && beta && mean && var && thr_host && flip_host, QNN_ERR_INVALID_ARG,
                "qnn_fold_bn: NULL argument");
    QNN_REQUIRE(N >= 0 && eps >= 0.0, QNN_ERR_INVALID_ARG, "qnn_fold_bn: N or eps negative");
    for (int64_t n = 0; n < N; ++n) {
        QNN_REQUIRE(var[n] + eps > 0.0, QNN_ERR_INVALID_ARG, "qnn_fold_bn: var[%lld] + eps is not positive",
                    (long long)n);
        const double sigma = std::sqrt(var[n] + eps);
        double t;
        uint8_t f;
        if (gamma[n] > 0.0) {
            t = std::ceil(mean[n] - beta[n] * sigma / gamma[n]);
            f = 0;
        } else if (gamma[n] < 0.0) {
            t = std::floor(mean[n] - beta[n] * sigma / gamma[n]) + 1.0;
            f = 1;
        } else {
            t = (double)INT32_MIN;
            f = (uint8_t)(beta[n] < 0.0);
        }
        if (!(t >= (double)INT32_MIN)) t = (double)INT32_MIN;   // also catches NaN
        if (t > (double)INT32_MAX) t = (double)INT32_MAX;
        thr_host[n] = (int32_t)t;
        flip_host[n] = f;
    }
    return QNN_OK;
}

}  // extern "C"

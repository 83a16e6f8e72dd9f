// Host-side state of the tilelens library: per-device control block and workspace, per-thread stream and caller
// workspace, the process-wide option table, error reporting.
#include "tl_common.cuh"

#include <cstdlib>
#include <mutex>

namespace tl {

namespace {

std::recursive_mutex& api_mutex() {
    static std::recursive_mutex m;
    return m;
}

struct Options {
    int64_t v[TL_OPT_COUNT_];
    Options() {
        set_defaults();
        // Initial values may come from the environment (read once, when the library is first used), so that a
        // measurement script can flip a switch without touching the program it runs.
        static const struct { const char* name; int id; int invert; } env[] = {
            {"TL_NO_PDL", TL_OPT_PDL, 1},           {"TL_PREFETCH_STAGES", TL_OPT_PREFETCH_STAGES, 0},
            {"TL_NO_PAIR", TL_OPT_PAIR_KERNEL, 1},  {"TL_BOX_PER_BLOCK", TL_OPT_BOX_PER_BLOCK, 0},
            {"TL_MAX_STAGES", TL_OPT_MAX_STAGES, 0}, {"TL_UMMA_M128", TL_OPT_UMMA_M128, 0},
            {"TL_RELAYOUT_NO_TMA", TL_OPT_RELAYOUT_TMA, 1}, {"TL_LOG", TL_OPT_LOG, 0},
        };
        for (const auto& e : env)
            if (const char* s = getenv(e.name)) v[e.id] = e.invert ? (atoi(s) != 0 ? 0 : 1) : atoi(s);
        if (const char* s = getenv("TL_PAIR_HALVES")) v[TL_OPT_PAIR_512] = atoi(s) == 1 ? 0 : 1;
    }
    void set_defaults() {
        for (auto& x : v) x = 0;
        v[TL_OPT_PDL] = 1;
        v[TL_OPT_PREFETCH_STAGES] = -1;
        v[TL_OPT_PAIR_KERNEL] = 1;
        v[TL_OPT_PAIR_512] = 1;
        v[TL_OPT_RELAYOUT_TMA] = 1;
        v[TL_OPT_WAIT_LIMIT_US] = 2000000;
        v[TL_OPT_MOE_ROW_CAP] = 0;
        v[TL_OPT_REDUCE_SPLIT] = 1;
        v[TL_OPT_NO_SCRATCH_PLANS] = 1;
        v[TL_OPT_PAIR_TMA_STORE] = 1;
        v[TL_OPT_GENERIC_RAW] = 1;
    }
};

Options& options() {
    static Options o;
    return o;
}

DeviceState g_devices[kMaxDevices];

}  // namespace

ApiLock::ApiLock() { api_mutex().lock(); }
ApiLock::~ApiLock() { api_mutex().unlock(); }

ThreadState& tls() {
    static thread_local ThreadState t;
    return t;
}

DeviceState& dev() {
    if (opt(TL_OPT_PLAN_AS_IF_SMS)) return g_devices[0];        // test hook: see ensure_device_info
    int d = 0;
    if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= kMaxDevices) {
        (void)cudaGetLastError();
        d = 0;
    }
    return g_devices[d];
}

int64_t opt(int option) { return option >= 0 && option < TL_OPT_COUNT_ ? options().v[option] : 0; }

uint64_t wait_limit_ns() {
    const int64_t us = opt(TL_OPT_WAIT_LIMIT_US);
    return uint64_t(us > 0 ? us : 1) * 1000ull;
}

int check_cuda(cudaError_t err) {
    if (err == cudaSuccess) return TL_OK;
    tls().last_cuda_error = static_cast<int>(err);
    (void)cudaGetLastError();   // clear the sticky-less error so later calls start clean
    return TL_ERR_CUDA;
}

int ensure_device_info() {
    if (const int64_t fake = opt(TL_OPT_PLAN_AS_IF_SMS)) {      // test hook: no CUDA call at all
        DeviceState& s = g_devices[0];
        if (s.sm_count != int(fake)) {
            s.sm_count = int(fake);
            s.pair_max_clusters = int(fake) / 2;
            static const int b200[9] = {0, 0, 74, 45, 33, 26, 22, 15, 15};
            for (int c = 2; c <= 8; ++c) s.cluster_cap[c] = fake == 148 ? b200[c] : (int(fake) / c > 0 ? int(fake) / c : -1);
        }
        return TL_OK;
    }
    int d = -1;
    if (int rc = check_cuda(cudaGetDevice(&d))) return rc;
    if (d < 0 || d >= kMaxDevices) return TL_ERR_UNSUPPORTED;
    DeviceState& s = g_devices[d];
    if (s.sm_count > 0) return TL_OK;
    int sms = 0;
    if (int rc = check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, d))) return rc;
    s.sm_count = sms;
    return TL_OK;
}

int ensure_control() {
    if (int rc = ensure_device_info()) return rc;
    DeviceState& s = dev();
    if (s.ctl.d_status) return TL_OK;
    void* p = nullptr;
    if (int rc = check_cuda(cudaMalloc(&p, 1024))) return rc;
    if (int rc = check_cuda(cudaMemset(p, 0, 1024))) return rc;
    void* h = nullptr;
    if (int rc = check_cuda(cudaHostAlloc(&h, 64, cudaHostAllocMapped))) return rc;
    void* h_dev = nullptr;
    if (int rc = check_cuda(cudaHostGetDevicePointer(&h_dev, h, 0))) return rc;
    s.ctl.d_status = static_cast<uint32_t*>(p);
    s.ctl.d_acc = reinterpret_cast<unsigned long long*>(static_cast<char*>(p) + 64);
    s.d_grid_counter = reinterpret_cast<unsigned long long*>(static_cast<char*>(p) + 960);   // after the 17 x 32 bytes of accumulators
    s.grid_arrivals = 0;
    s.ctl.h_acc = static_cast<unsigned long long*>(h);
    s.ctl.h_acc_dev = static_cast<unsigned long long*>(h_dev);
    return TL_OK;
}

int ensure_smem_attr(const void* kernel, int bytes) {
    DeviceState& s = dev();
    for (int i = 0; i < s.smem_attr_n; ++i)
        if (s.smem_attr_done[i] == kernel) return TL_OK;
    if (int rc = check_cuda(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes))) return rc;
    if (s.smem_attr_n < int(sizeof(s.smem_attr_done) / sizeof(s.smem_attr_done[0]))) s.smem_attr_done[s.smem_attr_n++] = kernel;
    return TL_OK;
}

bool stream_is_capturing(cudaStream_t stream) {
    cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &st) != cudaSuccess) {
        (void)cudaGetLastError();
        return true;                                      // a capture gone wrong: treat like one in progress
    }
    return st != cudaStreamCaptureStatusNone;
}

int get_workspace(size_t bytes, void** out, cudaStream_t stream) {
    if (bytes == 0) {
        *out = nullptr;
        return TL_OK;
    }
    ThreadState& t = tls();
    if (t.user_ws) {
        if (t.user_ws_bytes < bytes) return TL_ERR_WORKSPACE;
        *out = t.user_ws;
        return TL_OK;
    }
    // A captured launch would keep this address in its graph, while the internal buffer is replaced whenever a later
    // call needs a larger one (and growing it synchronises and allocates, which a capture forbids).
    if (stream_is_capturing(stream)) return TL_ERR_WORKSPACE;
    DeviceState& s = dev();
    if (s.own_ws_bytes < bytes) {
        // Work already enqueued may still use the old buffer: wait before replacing it.
        if (s.own_ws) {
            if (int rc = check_cuda(cudaDeviceSynchronize())) return rc;
            if (int rc = check_cuda(cudaFree(s.own_ws))) return rc;
            s.own_ws = nullptr;
            s.own_ws_bytes = 0;
        }
        size_t want = bytes + (bytes >> 2);
        void* p = nullptr;
        if (int rc = check_cuda(cudaMalloc(&p, want))) return rc;
        s.own_ws = p;
        s.own_ws_bytes = want;
    }
    *out = s.own_ws;
    return TL_OK;
}

}  // namespace tl

extern "C" {

const char* tl_status_string(int status) {
    switch (status) {
        case TL_OK: return "TL_OK";
        case TL_ERR_INVALID_ARG: return "TL_ERR_INVALID_ARG: bad pointer, size, block shape or divisibility";
        case TL_ERR_UNSUPPORTED: return "TL_ERR_UNSUPPORTED: valid request outside the instantiated kernels";
        case TL_ERR_ALIGNMENT: return "TL_ERR_ALIGNMENT: pointer or pitch misaligned";
        case TL_ERR_CUDA: return "TL_ERR_CUDA: a CUDA call failed (see tl_last_cuda_error)";
        case TL_ERR_TIMEOUT: return "TL_ERR_TIMEOUT: a bounded device-side wait expired";
        case TL_ERR_WORKSPACE: return "TL_ERR_WORKSPACE: caller-supplied workspace too small";
        default: return "unknown tl_status";
    }
}

int tl_last_cuda_error(void) { return tl::tls().last_cuda_error; }

int tl_set_stream(void* cuda_stream) {
    tl::tls().stream = static_cast<cudaStream_t>(cuda_stream);
    return TL_OK;
}

int tl_set_workspace(void* d_ptr, size_t bytes) {
    tl::ThreadState& t = tl::tls();
    if (d_ptr == nullptr) {
        t.user_ws = nullptr;
        t.user_ws_bytes = 0;
        return TL_OK;
    }
    if (reinterpret_cast<uintptr_t>(d_ptr) % 256 != 0) return TL_ERR_ALIGNMENT;
    t.user_ws = d_ptr;
    t.user_ws_bytes = bytes;
    return TL_OK;
}

int tl_set_option(int option, int64_t value) {
    tl::ApiLock lock;
    if (option < 0 || option >= TL_OPT_COUNT_) return TL_ERR_INVALID_ARG;
    switch (option) {
        case TL_OPT_PREFETCH_STAGES: if (value < -1 || value > 16) return TL_ERR_INVALID_ARG; break;
        case TL_OPT_MAX_STAGES: if (value != 0 && (value < 2 || value > 16)) return TL_ERR_INVALID_ARG; break;
        case TL_OPT_WAIT_LIMIT_US: if (value < 100 || value > 60000000) return TL_ERR_INVALID_ARG; break;
        case TL_OPT_STALL_ONCE: if (value < 0 || value > 4) return TL_ERR_INVALID_ARG; break;
        case TL_OPT_SM_LIMIT: if (value < 0 || value > 4096) return TL_ERR_INVALID_ARG; break;
        case TL_OPT_PLAN_AS_IF_SMS: if (value < 0 || value > 4096) return TL_ERR_INVALID_ARG; break;
        case TL_OPT_MOE_ROW_CAP: if (value != 0 && value != 16 && value != 32 && value != 64 && value != 128) return TL_ERR_INVALID_ARG; break;
        case TL_OPT_FFN_ONE_LAUNCH: if (value < 0 || value > 2) return TL_ERR_INVALID_ARG; break;
        default: if (value != 0 && value != 1) return TL_ERR_INVALID_ARG; break;
    }
    if (option == TL_OPT_PLAN_AS_IF_SMS && tl::options().v[option] != value) {
        // entering or leaving the hook: slot 0 forgets the SM count and the cluster numbers it held
        tl::g_devices[0].sm_count = 0;
        tl::g_devices[0].pair_max_clusters = -1;
        for (int& c : tl::g_devices[0].cluster_cap) c = 0;
    }
    tl::options().v[option] = value;
    return TL_OK;
}

int64_t tl_get_option(int option) {
    tl::ApiLock lock;
    if (option < 0 || option >= TL_OPT_COUNT_) return -1;
    return tl::options().v[option];
}

int tl_device_status(uint32_t* detail) {
    tl::ApiLock lock;
    if (int rc = tl::ensure_control()) return rc;
    if (int rc = tl::check_cuda(cudaDeviceSynchronize())) return rc;
    uint32_t word = 0;
    if (int rc = tl::check_cuda(cudaMemcpy(&word, tl::dev().ctl.d_status, 4, cudaMemcpyDeviceToHost))) return rc;
    if (detail) *detail = word;
    if (word == 0) return TL_OK;
    if (int rc = tl::check_cuda(cudaMemset(tl::dev().ctl.d_status, 0, 4))) return rc;
    // a kernel that gave up may have left the grid barrier's counter short of what later launches would wait for
    if (int rc = tl::check_cuda(cudaMemset(tl::dev().d_grid_counter, 0, 8))) return rc;
    tl::dev().grid_arrivals = 0;
    return TL_ERR_TIMEOUT;
}

}  // extern "C"

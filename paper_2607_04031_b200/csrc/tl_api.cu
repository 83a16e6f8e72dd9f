// Host-side state of the tilelens library: stream, workspace, control block, error reporting.
#include "tl_common.cuh"


namespace tl {

State& state() {
    static State s;
    return s;
}

int check_cuda(cudaError_t err) {
    if (err == cudaSuccess) return TL_OK;
    state().last_cuda_error = static_cast<int>(err);
    (void)cudaGetLastError();   // clear the sticky-less error so later calls start clean
    return TL_ERR_CUDA;
}

int ensure_device_info() {
    State& s = state();
    int dev = -1;
    if (int rc = check_cuda(cudaGetDevice(&dev))) return rc;
    if (dev == s.device && s.sm_count > 0) return TL_OK;
    int sms = 0;
    if (int rc = check_cuda(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev))) return rc;
    s.device = dev;
    s.sm_count = sms;
    return TL_OK;
}

int ensure_control() {
    State& s = state();
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
    s.ctl.h_acc = static_cast<unsigned long long*>(h);
    s.ctl.h_acc_dev = static_cast<unsigned long long*>(h_dev);
    return TL_OK;
}

int get_workspace(size_t bytes, void** out) {
    State& s = state();
    if (bytes == 0) {
        *out = nullptr;
        return TL_OK;
    }
    if (s.user_ws) {
        if (s.user_ws_bytes < bytes) return TL_ERR_WORKSPACE;
        *out = s.user_ws;
        return TL_OK;
    }
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

int tl_last_cuda_error(void) { return tl::state().last_cuda_error; }

int tl_set_stream(void* cuda_stream) {
    tl::state().stream = static_cast<cudaStream_t>(cuda_stream);
    return TL_OK;
}

int tl_set_workspace(void* d_ptr, size_t bytes) {
    tl::State& s = tl::state();
    if (d_ptr == nullptr) {
        s.user_ws = nullptr;
        s.user_ws_bytes = 0;
        return TL_OK;
    }
    if (reinterpret_cast<uintptr_t>(d_ptr) % 256 != 0) return TL_ERR_ALIGNMENT;
    s.user_ws = d_ptr;
    s.user_ws_bytes = bytes;
    return TL_OK;
}

int tl_device_status(uint32_t* detail) {
    if (int rc = tl::ensure_control()) return rc;
    if (int rc = tl::check_cuda(cudaDeviceSynchronize())) return rc;
    uint32_t word = 0;
    if (int rc = tl::check_cuda(cudaMemcpy(&word, tl::state().ctl.d_status, 4, cudaMemcpyDeviceToHost))) return rc;
    if (detail) *detail = word;
    if (word == 0) return TL_OK;
    if (int rc = tl::check_cuda(cudaMemset(tl::state().ctl.d_status, 0, 4))) return rc;
    return TL_ERR_TIMEOUT;
}

}  // extern "C"

// beagle_verify_greedy_static: greedy acceptance from target logits for callers that cannot hand
// the library any scratch memory.  The arg-max partial keys and the per-row ids live in one
// file-scope device array instead of a caller-provided workspace.
#include <cstdio>
#include <mutex>

#include "../../include/beagle.h"
#include "kernels.h"

using namespace beagle;

namespace {

constexpr int kStaticMaxRows = BEAGLE_STATIC_VERIFY_MAX_ROWS;
constexpr size_t kKeysBytes = (size_t)kStaticMaxRows * kRowArgmaxSplit * sizeof(unsigned long long);
constexpr size_t kIdsBytes = (size_t)kStaticMaxRows * sizeof(int32_t);
constexpr size_t kScratchBytes = kKeysBytes + kIdsBytes;

// Every GPU that loads the library holds this array (about 0.55 MB) until the process exits.
// In host code the NAME below is only a host-side handle of the symbol, not a device address:
// the address kernels may use comes from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_static_verify_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};

void set_error(char* buf, size_t len, const char* fmt, long long a = 0, long long b = 0) {
    if (buf != nullptr && len > 0) snprintf(buf, len, fmt, a, b);
}

// Device address of the scratch array on the CURRENT device (looked up on the first call there).
beagle_status scratch_address(void** out, char* err, size_t err_len) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        set_error(err, err_len, "verify_greedy_static: cannot identify the current device (cuda error %lld)", (long long)e);
        return BEAGLE_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_verify_scratch);
        if (e != cudaSuccess || p == nullptr) {
            set_error(err, err_len, "verify_greedy_static: cudaGetSymbolAddress failed on device %lld (cuda error %lld)", dev, (long long)e);
            return BEAGLE_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return BEAGLE_OK;
}

}  // namespace

extern "C" beagle_status beagle_verify_greedy_static(int32_t batch, int32_t gamma, int32_t vocab,
                                                     const int32_t* draft_tokens_dev, const void* target_logits_dev,
                                                     int32_t logits_dtype, int32_t* accept_len_dev,
                                                     int32_t* out_tokens_dev, void* stream_, char* err_buf,
                                                     size_t err_len) {
    if (err_buf != nullptr && err_len > 0) err_buf[0] = '\0';
    if (batch < 0 || gamma < 0 || vocab <= 0) {
        set_error(err_buf, err_len, "verify_greedy_static: batch and gamma must be >= 0 and vocab > 0");
        return BEAGLE_ERR_INVALID_ARG;
    }
    const long long rows = (long long)batch * ((long long)gamma + 1);
    if (rows > kStaticMaxRows) {
        set_error(err_buf, err_len,
                  "verify_greedy_static: batch*(gamma+1) = %lld logit rows exceed the built-in scratch of %lld rows; "
                  "use beagle_verify_greedy with a caller-provided workspace",
                  rows, (long long)kStaticMaxRows);
        return BEAGLE_ERR_CAPACITY;
    }
    if (logits_dtype != BEAGLE_FP32 && logits_dtype != BEAGLE_BF16) {
        set_error(err_buf, err_len, "verify_greedy_static: unknown logits_dtype");
        return BEAGLE_ERR_INVALID_ARG;
    }
    if (batch == 0) return BEAGLE_OK;
    if ((gamma > 0 && draft_tokens_dev == nullptr) || target_logits_dev == nullptr || accept_len_dev == nullptr ||
        out_tokens_dev == nullptr) {
        set_error(err_buf, err_len, "verify_greedy_static: NULL argument");
        return BEAGLE_ERR_INVALID_ARG;
    }
    void* scratch = nullptr;
    const beagle_status st = scratch_address(&scratch, err_buf, err_len);
    if (st != BEAGLE_OK) return st;
    // Nothing in the scratch has to start at zero: the partial pass writes every key of every row
    // it is given and the final pass reads only those, so the previous call's contents are dead.
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(scratch);
    int32_t* ids = reinterpret_cast<int32_t*>(static_cast<unsigned char*>(scratch) + kKeysBytes);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    launch_row_argmax(logits_dtype, target_logits_dev, (int)rows, vocab, keys, ids, stream);
    launch_accept(draft_tokens_dev, ids, batch, gamma, accept_len_dev, out_tokens_dev, stream);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_error(err_buf, err_len, "verify_greedy_static: launch failed (cuda error %lld)", (long long)e);
        return BEAGLE_ERR_CUDA;
    }
    return BEAGLE_OK;
}

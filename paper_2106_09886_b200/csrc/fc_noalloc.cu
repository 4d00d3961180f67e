// qnn_fc_forward_noalloc: one fully-connected layer (encode + contraction) whose only intermediate,
// the activation bit planes, lives in a buffer built into the library instead of one the caller allocates.
//
// Who needs this: code that is handed an input and an output pointer and nothing else -- a plug-in
// callback inside a host framework that owns all device memory and forbids its plug-ins to allocate,
// a hard-real-time control loop whose memory was fixed at start-up, a C program that links the library
// but carries no allocator of its own.  Such callers cannot provide the planes buffer that
// qnn_encode_pack + qnn_bgemm need between them, because they cannot call cudaMalloc (or any pool
// that might call it) at that point.
#include <mutex>

#include "qnn_internal.cuh"

namespace {

constexpr size_t kScratchWords = QNN_NOALLOC_SCRATCH_BYTES / sizeof(uint32_t);

// The built-in planes buffer.  Every GPU that loads the library carries these 8 MiB until the process ends.
// In host code this name is only a handle for the runtime, not a device address: the address a kernel
// can use is obtained once per device with cudaGetSymbolAddress below.
static __device__ __align__(256) uint32_t g_planes_scratch[kScratchWords];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
uint32_t *g_scratch_ptr[kMaxDevices] = {};   // device address of g_planes_scratch, per device ordinal

// Returns the device address of the scratch buffer on the current device, resolving it on first use.
int scratch_for_current_device(uint32_t **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return QNN_E_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_ptr[dev] == nullptr) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_planes_scratch) != cudaSuccess || p == nullptr) {
            (void)cudaGetLastError();
            return QNN_E_CUDA;
        }
        g_scratch_ptr[dev] = static_cast<uint32_t *>(p);
    }
    *out = g_scratch_ptr[dev];
    return QNN_OK;
}

}  // namespace

extern "C" int qnn_fc_forward_noalloc(const float *x, int64_t Mg, int Kg, int64_t ldx, int ab, float scale_a,
                                      unsigned flags, const void *w_packed, int wb, int Ng, float alpha, float *out,
                                      int64_t ldo, void *stream) {
    if (!x || !w_packed || !out || Mg <= 0 || Kg <= 0 || Ng <= 0 || !qnn_bits_ok(ab) || !qnn_bits_ok(wb))
        return QNN_E_ARG;
    // the planes of this problem must fit the built-in buffer
    const size_t need = qnn_planes_bytes(Mg, Kg, ab);
    if (need == 0 || need > (size_t)QNN_NOALLOC_SCRATCH_BYTES) return QNN_E_RANGE;
    // Every argument error of the two kernels is found here, before the encoder may overwrite the shared array (and
    // before the device is touched at all).  The checks only look at the planes pointer's alignment, which the
    // array's declaration fixes, so a stand-in with that alignment serves.
    const uint32_t *planes_stand_in = reinterpret_cast<const uint32_t *>(static_cast<uintptr_t>(256));
    int rc;
    if ((rc = qnn_check_encode_pack(x, Mg, Kg, ldx, ab, scale_a, flags, planes_stand_in, nullptr)) != QNN_OK) return rc;
    if ((rc = qnn_check_bgemm(planes_stand_in, ab, w_packed, wb, Mg, Ng, Kg, alpha, out, ldo, nullptr)) != QNN_OK) return rc;
    uint32_t *planes = nullptr;
    if ((rc = scratch_for_current_device(&planes)) != QNN_OK) return rc;
    // qnn_encode_pack writes every word of the region it uses (padding included), so nothing left
    // over from an earlier call can leak into this one and nothing needs clearing first.
    rc = qnn_encode_pack(x, Mg, Kg, ldx, ab, scale_a, flags, planes, nullptr, stream);
    if (rc != QNN_OK) return rc;
    return qnn_bgemm(planes, ab, w_packed, wb, Mg, Ng, Kg, alpha, out, ldo, nullptr, stream);
}

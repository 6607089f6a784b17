// lvspec_loose_accept_static: the loose acceptance pass for callers that must
// not allocate device memory.
//
// The context-based entry points take their scratch from cudaMalloc (at
// lvspec_create, and again whenever a larger shape arrives).  A serving loop
// that has handed all device memory to its own pool, a process running under a
// fixed memory budget, or code that has to stay clear of the implicit device
// synchronisation of cudaMalloc / cudaFree cannot use them.  This entry point
// needs no context and allocates nothing: its scratch (per-slice argmax
// partials, per-sequence tickets, a status word) lives in a fixed array in the
// library's device image, which every GPU that loads the library carries until
// the process exits.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "lvspec_internal.h"

namespace {

constexpr int kMaxDevices = 64;
constexpr size_t kSlots = LVSPEC_STATIC_MAX_SLOTS;
constexpr size_t kValOff = 0;                                   // float  [kSlots]
constexpr size_t kIdxOff = kValOff + kSlots * sizeof(float);    // int32  [kSlots]
constexpr size_t kCntOff = kIdxOff + kSlots * sizeof(int32_t);  // uint32 [LVSPEC_MAX_BATCH]
constexpr size_t kStatusOff = kCntOff + LVSPEC_MAX_BATCH * sizeof(uint32_t);
constexpr size_t kScratchBytes = (kStatusOff + sizeof(uint32_t) + 255) & ~size_t(255);

// The scratch itself.  In host code this name is only a handle for the
// runtime's symbol lookup, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

// Device code may name the array directly: zero the tickets and the status word.
__global__ void static_scratch_clear_kernel()
{
    uint32_t *words = reinterpret_cast<uint32_t *>(g_static_scratch + kCntOff);
    for (int i = threadIdx.x; i < LVSPEC_MAX_BATCH + 1; i += blockDim.x) words[i] = 0u;
}

struct DeviceSlot {
    unsigned char *scratch = nullptr;   // device address of g_static_scratch on this device
    int n_sm = 0;
};
DeviceSlot g_slots[kMaxDevices];
std::mutex g_mutex;

lvspec_status_t fail(char *err, size_t err_len, lvspec_status_t st, const char *msg)
{
    if (err && err_len) std::snprintf(err, err_len, "%s", msg);
    return st;
}

// First call on a device: ask the runtime where the array lives there.
lvspec_status_t device_slot(int device, DeviceSlot *out, char *err, size_t err_len)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceSlot &s = g_slots[device];
    if (!s.scratch) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || !ptr) {
            cudaGetLastError();
            char msg[160];
            std::snprintf(msg, sizeof msg, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
            return fail(err, err_len, LVSPEC_ERR_CUDA, msg);
        }
        int n_sm = 0;
        e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess || n_sm < 1) {
            cudaGetLastError();
            return fail(err, err_len, LVSPEC_ERR_CUDA, "cudaDeviceGetAttribute failed");
        }
        int major = 0;
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
        if (major != 10)
            return fail(err, err_len, LVSPEC_ERR_UNSUPPORTED, "this library holds sm_100a code only");
        s.n_sm = n_sm;
        s.scratch = static_cast<unsigned char *>(ptr);
    }
    *out = s;
    return LVSPEC_OK;
}

}  // namespace

extern "C" lvspec_status_t lvspec_loose_accept_static(
    void *cuda_stream, int32_t batch, int32_t gamma, int32_t vocab, int32_t n_mass_heads,
    const float *target_logits, const int32_t *draft_tokens, const float *visual_mass,
    const lvspec_thresholds_t *thresholds, int32_t shift_window, int32_t *accept_len,
    char *error_text, size_t error_text_len)
{
    using namespace lvspec;
    char *err = error_text;
    const size_t err_len = error_text_len;
    if (err && err_len) err[0] = '\0';
    if (!target_logits || !draft_tokens || !visual_mass || !thresholds || !accept_len)
        return fail(err, err_len, LVSPEC_ERR_INVALID_ARG, "null argument");
    if (batch < 1 || batch > LVSPEC_MAX_BATCH)
        return fail(err, err_len, LVSPEC_ERR_INVALID_ARG, "batch outside 1..LVSPEC_MAX_BATCH");
    if (gamma < 1 || gamma > LVSPEC_MAX_GAMMA)
        return fail(err, err_len, LVSPEC_ERR_INVALID_ARG, "gamma outside 1..LVSPEC_MAX_GAMMA");
    if (vocab < 1) return fail(err, err_len, LVSPEC_ERR_INVALID_ARG, "vocab < 1");
    if (n_mass_heads < 1) return fail(err, err_len, LVSPEC_ERR_INVALID_ARG, "n_mass_heads < 1");
    if (shift_window < 0) return fail(err, err_len, LVSPEC_ERR_INVALID_ARG, "shift_window < 0");
    if ((reinterpret_cast<uintptr_t>(target_logits) & 3u) ||
        (reinterpret_cast<uintptr_t>(draft_tokens) & 3u) ||
        (reinterpret_cast<uintptr_t>(visual_mass) & 3u) ||
        (reinterpret_cast<uintptr_t>(accept_len) & 3u))
        return fail(err, err_len, LVSPEC_ERR_INVALID_ARG, "misaligned device pointer");
    int n_loose = thresholds->n_loose;
    if (n_loose < 0) {
        if (!(thresholds->lambda >= 0.0 && thresholds->lambda <= 1.0))
            return fail(err, err_len, LVSPEC_ERR_INVALID_ARG, "lambda outside [0, 1]");
        n_loose = (int)std::floor(thresholds->lambda * (double)gamma + 1e-9);
    }
    if (n_loose > gamma) return fail(err, err_len, LVSPEC_ERR_INVALID_ARG, "n_loose > gamma");
    const int rows = batch * gamma;
    if (rows > LVSPEC_STATIC_MAX_ROWS) {
        char msg[160];
        std::snprintf(msg, sizeof msg,
                      "batch * gamma = %d exceeds LVSPEC_STATIC_MAX_ROWS = %d: the fixed scratch "
                      "array cannot hold this call; use lvspec_loose_accept",
                      rows, (int)LVSPEC_STATIC_MAX_ROWS);
        return fail(err, err_len, LVSPEC_ERR_UNSUPPORTED, msg);
    }

    int device = -1;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess || device < 0 || device >= kMaxDevices) {
        cudaGetLastError();
        return fail(err, err_len, LVSPEC_ERR_CUDA, "no current CUDA device");
    }
    DeviceSlot slot;
    lvspec_status_t st = device_slot(device, &slot, err, err_len);
    if (st != LVSPEC_OK) return st;

    // vocabulary slices: about two CTAs per SM, at least 4096 elements each, and
    // never more partials than the array holds
    int vs = (2 * slot.n_sm + rows - 1) / rows;
    const int by_vocab = (vocab + 4095) / 4096;
    const int by_array = (int)(kSlots / (size_t)rows);
    if (vs > by_vocab) vs = by_vocab;
    if (vs > by_array) vs = by_array;
    if (vs < 1) vs = 1;

    AcceptParams p;
    std::memset(&p, 0, sizeof p);
    p.logits = target_logits;
    p.draft = draft_tokens;
    p.mass = visual_mass;
    p.accept_len = accept_len;
    p.part_val = reinterpret_cast<float *>(slot.scratch + kValOff);
    p.part_idx = reinterpret_cast<int32_t *>(slot.scratch + kIdxOff);
    p.counters = reinterpret_cast<uint32_t *>(slot.scratch + kCntOff);
    p.status = reinterpret_cast<uint32_t *>(slot.scratch + kStatusOff);
    p.B = batch;
    p.gamma = gamma;
    p.V = vocab;
    p.Hm = n_mass_heads;
    p.n_loose = n_loose;
    p.window = shift_window > gamma ? gamma : shift_window;
    p.n_vsplit = vs;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // the tickets must start at zero whatever an earlier call left behind
    static_scratch_clear_kernel<<<1, 160, 0, stream>>>();
    e = cudaGetLastError();
    if (e != cudaSuccess)
        return fail(err, err_len, LVSPEC_ERR_CUDA, "launch of the scratch-clearing kernel failed");
    int launches = 0;
    e = launch_loose_accept(p, stream, &launches);
    if (e != cudaSuccess) {
        char msg[160];
        std::snprintf(msg, sizeof msg, "acceptance kernel launch: %s", cudaGetErrorString(e));
        return fail(err, err_len, LVSPEC_ERR_CUDA, msg);
    }
    return LVSPEC_OK;
}

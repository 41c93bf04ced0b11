// sk_select_static: the top-k selection of the last step, re-run without allocating anything.
//
// Some callers are not allowed to allocate device memory when they call into this library: code running while
// another library owns the allocator (a caching allocator that forbids foreign cudaMalloc calls), code on a
// latency path where cudaMalloc's implicit device synchronisation is unacceptable, or code running after the
// device has been filled on purpose.  For them this entry point keeps its scratch in a file-scope device array
// that is part of the loaded module (every GPU that loads the library holds it until the process exits).
#include "sk_state.h"

#include <cstdio>
#include <cstring>

namespace {

constexpr uint32_t kStaticMaxD = SK_STATIC_MAX_D;
// layout of the scratch, in bytes from its start (every part 256-byte aligned)
constexpr size_t kOffHist = 0;
constexpr size_t kOffHist2 = kOffHist + sk::kHistBins * 4;
constexpr size_t kOffSel = kOffHist2 + sk::kHistBins * 4;
constexpr size_t kOffKeys = kOffSel + 256;
constexpr size_t kOffCand = kOffKeys + (size_t)kStaticMaxD * 4;
constexpr size_t kOffCand2 = kOffCand + (size_t)kStaticMaxD * sizeof(sk::Cand);
constexpr size_t kScratchBytes = kOffCand2 + (size_t)kStaticMaxD * sizeof(sk::Cand);

// The scratch itself.  In host code this name is only a stand-in for the symbol, not a device address: the
// address every launch uses is looked up once per device with cudaGetSymbolAddress (see scratch_for_device).
static __device__ __align__(256) unsigned char g_select_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
unsigned char* g_scratch_ptr[kMaxDevices] = {nullptr};

// Set-up, once per device, with that device current: resolve the device address of the scratch array.
int scratch_for_device(unsigned char** out, char* msg, size_t msg_len) {
    int dev = -1;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        snprintf(msg, msg_len, "cudaGetDevice: %s", cudaGetErrorString(err));
        return SK_ECUDA;
    }
    if (!g_scratch_ptr[dev]) {
        unsigned char* p = nullptr;
        err = cudaGetSymbolAddress((void**)&p, g_select_scratch);
        if (err != cudaSuccess || !p) {
            snprintf(msg, msg_len, "cudaGetSymbolAddress(scratch): %s", cudaGetErrorString(err));
            return SK_ECUDA;
        }
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return SK_OK;
}

}  // namespace

// what the static selection found wrong is OR-ed into the handle's own status word, which sk_sync reads
__global__ void k_merge_status(const sk::Select* from, sk::Select* to) {
    if (from->status) atomicOr(&to->status, from->status);
}

// defined in sk_api.cu: records the message for sk_last_error() and returns `code`
int sk_fail_message(int code, const char* message);

// Called by sk_create (which may allocate): resolves the scratch address on the current device, so that loading the
// module that holds the array, whatever that costs, does not fall on the first sk_select_static call.
int sk_static_prepare(void) {
    char msg[200];
    unsigned char* base = nullptr;
    return scratch_for_device(&base, msg, sizeof msg);
}

extern "C" int sk_select_static(sk_state* s, uint32_t* idx_out) {
    if (!s || !idx_out) return sk_fail_message(SK_EINVAL, "sk_select_static: null argument");
    const sk::Params& P = s->P;
    if (P.d > kStaticMaxD) {
        char msg[160];
        snprintf(msg, sizeof msg, "sk_select_static: d = %u exceeds the static scratch limit SK_STATIC_MAX_D = %u",
                 P.d, kStaticMaxD);
        return sk_fail_message(SK_EINVAL, msg);
    }
    if (s->t == 0) return sk_fail_message(SK_ESTATE, "sk_select_static: no step has been taken yet");
    if (s->cand_mult > 1) return sk_fail_message(SK_ESTATE, "sk_select_static: not available with a second round (P > 1)");
    if (s->phase != 0) return sk_fail_message(SK_ESTATE, "sk_select_static: a partitioned step is in progress");
    char msg[200];
    unsigned char* base = nullptr;
    int rc = scratch_for_device(&base, msg, sizeof msg);
    if (rc) return sk_fail_message(rc, msg);

    uint32_t* hist = (uint32_t*)(base + kOffHist);
    uint32_t* hist2 = (uint32_t*)(base + kOffHist2);
    sk::Select* sel = (sk::Select*)(base + kOffSel);
    uint32_t* keys = (uint32_t*)(base + kOffKeys);
    sk::Cand* cand = (sk::Cand*)(base + kOffCand);
    sk::Cand* cand2 = (sk::Cand*)(base + kOffCand2);
    cudaStream_t st = s->stream;
    const bool vec = s->step_vec;       // the kernels of the last step: already loaded, nothing new is instantiated
    sk::Params Ps = P;
    Ps.status = &sel->status;           // the debug build's checks report into the scratch's own record

    // the array is shared by all calls and keeps the last call's contents: clear what must start at zero
    sk::launch_zero(base + kOffHist, kOffKeys - kOffHist, st);
    sk::MomentArgs A{};                 // members = 0: read vhat only, the step's own update is not repeated
    A.vhat = s->vhat;
    A.variant = (uint32_t)s->variant;
    sk::launch_unsketch_hist(Ps, A, s->sum, keys, hist, vec, s->sm_count, st);
    sk::launch_pick_bin(Ps, hist, sel, 0, st);
    sk::launch_emit(Ps, keys, nullptr, sel, idx_out, cand, hist2, s->sm_count, st);
    sk::launch_refine(Ps, sel, cand, cand2, hist2, idx_out, s->sm_count, st);
    k_merge_status<<<1, 1, 0, st>>>(sel, s->sel);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) {
        snprintf(msg, sizeof msg, "sk_select_static: launch failed: %s", cudaGetErrorString(err));
        return sk_fail_message(SK_ECUDA, msg);
    }
    return SK_OK;
}

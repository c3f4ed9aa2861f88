// hvd_verify_commit_noalloc: greedy verification and commit for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where a decoding step runs: a
// serving engine that has handed the whole device to its own memory pool, code running under a
// stream capture, or a plugin that is only ever given the caller's tensors.  hvd_create allocates
// the scratch memory of the kernels; this entry point needs no context.  Its scratch is the
// file-scope device array below, which every GPU that loads the library holds until the process
// exits (kScratchBytes, about 129 KB).
//
// In host code the array's name is only a stand-in: it is not a device address, and handing it to
// a kernel would make the kernel fault or use the wrong memory.  The device address is obtained
// once per device with cudaGetSymbolAddress (first call on that device, with the device current)
// and it is that pointer the kernels get.
#include <mutex>

#include "hvd_internal.cuh"

using namespace hvd;

namespace {

constexpr int64_t kMaxRows = HVD_NOALLOC_MAX_ROWS;
constexpr int32_t kMaxBatch = HVD_NOALLOC_MAX_BATCH;
constexpr size_t kCounterBytes = (size_t)kVerifyQueues * 32 * sizeof(uint32_t);
constexpr size_t kKeyBytes = (size_t)kMaxRows * sizeof(unsigned long long);
constexpr size_t kScratchBytes = kKeyBytes + kCounterBytes;

// [row keys: kMaxRows x 8 bytes][unit counters]; shared by every call on the device
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
struct DeviceSetup {
    bool ready;
    unsigned char* scratch;  // device address of g_scratch on this device
    hvd_ctx ctx;             // launch parameters only (no memory behind it)
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

// First call on a device: find the device address of the scratch array and the launch shape.
// Queries only; nothing is allocated.
hvd_status setup_device(int device, DeviceSetup** out, const char** why) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    DeviceSetup& s = g_setup[device];
    if (!s.ready) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_scratch);
        if (e != cudaSuccess) { *why = cudaGetErrorString(e); return HVD_ERR_CUDA; }
        s.scratch = static_cast<unsigned char*>(p);
        s.ctx = hvd_ctx();
        s.ctx.device = device;
        e = cudaDeviceGetAttribute(&s.ctx.num_sms, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess) { *why = cudaGetErrorString(e); return HVD_ERR_CUDA; }
        const size_t smem = verify_dyn_smem(kMaxBatch);
        s.ctx.vf_blocks_per_sm[0] = verify_occupancy(HVD_F32, smem);
        s.ctx.vf_blocks_per_sm[1] = verify_occupancy(HVD_BF16, smem);
        if (s.ctx.vf_blocks_per_sm[0] < 1 || s.ctx.vf_blocks_per_sm[1] < 1) {
            *why = "the verify kernels do not fit this device";
            return HVD_ERR_UNSUPPORTED;
        }
        s.ctx.pdl_commit = false;
        s.ctx.pdl_mask = 0;
        s.ctx.vf_small_bytes = kVerifySmallBytes;
        s.ready = true;
    }
    *out = &s;
    return HVD_OK;
}

thread_local char g_noalloc_error[256] = "";

hvd_status reject(hvd_status st, const char* msg) {
    snprintf(g_noalloc_error, sizeof(g_noalloc_error), "%s", msg);
    return st;
}

}  // namespace

extern "C" {

const char* hvd_noalloc_last_error(void) { return g_noalloc_error; }

hvd_status hvd_verify_commit_noalloc(int32_t B, int32_t k_cap, const void* logits, hvd_dtype dtype, int64_t V,
                                     const int64_t* row_off, int32_t k_uniform, int64_t total_rows,
                                     const int32_t* sel_draft, const int32_t* sel_len, const int32_t* select,
                                     int32_t* hist, const int64_t* hist_off, const int32_t* hist_cap,
                                     int32_t* hist_len, hvd_req_state* state, int32_t* accepted,
                                     int32_t* committed, int32_t* n_commit, int32_t* target_tok,
                                     int32_t* status, void* stream) {
    g_noalloc_error[0] = 0;
    if (B < 1 || B > kMaxBatch)
        return reject(HVD_ERR_INVALID_ARG, "hvd_verify_commit_noalloc: B outside [1, HVD_NOALLOC_MAX_BATCH]");
    if (total_rows < 1 || total_rows > kMaxRows)
        return reject(HVD_ERR_INVALID_ARG, "hvd_verify_commit_noalloc: total_rows outside [1, HVD_NOALLOC_MAX_ROWS]: "
                                           "the static scratch array holds one key per logits row");
    if (k_cap < 1 || k_cap > HVD_MAX_K) return reject(HVD_ERR_INVALID_ARG, "hvd_verify_commit_noalloc: k_cap outside [1, 64]");
    if (dtype != HVD_F32 && dtype != HVD_BF16) return reject(HVD_ERR_INVALID_ARG, "hvd_verify_commit_noalloc: unknown dtype");
    if (V < 1 || V > 0x7fffffffLL) return reject(HVD_ERR_INVALID_ARG, "hvd_verify_commit_noalloc: V outside [1, 2^31)");
    if (!logits || !sel_draft || !sel_len || !select || !hist || !hist_off || !hist_cap || !hist_len || !state ||
        !accepted || !committed || !n_commit || !status)
        return reject(HVD_ERR_INVALID_ARG, "hvd_verify_commit_noalloc: NULL pointer");
    const size_t esz = dtype == HVD_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(logits) & (esz - 1))
        return reject(HVD_ERR_INVALID_ARG, "hvd_verify_commit_noalloc: logits not aligned to its element type");
    if (reinterpret_cast<uintptr_t>(state) & 7)
        return reject(HVD_ERR_INVALID_ARG, "hvd_verify_commit_noalloc: state must be 8-byte aligned");
    if (!row_off) {
        if (k_uniform < 0 || k_uniform > k_cap)
            return reject(HVD_ERR_INVALID_ARG, "hvd_verify_commit_noalloc: k_uniform outside [0, k_cap]");
        if (total_rows != (int64_t)B * (k_uniform + 1))
            return reject(HVD_ERR_INVALID_ARG, "hvd_verify_commit_noalloc: total_rows != B*(k_uniform+1)");
    }

    int device = -1;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return reject(HVD_ERR_CUDA, cudaGetErrorString(e));
    if (device < 0 || device >= kMaxDevices) return reject(HVD_ERR_UNSUPPORTED, "hvd_verify_commit_noalloc: device ordinal too large");
    DeviceSetup* s = nullptr;
    const char* why = "";
    const hvd_status st = setup_device(device, &s, &why);
    if (st != HVD_OK) return reject(st, why);

    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    unsigned long long* row_key = reinterpret_cast<unsigned long long*>(s->scratch);
    uint32_t* counters = reinterpret_cast<uint32_t*>(s->scratch + kKeyBytes);
    // The array keeps whatever the last call left (zero after a call that ran to its end, but not
    // after one that was aborted): everything this call reads before writing is cleared first.
    e = cudaMemsetAsync(row_key, 0, (size_t)total_rows * sizeof(unsigned long long), cs);
    if (e == cudaSuccess) e = cudaMemsetAsync(counters, 0, kCounterBytes, cs);
    if (e != cudaSuccess) return reject(HVD_ERR_CUDA, cudaGetErrorString(e));

    VerifyArgs a;
    a.B = B; a.logits = logits; a.V = V; a.row_off = row_off; a.k_uniform = k_uniform;
    a.sel_draft = sel_draft; a.sel_len = sel_len; a.parent = nullptr; a.select = select;
    a.hist = hist; a.hist_off = hist_off; a.hist_cap = hist_cap; a.hist_len = hist_len; a.state = state;
    a.accepted = accepted; a.committed = committed; a.n_commit = n_commit; a.target_tok = target_tok;
    a.status = status; a.k_cap = k_cap;
    a.next_unit = counters; a.dev_error = nullptr;
    a.row_key = row_key; a.total_rows = total_rows; a.ext_keys = nullptr;
    hvd_ctx call_ctx = s->ctx;  // private copy: the error text of a failed launch lands here
    call_ctx.cfg.k_cap = k_cap;
    const hvd_status r = launch_verify(&call_ctx, a, dtype, cs);
    if (r != HVD_OK) return reject(r, call_ctx.last_error);
    return HVD_OK;
}

}  // extern "C"

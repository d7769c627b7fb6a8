// vispec_tree_verify_attn_static: the verification attention for callers that cannot allocate.
//
// Some users of this library run where device allocation is off the table: inside a serving loop
// whose memory pool was sized and frozen at start-up, in a plugin that is handed tensors but no
// allocator, or on a stream where a cudaMalloc would force a device-wide synchronisation at the
// worst moment.  The regular entry point needs a context (created with a few small cudaMalloc calls)
// and a caller-supplied workspace.  This one needs neither: its split-KV scratch is the file-scope
// device array below, which exists in every process that loads the library, on every GPU it uses,
// from module load until exit.
#include "vispec_internal.h"

// 16 MiB: room for up to 502 partial results of 64 query rows at D = 128 (33,280 bytes each)
// behind the 64 KiB header the workspace layout reserves.
#define VISPEC_STATIC_SCRATCH_BYTES (16u << 20)

static __device__ __align__(256) unsigned char g_static_scratch[VISPEC_STATIC_SCRATCH_BYTES];
static __device__ int g_static_status;   // sink for the status word when the caller passes none

namespace {

constexpr int kMaxDevices = 64;
struct DeviceSetup {
    bool done = false;
    void* scratch = nullptr;   // DEVICE address of g_static_scratch on this device
    int* status = nullptr;     // DEVICE address of g_static_status on this device
    int sm_count = 0;
};
DeviceSetup g_setup[kMaxDevices];

// In host code the names g_static_scratch / g_static_status are only handles for the runtime, not
// device addresses, so they must never be handed to a kernel directly: ask the runtime where the
// symbols live on the current device.
// No lock: two host threads that make their first call on a device at the same moment both run the queries below
// and store the same addresses and the same SM count, and `done` is set last, so whichever thread reads it as true
// finds the fields filled; the worst case is that the queries run twice.
int setup_current_device(int dev) {
    DeviceSetup& s = g_setup[dev];
    if (s.done) return VISPEC_OK;
    void* p = nullptr;
    int* st = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess) return VISPEC_E_CUDA;
    if (cudaGetSymbolAddress((void**)&st, g_static_status) != cudaSuccess) return VISPEC_E_CUDA;
    if (cudaDeviceGetAttribute(&s.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return VISPEC_E_CUDA;
    if (vispec::init_attn_generic() != cudaSuccess) return VISPEC_E_CUDA;   // a function attribute, not an allocation
    s.scratch = p;
    s.status = st;
    s.done = true;
    return VISPEC_OK;
}

}  // namespace

extern "C" int vispec_tree_verify_attn_static(const void* q, const void* k_cache, const void* v_cache,
                                              const int32_t* kv_len, const uint64_t* tree_mask, int B, int N,
                                              int Hq, int Hkv, int D, int S_max, float scale, void* out,
                                              float* lse, int* status_word, void* stream) {
    if (!q || !k_cache || !v_cache || !kv_len || !tree_mask || !out) return VISPEC_E_NULL;
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(k_cache) |
         reinterpret_cast<uintptr_t>(v_cache)) & 15)
        return VISPEC_E_ALIGN;
    if (B < 0 || N < 1 || N > VISPEC_MAX_TREE_NODES || Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || (D != 64 && D != 128) ||
        S_max < N)
        return VISPEC_E_SHAPE;
    // Size limit: one partial of 64 query rows per (sequence, kv head, 64-row block) and KV split must
    // fit the static array with at least two splits, otherwise the call is refused, not truncated.
    const size_t units = (size_t)B * Hkv * (((size_t)(Hq / Hkv) * N + 63) / 64);
    const size_t half_slot = vispec::slot_bytes(D) / 2;
    if (vispec::kCounterBytes + 2 * units * half_slot > VISPEC_STATIC_SCRATCH_BYTES) return VISPEC_E_WORKSPACE;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return VISPEC_E_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return VISPEC_E_RANGE;
    const int rc = setup_current_device(dev);
    if (rc != VISPEC_OK) return rc;
    const DeviceSetup& s = g_setup[dev];

    vispec::AttnArgs a = {};
    a.q = q; a.k = k_cache; a.v = v_cache; a.kv_len = kv_len; a.mask = tree_mask; a.out = out; a.lse = lse;
    a.B = B; a.N = N; a.Hq = Hq; a.Hkv = Hkv; a.D = D; a.S_max = S_max; a.scale = scale;
    a.ws = s.scratch; a.ws_bytes = VISPEC_STATIC_SCRATCH_BYTES;
    a.status = status_word ? status_word : s.status;
    a.sm_count = s.sm_count;
    a.early_prefetch = false;
    a.tc5_path = 0;
    a.k_map = nullptr; a.v_map = nullptr;
    int n = 0;
    return vispec::launch_attn_generic(a, (cudaStream_t)stream, &n) == cudaSuccess ? VISPEC_OK : VISPEC_E_CUDA;
}

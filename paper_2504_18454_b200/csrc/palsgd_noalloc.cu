// palsgd_outer_sync_noalloc: the outer synchronisation for callers that must not
// allocate device memory (see include/palsgd.h).
//
// The ordinary path keeps its launch tables (chunk table, pointer tables) in a
// device allocation made by palsgd_init.  Here the same tables live in a
// file-scope __device__ array of fixed size, are rebuilt on every call from the
// caller's pointer lists, and are handed to the same outer-sync kernel.
//
// In host code the name of a __device__ array is only a host-side stand-in for
// the symbol: it is not an address the GPU can use.  The device address is
// obtained once per device with cudaGetSymbolAddress and cached.
#include "../../include/palsgd.h"

#include <cmath>
#include <cstring>
#include <mutex>

#include "palsgd_kernels.cuh"

using namespace palsgd;

namespace {

// Every GPU that loads this library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[PALSGD_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void* g_scratch_dev_ptr[kMaxDevices];          // device address of the array, per device ordinal
bool  g_scratch_ready[kMaxDevices];
std::mutex g_mutex;                            // guards the cache above and the staging buffer below

// Host-side staging of the tables: fixed size, so that a call allocates nothing
// on the host either.  cudaMemcpyAsync from pageable memory returns once the
// bytes have been staged, so the buffer is free again when the call returns;
// the runtime waits for the work already enqueued on the stream before it
// stages them, so the call blocks the host that long.
alignas(256) unsigned char g_stage[PALSGD_NOALLOC_SCRATCH_BYTES];

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Device address of g_noalloc_scratch on the current device (set-up on first use).
cudaError_t scratch_address(void** out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!g_scratch_ready[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_dev_ptr[dev] = p;
        g_scratch_ready[dev] = true;
    }
    *out = g_scratch_dev_ptr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" int palsgd_outer_sync_noalloc(uint32_t K, int32_t precision, size_t n_tensors,
                                         const uint64_t* numel, void* const* param,
                                         float* const* master, float* const* global,
                                         float* const* outer_mom, double outer_lr,
                                         double outer_momentum, int32_t outer_nesterov, void* stream)
{
    if (K == 0 || K > PALSGD_MAX_WORKERS) return PALSGD_EINVAL;
    if (precision != PALSGD_PREC_FP32 && precision != PALSGD_PREC_BF16_MASTER) return PALSGD_EINVAL;
    if (outer_nesterov != 0 && outer_nesterov != 1) return PALSGD_EINVAL;
    if (!std::isfinite(outer_lr) || !std::isfinite(outer_momentum) || outer_momentum < 0.0) return PALSGD_EINVAL;
    if (n_tensors == 0 || !numel || !param || !global || !outer_mom) return PALSGD_EINVAL;
    const bool bf = precision == PALSGD_PREC_BF16_MASTER;
    if (bf && !master) return PALSGD_EINVAL;

    // ---- validate pointers; count segments (one per non-empty tensor) and chunks
    size_t n_seg = 0, n_chunks = 0;
    for (size_t j = 0; j < n_tensors; ++j) {
        if (numel[j] > (1ull << 40)) return PALSGD_EINVAL;
        if (numel[j] == 0) continue;
        if (!global[j] || !outer_mom[j]) return PALSGD_EINVAL;
        if (!aligned(global[j], 4) || !aligned(outer_mom[j], 4)) return PALSGD_EALIGN;
        for (uint32_t k = 0; k < K; ++k) {
            const size_t idx = (size_t)k * n_tensors + j;
            if (!param[idx] || (bf && !master[idx])) return PALSGD_EINVAL;
            if (!aligned(param[idx], bf ? 2 : 4) || (bf && !aligned(master[idx], 4))) return PALSGD_EALIGN;
        }
        n_seg += 1;
        n_chunks += (size_t)((numel[j] + kChunkElems - 1) / kChunkElems);
        if (n_chunks > PALSGD_NOALLOC_SCRATCH_BYTES) return PALSGD_ETOOBIG;     // far beyond the limit already
    }
    if (n_seg == 0) return PALSGD_OK;

    // ---- layout of the tables inside the scratch: [chunks][xf][xw][global][outer_mom]
    const size_t per_slot = round_up((size_t)K * n_seg * sizeof(void*), 256);
    const size_t per_seg = round_up(n_seg * sizeof(void*), 256);
    const size_t off_xf = round_up(n_chunks * sizeof(Chunk), 256);
    const size_t off_xw = off_xf + per_slot;
    const size_t off_global = off_xw + (bf ? per_slot : 0);
    const size_t off_mom = off_global + per_seg;
    const size_t total = off_mom + per_seg;
    if (total > PALSGD_NOALLOC_SCRATCH_BYTES) return PALSGD_ETOOBIG;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // Not capturable: a captured copy node would re-read the shared host staging buffer, and a captured
    // kernel node would keep this call's table sizes, at every replay -- after later calls have put
    // other tables there.  A capturing stream is refused before anything is enqueued.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &cap) != cudaSuccess) { (void)cudaGetLastError(); return PALSGD_ECUDA; }
    if (cap != cudaStreamCaptureStatusNone) return PALSGD_ESTATE;
    std::lock_guard<std::mutex> lock(g_mutex);

    void* d_void = nullptr;
    if (scratch_address(&d_void) != cudaSuccess) { (void)cudaGetLastError(); return PALSGD_ECUDA; }
    unsigned char* d = static_cast<unsigned char*>(d_void);

    // ---- build the tables on the host
    std::memset(g_stage, 0, total);
    Chunk* chunks = reinterpret_cast<Chunk*>(g_stage);
    void** t_xf = reinterpret_cast<void**>(g_stage + off_xf);
    void** t_xw = reinterpret_cast<void**>(g_stage + off_xw);
    void** t_global = reinterpret_cast<void**>(g_stage + off_global);
    void** t_mom = reinterpret_cast<void**>(g_stage + off_mom);
    size_t seg = 0, c = 0;
    for (size_t j = 0; j < n_tensors; ++j) {
        if (numel[j] == 0) continue;
        bool vec = aligned(global[j], 16) && aligned(outer_mom[j], 16);
        for (uint32_t k = 0; k < K; ++k) {
            const size_t idx = (size_t)k * n_tensors + j;
            t_xf[(size_t)k * n_seg + seg] = bf ? static_cast<void*>(master[idx]) : param[idx];
            if (bf) t_xw[(size_t)k * n_seg + seg] = param[idx];
            vec = vec && aligned(param[idx], 16) && (!bf || aligned(master[idx], 16));
        }
        t_global[seg] = global[j];
        t_mom[seg] = outer_mom[j];
        for (uint64_t off = 0; off < numel[j]; off += kChunkElems) {
            const uint64_t len = numel[j] - off < kChunkElems ? numel[j] - off : kChunkElems;
            chunks[c++] = Chunk{off, (uint32_t)len, (uint32_t)seg | (vec ? kSegVecFlag : 0u)};
        }
        seg += 1;
    }

    // ---- tables -> the static device array (ordered on `stream` before the kernel)
    if (cudaMemcpyAsync(d, g_stage, total, cudaMemcpyHostToDevice, s) != cudaSuccess) {
        (void)cudaGetLastError();
        return PALSGD_ECUDA;
    }

    OuterArgs a{};
    a.tb.chunks = reinterpret_cast<const Chunk*>(d);
    a.tb.n_chunks = (uint32_t)n_chunks;
    a.tb.n_seg = (uint32_t)n_seg;
    a.tb.K = K;
    a.tb.chunk_elems = kChunkElems;
    a.tb.xf = reinterpret_cast<float* const*>(d + off_xf);
    a.tb.xw = bf ? reinterpret_cast<__nv_bfloat16* const*>(d + off_xw) : nullptr;
    a.tb.global = reinterpret_cast<float* const*>(d + off_global);
    a.tb.outer_mom = reinterpret_cast<float* const*>(d + off_mom);
    a.mu = (float)outer_momentum;
    a.lr = (float)outer_lr;
    a.Kf = (float)K;
    a.nesterov = outer_nesterov;
    a.items = a.tb.chunks;                 // one CTA per 8192-element block, 128-bit stores by every thread
    a.n_items = (uint32_t)n_chunks;
    a.sub_elems = kChunkElems;
    a.n_stage = 1;
    const unsigned grid = (unsigned)(n_chunks > 0x7FFFFFFFull ? 0x7FFFFFFFull : n_chunks);
    if (bf) palsgd_outer_kernel<1, 0, 0><<<grid, kThreads, 0, s>>>(a);
    else    palsgd_outer_kernel<0, 0, 0><<<grid, kThreads, 0, s>>>(a);
    if (cudaGetLastError() != cudaSuccess) return PALSGD_ECUDA;
    return PALSGD_OK;
}

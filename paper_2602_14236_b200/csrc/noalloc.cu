// salicache_saliency_noalloc: the spatial score for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc once they are running: a serving process that
// handed all of the GPU's memory to its own pool at start-up, code inside a region where the
// allocator is locked, a plug-in that is forbidden to grow the process' footprint.  For them the
// edge bit planes, the sRGB table and the status word that salicache_saliency keeps in a context's
// scratch live here in one file-scope device array of fixed size, which every GPU that loads the
// library carries until the process exits.  The kernels are the ones salicache_saliency runs.
#include <math.h>
#include <mutex>
#include <string.h>

#include "common.cuh"

int sc_saliency_init(int max_h, int max_words);

namespace {

constexpr int NA_MAX_FRAMES = SALICACHE_NOALLOC_MAX_FRAMES;
constexpr int NA_MAX_SIDE = SALICACHE_NOALLOC_MAX_SIDE;
constexpr int NA_WORDS = (NA_MAX_SIDE + 31) / 32;
constexpr size_t NA_PLANE_WORDS = (size_t)NA_MAX_FRAMES * NA_MAX_SIDE * NA_WORDS;   // one bit plane, all frames
constexpr size_t NA_LUT_OFF = 2 * NA_PLANE_WORDS * sizeof(uint32_t);                // 256 doubles
constexpr size_t NA_STATUS_OFF = NA_LUT_OFF + 256 * sizeof(double);
constexpr size_t NA_BYTES = NA_STATUS_OFF + 256;

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress: it is not
// a device address and must never be passed to a kernel as one.
static __device__ __align__(256) unsigned char g_noalloc_scratch[NA_BYTES];

constexpr int NA_MAX_DEVICES = 64;
std::mutex g_mu;
unsigned char* g_base[NA_MAX_DEVICES];    // device address of g_noalloc_scratch, per device, once set up
int g_sm_count[NA_MAX_DEVICES];

// Once per device, with that device current: resolve the array's device address, set the kernels'
// shared-memory limits and upload the sRGB -> linear table.  Synchronous, no allocation.
int setup_device(int dev, unsigned char** base) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_base[dev]) {
        *base = g_base[dev];
        return SALICACHE_OK;
    }
    unsigned char* ptr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return SALICACHE_E_CUDA;
    int rc = sc_saliency_init(NA_MAX_SIDE, NA_WORDS);
    if (rc != SALICACHE_OK) return rc;
    double lut[256];
    for (int i = 0; i < 256; ++i) {   // IEC 61966-2-1 transfer curve
        double v = i / 255.0;
        lut[i] = v <= 0.04045 ? v / 12.92 : pow((v + 0.055) / 1.055, 2.4);
    }
    if (cudaMemcpy(ptr + NA_LUT_OFF, lut, sizeof(lut), cudaMemcpyHostToDevice) != cudaSuccess) return SALICACHE_E_CUDA;
    // a copy from pageable memory may return before the table has landed, and only the legacy default stream is
    // ordered behind it: wait here, so that the caller's stream (any stream) sees the table
    if (cudaDeviceSynchronize() != cudaSuccess) return SALICACHE_E_CUDA;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return SALICACHE_E_CUDA;
    g_sm_count[dev] = sms;
    g_base[dev] = ptr;
    *base = ptr;
    return SALICACHE_OK;
}

}  // namespace

extern "C" int salicache_saliency_noalloc(const salicache_params* p, const uint8_t* d_frames, int B, float* d_s,
                                          int32_t* d_status_or_null, void* cuda_stream) {
    if (!p || !d_frames || !d_s) return SALICACHE_E_NULL;
    if (p->var_radius != 3 || p->patch != 14 || !(p->sigma_ref > 0) || p->canny_lo < 0 || p->canny_hi < p->canny_lo ||
        p->canny_hi > 1442 || p->hyst_max_iters < 1 || p->n_images != 1 || p->color_norm != 0)
        return SALICACHE_E_PARAM;
    if (p->H <= 0 || p->W <= 0 || p->H % 112 != 0 || p->W % 112 != 0) return SALICACHE_E_SHAPE;
    if (p->H > NA_MAX_SIDE || p->W > NA_MAX_SIDE || B < 0 || B > NA_MAX_FRAMES) return SALICACHE_E_SHAPE;
    if ((reinterpret_cast<uintptr_t>(d_frames) & 15u) || (reinterpret_cast<uintptr_t>(d_s) & 15u) ||
        (reinterpret_cast<uintptr_t>(d_status_or_null) & 3u))
        return SALICACHE_E_ALIGN;
    if (B == 0) return SALICACHE_OK;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SALICACHE_E_CUDA;
    if (dev < 0 || dev >= NA_MAX_DEVICES) return SALICACHE_E_PARAM;
    unsigned char* base = nullptr;
    int rc = setup_device(dev, &base);
    if (rc != SALICACHE_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // a context on the host stack whose scratch pointers lead into the static array
    salicache_ctx c;
    memset(&c, 0, sizeof(c));
    c.p = *p;
    c.chunk = NA_MAX_FRAMES;
    c.n_planes = 1;
    c.n_tok = (p->H / p->patch) * (p->W / p->patch);
    c.plane[0] = PlaneGeom{p->H, p->W, p->H / p->patch, p->W / p->patch, 0, 0, c.n_tok};
    c.bits_kept = reinterpret_cast<uint32_t*>(base);
    c.bits_edge = reinterpret_cast<uint32_t*>(base) + NA_PLANE_WORDS;
    c.lut = reinterpret_cast<double*>(base + NA_LUT_OFF);
    c.d_status = d_status_or_null ? d_status_or_null : reinterpret_cast<int*>(base + NA_STATUS_OFF);
    c.sm_count = g_sm_count[dev];
    // the status word keeps the last call's value: start this call from "ok"
    if (!d_status_or_null && cudaMemsetAsync(base + NA_STATUS_OFF, 0, sizeof(int), st) != cudaSuccess)
        return SALICACHE_E_CUDA;
    return sc_saliency(&c, c.plane[0], d_frames, (size_t)p->H * p->W * 3, B, d_s, nullptr, st);
}

// ckks_rescale_static: rescale without any caller-provided or freshly allocated scratch memory.
//
// Some callers cannot allocate device memory at the point where they need a rescale: code running between
// cudaStreamBeginCapture and cudaStreamEndCapture, code inside a serving loop whose memory pool is frozen after
// start-up, or a host application that hands this library a fixed set of buffers and nothing else.  The ordinary
// ckks_rescale asks them for a workspace; this variant instead uses a fixed array that lives in the library
// image itself.  Every GPU that loads the library carries the array (CKKS_STATIC_SCRATCH_BYTES) until the
// process exits, which is why it is kept small and why larger inputs are refused rather than served.
//
// The array's name is only a host-side handle here: launching a kernel on `g_static_scratch` as written would
// hand it a host address.  The device address is looked up once per device with cudaGetSymbolAddress while that
// device is current, cached, and passed to the same kernels ckks_rescale runs.
#include <mutex>

#include "common.cuh"

namespace {

constexpr size_t SCRATCH_WORDS = CKKS_STATIC_SCRATCH_BYTES / sizeof(u64);
static __device__ __align__(256) u64 g_static_scratch[SCRATCH_WORDS];

constexpr int MAX_DEVICES = 64;
u64 *g_scratch_ptr[MAX_DEVICES] = {};
std::mutex g_scratch_mutex;

struct CurrentDevice {
    int prev = 0;
    explicit CurrentDevice(int dev) { cudaGetDevice(&prev); cudaSetDevice(dev); }
    ~CurrentDevice() { cudaSetDevice(prev); }
};

// Device address of the scratch array on `device` (which must be current).  First call per device does the lookup.
cudaError_t scratch_address(int device, u64 **out) {
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[device]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[device] = (u64 *)p;
    }
    *out = g_scratch_ptr[device];
    return cudaSuccess;
}

}  // namespace

extern "C" int32_t ckks_rescale_static(ckks_ctx *c, const ckks_ct *in, ckks_ct *out, void *stream) {
    if (!c || !in || !in->data || !out || !in->ncomp || in->ncomp > 3) return CKKS_ERR_ARG;
    if (in->level < 2 || in->level > c->L) return CKKS_ERR_LEVEL;
    if (!out->data || (in->ncomp > 1 && in->data == out->data)) return CKKS_ERR_ARG;
    if (c->device < 0 || c->device >= MAX_DEVICES) return CKKS_ERR_UNSUPPORTED;
    const size_t need = (size_t)in->ncomp * in->level * c->N;        // words: last limbs + lifted limbs
    if (need > SCRATCH_WORDS) {
        c->cuda_error = "ckks_rescale_static: input needs " + std::to_string(need * sizeof(u64)) + " bytes of scratch, the built-in array holds " +
                        std::to_string((size_t)CKKS_STATIC_SCRATCH_BYTES) + "; use ckks_rescale with a caller workspace";
        return CKKS_ERR_WORKSPACE;
    }
    CurrentDevice guard(c->device);
    u64 *scratch = nullptr;
    cudaError_t e = scratch_address(c->device, &scratch);
    if (e != cudaSuccess) { c->cuda_error = cudaGetErrorString(e); return CKKS_ERR_CUDA; }
    // Nothing in the scratch has to start at zero: the last limbs are copied in and every lifted limb is written
    // before it is read, so whatever the previous call left there is simply overwritten.
    launch_rescale(c, (const u64 *)in->data, (u64 *)out->data, in->ncomp, in->level, scratch, (cudaStream_t)stream);
    e = cudaGetLastError();
    if (e != cudaSuccess) { c->cuda_error = cudaGetErrorString(e); return CKKS_ERR_CUDA; }
    out->ncomp = in->ncomp;
    out->scale = in->scale / (double)c->mod[in->level - 1];
    out->level = in->level - 1;
    return CKKS_OK;
}

// ampq_score_segment_noalloc (include/ampq.h): the scoring pass over one
// segment for callers that must not allocate.
//
// Some callers cannot go through cudaMalloc: code running while another
// library owns the whole device heap through its own pool, code inside a region
// where a device allocation would synchronise the device or fragment a
// carefully packed heap, or plug-ins that are handed fixed buffers and nothing
// else.  For them every table and every per-tile partial sum of the pass lives
// in one file-scope device array of fixed size, which each GPU that loads the
// library holds until the process exits.  The kernels are the ones ampq_score
// launches; only where their tables live differs.
//
// The array's name is a device symbol.  In host code it is a host-side
// stand-in, not a device address, so it is never handed to a kernel: the
// device address is looked up once per device with cudaGetSymbolAddress, with
// that device current, and that pointer is what the launches receive.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>
#include <mutex>

#include "../../include/ampq.h"
#include "ampq_device.h"
#include "ampq_kernels.h"

namespace ampq {
namespace {

constexpr long long kNoAllocMaxTiles = 4096;  // per-tile partial slots in the fixed array
static_assert(AMPQ_NOALLOC_MAX_NUMEL <= kNoAllocMaxTiles * (long long)kTileElems, "the largest segment fits in the slots at the largest tile");
constexpr int kNoAllocAcc = 2;  // S and D of the one low-precision format
constexpr int kMaxDevices = 64;

// Everything ampq_score would keep in its workspace, for one tensor.
struct NoAllocScratch {
    Tensor tensor;
    long long tile_begin[2];       // scoring tiles: {0, ntiles}
    long long amax_tile_begin[2];  // amax tiles: {0, n_amax_tiles}
    Segment segment;
    unsigned amax_bits;
    int flag;
    LaunchStatus status;
    float scales[2 * kMaxLow];
    double seg_out[kNoAllocAcc];
    alignas(256) double partials[kNoAllocMaxTiles * kNoAllocAcc];
};

// 64.25 KiB per GPU.  Shared by every call; it keeps the last call's contents.
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

std::mutex g_setup_mutex;
NoAllocScratch* g_scratch_ptr[kMaxDevices] = {};  // device address of the array, per device

// Fills the tables of the one-tensor problem.  Everything a previous call left
// in them is overwritten here; amax_bits, the flag and the status word are
// reset by init_amax_kernel and scales_kernel, and every partial slot that is
// read is written by this call's scoring launch first.
__global__ void noalloc_prepare_kernel(NoAllocScratch* s, const void* values, const void* grads, long long n,
                                       int dtype, float amax_preset, long long ntiles, long long namax) {
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    Tensor t;
    t.values = values;
    t.grads = grads;
    t.numel = n;
    t.seg_len = n;
    t.grad_stride = n;
    t.partial_base = 0;
    t.tiles_per_seg = (int)ntiles;
    t.R = 1;
    t.per_sample = 1;
    t.dtype = dtype;
    t.share_n = 1;
    t.seg_base = 0;
    t.amax_preset = amax_preset;
    t.causal_shift = 0;
    t.amax_src = 0;
    for (int k = 0; k < kMaxRB - 1; ++k) t.gstream[k] = nullptr;
    t.stream_slot_stride = ntiles;
    s->tensor = t;
    s->tile_begin[0] = 0;
    s->tile_begin[1] = ntiles;
    s->amax_tile_begin[0] = 0;
    s->amax_tile_begin[1] = namax;
    s->segment.first_slot = 0;
    s->segment.count = (int)ntiles;
    s->segment.pad = 0;
    s->seg_out[0] = 0.0;
    s->seg_out[1] = 0.0;
}

// out = {S, D, amax}; NaN sums when the operand held Inf or NaN (or a bounded
// wait of the scoring kernel ran out).
__global__ void noalloc_publish_kernel(const NoAllocScratch* s, double* out) {
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    const bool bad = s->flag != 0 || s->status.timeout != 0;
    const double nan = __longlong_as_double(0x7FF8000000000000LL);
    out[0] = bad ? nan : s->seg_out[0];
    out[1] = bad ? nan : s->seg_out[1];
    out[2] = (double)__uint_as_float(s->amax_bits);
}

// Device address of the scratch array on `device` (which must be current).
cudaError_t scratch_of(int device, NoAllocScratch** out) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[device] = static_cast<NoAllocScratch*>(p);
    }
    *out = g_scratch_ptr[device];
    return cudaSuccess;
}

struct CurrentDevice {
    int prev = -1;
    bool ok = true;
    explicit CurrentDevice(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~CurrentDevice() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

}  // namespace
}  // namespace ampq

using namespace ampq;

extern "C" {
#pragma GCC visibility push(default)

int ampq_score_segment_noalloc(int device, void* cuda_stream, int dtype, int fmt, const void* values,
                               const void* grads, long long numel, float amax, double* dev_out) {
    if (dtype != AMPQ_F32 && dtype != AMPQ_BF16) return AMPQ_ERR_INVALID;
    if (fmt != AMPQ_FMT_E4M3 && fmt != AMPQ_FMT_E5M2) return AMPQ_ERR_INVALID;
    if (numel < 0 || !dev_out || (numel > 0 && (!values || !grads))) return AMPQ_ERR_INVALID;
    if (amax != amax || std::isinf(amax)) return AMPQ_ERR_INVALID;
    if (numel > AMPQ_NOALLOC_MAX_NUMEL) return AMPQ_ERR_TOO_LARGE;
    const int es = dtype == AMPQ_F32 ? 4 : 2;
    if ((reinterpret_cast<uintptr_t>(values) % es) || (reinterpret_cast<uintptr_t>(grads) % es) ||
        (reinterpret_cast<uintptr_t>(dev_out) % 8))
        return AMPQ_ERR_ALIGN;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev <= 0) { cudaGetLastError(); return AMPQ_ERR_CUDA; }
    if (device < 0 || device >= ndev || device >= kMaxDevices) return AMPQ_ERR_INVALID;
    CurrentDevice cur(device);
    if (!cur.ok) return AMPQ_ERR_CUDA;
    NoAllocScratch* s = nullptr;
    if (scratch_of(device, &s) != cudaSuccess) { cudaGetLastError(); return AMPQ_ERR_CUDA; }

    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    const float preset = amax > 0.0f ? amax : (amax == 0.0f ? 0.0f : -1.0f);  // -0 -> +0
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 1) { cudaGetLastError(); return AMPQ_ERR_CUDA; }
    // the tile the ordinary pass would take for this size, enlarged until the tiles fit in the fixed slots
    int shift = pick_tile_shift(numel, kScoreCtasPerSm * sms);
    while (shift < kMaxTileShift && ((numel + (1LL << shift) - 1) >> shift) > kNoAllocMaxTiles) ++shift;
    const long long ntiles = (numel + (1LL << shift) - 1) >> shift;
    const long long namax = preset >= 0.0f ? 0 : (numel + kAmaxTileElems - 1) / kAmaxTileElems;
    const int fmask = fmt == AMPQ_FMT_E4M3 ? kMaskE4M3 : kMaskE5M2;
    noalloc_prepare_kernel<<<1, 32, 0, st>>>(s, values, grads, numel, dtype, preset, ntiles, namax);
    bool ok = cudaGetLastError() == cudaSuccess;
    ok = ok && launch_init_amax(&s->tensor, 1, &s->amax_bits, &s->status, st) == cudaSuccess;
    ok = ok && launch_amax(&s->tensor, s->amax_tile_begin, 1, namax, kAmaxTileElems, &s->amax_bits, st) == cudaSuccess;
    ok = ok && launch_scales(1, fmask, &s->tensor, &s->amax_bits, s->scales, &s->flag, &s->status, st) == cudaSuccess;
    ok = ok && launch_score(dtype == AMPQ_F32 ? 0 : 1, 1, &s->tensor, s->tile_begin, 1, ntiles, shift, kScoreCtasPerSm * sms, fmask, s->scales,
                            s->partials, &s->status, st) == cudaSuccess;
    ok = ok && launch_finalize(&s->segment, 1, kNoAllocAcc, s->partials, s->seg_out, st) == cudaSuccess;
    if (ok) {
        noalloc_publish_kernel<<<1, 32, 0, st>>>(s, dev_out);
        ok = cudaGetLastError() == cudaSuccess;
    }
    if (!ok) { cudaGetLastError(); return AMPQ_ERR_CUDA; }
    return AMPQ_OK;
}

#pragma GCC visibility pop
}  // extern "C"

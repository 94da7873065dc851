// Host-callable launchers of the kernels in ampq_kernels.cu.
#pragma once
#include <cuda_runtime.h>

#include "ampq_device.h"

namespace ampq {

// alpha[f] = 2^(-2 m_f)/12 of user format index f (entry 0 unused: the baseline
// costs 0); acc_of_fmt[f] = accumulator column (1 or 2) holding D of format f.
struct CombineParams {
    double alpha[1 + kMaxLow];
    int acc_of_fmt[1 + kMaxLow];
    int nacc;
};

// The scales step: scale and inverse scale of every tensor from its amax.  As a
// launch of its own (launch_scales), or as the tail of the amax kernel
// (launch_amax with counter set): the amax CTA that finishes last runs it.
struct ScalesArgs {
    unsigned* counter = nullptr;  // tail only: zeroed before the launch, counts finished amax CTAs
    int T = 0, fmask = 0, pow2 = 0;
    const Tensor* tens = nullptr;
    unsigned* amax_bits = nullptr;
    float* scales = nullptr;
    int* flags = nullptr;
    LaunchStatus* status = nullptr;
};

// The per-layer combine as the tail of the finalize kernel (counter set): the
// finalize CTA that finishes last runs it.
struct CombineArgs {
    unsigned* counter = nullptr;
    const Layer* layers = nullptr;
    int L = 0, F = 0;
    CombineParams prm{};
    double* layer_out = nullptr;
};

cudaError_t launch_init_amax(const Tensor* tens, int T, unsigned* amax_bits, LaunchStatus* status,
                             cudaStream_t st);
// One CTA per tile of tile_elems elements (kMinAmaxTileElems..kAmaxTileElems; tile_begin counts such tiles).
// Triangular operands need tile_elems = kAmaxTileElems (whole matrix rows per tile).
cudaError_t launch_amax(const Tensor* tens, const long long* tile_begin, int T, long long ntiles, int tile_elems,
                        unsigned* amax_bits, cudaStream_t st, const ScalesArgs& tail = ScalesArgs());
// Amax tile for a pass over `elems` elements on `sms` SMs: the largest that still gives every SM a few tiles.
int pick_amax_tile(long long elems, int sms);
// pow2 = 1: power-of-two scales instead of amax / fmax.  Tensors whose amax_src
// names another tensor take (and record) that tensor's amax.
cudaError_t launch_scales(int T, int fmask, const Tensor* tens, unsigned* amax_bits, float* scales, int* tensor_flags,
                          LaunchStatus* status, cudaStream_t st, int pow2 = 0);
inline ScalesArgs scales_args(int T, int fmask, const Tensor* tens, unsigned* amax_bits, float* scales, int* flags,
                              LaunchStatus* status, int pow2, unsigned* counter = nullptr) {
    ScalesArgs a;
    a.counter = counter; a.T = T; a.fmask = fmask; a.pow2 = pow2; a.tens = tens; a.amax_bits = amax_bits;
    a.scales = scales; a.flags = flags; a.status = status;
    return a;
}
// Only that alias step (after an amax pass that is not followed by a score).
cudaError_t launch_resolve_amax(int T, const Tensor* tens, unsigned* amax_bits, cudaStream_t st);
// One launch per element type (0 = fp32, 1 = bf16) and number of gradient
// streams per read of the values rb = 1..kMaxRB (samples of a shared operand, or
// layers reading one per-sample operand), each with its own tile table; causal = 1 (rb = 1 only): the
// table holds triangular operands (Tensor::causal_shift > 0).  fmask = 0 scores
// only S (no cast, scales unused).  out_stride = doubles per partial slot when
// that is more than the kernel's own accumulator count (0: exactly that count).
// Tiles hold 2^tile_shift elements; the persistent grid has at most max_ctas CTAs
// (two per SM is the intended residency).
cudaError_t launch_score(int dtype, int rb, const Tensor* tens, const long long* tile_begin, int T, long long ntiles,
                         int tile_shift, int max_ctas, int fmask, const float* scales, double* partials,
                         LaunchStatus* status, cudaStream_t st, int causal = 0, int out_stride = 0);
// Largest tile shift in [kMinTileShift, kMaxTileShift] that still gives a grid of
// max_ctas CTAs 16 tiles each (or the smallest shift when even that does not).
int pick_tile_shift(long long scored_elems, int max_ctas);
cudaError_t launch_finalize(const Segment* segs, int nseg, int nacc, const double* partials, double* seg_out,
                            cudaStream_t st, const CombineArgs& tail = CombineArgs());
cudaError_t launch_combine(const Layer* layers, int L, int F, const CombineParams& prm, const double* seg_out,
                           double* layer_out, cudaStream_t st);
// One-segment jobs.  launch_job_prepare fills a job's tables on the device and,
// when the amax is preset (no amax pass follows), forms the scales at once
// (fmask, pow2, status as for launch_scales).  launch_job_finish sums the job's
// per-tile partials into seg_out (nacc doubles) and folds its amax / flag /
// scales into the per-tensor arrays.
cudaError_t launch_job_prepare(SegmentJob* job, const void* values, const void* grads, long long n, int dtype,
                               float amax_preset, long long ntiles, long long namax, int fmask, int pow2,
                               LaunchStatus* status, cudaStream_t st);
cudaError_t launch_job_finish(const SegmentJob* job, int nacc, const double* partials, double* seg_out, int tensor,
                              unsigned* amax_bits, int* flags, float* scales, cudaStream_t st);
// scale_pair = {scale, inv_scale} on the device; out has the operand's dtype.
cudaError_t launch_fake_quant(int dtype, int fmt_mask, const void* values, long long n, const float* scale_pair,
                              void* out, cudaStream_t st);
cudaError_t launch_codes(int dtype, int fmt_mask, const void* values, long long n, const float* scale_pair,
                         unsigned char* out, cudaStream_t st);

}  // namespace ampq

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

cudaError_t launch_init_amax(const Tensor* tens, int T, unsigned* amax_bits, LaunchStatus* status,
                             cudaStream_t st);
cudaError_t launch_amax(const Tensor* tens, const long long* tile_begin, int T, long long ntiles,
                        unsigned* amax_bits, cudaStream_t st);
// pow2 = 1: power-of-two scales instead of amax / fmax.  Tensors whose amax_src
// names another tensor take (and record) that tensor's amax.
cudaError_t launch_scales(int T, int fmask, const Tensor* tens, unsigned* amax_bits, float* scales, int* tensor_flags,
                          LaunchStatus* status, cudaStream_t st, int pow2 = 0);
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
// max_ctas CTAs a few dozen tiles each (or the smallest shift when even that does not).
int pick_tile_shift(long long scored_elems, int max_ctas);
cudaError_t launch_finalize(const Segment* segs, int nseg, int nacc, const double* partials, double* seg_out,
                            cudaStream_t st);
cudaError_t launch_combine(const Layer* layers, int L, int F, const CombineParams& prm, const double* seg_out,
                           double* layer_out, cudaStream_t st);
// One-segment jobs: fill a job's tables on the device, fold its amax / flag /
// scales into per-tensor arrays afterwards.
cudaError_t launch_job_prepare(SegmentJob* job, const void* values, const void* grads, long long n, int dtype,
                               float amax_preset, long long ntiles, long long namax, cudaStream_t st);
cudaError_t launch_job_fold(const SegmentJob* job, int tensor, unsigned* amax_bits, int* flags, float* scales,
                            cudaStream_t st);
// scale_pair = {scale, inv_scale} on the device; out has the operand's dtype.
cudaError_t launch_fake_quant(int dtype, int fmt_mask, const void* values, long long n, const float* scale_pair,
                              void* out, cudaStream_t st);
cudaError_t launch_codes(int dtype, int fmt_mask, const void* values, long long n, const float* scale_pair,
                         unsigned char* out, cudaStream_t st);

}  // namespace ampq

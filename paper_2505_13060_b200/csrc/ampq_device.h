// Device-side tables shared by the kernels (ampq_kernels.cu) and the host
// library (ampq_lib.cu).  Plain structs, no torch types.
#pragma once
#include <cstdint>

namespace ampq {

#ifndef AMPQ_AMAX_TILE_ELEMS
#define AMPQ_AMAX_TILE_ELEMS 32768
#endif

constexpr int kThreads = 256;          // threads per CTA of the amax kernel
constexpr int kConsumers = 256;        // scoring threads of a scoring CTA (warps 0..7)
constexpr int kScoreThreads = kConsumers + 32;  // plus the producer warp that feeds the shared-memory ring
#ifndef AMPQ_SCORE_CTAS_PER_SM
#define AMPQ_SCORE_CTAS_PER_SM 2
#endif
constexpr int kScoreCtasPerSm = AMPQ_SCORE_CTAS_PER_SM;  // resident scoring CTAs per SM; the persistent grid is this many per SM
constexpr int kSubElems = 32768;       // direct path: elements between two flushes of the fp32 accumulators into fp64
constexpr int kFlushTerms = 64;        // ring path: terms an fp32 accumulator lane takes between two flushes into fp64
constexpr unsigned kSpinLimit = 1u << 22;  // polls of an mbarrier before a wait gives up
// A scoring tile (one partial sum per sample and accumulator) holds 2^shift
// elements of a segment; the host picks the shift per score so that small
// problems still spread over every SM and large ones pay few tile ends.
constexpr int kMinTileShift = 13;
#ifndef AMPQ_MAX_TILE_SHIFT
#define AMPQ_MAX_TILE_SHIFT 21
#endif
constexpr int kMaxTileShift = AMPQ_MAX_TILE_SHIFT;
constexpr int kTileElems = 1 << kMaxTileShift;        // largest scoring tile
constexpr int kAmaxTileElems = AMPQ_AMAX_TILE_ELEMS;  // elements of one amax tile of a large pass
constexpr int kMinAmaxTileElems = 4096;               // small passes take smaller tiles so that they still spread over the SMs
static_assert(kSubElems % (1 << kMinTileShift) == 0, "a flush block is a whole number of the smallest scoring tiles");
static_assert(kAmaxTileElems >= (1 << 15), "an amax tile holds whole rows of the largest triangular matrix");
constexpr int kMaxLow = 2;             // low-precision formats scored in one pass
constexpr int kMaxAcc = 1 + kMaxLow;   // accumulators per segment: S, D_0, D_1
constexpr int kMaxRB = 4;              // gradient streams per read of the values: samples of a shared operand, or layers reading one input
constexpr int kScoreClasses = 2 * kMaxRB + 2;  // scoring launches of one score: element type x streams per read,
                                               // plus one class per element type for causal (triangular) operands
constexpr int kMinCausalShift = 6, kMaxCausalShift = 15;  // T between 64 and 32768

// internal low-precision slots: bit 0 = E4M3, bit 1 = E5M2.  With both present
// slot 0 is E4M3 and slot 1 is E5M2; with one present it is slot 0.
constexpr int kMaskE4M3 = 1;
constexpr int kMaskE5M2 = 2;

// One bound operand of a scored layer.
struct Tensor {
    const void* values;      // device pointer, numel elements
    const void* grads;       // device pointer; sample r at grads + r*grad_stride
    long long numel;         // value elements in total
    long long seg_len;       // elements of one segment: numel/R (per-sample) or numel (shared)
    long long grad_stride;   // elements between consecutive samples' gradients
    long long partial_base;  // partial slot of (r, i) = partial_base + r*tiles_per_seg + i
    int tiles_per_seg;       // ceil(seg_len / tile elements of this score)
    int R;                   // calibration samples
    int per_sample;          // 1: values are [R, seg_len]; 0: shared by all samples
    int dtype;               // AMPQ_F32 / AMPQ_BF16
    int share_n;             // layers that read one per-sample operand are scored in one read of its values:
                             // 1: on its own; n = 2..kMaxRB: first of n such tensors, its tiles carry the
                             // gradient streams of all n; 0: one of the others (no tiles of its own)
    int seg_base;            // index of segment (this tensor, r = 0) in the segment outputs
    float amax_preset;       // >= 0: use instead of measuring
    int causal_shift;        // > 0: segments are stacks of T x T matrices, T = 2^causal_shift, whose strictly
                             // upper triangles are exactly zero and are not read; 0: dense
    int amax_src;            // index of the tensor whose measured amax this one takes (a tensor bound to the
                             // very same values); its own index otherwise
    // Gradient streams 1..kMaxRB-1 of a tile that reads its values once for several
    // streams (stream 0 is `grads`); stream j of a tile at sample r0 starts at
    // gstream[j-1] + r0*grad_stride.  Shared values (weights): grads + j*grad_stride,
    // the next samples' gradients.  share_n > 1: the gradients of tensors
    // 1..share_n-1 of the group.  stream_slot_stride = partial slots between two
    // streams: tiles_per_seg (next sample) or R*tiles_per_seg (next tensor).
    const void* gstream[kMaxRB - 1];
    long long stream_slot_stride;
};

// One segment = (tensor, sample): its partial slots are contiguous.
struct Segment {
    long long first_slot;
    int count;
    int pad;
};

// One scored layer for the combine step.
struct Layer {
    int seg_base0, seg_base1;  // segment index of (operand, r = 0)
    int tensor0, tensor1;
    int R;
    int out_off;               // offset (doubles) of this layer's block in the layer outputs
};

// Layer output block layout (doubles): s_r[R], s_mean, d_meas_r[R*F], d_model[F], d_meas[F]
inline int layer_block_doubles(int R, int F) { return R + 1 + R * F + 2 * F; }

// The tables of a one-tensor, one-sample scoring job (streaming calibration,
// fake quantisation): what a full score keeps in separate arrays, for one segment.
struct SegmentJob {
    Tensor tensor;
    long long tile_begin[2];       // scoring tiles {0, ntiles}
    long long amax_tile_begin[2];  // amax tiles {0, n_amax_tiles}
    Segment segment;
    unsigned amax_bits;
    int flag;                      // 1: the tensor held Inf/NaN
    float scales[2 * kMaxLow];
    unsigned amax_done;            // amax CTAs that have finished (the last one forms the scales)
};

struct LaunchStatus {
    int nonfinite;  // set when some tensor's amax is Inf/NaN
    int timeout;    // set when a wait inside the scoring kernel ran out
    int bounds;     // set by a -DAMPQ_BOUNDS_CHECK build when a tile falls outside its tensor
    unsigned amax_done;      // amax CTAs that have finished: the last one forms the scales
    unsigned finalize_done;  // finalize CTAs that have finished: the last one combines the layers
};

}  // namespace ampq

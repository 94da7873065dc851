// C ABI of the sensitivity pass (include/ampq.h): registry of layers, operands
// and groups, the device work tables, the launch sequence, result read-back,
// sub-graph sums and the selection call.  Host code; the arithmetic of the hot
// path is in ampq_kernels.cu.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/ampq.h"
#include "ampq_device.h"
#include "ampq_kernels.h"
#include "ampq_select.h"

using namespace ampq;

namespace {

struct Operand {
    bool bound = false;
    int dtype = 0, mem = 0, per_sample = 0;
    const void* values = nullptr;
    const void* grads = nullptr;
    long long numel = 0, grad_stride = 0;
    float amax_preset = -1.0f;
    long long causal_T = 0;  // > 0: declared a stack of T x T lower-triangular matrices
    void* stage = nullptr;  // device staging for host-bound operands
    size_t stage_bytes = 0;
    int tensor = -1;        // index in the tables of the last score, or -1
};

struct LayerRec {
    int kind = 0, R = 1;
    std::string name;
    Operand op[2];
    int scored = -1;  // index among the layers of the last score, or -1
};

struct Group {
    std::vector<int> layers;
    std::vector<unsigned char> Q;
    std::vector<double> c;
    int P = 0;
};

template <typename T>
struct DevBuf {
    T* p = nullptr;
    size_t cap = 0;
    cudaError_t ensure(size_t n) {
        if (n <= cap) return cudaSuccess;
        if (p) cudaFree(p);
        p = nullptr;
        cap = 0;
        size_t want = n + n / 4 + 16;
        cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&p), want * sizeof(T));
        if (e == cudaSuccess) cap = want;
        return e;
    }
    void release() {
        if (p) cudaFree(p);
        p = nullptr;
        cap = 0;
    }
};

template <typename T>
struct PinBuf {
    T* p = nullptr;
    size_t cap = 0;
    cudaError_t ensure(size_t n) {
        if (n <= cap) return cudaSuccess;
        if (p) cudaFreeHost(p);
        p = nullptr;
        cap = 0;
        size_t want = n + n / 4 + 16;
        cudaError_t e = cudaMallocHost(reinterpret_cast<void**>(&p), want * sizeof(T));
        if (e == cudaSuccess) cap = want;
        return e;
    }
    void release() {
        if (p) cudaFreeHost(p);
        p = nullptr;
        cap = 0;
    }
};

// A typed window into the result arena (see ensure_results).
template <typename T>
struct View {
    T* p = nullptr;
};

int mantissa_bits_of(int fmt) { return fmt == AMPQ_FMT_E4M3 ? 3 : (fmt == AMPQ_FMT_E5M2 ? 2 : 7); }

}  // namespace

struct ampq_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    int F = 2;
    int fmt[1 + kMaxLow] = {AMPQ_FMT_BASE, AMPQ_FMT_E4M3, 0};
    int fmask = kMaskE4M3;
    int slot_of_fmt[1 + kMaxLow] = {-1, 0, -1};  // user format index -> internal low slot
    std::vector<LayerRec> layers;
    std::vector<Group> groups;
    int scale_pow2 = 0;    // AMPQ_SCALE_POW2: power-of-two scales
    bool measured = true;  // false: only the model term S is scored (no amax pass, no cast)
    bool sharing = true;   // layers bound to the very same values share its amax and one read of it
    bool amax_ready = false;  // ampq_measure_amax (or a score) has filled the amax mirror
    bool dirty = true;     // bindings changed since the tables were built
    bool scored = false;   // a score has been issued
    bool pending = false;  // its results have not been synchronised yet
    int launches = 0;
    int max_ctas = kScoreCtasPerSm;  // persistent scoring grid: kScoreCtasPerSm CTAs per SM
    int tile_shift = kMaxTileShift;  // log2 of the scoring tile of the last score
    int amax_tile = kAmaxTileElems;  // elements of an amax tile of the last pass
    int sms = 1;
    std::string err;

    // tables of the last score (host copies)
    std::vector<Tensor> tens;
    // tile_begin[dtype * kMaxRB + rb - 1]: tiles of `dtype` operands scored with rb gradient streams per read
    std::vector<long long> tile_begin[kScoreClasses], amax_tile_begin;
    std::vector<Segment> segs;
    std::vector<Layer> lay;
    std::vector<int> scored_layer_ids;
    long long ntiles[kScoreClasses] = {}, namax_tiles = 0, nslots = 0;
    int n_amax_alias = 0;     // tensors that take an earlier tensor's amax (bound to the very same values)
    int n_share_groups = 0;   // groups of layers scored in one read of a per-sample operand they share
    long long amax_bytes = 0, score_bytes = 0;  // bytes of bound tensors the two passes of a score read
    int layer_out_doubles = 0;

    DevBuf<Tensor> d_tens;
    DevBuf<long long> d_tile_begin[kScoreClasses], d_amax_tile_begin;
    DevBuf<Segment> d_segs;
    DevBuf<Layer> d_lay;
    DevBuf<double> d_partials;
    // Every small result of a pass lives in ONE device arena with ONE pinned host
    // mirror of the same layout, so that reading a pass back is a single copy:
    // status | amax_bits[T] | flags[T] | scales[T][2][kMaxLow] | seg_out | layer_out
    DevBuf<unsigned char> d_arena;
    PinBuf<unsigned char> h_arena;
    size_t arena_bytes = 0;  // bytes of the current layout
    View<LaunchStatus> d_status, h_status;
    View<unsigned> d_amax_bits, h_amax_bits;
    View<int> d_flags, h_flags;
    View<float> d_scales, h_scales;
    View<double> d_seg_out, h_seg_out, d_layer_out, h_layer_out;
    DevBuf<LaunchStatus> d_fq_status;  // status word of fake-quantisation calls (outside any pass)

    // streaming calibration (ampq_stream_*) and fake quantisation
    bool streaming = false;
    std::vector<int> stream_seg_base;   // [2*layer + operand] -> first segment (sample 0)
    DevBuf<SegmentJob> d_jobs;          // one job per (tensor, sample) of a streaming pass
    DevBuf<double> d_job_partials;      // per-tile partials of the job in flight (jobs are ordered on the stream)
    DevBuf<SegmentJob> d_fq_job;        // tables of a fake-quantisation call
    std::vector<void*> retired;         // outgrown job-partial buffers, freed when no job can be in flight
    size_t job_partials_hint = 0;       // doubles of the last job-partial allocation

    bool timing = false;            // record CUDA events around the kernels of a score
    cudaEvent_t ev[6] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    bool ev_valid = false;
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

int fail(ampq_ctx* ctx, int code, const std::string& msg) {
    if (ctx) ctx->err = msg;
    return code;
}

int cuda_fail(ampq_ctx* ctx, cudaError_t e, const char* where) {
    if (ctx) ctx->err = std::string(where) + ": " + cudaGetErrorString(e);
    return AMPQ_ERR_CUDA;
}

#define AMPQ_CUDA(call, where)                         \
    do {                                               \
        cudaError_t e__ = (call);                      \
        if (e__ != cudaSuccess) return cuda_fail(ctx, e__, where); \
    } while (0)

bool layer_ready(const LayerRec& l) { return l.op[0].bound && l.op[1].bound; }

long long extent_of(const LayerRec& l, const Operand& o) { return o.per_sample ? o.numel / l.R : o.numel; }

// Lays the result arena out for T tensors, S segments of nacc doubles and
// layer_doubles doubles of layer blocks, growing the two allocations if needed.
// Only called when no pass is pending.
int ensure_results(ampq_ctx* ctx, size_t T, size_t S, int nacc, size_t layer_doubles) {
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    const size_t o_status = 0;
    const size_t o_amax = up(sizeof(LaunchStatus));
    const size_t o_flags = o_amax + up(T * sizeof(unsigned));
    const size_t o_scales = o_flags + up(T * sizeof(int));
    const size_t o_seg = o_scales + up(T * 2 * kMaxLow * sizeof(float));
    const size_t o_layer = o_seg + up(S * nacc * sizeof(double));
    const size_t total = o_layer + up(layer_doubles * sizeof(double));
    AMPQ_CUDA(ctx->d_arena.ensure(total), "cudaMalloc(results)");
    AMPQ_CUDA(ctx->h_arena.ensure(total), "cudaMallocHost(results)");
    ctx->arena_bytes = total;
    unsigned char *d = ctx->d_arena.p, *h = ctx->h_arena.p;
    ctx->d_status.p = reinterpret_cast<LaunchStatus*>(d + o_status);
    ctx->h_status.p = reinterpret_cast<LaunchStatus*>(h + o_status);
    ctx->d_amax_bits.p = reinterpret_cast<unsigned*>(d + o_amax);
    ctx->h_amax_bits.p = reinterpret_cast<unsigned*>(h + o_amax);
    ctx->d_flags.p = reinterpret_cast<int*>(d + o_flags);
    ctx->h_flags.p = reinterpret_cast<int*>(h + o_flags);
    ctx->d_scales.p = reinterpret_cast<float*>(d + o_scales);
    ctx->h_scales.p = reinterpret_cast<float*>(h + o_scales);
    ctx->d_seg_out.p = reinterpret_cast<double*>(d + o_seg);
    ctx->h_seg_out.p = reinterpret_cast<double*>(h + o_seg);
    ctx->d_layer_out.p = reinterpret_cast<double*>(d + o_layer);
    ctx->h_layer_out.p = reinterpret_cast<double*>(h + o_layer);
    return AMPQ_OK;
}

// log2 T when the operand may be scored as a stack of lower-triangular T x T
// matrices, else 0 (scored densely, which gives the same sums).  The triangular
// path needs a power-of-two T in [64, 32768], whole matrices per sample, and
// 16-byte aligned sample slices of values and gradients.
int causal_shift_of(const LayerRec& l, const Operand& o) {
    const long long T = o.causal_T;
    if (T <= 0 || !o.per_sample || (T & (T - 1))) return 0;
    int shift = 0;
    while ((1LL << shift) < T) ++shift;
    if (shift < kMinCausalShift || shift > kMaxCausalShift) return 0;
    const long long seg_len = extent_of(l, o);
    if (seg_len == 0 || seg_len % (T * T)) return 0;
    if (o.mem == AMPQ_MEM_HOST) return shift;  // staged: 256-byte aligned, samples back to back
    const int es = o.dtype == AMPQ_F32 ? 4 : 2;
    if ((reinterpret_cast<uintptr_t>(o.values) & 15) || (reinterpret_cast<uintptr_t>(o.grads) & 15)) return 0;
    if ((seg_len * es) % 16) return 0;
    if (l.R > 1 && (o.grad_stride * es) % 16) return 0;
    return shift;
}

// What makes two per-sample operands "the same input read by several layers".
struct ShareKey {
    const void* values;
    long long numel, grad_stride;
    int dtype, R;
    unsigned preset_bits;
    bool operator==(const ShareKey& o) const {
        return values == o.values && numel == o.numel && grad_stride == o.grad_stride && dtype == o.dtype && R == o.R &&
               preset_bits == o.preset_bits;
    }
};

struct ShareGroup {
    ShareKey key;
    std::vector<const Operand*> members;  // in registration order; members[0] carries the tiles
    int leader_tensor = -1;
    long long leader_base = 0;
    int leader_amax_src = -1;
};

// Builds the host tables for every layer whose two operands are bound.
int build_tables(ampq_ctx* ctx) {
    ctx->tens.clear(); ctx->amax_tile_begin.clear();
    ctx->n_amax_alias = 0; ctx->n_share_groups = 0;
    ctx->amax_bytes = 0; ctx->score_bytes = 0;
    for (auto& tb : ctx->tile_begin) tb.clear();
    ctx->segs.clear(); ctx->lay.clear(); ctx->scored_layer_ids.clear();
    for (auto& l : ctx->layers) { l.scored = -1; l.op[0].tensor = l.op[1].tensor = -1; }
    long long tiles[kScoreClasses] = {}, atiles = 0, slots = 0;
    int out_off = 0;
    std::vector<char> measures_amax;  // per tensor: it has amax tiles of its own

    // Layers that read one input (q, k, v or gate, up of a transformer block) bind
    // the very same per-sample values with gradients of their own.  Up to kMaxRB
    // of them form a group that is scored like a weight with several per-sample
    // gradients: the values are read and cast once per tile, every member's
    // gradient is one more stream of that tile.
    std::vector<ShareGroup> groups;
    std::vector<std::pair<int, int>> role(ctx->layers.size() * 2, {-1, 0});  // (group, position) per operand
    if (ctx->sharing) {
        for (size_t li = 0; li < ctx->layers.size(); ++li) {
            const LayerRec& l = ctx->layers[li];
            if (!layer_ready(l)) continue;
            for (int k = 0; k < 2; ++k) {
                const Operand& o = l.op[k];
                if (o.mem != AMPQ_MEM_DEVICE || !o.per_sample || o.numel == 0 || o.causal_T != 0) continue;
                unsigned pb;
                std::memcpy(&pb, &o.amax_preset, sizeof pb);
                const ShareKey key{o.values, o.numel, o.grad_stride, o.dtype, l.R, pb};
                int g = -1;
                for (size_t e = groups.size(); e-- > 0;)  // the latest group of this key that still has room
                    if (groups[e].key == key) { if ((int)groups[e].members.size() < kMaxRB) g = (int)e; break; }
                if (g < 0) { groups.push_back(ShareGroup{key, {}, -1, 0, -1}); g = (int)groups.size() - 1; }
                role[2 * li + k] = {g, (int)groups[g].members.size()};
                groups[g].members.push_back(&o);
            }
        }
    }
    long long scored_elems = 0;  // value elements the scoring launches walk (shared values once per sample group)
    for (size_t li = 0; li < ctx->layers.size(); ++li) {
        const LayerRec& l = ctx->layers[li];
        if (!layer_ready(l)) continue;
        for (int k = 0; k < 2; ++k) {
            if (role[2 * li + k].first >= 0 && role[2 * li + k].second > 0) continue;  // read with its group's first member
            scored_elems += l.op[k].per_sample ? l.op[k].numel : l.op[k].numel * ((l.R + kMaxRB - 1) / kMaxRB);
        }
    }
    ctx->tile_shift = pick_tile_shift(scored_elems, ctx->max_ctas);
    {   // amax tiles: smaller for a small pass; whole matrix rows per tile when a triangular operand is present
        long long measured_elems = 0;
        bool triangular = false;
        for (const auto& l : ctx->layers) {
            if (!layer_ready(l)) continue;
            for (int k = 0; k < 2; ++k) {
                if (l.op[k].amax_preset < 0.0f) measured_elems += l.op[k].numel;
                triangular = triangular || causal_shift_of(l, l.op[k]) > 0;
            }
        }
        ctx->amax_tile = triangular ? kAmaxTileElems : pick_amax_tile(measured_elems, ctx->sms);
        if (triangular && ctx->tile_shift < kMaxCausalShift) ctx->tile_shift = kMaxCausalShift;  // a scoring tile holds whole rows too
    }
    const long long tile_elems = 1LL << ctx->tile_shift;
    for (size_t li = 0; li < ctx->layers.size(); ++li) {
        LayerRec& l = ctx->layers[li];
        if (!layer_ready(l)) continue;
        Layer ly{};
        ly.R = l.R;
        ly.out_off = out_off;
        out_off += layer_block_doubles(l.R, ctx->F);
        for (int k = 0; k < 2; ++k) {
            Operand& o = l.op[k];
            Tensor t{};
            const long long ext = extent_of(l, o);
            const int es = o.dtype == AMPQ_F32 ? 4 : 2;
            if (o.mem == AMPQ_MEM_HOST) {
                // staging: values, then R gradient slices back to back
                const size_t vbytes = (((size_t)o.numel * es) + 255) / 256 * 256;  // keeps the gradients 256-byte aligned
                const size_t need = vbytes + (size_t)l.R * ext * es;
                if (need > o.stage_bytes) {
                    if (o.stage) cudaFree(o.stage);
                    o.stage = nullptr; o.stage_bytes = 0;
                    if (need) {
                        AMPQ_CUDA(cudaMalloc(&o.stage, need), "cudaMalloc(staging)");
                        o.stage_bytes = need;
                    }
                }
                t.values = o.stage;
                t.grads = reinterpret_cast<const char*>(o.stage) + vbytes;
                t.grad_stride = ext;
            } else {
                t.values = o.values;
                t.grads = o.grads;
                t.grad_stride = o.grad_stride;
            }
            t.numel = o.numel;
            t.seg_len = ext;
            t.R = l.R;
            t.per_sample = o.per_sample;
            t.dtype = o.dtype;
            if ((ext + tile_elems - 1) / tile_elems > 0x7FFFFFFFLL)
                return fail(ctx, AMPQ_ERR_TOO_LARGE, "an operand has more than 2^31-1 tiles per sample");
            t.tiles_per_seg = (int)((ext + tile_elems - 1) / tile_elems);
            t.share_n = 1;
            t.stream_slot_stride = t.tiles_per_seg;
            for (int j = 1; j < kMaxRB; ++j)  // never read past the R samples: a tile of a shared operand has at most R streams
                t.gstream[j - 1] = reinterpret_cast<const char*>(t.grads) + (long long)j * t.grad_stride * es;
            t.seg_base = (int)ctx->segs.size();
            t.amax_preset = o.amax_preset;
            t.causal_shift = causal_shift_of(l, o);
            const int me = (int)ctx->tens.size();
            t.amax_src = me;
            const long long per_tensor_slots = (long long)l.R * t.tiles_per_seg;
            ShareGroup* grp = role[2 * li + k].first >= 0 ? &groups[role[2 * li + k].first] : nullptr;
            const int pos = role[2 * li + k].second;
            if (grp && grp->members.size() < 2) grp = nullptr;
            // per-sample operands: one single-sample tile per (sample, value tile);
            // shared operands: value tiles x full groups of kMaxRB samples, plus one
            // remainder group of R mod kMaxRB samples; an input read by n layers: the
            // first layer's tensor has one n-stream tile per (sample, value tile)
            long long my_tiles[kScoreClasses] = {};
            const int c0 = (o.dtype == AMPQ_F32 ? 0 : 1) * kMaxRB;  // classes of this operand's dtype
            long long my_atiles = o.amax_preset >= 0.0f ? 0 : (o.numel + ctx->amax_tile - 1) / ctx->amax_tile;
            if (grp && pos > 0) {
                t.share_n = 0;
                t.partial_base = grp->leader_base + pos * per_tensor_slots;
                if (my_atiles > 0) { t.amax_src = grp->leader_amax_src; ++ctx->n_amax_alias; }
                my_atiles = 0;
            } else {
                t.partial_base = slots;
                if (grp) {
                    const int n = (int)grp->members.size();
                    t.share_n = n;
                    for (int j = 1; j < n; ++j) t.gstream[j - 1] = grp->members[j]->grads;
                    t.stream_slot_stride = per_tensor_slots;
                    my_tiles[c0 + n - 1] = per_tensor_slots;
                    grp->leader_tensor = me;
                    grp->leader_base = slots;
                    slots += (long long)n * per_tensor_slots;
                    ++ctx->n_share_groups;
                } else {
                    if (t.causal_shift > 0) my_tiles[2 * kMaxRB + (o.dtype == AMPQ_F32 ? 0 : 1)] = per_tensor_slots;
                    else if (o.per_sample) my_tiles[c0] = per_tensor_slots;
                    else {
                        my_tiles[c0 + kMaxRB - 1] = (long long)t.tiles_per_seg * (l.R / kMaxRB);
                        if (l.R % kMaxRB) my_tiles[c0 + l.R % kMaxRB - 1] += t.tiles_per_seg;
                    }
                    slots += per_tensor_slots;
                }
                // A tensor bound to the very same device values as an earlier one needs no
                // amax pass of its own: it takes the earlier one's.
                if (ctx->sharing && my_atiles > 0 && o.mem == AMPQ_MEM_DEVICE) {
                    for (size_t e = 0; e < ctx->tens.size(); ++e) {
                        const Tensor& u = ctx->tens[e];
                        if (measures_amax[e] && u.values == t.values && u.numel == t.numel && u.dtype == t.dtype &&
                            u.causal_shift == t.causal_shift) {
                            t.amax_src = (int)e;
                            ++ctx->n_amax_alias;
                            my_atiles = 0;
                            break;
                        }
                    }
                }
                if (grp) grp->leader_amax_src = t.amax_src;
            }
            {
                // bytes read: a triangular operand keeps, of row i, the 16-byte vectors up to the diagonal
                long long kept = o.numel;
                if (t.causal_shift > 0) {
                    const long long T = 1LL << t.causal_shift, per = 16 / es, g = T / per;
                    kept = o.numel / (T * T) * (per * per * g * (g + 1) / 2);
                }
                if (my_atiles > 0) ctx->amax_bytes += kept * es;
                if (t.share_n > 0) {
                    const long long value_reads = o.per_sample ? 1 : (l.R + kMaxRB - 1) / kMaxRB;
                    const long long grad_streams = o.per_sample ? t.share_n : l.R;
                    ctx->score_bytes += kept * es * (value_reads + grad_streams);
                }
            }
            for (int c = 0; c < kScoreClasses; ++c) {
                ctx->tile_begin[c].push_back(tiles[c]);
                tiles[c] += my_tiles[c];
            }
            ctx->amax_tile_begin.push_back(atiles);
            atiles += my_atiles;
            measures_amax.push_back(my_atiles > 0);
            for (int r = 0; r < l.R; ++r) {
                Segment sg{};
                sg.first_slot = t.partial_base + (long long)r * t.tiles_per_seg;
                sg.count = t.tiles_per_seg;
                ctx->segs.push_back(sg);
            }
            o.tensor = me;
            if (k == 0) { ly.seg_base0 = t.seg_base; ly.tensor0 = o.tensor; }
            else { ly.seg_base1 = t.seg_base; ly.tensor1 = o.tensor; }
            ctx->tens.push_back(t);
        }
        l.scored = (int)ctx->lay.size();
        ctx->lay.push_back(ly);
        ctx->scored_layer_ids.push_back((int)li);
    }
    long long most = atiles;
    for (int c = 0; c < kScoreClasses; ++c) {
        ctx->tile_begin[c].push_back(tiles[c]);
        ctx->ntiles[c] = tiles[c];
        if (tiles[c] > most) most = tiles[c];
    }
    ctx->amax_tile_begin.push_back(atiles);
    ctx->namax_tiles = atiles;
    ctx->nslots = slots;
    ctx->layer_out_doubles = out_off;
    if (most > 0x7FFFFFFFLL)
        return fail(ctx, AMPQ_ERR_TOO_LARGE, "more than 2^31-1 tiles in one score");
    return AMPQ_OK;
}

int upload_tables(ampq_ctx* ctx) {
    const size_t T = ctx->tens.size(), L = ctx->lay.size(), S = ctx->segs.size();
    const int nacc = 1 + (ctx->F - 1);
    AMPQ_CUDA(ctx->d_tens.ensure(T), "cudaMalloc(tensors)");
    for (int c = 0; c < kScoreClasses; ++c) AMPQ_CUDA(ctx->d_tile_begin[c].ensure(T + 1), "cudaMalloc(tile_begin)");
    AMPQ_CUDA(ctx->d_amax_tile_begin.ensure(T + 1), "cudaMalloc(amax_tile_begin)");
    AMPQ_CUDA(ctx->d_segs.ensure(S), "cudaMalloc(segments)");
    AMPQ_CUDA(ctx->d_lay.ensure(L), "cudaMalloc(layers)");
    AMPQ_CUDA(ctx->d_partials.ensure((size_t)ctx->nslots * nacc), "cudaMalloc(partials)");
    {
        const int rc = ensure_results(ctx, T, S, nacc, (size_t)ctx->layer_out_doubles);
        if (rc) return rc;
    }
    cudaStream_t st = ctx->stream;
    if (T) {
        AMPQ_CUDA(cudaMemcpyAsync(ctx->d_tens.p, ctx->tens.data(), T * sizeof(Tensor), cudaMemcpyHostToDevice, st), "H2D tensors");
        AMPQ_CUDA(cudaMemsetAsync(ctx->d_scales.p, 0, T * 2 * kMaxLow * sizeof(float), st), "memset scales");
    }
    for (int c = 0; c < kScoreClasses; ++c)
        AMPQ_CUDA(cudaMemcpyAsync(ctx->d_tile_begin[c].p, ctx->tile_begin[c].data(), (T + 1) * sizeof(long long), cudaMemcpyHostToDevice, st), "H2D tile_begin");
    AMPQ_CUDA(cudaMemcpyAsync(ctx->d_amax_tile_begin.p, ctx->amax_tile_begin.data(), (T + 1) * sizeof(long long), cudaMemcpyHostToDevice, st), "H2D amax_tile_begin");
    if (S) AMPQ_CUDA(cudaMemcpyAsync(ctx->d_segs.p, ctx->segs.data(), S * sizeof(Segment), cudaMemcpyHostToDevice, st), "H2D segments");
    if (L) AMPQ_CUDA(cudaMemcpyAsync(ctx->d_lay.p, ctx->lay.data(), L * sizeof(Layer), cudaMemcpyHostToDevice, st), "H2D layers");
    return AMPQ_OK;
}

// Copies host-bound operands into their device staging on the stream.
int stage_host_operands(ampq_ctx* ctx) {
    for (auto& l : ctx->layers) {
        if (l.scored < 0) continue;
        for (int k = 0; k < 2; ++k) {
            Operand& o = l.op[k];
            if (o.mem != AMPQ_MEM_HOST || o.numel == 0) continue;
            const int es = o.dtype == AMPQ_F32 ? 4 : 2;
            const long long ext = extent_of(l, o);
            char* dst = reinterpret_cast<char*>(o.stage);
            AMPQ_CUDA(cudaMemcpyAsync(dst, o.values, (size_t)o.numel * es, cudaMemcpyHostToDevice, ctx->stream), "H2D values");
            dst += (((size_t)o.numel * es) + 255) / 256 * 256;
            if (o.grad_stride == ext) {
                AMPQ_CUDA(cudaMemcpyAsync(dst, o.grads, (size_t)l.R * ext * es, cudaMemcpyHostToDevice, ctx->stream), "H2D grads");
            } else {
                for (int r = 0; r < l.R; ++r)
                    AMPQ_CUDA(cudaMemcpyAsync(dst + (size_t)r * ext * es,
                                              reinterpret_cast<const char*>(o.grads) + (size_t)r * o.grad_stride * es,
                                              (size_t)ext * es, cudaMemcpyHostToDevice, ctx->stream), "H2D grads");
            }
        }
    }
    return AMPQ_OK;
}

void free_retired(ampq_ctx* ctx) {
    for (void* p : ctx->retired) cudaFree(p);
    ctx->retired.clear();
}

int sync_results(ampq_ctx* ctx) {
    if (!ctx->scored) return fail(ctx, AMPQ_ERR_STATE, "no score has been issued");
    if (ctx->pending) {
        AMPQ_CUDA(cudaStreamSynchronize(ctx->stream), "cudaStreamSynchronize");
        ctx->pending = false;
        free_retired(ctx);  // every job that could use them has finished
    }
    if (!ctx->tens.empty() && ctx->h_status.p->bounds)
        return fail(ctx, AMPQ_ERR_CUDA, "bounds check: a scoring tile fell outside its tensor (library bug); the results of this score are invalid");
    if (!ctx->tens.empty() && ctx->h_status.p->timeout)
        return fail(ctx, AMPQ_ERR_TIMEOUT, "a bounded wait inside the scoring kernel ran out; the results of this score are invalid");
    return AMPQ_OK;
}

int check_layer(ampq_ctx* ctx, int layer_id) {
    if (!ctx) return AMPQ_ERR_INVALID;
    if (layer_id < 0 || layer_id >= (int)ctx->layers.size()) return fail(ctx, AMPQ_ERR_INVALID, "unknown layer id");
    return AMPQ_OK;
}

const double* layer_block(const ampq_ctx* ctx, int scored) {
    return ctx->h_layer_out.p + ctx->lay[scored].out_off;
}

// d_{l,f} of a scored layer from the last score.
double layer_d(const ampq_ctx* ctx, int scored, int f, int d_mode) {
    const int R = ctx->lay[scored].R, F = ctx->F;
    const double* o = layer_block(ctx, scored);
    const double* d_model = o + R + 1 + (long long)R * F;
    const double* d_meas = d_model + F;
    return d_mode == AMPQ_D_MEASURED ? d_meas[f] : d_model[f];
}

int group_costs_impl(ampq_ctx* ctx, const Group& g, int d_mode, double* d_out) {
    const int Lj = (int)g.layers.size();
    for (int l = 0; l < Lj; ++l) {
        if (ctx->layers[g.layers[l]].scored < 0)
            return fail(ctx, AMPQ_ERR_STATE, "a layer of the group was not part of the last score");
        const int sc = ctx->layers[g.layers[l]].scored;
        if (ctx->h_flags.p[ctx->lay[sc].tensor0] || ctx->h_flags.p[ctx->lay[sc].tensor1])
            return fail(ctx, AMPQ_ERR_NONFINITE, "layer '" + ctx->layers[g.layers[l]].name + "' holds Inf/NaN");
    }
    for (int p = 0; p < g.P; ++p) {
        double d = 0.0;
        for (int l = 0; l < Lj; ++l)
            d += layer_d(ctx, ctx->layers[g.layers[l]].scored, g.Q[l + (size_t)Lj * p], d_mode);
        d_out[p] = d;
    }
    return AMPQ_OK;
}

// Common start of a full pass: wait for the previous read-back, end any
// streaming pass, rebuild and upload the tables when the bindings changed.
int prepare_tables(ampq_ctx* ctx) {
    int rc;
    if (ctx->pending) {  // the previous pass's read-back still owns the pinned mirrors
        AMPQ_CUDA(cudaStreamSynchronize(ctx->stream), "cudaStreamSynchronize");
        ctx->pending = false;
    }
    ctx->streaming = false;
    if (ctx->dirty) {
        ctx->scored = false;
        ctx->amax_ready = false;
        if ((rc = build_tables(ctx))) return rc;
        if ((rc = upload_tables(ctx))) return rc;
        ctx->dirty = false;
    }
    return AMPQ_OK;
}

// alpha_f = 2^(-2 m_f)/12 (Sec. 2.2) and the accumulator column of every format.
CombineParams combine_params(const ampq_ctx* ctx) {
    CombineParams prm{};
    prm.nacc = ctx->F;
    for (int f = 1; f < ctx->F; ++f) {
        prm.alpha[f] = std::ldexp(1.0, -2 * mantissa_bits_of(ctx->fmt[f])) / 12.0;
        prm.acc_of_fmt[f] = 1 + ctx->slot_of_fmt[f];
    }
    return prm;
}

// The asynchronous read-back of every small result of a pass.
int read_back(ampq_ctx* ctx) {
    AMPQ_CUDA(cudaMemcpyAsync(ctx->h_arena.p, ctx->d_arena.p, ctx->arena_bytes, cudaMemcpyDeviceToHost, ctx->stream), "D2H results");
    return AMPQ_OK;
}

// Per-tile partials of a streamed sample.  Jobs are ordered on the stream, so
// one buffer serves them all; when a larger sample arrives the buffer grows
// geometrically and the old one, which earlier jobs in flight may still use, is
// kept until the pass ends instead of being freed (a free would synchronise).
int ensure_job_partials(ampq_ctx* ctx, size_t n) {
    if (n <= ctx->d_job_partials.cap) return AMPQ_OK;
    if (ctx->d_job_partials.p) ctx->retired.push_back(ctx->d_job_partials.p);
    ctx->d_job_partials.p = nullptr;
    ctx->d_job_partials.cap = 0;
    size_t want = n > 2 * ctx->job_partials_hint ? n : 2 * ctx->job_partials_hint;
    AMPQ_CUDA(cudaMalloc(reinterpret_cast<void**>(&ctx->d_job_partials.p), want * sizeof(double)), "cudaMalloc(job partials)");
    ctx->d_job_partials.cap = want;
    ctx->job_partials_hint = want;
    return AMPQ_OK;
}

// Runs one (tensor, sample) job through amax / scales on the stream; the
// caller launches what follows.  job is a device pointer.
int job_amax_and_scales(ampq_ctx* ctx, SegmentJob* job, LaunchStatus* status, int dtype, const void* values,
                        const void* grads, long long numel, float preset, long long ntiles) {
    cudaStream_t st = ctx->stream;
    const int atile = pick_amax_tile(numel, ctx->sms);
    const long long namax = preset >= 0.0f ? 0 : (numel + atile - 1) / atile;
    // with a preset the scales are formed while the tables are filled; otherwise by the last CTA of the amax pass
    AMPQ_CUDA(launch_job_prepare(job, values, grads, numel, dtype, preset, ntiles, namax, ctx->fmask, ctx->scale_pow2, status, st), "job_prepare");
    ++ctx->launches;
    if (namax > 0) {
        AMPQ_CUDA(launch_amax(&job->tensor, job->amax_tile_begin, 1, namax, atile, &job->amax_bits, st,
                              scales_args(1, ctx->fmask, &job->tensor, &job->amax_bits, job->scales, &job->flag, status,
                                          ctx->scale_pow2, &job->amax_done)), "amax");
        ++ctx->launches;
    }
    return AMPQ_OK;
}

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

const char* ampq_strerror(int status) {
    switch (status) {
        case AMPQ_OK: return "ok";
        case AMPQ_ERR_INVALID: return "invalid argument";
        case AMPQ_ERR_ALIGN: return "tensor pointer not aligned to its element size";
        case AMPQ_ERR_STATE: return "call out of order";
        case AMPQ_ERR_CUDA: return "CUDA error";
        case AMPQ_ERR_NONFINITE: return "operand holds Inf or NaN";
        case AMPQ_ERR_INFEASIBLE: return "no assignment meets the budget";
        case AMPQ_ERR_TOO_LARGE: return "problem too large";
        case AMPQ_ERR_NOMEM: return "out of memory";
        case AMPQ_ERR_TIMEOUT: return "a device-side wait timed out";
        default: return "unknown status";
    }
}

const char* ampq_last_error(const ampq_ctx* ctx) { return ctx ? ctx->err.c_str() : ""; }

int ampq_create(ampq_ctx** out, int device, void* cuda_stream) {
    if (!out) return AMPQ_ERR_INVALID;
    *out = nullptr;
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || n <= 0) { cudaGetLastError(); return AMPQ_ERR_CUDA; }
    if (device < 0 || device >= n) return AMPQ_ERR_INVALID;
    ampq_ctx* ctx = new (std::nothrow) ampq_ctx();
    if (!ctx) return AMPQ_ERR_NOMEM;
    ctx->device = device;
    ctx->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    DeviceGuard g(device);
    if (!g.ok || cudaFree(nullptr) != cudaSuccess) { delete ctx; return AMPQ_ERR_CUDA; }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 1) {
        delete ctx;
        return AMPQ_ERR_CUDA;
    }
    ctx->max_ctas = kScoreCtasPerSm * sms;
    ctx->sms = sms;
    *out = ctx;
    return AMPQ_OK;
}

int ampq_destroy(ampq_ctx* ctx) {
    if (!ctx) return AMPQ_OK;
    {
        DeviceGuard g(ctx->device);
        if (ctx->pending || !ctx->retired.empty()) cudaStreamSynchronize(ctx->stream);
        free_retired(ctx);
        for (auto& l : ctx->layers)
            for (int k = 0; k < 2; ++k)
                if (l.op[k].stage) cudaFree(l.op[k].stage);
        ctx->d_tens.release(); ctx->d_amax_tile_begin.release();
        for (auto& b : ctx->d_tile_begin) b.release();
        ctx->d_segs.release(); ctx->d_lay.release(); ctx->d_partials.release();
        ctx->d_arena.release(); ctx->h_arena.release(); ctx->d_fq_status.release();
        ctx->d_jobs.release(); ctx->d_job_partials.release(); ctx->d_fq_job.release();
        for (int i = 0; i < 6; ++i)
            if (ctx->ev[i]) cudaEventDestroy(ctx->ev[i]);
    }
    delete ctx;
    return AMPQ_OK;
}

int ampq_set_formats(ampq_ctx* ctx, const int* fmt, int F) {
    if (!ctx || !fmt) return AMPQ_ERR_INVALID;
    if (F < 2 || F > 1 + kMaxLow) return fail(ctx, AMPQ_ERR_INVALID, "F must be 2 or 3");
    if (fmt[0] != AMPQ_FMT_BASE) return fail(ctx, AMPQ_ERR_INVALID, "fmt[0] must be AMPQ_FMT_BASE");
    if (ctx->streaming) return fail(ctx, AMPQ_ERR_STATE, "the formats cannot change inside a streaming pass");
    int mask = 0;
    for (int f = 1; f < F; ++f) {
        if (fmt[f] != AMPQ_FMT_E4M3 && fmt[f] != AMPQ_FMT_E5M2) return fail(ctx, AMPQ_ERR_INVALID, "unknown low-precision format");
        const int bit = fmt[f] == AMPQ_FMT_E4M3 ? kMaskE4M3 : kMaskE5M2;
        if (mask & bit) return fail(ctx, AMPQ_ERR_INVALID, "duplicate format");
        mask |= bit;
    }
    ctx->F = F;
    ctx->fmask = mask;
    for (int f = 0; f < 1 + kMaxLow; ++f) { ctx->fmt[f] = f < F ? fmt[f] : 0; ctx->slot_of_fmt[f] = -1; }
    for (int f = 1; f < F; ++f) ctx->slot_of_fmt[f] = (mask == 3 && fmt[f] == AMPQ_FMT_E5M2) ? 1 : 0;
    ctx->dirty = true;
    ctx->scored = false;
    return AMPQ_OK;
}

int ampq_register_layer(ampq_ctx* ctx, int kind, const char* name, int R, int* layer_id) {
    if (!ctx || !layer_id) return AMPQ_ERR_INVALID;
    if (kind != AMPQ_LINEAR && kind != AMPQ_BGEMM) return fail(ctx, AMPQ_ERR_INVALID, "unknown layer kind");
    if (R < 1) return fail(ctx, AMPQ_ERR_INVALID, "R must be at least 1");
    LayerRec l;
    l.kind = kind;
    l.R = R;
    if (name) l.name = name;
    ctx->layers.push_back(l);
    *layer_id = (int)ctx->layers.size() - 1;
    return AMPQ_OK;
}

int ampq_bind_operand(ampq_ctx* ctx, int layer_id, int operand, int dtype, int mem, const void* values,
                      long long numel, int per_sample_values, const void* grads, long long grad_stride) {
    int rc = check_layer(ctx, layer_id);
    if (rc) return rc;
    if (operand != 0 && operand != 1) return fail(ctx, AMPQ_ERR_INVALID, "operand must be 0 or 1");
    if (dtype != AMPQ_F32 && dtype != AMPQ_BF16) return fail(ctx, AMPQ_ERR_INVALID, "unknown dtype");
    if (mem != AMPQ_MEM_DEVICE && mem != AMPQ_MEM_HOST) return fail(ctx, AMPQ_ERR_INVALID, "unknown memory kind");
    if (numel < 0) return fail(ctx, AMPQ_ERR_INVALID, "negative numel");
    LayerRec& l = ctx->layers[layer_id];
    if (numel > 0 && (!values || !grads)) return fail(ctx, AMPQ_ERR_INVALID, "null tensor pointer");
    if (per_sample_values && numel % l.R != 0) return fail(ctx, AMPQ_ERR_INVALID, "numel is not a multiple of R");
    const long long ext = per_sample_values ? numel / l.R : numel;
    if (l.R > 1 && grad_stride < ext) return fail(ctx, AMPQ_ERR_INVALID, "grad_stride is smaller than one sample's gradient");
    const int es = dtype == AMPQ_F32 ? 4 : 2;
    if ((reinterpret_cast<uintptr_t>(values) % es) || (reinterpret_cast<uintptr_t>(grads) % es))
        return fail(ctx, AMPQ_ERR_ALIGN, "tensor pointer not aligned to its element size");
    Operand& o = l.op[operand];
    o.bound = true;
    o.dtype = dtype; o.mem = mem; o.per_sample = per_sample_values ? 1 : 0;
    o.values = values; o.grads = grads; o.numel = numel; o.grad_stride = grad_stride;
    ctx->dirty = true;
    return AMPQ_OK;
}

int ampq_set_amax(ampq_ctx* ctx, int layer_id, int operand, float amax) {
    int rc = check_layer(ctx, layer_id);
    if (rc) return rc;
    if (operand != 0 && operand != 1) return fail(ctx, AMPQ_ERR_INVALID, "operand must be 0 or 1");
    if (amax != amax || std::isinf(amax)) return fail(ctx, AMPQ_ERR_INVALID, "amax must be finite");
    ctx->layers[layer_id].op[operand].amax_preset = amax > 0.0f ? amax : (amax == 0.0f ? 0.0f : -1.0f);  // -0 -> +0
    ctx->dirty = true;
    return AMPQ_OK;
}

int ampq_set_scale_mode(ampq_ctx* ctx, int mode) {
    if (!ctx) return AMPQ_ERR_INVALID;
    if (mode != AMPQ_SCALE_AMAX && mode != AMPQ_SCALE_POW2) return fail(ctx, AMPQ_ERR_INVALID, "unknown scale mode");
    if (ctx->streaming) return fail(ctx, AMPQ_ERR_STATE, "the scale mode cannot change inside a streaming pass");
    ctx->scale_pow2 = mode == AMPQ_SCALE_POW2 ? 1 : 0;
    ctx->scored = false;
    return AMPQ_OK;
}

int ampq_set_measured(ampq_ctx* ctx, int on) {
    if (!ctx) return AMPQ_ERR_INVALID;
    if (ctx->streaming) return fail(ctx, AMPQ_ERR_STATE, "the scored terms cannot change inside a streaming pass");
    ctx->measured = on != 0;
    ctx->scored = false;
    return AMPQ_OK;
}

int ampq_set_sharing(ampq_ctx* ctx, int on) {
    if (!ctx) return AMPQ_ERR_INVALID;
    ctx->sharing = on != 0;
    ctx->dirty = true;
    return AMPQ_OK;
}

int ampq_measure_amax(ampq_ctx* ctx) {
    if (!ctx) return AMPQ_ERR_INVALID;
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail(ctx, AMPQ_ERR_CUDA, "cudaSetDevice failed");
    int rc;
    if ((rc = prepare_tables(ctx))) return rc;
    ctx->scored = false;
    const int T = (int)ctx->tens.size();
    cudaStream_t st = ctx->stream;
    ctx->launches = 0;
    ctx->ev_valid = false;
    if ((rc = stage_host_operands(ctx))) return rc;
    if (T > 0) {
        AMPQ_CUDA(launch_init_amax(ctx->d_tens.p, T, ctx->d_amax_bits.p, ctx->d_status.p, st), "init_amax");
        AMPQ_CUDA(launch_amax(ctx->d_tens.p, ctx->d_amax_tile_begin.p, T, ctx->namax_tiles, ctx->amax_tile, ctx->d_amax_bits.p, st), "amax");
        ctx->launches = ctx->namax_tiles > 0 ? 2 : 1;
        if (ctx->n_amax_alias > 0) {
            AMPQ_CUDA(launch_resolve_amax(T, ctx->d_tens.p, ctx->d_amax_bits.p, st), "resolve_amax");
            ++ctx->launches;
        }
        AMPQ_CUDA(cudaMemcpyAsync(ctx->h_amax_bits.p, ctx->d_amax_bits.p, T * sizeof(unsigned), cudaMemcpyDeviceToHost, st), "D2H amax");
    }
    ctx->amax_ready = true;
    ctx->pending = T > 0;
    return AMPQ_OK;
}

int ampq_get_amax(ampq_ctx* ctx, int layer_id, float* amax) {
    int rc = check_layer(ctx, layer_id);
    if (rc) return rc;
    if (!amax) return fail(ctx, AMPQ_ERR_INVALID, "null output");
    if (!ctx->amax_ready || ctx->dirty) return fail(ctx, AMPQ_ERR_STATE, "no amax has been measured for the current bindings");
    DeviceGuard g(ctx->device);
    if (ctx->pending) {
        AMPQ_CUDA(cudaStreamSynchronize(ctx->stream), "cudaStreamSynchronize");
        ctx->pending = false;
    }
    const LayerRec& l = ctx->layers[layer_id];
    if (l.scored < 0) return fail(ctx, AMPQ_ERR_STATE, "layer has an unbound operand");
    for (int k = 0; k < 2; ++k) std::memcpy(&amax[k], &ctx->h_amax_bits.p[l.op[k].tensor], sizeof(float));
    return AMPQ_OK;
}

int ampq_set_causal(ampq_ctx* ctx, int layer_id, int operand, long long T) {
    int rc = check_layer(ctx, layer_id);
    if (rc) return rc;
    if (operand != 0 && operand != 1) return fail(ctx, AMPQ_ERR_INVALID, "operand must be 0 or 1");
    if (T < 0) return fail(ctx, AMPQ_ERR_INVALID, "T must not be negative");
    ctx->layers[layer_id].op[operand].causal_T = T;
    ctx->dirty = true;
    return AMPQ_OK;
}

int ampq_score(ampq_ctx* ctx) {
    if (!ctx) return AMPQ_ERR_INVALID;
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail(ctx, AMPQ_ERR_CUDA, "cudaSetDevice failed");
    int rc;
    if ((rc = prepare_tables(ctx))) return rc;
    const int T = (int)ctx->tens.size(), L = (int)ctx->lay.size(), S = (int)ctx->segs.size();
    const int nacc = ctx->F;  // S plus one D per low-precision format
    cudaStream_t st = ctx->stream;
    ctx->launches = 0;
    ctx->ev_valid = false;
    const bool tm = ctx->timing && T > 0;
    if (tm) AMPQ_CUDA(cudaEventRecord(ctx->ev[0], st), "cudaEventRecord");
    if ((rc = stage_host_operands(ctx))) return rc;
    if (T > 0) {
        AMPQ_CUDA(launch_init_amax(ctx->d_tens.p, T, ctx->d_amax_bits.p, ctx->d_status.p, st), "init_amax");
        ++ctx->launches;
        if (tm) AMPQ_CUDA(cudaEventRecord(ctx->ev[1], st), "cudaEventRecord");
        // scale and inverse scale of every tensor: by the last CTA of the amax pass, or, when
        // nothing is measured, by a small launch of their own
        const ScalesArgs sa = scales_args(T, ctx->fmask, ctx->d_tens.p, ctx->d_amax_bits.p, ctx->d_scales.p, ctx->d_flags.p,
                                          ctx->d_status.p, ctx->scale_pow2, &ctx->d_status.p->amax_done);
        // (the tail costs every amax CTA one atomic on a single word: only worth it for a small pass)
        const bool amax_pass = ctx->namax_tiles > 0 && ctx->measured;
        const bool tail = amax_pass && ctx->namax_tiles <= 4096;
        if (amax_pass) {
            AMPQ_CUDA(launch_amax(ctx->d_tens.p, ctx->d_amax_tile_begin.p, T, ctx->namax_tiles, ctx->amax_tile, ctx->d_amax_bits.p, st,
                                  tail ? sa : ScalesArgs()), "amax");
            ++ctx->launches;
        }
        if (!ctx->measured && ctx->nslots > 0)  // the S-only kernels leave the D columns of a slot untouched
            AMPQ_CUDA(cudaMemsetAsync(ctx->d_partials.p, 0, (size_t)ctx->nslots * nacc * sizeof(double), st), "memset partials");
        if (tm) AMPQ_CUDA(cudaEventRecord(ctx->ev[2], st), "cudaEventRecord");
        if (!tail) {
            AMPQ_CUDA(launch_scales(T, ctx->fmask, ctx->d_tens.p, ctx->d_amax_bits.p, ctx->d_scales.p, ctx->d_flags.p, ctx->d_status.p, st, ctx->scale_pow2), "scales");
            ++ctx->launches;
        }
        if (tm) AMPQ_CUDA(cudaEventRecord(ctx->ev[3], st), "cudaEventRecord");
        for (int c = 0; c < kScoreClasses; ++c) {
            if (ctx->ntiles[c] <= 0) continue;
            const bool causal = c >= 2 * kMaxRB;  // the last two classes: triangular operands, fp32 and bf16
            AMPQ_CUDA(launch_score(causal ? c - 2 * kMaxRB : c / kMaxRB, causal ? 1 : c % kMaxRB + 1, ctx->d_tens.p,
                                   ctx->d_tile_begin[c].p, T, ctx->ntiles[c], ctx->tile_shift, ctx->max_ctas,
                                   ctx->measured ? ctx->fmask : 0, ctx->d_scales.p, ctx->d_partials.p, ctx->d_status.p, st,
                                   causal ? 1 : 0, nacc), "score");
            ++ctx->launches;
        }
        if (tm) AMPQ_CUDA(cudaEventRecord(ctx->ev[4], st), "cudaEventRecord");
        {   // ordered sums per segment; the CTA that finishes last combines the layers
            CombineArgs ca;
            ca.counter = &ctx->d_status.p->finalize_done;
            ca.layers = ctx->d_lay.p; ca.L = L; ca.F = ctx->F; ca.prm = combine_params(ctx); ca.layer_out = ctx->d_layer_out.p;
            AMPQ_CUDA(launch_finalize(ctx->d_segs.p, S, nacc, ctx->d_partials.p, ctx->d_seg_out.p, st, ca), "finalize");
            ++ctx->launches;
        }
        if ((rc = read_back(ctx))) return rc;
        if (tm) {
            AMPQ_CUDA(cudaEventRecord(ctx->ev[5], st), "cudaEventRecord");
            ctx->ev_valid = true;
        }
    }
    ctx->scored = true;
    ctx->amax_ready = true;
    ctx->pending = T > 0;
    return AMPQ_OK;
}

int ampq_stream_begin(ampq_ctx* ctx) {
    if (!ctx) return AMPQ_ERR_INVALID;
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail(ctx, AMPQ_ERR_CUDA, "cudaSetDevice failed");
    if (ctx->pending) {
        AMPQ_CUDA(cudaStreamSynchronize(ctx->stream), "cudaStreamSynchronize");
        ctx->pending = false;
    }
    if (!ctx->retired.empty()) {  // left by a streaming pass that was never ended
        AMPQ_CUDA(cudaStreamSynchronize(ctx->stream), "cudaStreamSynchronize");
        free_retired(ctx);
    }
    // tables over EVERY registered layer: tensor 2*l + operand, one segment per sample
    ctx->tens.clear(); ctx->segs.clear(); ctx->lay.clear(); ctx->scored_layer_ids.clear();
    ctx->stream_seg_base.clear();
    int out_off = 0, nseg = 0;
    for (size_t li = 0; li < ctx->layers.size(); ++li) {
        LayerRec& l = ctx->layers[li];
        Layer ly{};
        ly.R = l.R;
        ly.out_off = out_off;
        out_off += layer_block_doubles(l.R, ctx->F);
        for (int k = 0; k < 2; ++k) {
            Tensor t{};
            t.R = l.R;
            t.seg_base = nseg;
            t.amax_preset = l.op[k].amax_preset;
            l.op[k].tensor = (int)ctx->tens.size();
            ctx->stream_seg_base.push_back(nseg);
            if (k == 0) { ly.seg_base0 = nseg; ly.tensor0 = l.op[k].tensor; }
            else { ly.seg_base1 = nseg; ly.tensor1 = l.op[k].tensor; }
            ctx->tens.push_back(t);
            nseg += l.R;
        }
        l.scored = (int)ctx->lay.size();
        ctx->lay.push_back(ly);
        ctx->scored_layer_ids.push_back((int)li);
    }
    ctx->layer_out_doubles = out_off;
    const size_t T = ctx->tens.size(), L = ctx->lay.size(), S = (size_t)nseg;
    const int nacc = ctx->F;
    AMPQ_CUDA(ctx->d_lay.ensure(L), "cudaMalloc(layers)");
    AMPQ_CUDA(ctx->d_jobs.ensure(S), "cudaMalloc(jobs)");
    {
        int rc = ensure_results(ctx, T, S, nacc, (size_t)out_off);
        if (rc) return rc;
        // room for the per-tile partials of the largest operand that is bound (a hint: samples
        // of operands that are not bound, or larger ones, make the buffer grow later)
        long long most = 0;
        for (const auto& l : ctx->layers)
            for (int k = 0; k < 2; ++k)
                if (l.op[k].bound) {
                    const long long ext = extent_of(l, l.op[k]);
                    const int shift = pick_tile_shift(ext, ctx->max_ctas);
                    most = std::max(most, (ext + (1LL << shift) - 1) >> shift);
                }
        if (most > 0 && most <= 0x7FFFFFFFLL && (rc = ensure_job_partials(ctx, (size_t)most * nacc + 1))) return rc;
    }
    cudaStream_t st = ctx->stream;
    if (L) AMPQ_CUDA(cudaMemcpyAsync(ctx->d_lay.p, ctx->lay.data(), L * sizeof(Layer), cudaMemcpyHostToDevice, st), "H2D layers");
    // amax, flags, scales, every per-sample sum and the status word start at zero
    AMPQ_CUDA(cudaMemsetAsync(ctx->d_arena.p, 0, ctx->arena_bytes, st), "memset results");
    ctx->streaming = true;
    ctx->scored = false;
    ctx->dirty = true;  // a later ampq_score rebuilds its own tables
    ctx->launches = 0;
    ctx->ev_valid = false;
    return AMPQ_OK;
}

int ampq_stream_sample(ampq_ctx* ctx, int layer_id, int operand, int r, int dtype, const void* values,
                       const void* grads, long long numel) {
    int rc = check_layer(ctx, layer_id);
    if (rc) return rc;
    if (!ctx->streaming) return fail(ctx, AMPQ_ERR_STATE, "ampq_stream_sample outside ampq_stream_begin / ampq_stream_end");
    if (operand != 0 && operand != 1) return fail(ctx, AMPQ_ERR_INVALID, "operand must be 0 or 1");
    if (dtype != AMPQ_F32 && dtype != AMPQ_BF16) return fail(ctx, AMPQ_ERR_INVALID, "unknown dtype");
    const LayerRec& l = ctx->layers[layer_id];
    if (l.scored < 0 || 2 * (size_t)layer_id + 1 >= ctx->stream_seg_base.size())
        return fail(ctx, AMPQ_ERR_STATE, "layer was registered after ampq_stream_begin");
    if (r < 0 || r >= l.R) return fail(ctx, AMPQ_ERR_INVALID, "sample index outside [0, R)");
    if (numel < 0 || (numel > 0 && (!values || !grads))) return fail(ctx, AMPQ_ERR_INVALID, "bad tensor");
    const int es = dtype == AMPQ_F32 ? 4 : 2;
    if ((reinterpret_cast<uintptr_t>(values) % es) || (reinterpret_cast<uintptr_t>(grads) % es))
        return fail(ctx, AMPQ_ERR_ALIGN, "tensor pointer not aligned to its element size");
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail(ctx, AMPQ_ERR_CUDA, "cudaSetDevice failed");
    const int nacc = ctx->F;
    const int tensor = 2 * layer_id + operand;
    const int seg = ctx->stream_seg_base[tensor] + r;
    const int shift = pick_tile_shift(numel, ctx->max_ctas);
    const long long ntiles = (numel + (1LL << shift) - 1) >> shift;
    if (ntiles > 0x7FFFFFFFLL) return fail(ctx, AMPQ_ERR_TOO_LARGE, "more than 2^31-1 tiles in one sample");
    if ((rc = ensure_job_partials(ctx, (size_t)ntiles * nacc + 1))) return rc;
    SegmentJob* job = ctx->d_jobs.p + seg;
    cudaStream_t st = ctx->stream;
    // S only: a preset of 0 keeps the amax pass away; the D columns of the slots are cleared instead of written
    const float preset = ctx->measured ? l.op[operand].amax_preset : 0.0f;
    if ((rc = job_amax_and_scales(ctx, job, ctx->d_status.p, dtype, values, grads, numel, preset, ntiles))) return rc;
    if (!ctx->measured && ntiles > 0)
        AMPQ_CUDA(cudaMemsetAsync(ctx->d_job_partials.p, 0, (size_t)ntiles * nacc * sizeof(double), st), "memset partials");
    AMPQ_CUDA(launch_score(dtype == AMPQ_F32 ? 0 : 1, 1, &job->tensor, job->tile_begin, 1, ntiles, shift, ctx->max_ctas,
                           ctx->measured ? ctx->fmask : 0, job->scales, ctx->d_job_partials.p, ctx->d_status.p, st, 0, nacc), "score");
    if (ntiles > 0) ++ctx->launches;
    AMPQ_CUDA(launch_job_finish(job, nacc, ctx->d_job_partials.p, ctx->d_seg_out.p + (size_t)seg * nacc, tensor,
                                ctx->d_amax_bits.p, ctx->d_flags.p, ctx->d_scales.p, st), "job_finish");
    ++ctx->launches;
    return AMPQ_OK;
}

int ampq_stream_end(ampq_ctx* ctx) {
    if (!ctx) return AMPQ_ERR_INVALID;
    if (!ctx->streaming) return fail(ctx, AMPQ_ERR_STATE, "ampq_stream_end without ampq_stream_begin");
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail(ctx, AMPQ_ERR_CUDA, "cudaSetDevice failed");
    int nseg = 0;
    for (const auto& ly : ctx->lay) nseg += 2 * ly.R;
    const int T = (int)ctx->tens.size(), L = (int)ctx->lay.size();
    int rc = AMPQ_OK;
    if (T > 0) {
        AMPQ_CUDA(launch_combine(ctx->d_lay.p, L, ctx->F, combine_params(ctx), ctx->d_seg_out.p, ctx->d_layer_out.p, ctx->stream), "combine");
        ++ctx->launches;
        if ((rc = read_back(ctx))) return rc;
    }
    (void)nseg;
    ctx->streaming = false;
    ctx->scored = true;
    ctx->pending = T > 0;
    return AMPQ_OK;
}

int ampq_fake_quant(ampq_ctx* ctx, int dtype, int fmt, const void* values, long long numel, float amax, void* dev_out) {
    if (!ctx) return AMPQ_ERR_INVALID;
    if (dtype != AMPQ_F32 && dtype != AMPQ_BF16) return fail(ctx, AMPQ_ERR_INVALID, "unknown dtype");
    if (numel < 0 || (numel > 0 && (!values || !dev_out))) return fail(ctx, AMPQ_ERR_INVALID, "bad tensor");
    if (amax != amax || std::isinf(amax)) return fail(ctx, AMPQ_ERR_INVALID, "amax must be finite");
    int f = -1;
    for (int k = 1; k < ctx->F; ++k)
        if (ctx->fmt[k] == fmt) f = k;
    if (f < 0) return fail(ctx, AMPQ_ERR_INVALID, "format is not in the context's format list");
    const int es = dtype == AMPQ_F32 ? 4 : 2;
    if ((reinterpret_cast<uintptr_t>(values) % es) || (reinterpret_cast<uintptr_t>(dev_out) % es))
        return fail(ctx, AMPQ_ERR_ALIGN, "tensor pointer not aligned to its element size");
    DeviceGuard g(ctx->device);
    if (!g.ok) return fail(ctx, AMPQ_ERR_CUDA, "cudaSetDevice failed");
    AMPQ_CUDA(ctx->d_fq_job.ensure(1), "cudaMalloc(job)");
    AMPQ_CUDA(ctx->d_fq_status.ensure(1), "cudaMalloc(status)");
    int rc = job_amax_and_scales(ctx, ctx->d_fq_job.p, ctx->d_fq_status.p, dtype, values, values, numel,
                                 amax > 0.0f ? amax : (amax == 0.0f ? 0.0f : -1.0f), 0);
    if (rc) return rc;
    const float* pair = ctx->d_fq_job.p->scales + ctx->slot_of_fmt[f] * 2;
    AMPQ_CUDA(launch_fake_quant(dtype, fmt == AMPQ_FMT_E4M3 ? kMaskE4M3 : kMaskE5M2, values, numel, pair, dev_out, ctx->stream), "fake_quant");
    return AMPQ_OK;
}

int ampq_last_launch_count(const ampq_ctx* ctx) { return ctx ? ctx->launches : 0; }

int ampq_last_tile_shift(const ampq_ctx* ctx) { return ctx && !ctx->dirty && !ctx->tens.empty() ? ctx->tile_shift : 0; }

int ampq_get_pass_bytes(ampq_ctx* ctx, long long* bytes) {
    if (!ctx || !bytes) return AMPQ_ERR_INVALID;
    if (ctx->dirty || ctx->streaming || !(ctx->scored || ctx->amax_ready))
        return fail(ctx, AMPQ_ERR_STATE, "no pass has been issued for the current bindings");
    bytes[0] = ctx->measured ? ctx->amax_bytes : 0;
    bytes[1] = ctx->score_bytes;
    return AMPQ_OK;
}

int ampq_set_timing(ampq_ctx* ctx, int on) {
    if (!ctx) return AMPQ_ERR_INVALID;
    DeviceGuard g(ctx->device);
    if (on && !ctx->ev[0]) {
        for (int i = 0; i < 6; ++i) AMPQ_CUDA(cudaEventCreate(&ctx->ev[i]), "cudaEventCreate");
    }
    ctx->timing = on != 0;
    ctx->ev_valid = false;
    return AMPQ_OK;
}

int ampq_get_timing(ampq_ctx* ctx, float* ms) {
    if (!ctx || !ms) return AMPQ_ERR_INVALID;
    DeviceGuard g(ctx->device);
    int rc = sync_results(ctx);
    if (rc) return rc;
    if (!ctx->ev_valid) return fail(ctx, AMPQ_ERR_STATE, "timing was not enabled for the last score");
    AMPQ_CUDA(cudaEventSynchronize(ctx->ev[5]), "cudaEventSynchronize");
    AMPQ_CUDA(cudaEventElapsedTime(&ms[0], ctx->ev[1], ctx->ev[2]), "cudaEventElapsedTime");
    AMPQ_CUDA(cudaEventElapsedTime(&ms[1], ctx->ev[3], ctx->ev[4]), "cudaEventElapsedTime");
    AMPQ_CUDA(cudaEventElapsedTime(&ms[2], ctx->ev[0], ctx->ev[5]), "cudaEventElapsedTime");
    return AMPQ_OK;
}

int ampq_get_layer(ampq_ctx* ctx, int layer_id, float* amax, float* scale, float* inv_scale,
                   double* s_per_sample, double* s_mean, double* d_meas_per_sample, double* d_model,
                   double* d_meas) {
    int rc = check_layer(ctx, layer_id);
    if (rc) return rc;
    DeviceGuard g(ctx->device);
    if ((rc = sync_results(ctx))) return rc;
    const LayerRec& l = ctx->layers[layer_id];
    if (l.scored < 0) return fail(ctx, AMPQ_ERR_STATE, "layer was not part of the last score");
    const Layer& ly = ctx->lay[l.scored];
    const int F = ctx->F, R = ly.R;
    const int tix[2] = {ly.tensor0, ly.tensor1};
    bool bad = false;
    for (int k = 0; k < 2; ++k) {
        const int t = tix[k];
        bad = bad || ctx->h_flags.p[t] != 0;
        if (amax) std::memcpy(&amax[k], &ctx->h_amax_bits.p[t], sizeof(float));
        for (int f = 0; f < F; ++f) {
            float sc = 1.0f, iv = 1.0f;
            if (f > 0) {
                sc = ctx->h_scales.p[t * 2 * kMaxLow + ctx->slot_of_fmt[f] * 2 + 0];
                iv = ctx->h_scales.p[t * 2 * kMaxLow + ctx->slot_of_fmt[f] * 2 + 1];
            }
            if (scale) scale[k * F + f] = sc;
            if (inv_scale) inv_scale[k * F + f] = iv;
        }
    }
    const double* o = layer_block(ctx, l.scored);
    if (s_per_sample) std::memcpy(s_per_sample, o, sizeof(double) * R);
    if (s_mean) *s_mean = o[R];
    if (d_meas_per_sample) std::memcpy(d_meas_per_sample, o + R + 1, sizeof(double) * R * F);
    if (d_model) std::memcpy(d_model, o + R + 1 + (long long)R * F, sizeof(double) * F);
    if (d_meas) std::memcpy(d_meas, o + R + 1 + (long long)R * F + F, sizeof(double) * F);
    if (bad) return fail(ctx, AMPQ_ERR_NONFINITE, "layer '" + l.name + "' holds Inf/NaN");
    return AMPQ_OK;
}

int ampq_get_layer_table(ampq_ctx* ctx, const int* layer_ids, int n, double* out) {
    if (!ctx || n < 0 || (n > 0 && (!layer_ids || !out))) return AMPQ_ERR_INVALID;
    DeviceGuard g(ctx->device);
    int rc = sync_results(ctx);
    if (rc) return rc;
    const int F = ctx->F, K = 1 + 2 * F;
    bool bad = false;
    for (int i = 0; i < n; ++i) {
        if ((rc = check_layer(ctx, layer_ids[i]))) return rc;
        const LayerRec& l = ctx->layers[layer_ids[i]];
        if (l.scored < 0) return fail(ctx, AMPQ_ERR_STATE, "layer '" + l.name + "' was not part of the last score");
        const Layer& ly = ctx->lay[l.scored];
        bad = bad || ctx->h_flags.p[ly.tensor0] != 0 || ctx->h_flags.p[ly.tensor1] != 0;
        const double* o = layer_block(ctx, l.scored);
        double* row = out + (size_t)i * K;
        row[0] = o[ly.R];
        std::memcpy(row + 1, o + ly.R + 1 + (long long)ly.R * F, sizeof(double) * 2 * F);  // d_model[F], d_meas[F]
    }
    if (bad) return fail(ctx, AMPQ_ERR_NONFINITE, "a layer of the table holds Inf/NaN");
    return AMPQ_OK;
}

int ampq_get_operand(ampq_ctx* ctx, int layer_id, int operand, double* out) {
    int rc = check_layer(ctx, layer_id);
    if (rc) return rc;
    if ((operand != 0 && operand != 1) || !out) return fail(ctx, AMPQ_ERR_INVALID, "bad operand or null output");
    DeviceGuard g(ctx->device);
    if ((rc = sync_results(ctx))) return rc;
    const LayerRec& l = ctx->layers[layer_id];
    if (l.scored < 0) return fail(ctx, AMPQ_ERR_STATE, "layer was not part of the last score");
    const Layer& ly = ctx->lay[l.scored];
    const int F = ctx->F, nacc = F;
    const int sb = operand == 0 ? ly.seg_base0 : ly.seg_base1;
    for (int r = 0; r < ly.R; ++r) {
        out[r * F] = ctx->h_seg_out.p[(size_t)(sb + r) * nacc];
        for (int f = 1; f < F; ++f)
            out[r * F + f] = ctx->h_seg_out.p[(size_t)(sb + r) * nacc + 1 + ctx->slot_of_fmt[f]];
    }
    return AMPQ_OK;
}

int ampq_export_codes(ampq_ctx* ctx, int layer_id, int operand, int fmt, unsigned char* dev_out) {
    int rc = check_layer(ctx, layer_id);
    if (rc) return rc;
    if (operand != 0 && operand != 1) return fail(ctx, AMPQ_ERR_INVALID, "operand must be 0 or 1");
    if (!ctx->scored || ctx->dirty) return fail(ctx, AMPQ_ERR_STATE, "export needs the scales of a score of the current bindings");
    const LayerRec& l = ctx->layers[layer_id];
    const Operand& o = l.op[operand];
    if (l.scored < 0 || o.tensor < 0) return fail(ctx, AMPQ_ERR_STATE, "layer was not part of the last score");
    if (o.mem != AMPQ_MEM_DEVICE) return fail(ctx, AMPQ_ERR_INVALID, "export needs a device-bound operand");
    int f = -1;
    for (int k = 1; k < ctx->F; ++k)
        if (ctx->fmt[k] == fmt) f = k;
    if (f < 0) return fail(ctx, AMPQ_ERR_INVALID, "format is not in the context's format list");
    if (o.numel > 0 && !dev_out) return fail(ctx, AMPQ_ERR_INVALID, "null output");
    DeviceGuard g(ctx->device);
    const float* pair = ctx->d_scales.p + (size_t)o.tensor * 2 * kMaxLow + ctx->slot_of_fmt[f] * 2;
    AMPQ_CUDA(launch_codes(o.dtype, fmt == AMPQ_FMT_E4M3 ? kMaskE4M3 : kMaskE5M2, o.values, o.numel, pair, dev_out, ctx->stream), "codes");
    return AMPQ_OK;
}

int ampq_define_group(ampq_ctx* ctx, const int* layer_ids, int Lj, const unsigned char* Q, const double* c,
                      int Pj, int* group_id) {
    if (!ctx || !layer_ids || !Q || !c || !group_id) return AMPQ_ERR_INVALID;
    if (Lj < 1 || Pj < 1) return fail(ctx, AMPQ_ERR_INVALID, "a group needs at least one layer and one configuration");
    Group g;
    for (int l = 0; l < Lj; ++l) {
        if (layer_ids[l] < 0 || layer_ids[l] >= (int)ctx->layers.size()) return fail(ctx, AMPQ_ERR_INVALID, "unknown layer id in group");
        g.layers.push_back(layer_ids[l]);
    }
    for (long long i = 0; i < (long long)Lj * Pj; ++i)
        if (Q[i] >= ctx->F) return fail(ctx, AMPQ_ERR_INVALID, "Q entry outside the format list");
    for (int p = 0; p < Pj; ++p)
        if (c[p] != c[p]) return fail(ctx, AMPQ_ERR_INVALID, "metric is NaN");
    g.Q.assign(Q, Q + (size_t)Lj * Pj);
    g.c.assign(c, c + Pj);
    g.P = Pj;
    ctx->groups.push_back(std::move(g));
    *group_id = (int)ctx->groups.size() - 1;
    return AMPQ_OK;
}

int ampq_clear_groups(ampq_ctx* ctx) {
    if (!ctx) return AMPQ_ERR_INVALID;
    ctx->groups.clear();
    return AMPQ_OK;
}

int ampq_group_costs(ampq_ctx* ctx, int group_id, int d_mode, double* d_out) {
    if (!ctx || !d_out) return AMPQ_ERR_INVALID;
    if (group_id < 0 || group_id >= (int)ctx->groups.size()) return fail(ctx, AMPQ_ERR_INVALID, "unknown group id");
    if (d_mode != AMPQ_D_MODEL && d_mode != AMPQ_D_MEASURED) return fail(ctx, AMPQ_ERR_INVALID, "unknown d_mode");
    DeviceGuard g(ctx->device);
    int rc = sync_results(ctx);
    if (rc) return rc;
    return group_costs_impl(ctx, ctx->groups[group_id], d_mode, d_out);
}

int ampq_group_costs_table(const int* layer_ids, int Lj, const unsigned char* Q, int Pj, const double* d_layer,
                           int L, int F, double* d_out) {
    if (!layer_ids || !Q || !d_layer || !d_out || Lj < 1 || Pj < 1 || L < 1 || F < 1) return AMPQ_ERR_INVALID;
    for (int l = 0; l < Lj; ++l)
        if (layer_ids[l] < 0 || layer_ids[l] >= L) return AMPQ_ERR_INVALID;
    for (long long i = 0; i < (long long)Lj * Pj; ++i)
        if (Q[i] >= F) return AMPQ_ERR_INVALID;
    for (int p = 0; p < Pj; ++p) {
        double d = 0.0;
        for (int l = 0; l < Lj; ++l) d += d_layer[(size_t)layer_ids[l] * F + Q[l + (size_t)Lj * p]];
        d_out[p] = d;
    }
    return AMPQ_OK;
}

int ampq_budget_from_tau(double tau, const double* losses, int R, double* budget) {
    if (!losses || !budget || R < 1 || !(tau >= 0.0)) return AMPQ_ERR_INVALID;
    double a = 0.0;
    for (int r = 0; r < R; ++r) a += losses[r] * losses[r];
    *budget = tau * tau * (a / (double)R);
    return AMPQ_OK;
}

int ampq_all_lowp_cost(ampq_ctx* ctx, int d_mode, int f, double* d_all) {
    if (!ctx || !d_all) return AMPQ_ERR_INVALID;
    if (f < 1 || f >= ctx->F) return fail(ctx, AMPQ_ERR_INVALID, "format index must be 1..F-1");
    if (d_mode != AMPQ_D_MODEL && d_mode != AMPQ_D_MEASURED) return fail(ctx, AMPQ_ERR_INVALID, "unknown d_mode");
    DeviceGuard g(ctx->device);
    int rc = sync_results(ctx);
    if (rc) return rc;
    double d = 0.0;
    for (size_t s = 0; s < ctx->lay.size(); ++s) {
        if (ctx->h_flags.p[ctx->lay[s].tensor0] || ctx->h_flags.p[ctx->lay[s].tensor1])
            return fail(ctx, AMPQ_ERR_NONFINITE, "a scored layer holds Inf/NaN");
        d += layer_d(ctx, (int)s, f, d_mode);
    }
    *d_all = d;
    return AMPQ_OK;
}

int ampq_select_tables(int J, const int* P, const long long* off, const double* c, const double* d,
                       double budget, int* p_out, double* c_total, double* d_total) {
    if (J < 0 || (J > 0 && (!P || !off || !c || !d || !p_out))) return AMPQ_ERR_INVALID;
    const int rc = select_mckp(J, P, off, c, d, budget, 50000000LL, p_out, c_total, d_total);
    switch (rc) {
        case kSelectOk: return AMPQ_OK;
        case kSelectInfeasible: return AMPQ_ERR_INFEASIBLE;
        case kSelectTooLarge: return AMPQ_ERR_TOO_LARGE;
        default: return AMPQ_ERR_INVALID;
    }
}

int ampq_select(ampq_ctx* ctx, int d_mode, double budget, int* p_out, double* c_total, double* d_total) {
    if (!ctx || !p_out) return AMPQ_ERR_INVALID;
    if (d_mode != AMPQ_D_MODEL && d_mode != AMPQ_D_MEASURED) return fail(ctx, AMPQ_ERR_INVALID, "unknown d_mode");
    DeviceGuard g(ctx->device);
    int rc = sync_results(ctx);
    if (rc) return rc;
    const int J = (int)ctx->groups.size();
    std::vector<int> P(J);
    std::vector<long long> off(J);
    std::vector<double> c, d;
    for (int j = 0; j < J; ++j) {
        const Group& gr = ctx->groups[j];
        P[j] = gr.P;
        off[j] = (long long)c.size();
        c.insert(c.end(), gr.c.begin(), gr.c.end());
        d.resize(d.size() + gr.P);
        if ((rc = group_costs_impl(ctx, gr, d_mode, d.data() + off[j]))) return rc;
    }
    rc = ampq_select_tables(J, P.data(), off.data(), c.data(), d.data(), budget, p_out, c_total, d_total);
    if (rc == AMPQ_ERR_INFEASIBLE) ctx->err = "no assignment meets the budget";
    if (rc == AMPQ_ERR_TOO_LARGE) ctx->err = "selection exceeded its state limit";
    return rc;
}

#pragma GCC visibility pop
}  // extern "C"

// CUDA kernels of the loss-MSE sensitivity pass for sm_100a.
//
// The pass is a stream-reduce: every operand element and its gradient are read
// once from HBM, all arithmetic happens in registers, and a few doubles per
// tile are written back.  The kernels are therefore shaped for HBM bandwidth:
// the scoring kernel is persistent and stages operand and gradient chunks in a
// shared-memory ring with bulk asynchronous copies (TMA) so that the bytes in
// flight do not depend on the arithmetic; the amax kernel uses 128-bit
// coalesced non-allocating loads; packed two-wide fp32 arithmetic (fma.rn.f32x2)
// and the hardware FP8 converts so that the instruction count per element stays
// below what 148 SMs can issue at full memory speed.  No tensor cores: there is
// no contraction anywhere on this path.
//
//   amax_kernel     max_k |z_k| per tensor (integer max of the bit patterns,
//                   warp redux + one atomicMax per CTA)
//   scales_kernel   scale = amax/fmax, inv = fmax/amax per tensor and format
//   score_kernel    fused cast / error / weighting / per-tile reduction
//   finalize_kernel ordered fp64 sum of the per-tile partials per segment
//   combine_kernel  per-layer sensitivities and loss-MSE terms (Sec. 2.2)
//   codes_kernel    test hook: the FP8 codes the scoring kernel sees
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <atomic>
#include <cstdint>
#include <type_traits>

#include "ampq_device.h"
#include "ampq_kernels.h"

namespace ampq {

// ---------------------------------------------------------------------------
// small device helpers

__device__ __forceinline__ uint4 ld_stream_v4(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// Two fp32 values -> two FP8 codes (round to nearest even, saturate to the
// largest finite value), first argument in the low byte.
template <int FMT>
__device__ __forceinline__ unsigned short cast_pair(float lo, float hi) {
    unsigned short r;
    if (FMT == kMaskE4M3)
        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    else
        asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

// Two FP8 codes -> their exact values as fp32 (every FP8 value is an fp16 value).
template <int FMT>
__device__ __forceinline__ float2 decode_pair(unsigned short c) {
    unsigned h;
    if (FMT == kMaskE4M3)
        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h) : "h"(c));
    else
        asm("cvt.rn.f16x2.e5m2x2 %0, %1;" : "=r"(h) : "h"(c));
    __half2 hh = *reinterpret_cast<__half2*>(&h);
    return __half22float2(hh);
}

// -(dec(Q(z*inv))*scale - z) for a pair: the negated quantisation error; only
// its square is used.  One fp32 rounding in y = z*inv, one in the fma.
template <int FMT>
__device__ __forceinline__ float2 neg_err_pair(float2 z, float2 inv2, float2 nscale2) {
    float2 y = __fmul2_rn(z, inv2);
    float2 dq = decode_pair<FMT>(cast_pair<FMT>(y.x, y.y));
    return __ffma2_rn(dq, nscale2, z);
}

template <int DT>
struct Elem;
template <>
struct Elem<0> {  // fp32
    static constexpr int kPerVec = 4;
    static constexpr int kBytes = 4;
    __device__ static __forceinline__ void unpack(const uint4& v, float2 (&out)[2]) {
        out[0] = make_float2(__uint_as_float(v.x), __uint_as_float(v.y));
        out[1] = make_float2(__uint_as_float(v.z), __uint_as_float(v.w));
    }
    __device__ static __forceinline__ float load(const void* p, long long i) {
        return __ldg(reinterpret_cast<const float*>(p) + i);
    }
};
template <>
struct Elem<1> {  // bf16: the upper half of an fp32
    static constexpr int kPerVec = 8;
    static constexpr int kBytes = 2;
    __device__ static __forceinline__ float2 two(unsigned w) {
        return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
    }
    __device__ static __forceinline__ void unpack(const uint4& v, float2 (&out)[4]) {
        out[0] = two(v.x); out[1] = two(v.y); out[2] = two(v.z); out[3] = two(v.w);
    }
    __device__ static __forceinline__ float load(const void* p, long long i) {
        unsigned short b = __ldg(reinterpret_cast<const unsigned short*>(p) + i);
        return __uint_as_float(static_cast<unsigned>(b) << 16);
    }
};

// Which tensor owns global tile `tile`: begin[j] <= tile < begin[j+1].  All
// threads of the CTA take part; the answer is broadcast through shared memory.
__device__ __forceinline__ int find_tensor(const long long* __restrict__ begin, int T,
                                           long long tile, int* s_slot) {
    for (int j = threadIdx.x; j < T; j += blockDim.x) {
        if (tile >= __ldg(begin + j) && tile < __ldg(begin + j + 1)) *s_slot = j;
    }
    __syncthreads();
    return *s_slot;
}

// Causal operands: element e of a segment sits in row (e >> shift) of a stack of
// T x T matrices (T = 2^shift), at column e & (T-1) of matrix row
// (e >> shift) & (T-1); everything right of the diagonal is exactly zero and is
// never read.  Reads go in whole 16-byte vectors: matrix row i keeps its first
// i / kPerVec + 1 vectors.
__device__ __forceinline__ int causal_row_vectors(long long row, int shift, int per_vec) {
    return (int)(row & ((1 << shift) - 1)) / per_vec + 1;
}

// ---------------------------------------------------------------------------
// amax

__global__ void init_amax_kernel(const Tensor* __restrict__ tens, int T,
                                 unsigned* __restrict__ amax_bits, LaunchStatus* status) {
    int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t == 0) {
        status->nonfinite = 0;
        status->timeout = 0;
        status->bounds = 0;
        status->amax_done = 0;
        status->finalize_done = 0;
    }
    if (t < T) {
        float p = tens[t].amax_preset;
        amax_bits[t] = (p >= 0.0f) ? __float_as_uint(p) : 0u;
    }
}

// scale = fl32(amax / fmax), inv = fl32(fmax / amax), IEEE divisions; the
// neutral pair (1, 1) when amax is 0 or fmax/amax is not a finite fp32.
// pow2 mode: scale = the smallest power of two p with fmax * p >= amax, inv =
// 1/p.  With fmax = 1.75 * 2^ef and amax = m * 2^ea (1 <= m < 2) that is
// 2^(ea - ef) when m <= 1.75 and 2^(ea - ef + 1) otherwise, read off the bits;
// neutral when p or 1/p is not a normal fp32.
//
// A tensor bound to the same values as an earlier one (Tensor::amax_src) takes
// that tensor's amax and records it as its own; the source always holds its own
// amax, so no thread reads a word another one writes.
__device__ __forceinline__ void scales_of_tensor(int t, int fmask, const Tensor* __restrict__ tens, unsigned* amax_bits,
                                                 float* __restrict__ scales, int* __restrict__ tensor_flags,
                                                 LaunchStatus* status, int pow2) {
    const int src = tens[t].amax_src;
    unsigned bits = *reinterpret_cast<volatile unsigned*>(amax_bits + src);
    if (src != t) amax_bits[t] = bits;
    int bad = bits >= 0x7F800000u;
    tensor_flags[t] = bad;
    if (bad) atomicExch(&status->nonfinite, 1);
    float amax = __uint_as_float(bits);
    int slot = 0;
#pragma unroll
    for (int f = 1; f <= 2; ++f) {
        if (!(fmask & f)) continue;
        float fmax = (f == kMaskE4M3) ? 448.0f : 57344.0f;
        float scale = 1.0f, inv = 1.0f;
        if (!bad && amax > 0.0f && pow2) {
            const int ef = (f == kMaskE4M3) ? 8 : 15;
            const int field = (int)(bits >> 23);  // 0 for a subnormal amax: far below the range anyway
            const int k = field - 127 - ef + ((bits & 0x7FFFFFu) > 0x600000u ? 1 : 0);
            if (field > 0 && k >= -126 && k <= 126) {
                scale = __uint_as_float((unsigned)(k + 127) << 23);
                inv = __uint_as_float((unsigned)(127 - k) << 23);
            }
        } else if (!bad && amax > 0.0f) {
            float i = __fdiv_rn(fmax, amax);
            if (i <= 3.402823466e+38f) {
                inv = i;
                scale = __fdiv_rn(amax, fmax);
            }
        }
        scales[t * 2 * kMaxLow + slot * 2 + 0] = scale;
        scales[t * 2 * kMaxLow + slot * 2 + 1] = inv;
        ++slot;
    }
}

__global__ void scales_kernel(ScalesArgs a) {
    int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t < a.T) scales_of_tensor(t, a.fmask, a.tens, a.amax_bits, a.scales, a.flags, a.status, a.pow2);
}

// The alias step of scales_kernel alone, for passes that stop after the amax.
__global__ void resolve_amax_kernel(int T, const Tensor* __restrict__ tens, unsigned* __restrict__ amax_bits) {
    int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const int src = tens[t].amax_src;
    if (src != t) amax_bits[t] = amax_bits[src];
}

__global__ void __launch_bounds__(kThreads)
amax_kernel(const Tensor* __restrict__ tens, const long long* __restrict__ tile_begin, int T, int tile_elems,
            unsigned* amax_bits, ScalesArgs tail) {
    __shared__ int s_slot;
    __shared__ int s_last;
    __shared__ unsigned s_warp[kThreads / 32];
    const long long tile = blockIdx.x;
    const int t = find_tensor(tile_begin, T, tile, &s_slot);
    const Tensor& tn = tens[t];
    const long long first = (tile - __ldg(tile_begin + t)) * (long long)tile_elems;
    const long long left = tn.numel - first;
    int n = left < tile_elems ? (int)left : tile_elems;
#ifdef AMPQ_BOUNDS_CHECK
    if (first < 0 || left <= 0) n = 0;  // a tile outside its tensor is not read (the scoring pass reports it)
#endif
    const int es = tn.dtype == 0 ? 4 : 2;
    const char* base = reinterpret_cast<const char*>(tn.values) + first * es;
    unsigned m = 0;  // fp32 bit pattern of the running max |x|
    if (tn.causal_shift > 0) {
        // triangular operand (16-byte aligned, whole rows per tile): warp w takes
        // rows w, w + 8, ... of the tile and its lanes stride over the vectors the
        // row keeps, four loads in flight per lane
        const int per = 16 / es;
        const int shift = tn.causal_shift;
        const int nrows = n >> shift;
        const long long row0 = first >> shift;
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        for (int r = warp; r < nrows; r += kThreads / 32) {
            const int nv = causal_row_vectors(row0 + r, shift, per);
            const uint4* vp = reinterpret_cast<const uint4*>(base + ((long long)r << shift) * es);
            for (int c = lane; c < nv; c += 32 * 4) {
                uint4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    v[u] = c + 32 * u < nv ? ld_stream_v4(vp + c + 32 * u) : make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const unsigned w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        if (tn.dtype == 0) {
                            m = max(m, w[k] & 0x7FFFFFFFu);
                        } else {
                            m = max(m, (w[k] & 0x7FFFu) << 16);
                            m = max(m, w[k] & 0x7FFF0000u);
                        }
                    }
                }
            }
        }
    } else if ((reinterpret_cast<uintptr_t>(base) & 15) == 0) {
        const int per = 16 / es;
        const int nvec = n / per;
        const uint4* vp = reinterpret_cast<const uint4*>(base);
        if (tn.dtype == 0) {
            for (int i = threadIdx.x; i < nvec; i += kThreads * 4) {
                uint4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    int idx = i + u * kThreads;
                    v[u] = idx < nvec ? ld_stream_v4(vp + idx) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    m = max(m, v[u].x & 0x7FFFFFFFu); m = max(m, v[u].y & 0x7FFFFFFFu);
                    m = max(m, v[u].z & 0x7FFFFFFFu); m = max(m, v[u].w & 0x7FFFFFFFu);
                }
            }
        } else {
            unsigned lo = 0, hi = 0;  // 16-bit patterns of |x|
            for (int i = threadIdx.x; i < nvec; i += kThreads * 4) {
                uint4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    int idx = i + u * kThreads;
                    v[u] = idx < nvec ? ld_stream_v4(vp + idx) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const unsigned w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        lo = max(lo, w[k] & 0x7FFFu);
                        hi = max(hi, w[k] & 0x7FFF0000u);
                    }
                }
            }
            m = max(lo << 16, hi);
        }
        for (int i = nvec * per + threadIdx.x; i < n; i += kThreads) {
            float x = tn.dtype == 0 ? Elem<0>::load(base, i) : Elem<1>::load(base, i);
            m = max(m, __float_as_uint(x) & 0x7FFFFFFFu);
        }
    } else {
        for (int i = threadIdx.x; i < n; i += kThreads) {
            float x = tn.dtype == 0 ? Elem<0>::load(base, i) : Elem<1>::load(base, i);
            m = max(m, __float_as_uint(x) & 0x7FFFFFFFu);
        }
    }
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned r = s_warp[0];
#pragma unroll
        for (int w = 1; w < kThreads / 32; ++w) r = max(r, s_warp[w]);
        atomicMax(amax_bits + t, r);
    }
    // With a tail, the CTA that finishes last (a counter, nobody waits) forms the
    // scales of all tensors, which saves the launch of scales_kernel.
    if (tail.counter != nullptr) {
        if (threadIdx.x == 0) {
            __threadfence();
            s_last = atomicAdd(tail.counter, 1u) == gridDim.x - 1;
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            for (int u = threadIdx.x; u < tail.T; u += kThreads)
                scales_of_tensor(u, tail.fmask, tail.tens, tail.amax_bits, tail.scales, tail.flags, tail.status, tail.pow2);
        }
    }
}

// ---------------------------------------------------------------------------
// fused scoring

template <int FMASK>
struct Fm {
    static constexpr int kLow = (FMASK & 1) + ((FMASK >> 1) & 1);
    static constexpr int kAcc = 1 + kLow;
    static constexpr int kFmt0 = (FMASK & 1) ? kMaskE4M3 : kMaskE5M2;  // unused when FMASK = 0 (S only)
    static constexpr int kFmt1 = kMaskE5M2;
};

// Accumulators of one sample: S and D per low format, two fp32 lanes each.
template <int NACC>
struct Acc {
    float2 v[NACC];
};

template <int FMASK, int RB, int NP>
__device__ __forceinline__ void accumulate_pairs(const float2 (&z)[NP], const float2 (&g)[RB][NP],
                                                 const float2 (&inv2)[2], const float2 (&nsc2)[2],
                                                 Acc<Fm<FMASK>::kAcc> (&acc)[RB]) {
#pragma unroll
    for (int k = 0; k < NP; ++k) {
        float2 ne0, ne1;
        if constexpr (Fm<FMASK>::kLow >= 1) ne0 = neg_err_pair<Fm<FMASK>::kFmt0>(z[k], inv2[0], nsc2[0]);
        if constexpr (Fm<FMASK>::kLow == 2) ne1 = neg_err_pair<Fm<FMASK>::kFmt1>(z[k], inv2[1], nsc2[1]);
#pragma unroll
        for (int r = 0; r < RB; ++r) {
            float2 p = __fmul2_rn(z[k], g[r][k]);
            acc[r].v[0] = __ffma2_rn(p, p, acc[r].v[0]);
            if constexpr (Fm<FMASK>::kLow >= 1) {
                float2 t0 = __fmul2_rn(ne0, g[r][k]);
                acc[r].v[1] = __ffma2_rn(t0, t0, acc[r].v[1]);
            }
            if constexpr (Fm<FMASK>::kLow == 2) {
                float2 t1 = __fmul2_rn(ne1, g[r][k]);
                acc[r].v[Fm<FMASK>::kAcc - 1] = __ffma2_rn(t1, t1, acc[r].v[Fm<FMASK>::kAcc - 1]);
            }
        }
    }
}

// One tile: n elements of values at vbase weighted by RB gradient streams.
template <int DT, int FMASK, int RB>
__device__ __forceinline__ void score_tile(const char* vbase, const char* const (&gbase)[RB], int n,
                                           const float2 (&inv2)[2], const float2 (&nsc2)[2],
                                           Acc<Fm<FMASK>::kAcc> (&acc)[RB]) {
    using E = Elem<DT>;
    constexpr int NP = E::kPerVec / 2;
    constexpr int U = RB == 1 ? 4 : (RB == 2 ? 2 : 1);
    bool aligned = (reinterpret_cast<uintptr_t>(vbase) & 15) == 0;
#pragma unroll
    for (int r = 0; r < RB; ++r) aligned = aligned && (reinterpret_cast<uintptr_t>(gbase[r]) & 15) == 0;
    int done = 0;
    if (aligned) {
        const int nvec = n / E::kPerVec;
        const uint4* vp = reinterpret_cast<const uint4*>(vbase);
        for (int i = threadIdx.x; i < nvec; i += kThreads * U) {
            uint4 v[U], g[RB][U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int idx = i + u * kThreads;
                if (idx < nvec) {
                    v[u] = ld_stream_v4(vp + idx);
#pragma unroll
                    for (int r = 0; r < RB; ++r)
                        g[r][u] = ld_stream_v4(reinterpret_cast<const uint4*>(gbase[r]) + idx);
                } else {  // zeros add nothing to any sum
                    v[u] = make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int r = 0; r < RB; ++r) g[r][u] = make_uint4(0, 0, 0, 0);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float2 z[NP], gg[RB][NP];
                E::unpack(v[u], z);
#pragma unroll
                for (int r = 0; r < RB; ++r) E::unpack(g[r][u], gg[r]);
                accumulate_pairs<FMASK, RB, NP>(z, gg, inv2, nsc2, acc);
            }
        }
        done = nvec * E::kPerVec;
    }
    // ragged tail of an aligned tile, or the whole of a misaligned one
    for (int i = done + threadIdx.x; i < n; i += kThreads) {
        float2 z[1], gg[RB][1];
        z[0] = make_float2(E::load(vbase, i), 0.0f);
#pragma unroll
        for (int r = 0; r < RB; ++r) gg[r][0] = make_float2(E::load(gbase[r], i), 0.0f);
        accumulate_pairs<FMASK, RB, 1>(z, gg, inv2, nsc2, acc);
    }
}

// ---------------------------------------------------------------------------
// shared-memory ring fed by bulk asynchronous copies (TMA, untiled form)

__device__ __forceinline__ unsigned smem_u32(const void* p) {
    return (unsigned)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(unsigned long long* b, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* b) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* b, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
// One poll of a phase; the hardware may park the thread for up to `hint_ns`
// before it answers, which keeps a waiting warp out of the issue slots.
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* b, unsigned parity, unsigned hint_ns = 2000u) {
    unsigned ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(b)), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}
// Global -> this CTA's shared memory, completion counted in bytes on an
// mbarrier.  Both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned bytes, unsigned long long* b) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(b))
                 : "memory");
}
__device__ __forceinline__ uint4 lds_v4(const void* p) {
    uint4 r;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "r"(smem_u32(p)));
    return r;
}
__device__ __forceinline__ void consumer_barrier() {  // the kConsumers scoring threads only
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
}

// Polls and suspend hint of the stage waits (scoring warps waiting for a full
// stage, the producer waiting for an empty one).  A test build
// (-DAMPQ_TEST_SHORT_WAITS) makes them give up after a handful of polls, long
// before the copy they wait for can land, to exercise the time-out path: every
// copy still completes, because the producer's final drain below keeps the full
// limit.
#ifdef AMPQ_TEST_SHORT_WAITS
constexpr unsigned kStageSpinLimit = 2u;
constexpr unsigned kStageHintNs = 0u;
#else
constexpr unsigned kStageSpinLimit = kSpinLimit;
constexpr unsigned kStageHintNs = 2000u;
#endif

// Waits for a phase of an mbarrier, at most kStageSpinLimit polls.  A wait that
// runs out raises the CTA's abort flag; once that is up every wait returns
// false after one poll, so that all threads still walk the same control flow to
// the end.
__device__ __forceinline__ bool mbar_wait(unsigned long long* b, unsigned parity, volatile int* s_abort) {
    if (mbar_try_wait(b, parity, kStageHintNs)) return true;
    for (unsigned spin = 0; spin < kStageSpinLimit; ++spin) {
        if (*s_abort) return false;
        if (mbar_try_wait(b, parity, kStageHintNs)) return true;
    }
    *s_abort = 1;
    return false;
}

// Position in the ring: stage index and the parity of the lap it is in.
template <int STAGES>
struct RingPos {
    unsigned stage = 0, parity = 0;
    __device__ __forceinline__ void advance() {
        if (++stage == STAGES) {
            stage = 0;
            parity ^= 1u;
        }
    }
};

// CTA-wide sum of RB*NACC values in a fixed order over the scoring warps;
// thread a < RB*NACC writes partial (r, a) of the tile.  s_red holds one
// kConsumers/32 x RB*NACC block; the caller alternates two blocks from tile to
// tile so that a tile's readers never meet the next tile's writers.
template <int NACC, int RB, class A64>
__device__ __forceinline__ void reduce_and_store(const A64& acc, double* s_red,
                                                 double* __restrict__ partials, long long slot0,
                                                 long long slot_stride, int out_stride) {
    constexpr int NV = RB * NACC;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int r = 0; r < RB; ++r) {
#pragma unroll
        for (int a = 0; a < NACC; ++a) {
            double x = acc.get(r, a);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
            if (lane == 0) s_red[warp * NV + r * NACC + a] = x;
        }
    }
    consumer_barrier();
    if (threadIdx.x < NV) {
        double x = 0.0;
#pragma unroll
        for (int w = 0; w < kConsumers / 32; ++w) x += s_red[w * NV + threadIdx.x];
        const int r = threadIdx.x / NACC, a = threadIdx.x % NACC;
        partials[(slot0 + r * slot_stride) * out_stride + a] = x;  // out_stride >= NACC doubles per slot
    }
}

// The fp64 accumulators of a tile, one set per scoring thread: in registers, or,
// with three and four gradient streams, where the registers run out, in this
// thread's column of a shared-memory block (entry (r, a) of thread t at
// [(r * NACC + a) * kConsumers + t]: consecutive threads, consecutive words).
template <int NACC, int RB>
struct Acc64Reg {
    double v[RB][NACC];
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int r = 0; r < RB; ++r)
#pragma unroll
            for (int a = 0; a < NACC; ++a) v[r][a] = 0.0;
    }
    __device__ __forceinline__ void add(int r, int a, double x) { v[r][a] += x; }
    __device__ __forceinline__ double get(int r, int a) const { return v[r][a]; }
};
template <int NACC, int RB>
struct Acc64Smem {
    double* col;
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int k = 0; k < RB * NACC; ++k) col[k * kConsumers] = 0.0;
    }
    __device__ __forceinline__ void add(int r, int a, double x) { col[(r * NACC + a) * kConsumers] += x; }
    __device__ __forceinline__ double get(int r, int a) const { return col[(r * NACC + a) * kConsumers]; }
};
#ifndef AMPQ_ACC64_SMEM_FROM
#define AMPQ_ACC64_SMEM_FROM 3   // gradient streams from which the fp64 accumulators live in shared memory
#endif
template <int RB>
constexpr bool kAcc64InSmem = RB >= AMPQ_ACC64_SMEM_FROM;
template <int NACC, int RB>
using Acc64 = typename std::conditional<kAcc64InSmem<RB>, Acc64Smem<NACC, RB>, Acc64Reg<NACC, RB>>::type;

template <int NACC, int RB, class A64>
__device__ __forceinline__ void flush_acc(Acc<NACC> (&acc)[RB], A64& acc64) {
#pragma unroll
    for (int r = 0; r < RB; ++r)
#pragma unroll
        for (int a = 0; a < NACC; ++a) {
            acc64.add(r, a, (double)acc[r].v[a].x + (double)acc[r].v[a].y);
            acc[r].v[a] = make_float2(0.0f, 0.0f);
        }
}

// n elements straight from global memory (what the ring does not carry: ragged
// ends and tensors that are not 16-byte aligned), in blocks of kSubElems so that
// an fp32 accumulator lane never sees more than kSubElems / kConsumers terms.
template <int DT, int FMASK, int RB, class A64>
__device__ __forceinline__ void score_direct(const char* vbase, const char* const (&gbase)[RB], int n,
                                             const float2 (&inv2)[2], const float2 (&nsc2)[2], A64& acc64) {
    constexpr int NACC = Fm<FMASK>::kAcc;
    const int es = Elem<DT>::kBytes;
    for (int sub = 0; sub < n; sub += kSubElems) {
        Acc<NACC> acc[RB];
#pragma unroll
        for (int r = 0; r < RB; ++r)
#pragma unroll
            for (int a = 0; a < NACC; ++a) acc[r].v[a] = make_float2(0.0f, 0.0f);
        const int m = n - sub < kSubElems ? n - sub : kSubElems;
        const char* gsub[RB];
#pragma unroll
        for (int r = 0; r < RB; ++r) gsub[r] = gbase[r] + (long long)sub * es;
        score_tile<DT, FMASK, RB>(vbase + (long long)sub * es, gsub, m, inv2, nsc2, acc);
        flush_acc<NACC, RB>(acc, acc64);
    }
}

// One tile of a causal operand (one sample per read): whole matrix rows, of
// which only the vectors on or left of the diagonal are read -- straight from
// global memory, because a row's kept part is one short contiguous run and the
// ring would need one bulk copy per row and stream (the copy rate, not the
// bytes, then sets the pace).  A warp takes groups of consecutive rows (groups
// strided over the warps).  Its work items are (row, slot of 32 vectors); every
// lane keeps kU items per stream in flight, and the items run on from one row
// of the group into the next, so that a short row, or the ragged end of a long
// one, leaves at most 31 lanes of one item idle instead of most of kU items.
template <int DT, int FMASK>
__device__ __forceinline__ void score_causal_rows(const char* vbase, const char* gbase, int n, long long row0,
                                                  int shift, const float2 (&inv2)[2], const float2 (&nsc2)[2],
                                                  Acc64Reg<Fm<FMASK>::kAcc, 1>& acc64) {
    using E = Elem<DT>;
    constexpr int NACC = Fm<FMASK>::kAcc;
    constexpr int NP = E::kPerVec / 2;
    constexpr int kU = 4;
    constexpr int kWarps = kConsumers / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nrows = n >> shift;
    // rows per group: up to 8, fewer when the tile has too few rows to give every warp a group
    int group = nrows / kWarps;
    group = group < 1 ? 1 : (group > 8 ? 8 : group);
    Acc<NACC> acc[1];
#pragma unroll
    for (int a = 0; a < NACC; ++a) acc[0].v[a] = make_float2(0.0f, 0.0f);
    int since_flush = 0;
    for (int r0 = warp * group; r0 < nrows; r0 += kWarps * group) {
        const int r1 = r0 + group < nrows ? r0 + group : nrows;
        int r = r0;                                                     // the next item: row r, vectors c .. c + 31
        int c = 0;
        int nv = causal_row_vectors(row0 + r, shift, E::kPerVec);
        while (r < r1) {
            uint4 v[kU], g[kU];
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const bool live = r < r1 && c + lane < nv;
                const long long off = (((long long)r << shift) * E::kBytes) + (long long)(c + lane) * 16;
                v[u] = live ? ld_stream_v4(vbase + off) : make_uint4(0, 0, 0, 0);
                g[u] = live ? ld_stream_v4(gbase + off) : make_uint4(0, 0, 0, 0);
                c += 32;
                if (r < r1 && c >= nv) {  // on to the next row of the group (uniform over the warp)
                    ++r;
                    c = 0;
                    if (r < r1) nv = causal_row_vectors(row0 + r, shift, E::kPerVec);
                }
            }
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                float2 z[NP], gg[1][NP];
                E::unpack(v[u], z);
                E::unpack(g[u], gg[0]);
                accumulate_pairs<FMASK, 1, NP>(z, gg, inv2, nsc2, acc);
            }
            since_flush += kU * NP;
            if (since_flush + kU * NP > kFlushTerms) {  // at most kFlushTerms terms per fp32 lane
                flush_acc<NACC, 1>(acc, acc64);
                since_flush = 0;
            }
        }
    }
    flush_acc<NACC, 1>(acc, acc64);
}

// Geometry of the ring for RB gradient streams per value stream.  The
// compile-time knobs exist for tuning builds; the defaults are what was
// measured best on B200.
#ifndef AMPQ_RING_U12
#define AMPQ_RING_U12 2   // 16-byte vectors per thread, stream and chunk, RB <= 2
#endif
#ifndef AMPQ_RING_U34
#define AMPQ_RING_U34 1   // the same for RB >= 3
#endif
#ifndef AMPQ_RING_BYTES
#define AMPQ_RING_BYTES (64 * 1024)  // ring budget per CTA; deeper rings measured no faster
#endif
template <int RB>
struct Ring {
    static constexpr int kU = RB <= 2 ? AMPQ_RING_U12 : AMPQ_RING_U34;
    static constexpr int kChunkBytes = kU * kConsumers * 16;          // bytes of one stream in one stage
    static constexpr int kStageBytes = (1 + RB) * kChunkBytes;
#if defined(AMPQ_STAGES_RB1) && defined(AMPQ_STAGES_RB2)
    static constexpr int kStages = RB == 1 ? AMPQ_STAGES_RB1 : (RB == 2 ? AMPQ_STAGES_RB2 : AMPQ_RING_BYTES / kStageBytes);
#else
    static constexpr int kStages = AMPQ_RING_BYTES / kStageBytes;
#endif
    static_assert(kStages >= 2, "the ring needs at least two stages");
    static constexpr int kRingBytes = kStages * kStageBytes;
    static constexpr int kRedDoubles = 2 * (kConsumers / 32) * RB * kMaxAcc;
    static constexpr int kAcc64Doubles = kAcc64InSmem<RB> ? RB * kMaxAcc * kConsumers : 0;  // fp64 accumulators kept in shared memory
    // ring | full[kStages] empty[kStages] | reduction blocks | fp64 accumulators | abort flag
    static constexpr int kSmemBytes = kRingBytes + 2 * kStages * 8 + (kRedDoubles + kAcc64Doubles) * 8 + 16;
};

// The scoring warps' side of the ring for one tile: nchunks stages, each
// taken into registers, handed back, then scored.
template <int DT, int FMASK, int RB, class A64>
__device__ __forceinline__ void consume_chunks(int nchunks, const unsigned char* ring, unsigned long long* full,
                                               unsigned long long* empty, RingPos<Ring<RB>::kStages>& pos,
                                               volatile int* s_abort, const float2 (&inv2)[2],
                                               const float2 (&nsc2)[2], Acc<Fm<FMASK>::kAcc> (&acc)[RB],
                                               A64& acc64) {
    using RG = Ring<RB>;
    using E = Elem<DT>;
    constexpr int NACC = Fm<FMASK>::kAcc;
    constexpr int U = RG::kU;
    constexpr int NP = E::kPerVec / 2;
    const int tid = threadIdx.x;
    int since_flush = 0;
    for (int c = 0; c < nchunks; ++c) {
        const bool ok = mbar_wait(full + pos.stage, pos.parity, s_abort);
        uint4 v[U], g[RB][U];
        if (ok) {
            const unsigned char* st = ring + pos.stage * RG::kStageBytes + tid * 16;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                v[u] = lds_v4(st + u * kConsumers * 16);
#pragma unroll
                for (int r = 0; r < RB; ++r) g[r][u] = lds_v4(st + (1 + r) * RG::kChunkBytes + u * kConsumers * 16);
            }
        }
        __syncwarp();
        if (ok && (tid & 31) == 0) mbar_arrive(empty + pos.stage);  // the warp's vectors are in registers
        pos.advance();
        if (ok) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float2 z[NP], gg[RB][NP];
                E::unpack(v[u], z);
#pragma unroll
                for (int r = 0; r < RB; ++r) E::unpack(g[r][u], gg[r]);
                accumulate_pairs<FMASK, RB, NP>(z, gg, inv2, nsc2, acc);
            }
        }
        // at most kFlushTerms terms per fp32 lane between two flushes
        since_flush += U * NP;
        if (since_flush >= kFlushTerms) {
            flush_acc<NACC, RB>(acc, acc64);
            since_flush = 0;
        }
    }
}

// Where a tile lives.
struct TileGeom {
    long long voff, goff, slot0;
    int r0, n;
};

template <int RB, bool CAUSAL>
__device__ __forceinline__ TileGeom tile_geometry(const Tensor& tn, int local, int tile_shift) {
    TileGeom q;
    int i;  // value tile within the segment
    if (tn.per_sample) {  // one sample per tile; RB > 1: the RB streams are RB layers' gradients of that sample
        q.r0 = local / tn.tiles_per_seg;
        i = local - q.r0 * tn.tiles_per_seg;
        q.voff = (long long)q.r0 * tn.seg_len + ((long long)i << tile_shift);
    } else if (RB == kMaxRB) {  // full groups of four samples
        const int nfull = tn.R / kMaxRB;
        i = local / nfull;
        q.r0 = (local - i * nfull) * kMaxRB;
        q.voff = (long long)i << tile_shift;
    } else {  // the remainder group: the last R mod 4 samples
        i = local;
        q.r0 = (tn.R / kMaxRB) * kMaxRB;
        q.voff = (long long)i << tile_shift;
    }
    if (CAUSAL && 2 * tn.causal_shift > tile_shift) {
        // A T x T triangular matrix spans P = T^2 / tile tiles whose work grows with
        // their position k in the matrix (tile k holds rows whose kept prefix is
        // about k/P of a row).  A persistent CTA walks the tiles with a fixed
        // stride, which for common P would always land it on the same k; rotating k
        // by a hash of the matrix index gives every CTA every k.  The partial slot
        // follows the tile's true position, so the sums do not change.
        const int lp = 2 * tn.causal_shift - tile_shift;
        const unsigned m = (unsigned)i >> lp, k = (unsigned)i & ((1u << lp) - 1u);
        const unsigned rot = (m * 0x9E3779B1u) >> (32 - lp);
        i = (int)((m << lp) | ((k + rot) & ((1u << lp) - 1u)));
        q.voff = (long long)q.r0 * tn.seg_len + ((long long)i << tile_shift);
    }
    q.goff = (long long)i << tile_shift;  // offset inside a sample's gradient
    const long long left = tn.seg_len - q.goff;
    q.n = left < (1LL << tile_shift) ? (int)left : (1 << tile_shift);
    q.slot0 = tn.partial_base + (long long)q.r0 * tn.tiles_per_seg + i;
    return q;
}

// Gradient streams of a tile (Tensor::gstream): the next samples of a shared
// operand's own gradients, or the gradients of the other layers that read this
// per-sample operand.
template <int RB, int ES>
__device__ __forceinline__ void grad_bases(const Tensor& tn, const TileGeom& q, const char* (&gb)[RB]) {
    const long long off = (q.goff + (long long)q.r0 * tn.grad_stride) * ES;
    gb[0] = reinterpret_cast<const char*>(tn.grads) + off;
#pragma unroll
    for (int r = 1; r < RB; ++r) gb[r] = reinterpret_cast<const char*>(tn.gstream[r - 1]) + off;
}

// Debug builds (-DAMPQ_BOUNDS_CHECK): a tile whose element range, samples or
// partial slots fall outside what its tensor owns is reported in the status
// word and skipped by the producer and the scoring warps alike, instead of
// being read.  The check costs a few compares per tile and is compiled out of
// release builds.
template <int RB>
__device__ __forceinline__ bool tile_in_bounds(const Tensor& tn, const TileGeom& q) {
#ifdef AMPQ_BOUNDS_CHECK
    const long long vals = tn.per_sample ? tn.numel : tn.seg_len;
    const long long per_tensor = (long long)tn.R * tn.tiles_per_seg;
    const bool shared_input = RB > 1 && tn.per_sample;
    const int last_r = shared_input ? q.r0 : q.r0 + RB - 1;
    const long long owned = shared_input ? RB * per_tensor : per_tensor;
    return q.n > 0 && q.goff >= 0 && q.goff + q.n <= tn.seg_len && q.voff >= 0 && q.voff + q.n <= vals &&
           q.r0 >= 0 && last_r < tn.R && (!shared_input || tn.share_n == RB) && q.slot0 >= tn.partial_base &&
           q.slot0 + (long long)(RB - 1) * tn.stream_slot_stride < tn.partial_base + owned;
#else
    return true;
#endif
}

// The scoring warps' walk over the tiles of the launch (see score_kernel).
template <int DT, int FMASK, int RB, bool CAUSAL>
__device__ __forceinline__ void score_tiles(const Tensor* __restrict__ tens, const long long* __restrict__ tile_begin,
                                            long long ntiles, int tile_shift, const float* __restrict__ scales,
                                            double* __restrict__ partials, LaunchStatus* __restrict__ status,
                                            int out_stride, const unsigned char* ring, unsigned long long* full,
                                            unsigned long long* empty, double* s_red, double* s_acc64,
                                            volatile int* s_abort) {
    using RG = Ring<RB>;
    constexpr int NACC = Fm<FMASK>::kAcc;
    RingPos<RG::kStages> pos;  // the same walk of the ring as the producer's
    int t = 0;                 // tensor of the current tile; tiles only move forward
    int red_block = 0;
    for (long long tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        while (tile >= __ldg(tile_begin + t + 1)) ++t;
        const Tensor& tn = tens[t];
        const TileGeom q = tile_geometry<RB, CAUSAL>(tn, (int)(tile - __ldg(tile_begin + t)), tile_shift);
        constexpr int es = Elem<DT>::kBytes;
        float2 inv2[2], nsc2[2];
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            const float sc = __ldg(scales + t * 2 * kMaxLow + s * 2 + 0);
            const float iv = __ldg(scales + t * 2 * kMaxLow + s * 2 + 1);
            inv2[s] = make_float2(iv, iv);
            nsc2[s] = make_float2(-sc, -sc);
        }
        const char* vb = reinterpret_cast<const char*>(tn.values) + q.voff * es;
        const char* gb[RB];
        grad_bases<RB, es>(tn, q, gb);
        bool aligned = (reinterpret_cast<uintptr_t>(vb) & 15) == 0;
#pragma unroll
        for (int r = 0; r < RB; ++r) aligned = aligned && (reinterpret_cast<uintptr_t>(gb[r]) & 15) == 0;
        const bool inside = tile_in_bounds<RB>(tn, q);
        if (!inside) {  // only in a bounds-checking build: report, score nothing, move on
            if (threadIdx.x == 0) atomicExch(&status->bounds, 1);
            continue;
        }
        const int nchunks = aligned && !CAUSAL ? (int)(((long long)q.n * es) / RG::kChunkBytes) : 0;

        Acc64<NACC, RB> acc64;
        if constexpr (kAcc64InSmem<RB>) acc64.col = s_acc64 + threadIdx.x;
        acc64.zero();
        Acc<NACC> acc[RB];
#pragma unroll
        for (int r = 0; r < RB; ++r)
#pragma unroll
            for (int a = 0; a < NACC; ++a) acc[r].v[a] = make_float2(0.0f, 0.0f);
        consume_chunks<DT, FMASK, RB>(nchunks, ring, full, empty, pos, s_abort, inv2, nsc2, acc, acc64);
        flush_acc<NACC, RB>(acc, acc64);
        // what the ring did not carry
        const int done = (int)(((long long)nchunks * RG::kChunkBytes) / es);
        if constexpr (CAUSAL) {
            score_causal_rows<DT, FMASK>(vb, gb[0], q.n, q.goff >> tn.causal_shift, tn.causal_shift, inv2, nsc2, acc64);
        } else if (done < q.n) {
            const char* gt[RB];
#pragma unroll
            for (int r = 0; r < RB; ++r) gt[r] = gb[r] + (long long)done * es;
            score_direct<DT, FMASK, RB>(vb + (long long)done * es, gt, q.n - done, inv2, nsc2, acc64);
        }
        reduce_and_store<NACC, RB>(acc64, s_red + red_block * (kConsumers / 32) * RB * NACC, partials, q.slot0,
                                   tn.stream_slot_stride, out_stride);
        red_block ^= 1;
    }
}

// The scoring kernel.  Persistent: CTA b takes tiles b, b + gridDim.x, ... of
// the launch's tile table.  Warps 0..7 score; warp 8 is the producer: one lane
// streams every full 16-byte-aligned chunk of the value tile and of its RB
// gradient tiles into a ring of shared-memory stages with bulk asynchronous
// copies, running as far ahead as the ring is deep, tile after tile, so that
// the bytes in flight do not depend on how long the arithmetic of a chunk
// takes.  A scoring thread takes its 16-byte vectors of a stage into
// registers, hands the stage back and then does the arithmetic.  fp32 sums are
// flushed into fp64 every kFlushTerms terms; a tile ends with the CTA-wide
// ordered sum and one partial per (sample, accumulator).
//
// One launch per element type DT and number RB (1..4) of gradient streams per
// read of the values: per-sample operands and the single-sample remainder of
// shared operands run with RB = 1; shared operands (weights) are read once per
// group of up to four samples; a per-sample operand that several layers read is
// read once per group of up to four layers.
template <int DT, int FMASK, int RB, bool CAUSAL>
__global__ void __launch_bounds__(kScoreThreads, kScoreCtasPerSm)
score_kernel(const Tensor* __restrict__ tens, const long long* __restrict__ tile_begin, int T, long long ntiles,
             int tile_shift, const float* __restrict__ scales, double* __restrict__ partials,
             LaunchStatus* __restrict__ status, int out_stride) {
    using RG = Ring<RB>;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* ring = smem;
    unsigned long long* full = reinterpret_cast<unsigned long long*>(smem + RG::kRingBytes);
    unsigned long long* empty = full + RG::kStages;
    double* s_red = reinterpret_cast<double*>(empty + RG::kStages);
    double* s_acc64 = s_red + RG::kRedDoubles;
    volatile int* s_abort = reinterpret_cast<volatile int*>(s_acc64 + RG::kAcc64Doubles);

    if (threadIdx.x == 0) {
        for (int s = 0; s < RG::kStages; ++s) {
            mbar_init(full + s, 1);
            mbar_init(empty + s, kConsumers / 32);
        }
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const bool producer = threadIdx.x >= kConsumers;
    unsigned it = 0;  // chunks the producer has put into the ring so far
    RingPos<RG::kStages> pos;  // both sides walk the ring in the same order
    int t = 0;        // tensor of the current tile; tiles only move forward
    if (producer) {
        if (!CAUSAL && threadIdx.x == kConsumers) {  // causal tiles do not go through the ring
            for (long long tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
                while (tile >= __ldg(tile_begin + t + 1)) ++t;
                const Tensor& tn = tens[t];
                const TileGeom q = tile_geometry<RB, CAUSAL>(tn, (int)(tile - __ldg(tile_begin + t)), tile_shift);
                constexpr int es = Elem<DT>::kBytes;
                const char* vb = reinterpret_cast<const char*>(tn.values) + q.voff * es;
                const char* gb[RB];
                grad_bases<RB, es>(tn, q, gb);
                bool aligned = (reinterpret_cast<uintptr_t>(vb) & 15) == 0;
#pragma unroll
                for (int r = 0; r < RB; ++r) aligned = aligned && (reinterpret_cast<uintptr_t>(gb[r]) & 15) == 0;
                const int nchunks = aligned && tile_in_bounds<RB>(tn, q) ? (int)(((long long)q.n * es) / RG::kChunkBytes) : 0;
                for (int c = 0; c < nchunks; ++c) {
                    // the stage must have been handed back once per earlier lap
                    if (it >= (unsigned)RG::kStages && !mbar_wait(empty + pos.stage, pos.parity ^ 1u, s_abort)) break;
                    unsigned char* dst = ring + pos.stage * RG::kStageBytes;
                    mbar_arrive_expect_tx(full + pos.stage, RG::kStageBytes);
                    bulk_load(dst, vb + (long long)c * RG::kChunkBytes, RG::kChunkBytes, full + pos.stage);
#pragma unroll
                    for (int r = 0; r < RB; ++r)
                        bulk_load(dst + (1 + r) * RG::kChunkBytes, gb[r] + (long long)c * RG::kChunkBytes,
                                  RG::kChunkBytes, full + pos.stage);
                    pos.advance();
                    ++it;
                }
                if (*s_abort) break;
            }
        }
    } else {
        score_tiles<DT, FMASK, RB, CAUSAL>(tens, tile_begin, ntiles, tile_shift, scales, partials, status, out_stride,
                                           ring, full, empty, s_red, s_acc64, s_abort);
    }
    // Every thread of the CTA meets here: the producer has stopped issuing and the
    // scoring warps have stopped taking stages.  If a wait ran out on either side,
    // every copy issued so far must still land before the CTA gives its shared
    // memory back: the producer lane waits (bounded, at the full limit) for the
    // last lap of each stage; a stage's earlier laps had completed before it was
    // refilled.  Then the time-out is reported.
    __syncthreads();
    if (*s_abort && threadIdx.x == kConsumers) {
        for (unsigned k = 0; k < (unsigned)RG::kStages && k < it; ++k) {
            const unsigned j = it - 1 - k;
            for (unsigned spin = 0; spin < kSpinLimit; ++spin)
                if (mbar_try_wait(full + j % RG::kStages, (j / RG::kStages) & 1)) break;
        }
        atomicExch(&status->timeout, 1);
    }
}

// ---------------------------------------------------------------------------
// Per layer (Sec. 2.2): s^r = S(op0,r) + S(op1,r); s = (1/R) sum_r s^r;
// d_model_f = alpha_f s; d_meas^r_f = D_f(op0,r) + D_f(op1,r); d_meas_f = mean_r.
// Format index f = 0 is the high-precision baseline and costs 0.
__device__ __forceinline__ void combine_layer(const Layer& ly, int F, const CombineParams& prm,
                                              const double* seg_out, double* __restrict__ layer_out) {
    const int nacc = prm.nacc, R = ly.R;
    double* o = layer_out + ly.out_off;
    double* s_r = o;
    double* s_mean = o + R;
    double* d_meas_r = o + R + 1;
    double* d_model = d_meas_r + (long long)R * F;
    double* d_meas = d_model + F;
    double acc = 0.0;
    for (int r = 0; r < R; ++r) {
        double v = seg_out[(long long)(ly.seg_base0 + r) * nacc] + seg_out[(long long)(ly.seg_base1 + r) * nacc];
        s_r[r] = v;
        acc += v;
    }
    const double sm = acc / (double)R;
    *s_mean = sm;
    d_model[0] = 0.0;
    d_meas[0] = 0.0;
    for (int r = 0; r < R; ++r) d_meas_r[(long long)r * F] = 0.0;
    for (int f = 1; f < F; ++f) {
        const int a = prm.acc_of_fmt[f];
        d_model[f] = prm.alpha[f] * sm;
        double s = 0.0;
        for (int r = 0; r < R; ++r) {
            double v = seg_out[(long long)(ly.seg_base0 + r) * nacc + a] +
                       seg_out[(long long)(ly.seg_base1 + r) * nacc + a];
            d_meas_r[(long long)r * F + f] = v;
            s += v;
        }
        d_meas[f] = s / (double)R;
    }
}

__global__ void combine_kernel(const Layer* __restrict__ layers, int L, int F, CombineParams prm,
                               const double* __restrict__ seg_out, double* __restrict__ layer_out) {
    int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l < L) combine_layer(layers[l], F, prm, seg_out, layer_out);
}

// Ordered fp64 sum of the per-tile partials of one segment by one warp: lane j
// sums slots j, j+32, ... in order, then a fixed shuffle tree.
__device__ __forceinline__ void finalize_segment(const Segment& sg, int nacc, const double* __restrict__ partials,
                                                 double* out) {
    const int lane = threadIdx.x & 31;
    for (int a = 0; a < nacc; ++a) {
        double x = 0.0;
        for (int j = lane; j < sg.count; j += 32) x += partials[(sg.first_slot + j) * nacc + a];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
        if (lane == 0) out[a] = x;
    }
}

// One warp per segment.  With a tail, the CTA that finishes last (a counter,
// nobody waits) combines the layers, which saves the launch of combine_kernel.
__global__ void finalize_kernel(const Segment* __restrict__ segs, int nseg, int nacc,
                                const double* __restrict__ partials, double* seg_out, CombineArgs tail) {
    __shared__ int s_last;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (warp < nseg) finalize_segment(segs[warp], nacc, partials, seg_out + (long long)warp * nacc);
    if (tail.counter != nullptr) {
        __syncthreads();
        if (threadIdx.x == 0) {
            __threadfence();
            s_last = atomicAdd(tail.counter, 1u) == gridDim.x - 1;
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            for (int l = threadIdx.x; l < tail.L; l += blockDim.x)  // reads what every other CTA wrote before its count
                combine_layer(tail.layers[l], tail.F, tail.prm, seg_out, tail.layer_out);
        }
    }
}

// Test hook: codes of n elements with the scoring kernel's own cast.
template <int DT, int FMT>
__global__ void codes_kernel(const void* __restrict__ values, long long n, const float* __restrict__ scale_pair,
                             unsigned char* __restrict__ out) {
    const float inv = scale_pair[1];
    const long long npairs = (n + 1) / 2;
    for (long long p = blockIdx.x * (long long)blockDim.x + threadIdx.x; p < npairs;
         p += (long long)gridDim.x * blockDim.x) {
        const long long i = 2 * p;
        float2 z = make_float2(Elem<DT>::load(values, i), i + 1 < n ? Elem<DT>::load(values, i + 1) : 0.0f);
        float2 y = __fmul2_rn(z, make_float2(inv, inv));
        unsigned short c = cast_pair<FMT>(y.x, y.y);
        out[i] = (unsigned char)(c & 0xFF);
        if (i + 1 < n) out[i + 1] = (unsigned char)(c >> 8);
    }
}

// ---------------------------------------------------------------------------
// one-segment jobs (streaming calibration, fake quantisation)

__global__ void job_prepare_kernel(SegmentJob* job, const void* values, const void* grads, long long n, int dtype,
                                   float amax_preset, long long ntiles, long long namax, int fmask, int pow2,
                                   LaunchStatus* status) {
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
    job->tensor = t;
    job->tile_begin[0] = 0;
    job->tile_begin[1] = ntiles;
    job->amax_tile_begin[0] = 0;
    job->amax_tile_begin[1] = namax;
    job->segment.first_slot = 0;
    job->segment.count = (int)ntiles;
    job->segment.pad = 0;
    job->amax_bits = amax_preset >= 0.0f ? __float_as_uint(amax_preset) : 0u;
    job->flag = 0;
    job->amax_done = 0;
    // no amax pass follows (preset, or nothing to measure): the scales are known now
    if (namax == 0) scales_of_tensor(0, fmask, &job->tensor, &job->amax_bits, job->scales, &job->flag, status, pow2);
}

// Ends a job: the ordered sum of its per-tile partials (one warp), then the fold
// into the per-tensor arrays of the context: the largest amax any sample used,
// a sticky non-finite flag, the scales of the last sample.
__global__ void job_finish_kernel(const SegmentJob* job, int nacc, const double* __restrict__ partials,
                                  double* seg_out, int tensor, unsigned* amax_bits, int* flags, float* scales) {
    if (blockIdx.x != 0 || threadIdx.x >= 32) return;
    finalize_segment(job->segment, nacc, partials, seg_out);
    if (threadIdx.x != 0) return;
    atomicMax(amax_bits + tensor, job->amax_bits);
    if (job->flag) flags[tensor] = 1;
    for (int k = 0; k < 2 * kMaxLow; ++k) scales[tensor * 2 * kMaxLow + k] = job->scales[k];
}

// The quantised operand itself: out_k = dec(Q(z_k * inv)) * scale as one fp32
// product, stored in the operand's own type (bf16: round to nearest even).
template <int DT, int FMT>
__global__ void fake_quant_kernel(const void* __restrict__ values, long long n, const float* __restrict__ scale_pair,
                                  void* __restrict__ out) {
    const float scale = scale_pair[0], inv = scale_pair[1];
    const long long npairs = (n + 1) / 2;
    for (long long p = blockIdx.x * (long long)blockDim.x + threadIdx.x; p < npairs;
         p += (long long)gridDim.x * blockDim.x) {
        const long long i = 2 * p;
        const bool two = i + 1 < n;
        float2 z = make_float2(Elem<DT>::load(values, i), two ? Elem<DT>::load(values, i + 1) : 0.0f);
        float2 y = __fmul2_rn(z, make_float2(inv, inv));
        float2 dq = decode_pair<FMT>(cast_pair<FMT>(y.x, y.y));
        float2 zh = __fmul2_rn(dq, make_float2(scale, scale));
        if (DT == 0) {
            float* o = reinterpret_cast<float*>(out);
            o[i] = zh.x;
            if (two) o[i + 1] = zh.y;
        } else {
            unsigned short* o = reinterpret_cast<unsigned short*>(out);
            unsigned short lo, hi;
            asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(lo) : "f"(zh.x));
            asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(hi) : "f"(zh.y));
            o[i] = lo;
            if (two) o[i + 1] = hi;
        }
    }
}

// ---------------------------------------------------------------------------
// host launchers

cudaError_t launch_init_amax(const Tensor* tens, int T, unsigned* amax_bits, LaunchStatus* status,
                             cudaStream_t st) {
    init_amax_kernel<<<(T + 255) / 256 > 0 ? (T + 255) / 256 : 1, 256, 0, st>>>(tens, T, amax_bits, status);
    return cudaGetLastError();
}

cudaError_t launch_amax(const Tensor* tens, const long long* tile_begin, int T, long long ntiles, int tile_elems,
                        unsigned* amax_bits, cudaStream_t st, const ScalesArgs& tail) {
    if (ntiles <= 0) return cudaSuccess;
    if (tile_elems < kMinAmaxTileElems || tile_elems > kAmaxTileElems) return cudaErrorInvalidValue;
    amax_kernel<<<(unsigned)ntiles, kThreads, 0, st>>>(tens, tile_begin, T, tile_elems, amax_bits, tail);
    return cudaGetLastError();
}

int pick_amax_tile(long long elems, int sms) {
    int tile = kAmaxTileElems;
    while (tile > kMinAmaxTileElems && elems / tile < 4LL * sms) tile /= 2;
    return tile;
}

cudaError_t launch_scales(int T, int fmask, const Tensor* tens, unsigned* amax_bits, float* scales, int* tensor_flags,
                          LaunchStatus* status, cudaStream_t st, int pow2) {
    if (T <= 0) return cudaSuccess;
    scales_kernel<<<(T + 255) / 256, 256, 0, st>>>(scales_args(T, fmask, tens, amax_bits, scales, tensor_flags, status, pow2));
    return cudaGetLastError();
}

cudaError_t launch_resolve_amax(int T, const Tensor* tens, unsigned* amax_bits, cudaStream_t st) {
    if (T <= 0) return cudaSuccess;
    resolve_amax_kernel<<<(T + 255) / 256, 256, 0, st>>>(T, tens, amax_bits);
    return cudaGetLastError();
}

#ifndef AMPQ_TILES_PER_CTA
#define AMPQ_TILES_PER_CTA 16   // tiles a CTA of the persistent grid should get before tiles stop shrinking
#endif
int pick_tile_shift(long long scored_elems, int max_ctas) {
    int shift = kMaxTileShift;
    while (shift > kMinTileShift && (scored_elems >> shift) < (long long)AMPQ_TILES_PER_CTA * max_ctas) --shift;
    return shift;
}

template <int DT, int FMASK, int RB, bool CAUSAL>
static cudaError_t launch_score_inst(const Tensor* tens, const long long* tile_begin, int T, long long ntiles,
                                     int tile_shift, int max_ctas, const float* scales, double* partials,
                                     LaunchStatus* status, cudaStream_t st, int out_stride) {
    constexpr int smem = Ring<RB>::kSmemBytes;
    if (out_stride < Fm<FMASK>::kAcc) out_stride = Fm<FMASK>::kAcc;
    // the shared-memory opt-in of an instantiation is set once per device
    static std::atomic<unsigned long long> opted_in{0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 64 || !(opted_in.load(std::memory_order_acquire) >> dev & 1ULL)) {
        e = cudaFuncSetAttribute(score_kernel<DT, FMASK, RB, CAUSAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        if (dev < 64) opted_in.fetch_or(1ULL << dev, std::memory_order_release);
    }
    const unsigned grid = (unsigned)(ntiles < (long long)max_ctas ? ntiles : (long long)max_ctas);
    score_kernel<DT, FMASK, RB, CAUSAL><<<grid, kScoreThreads, smem, st>>>(tens, tile_begin, T, ntiles, tile_shift,
                                                                           scales, partials, status, out_stride);
    return cudaGetLastError();
}

template <int DT, int RB, bool CAUSAL>
static cudaError_t launch_score_rb(const Tensor* tens, const long long* tile_begin, int T, long long ntiles,
                                   int tile_shift, int max_ctas, int fmask, const float* scales, double* partials,
                                   LaunchStatus* status, cudaStream_t st, int out_stride) {
    switch (fmask) {
        case 0: return launch_score_inst<DT, 0, RB, CAUSAL>(tens, tile_begin, T, ntiles, tile_shift, max_ctas, scales, partials, status, st, out_stride);
        case 1: return launch_score_inst<DT, 1, RB, CAUSAL>(tens, tile_begin, T, ntiles, tile_shift, max_ctas, scales, partials, status, st, out_stride);
        case 2: return launch_score_inst<DT, 2, RB, CAUSAL>(tens, tile_begin, T, ntiles, tile_shift, max_ctas, scales, partials, status, st, out_stride);
        case 3: return launch_score_inst<DT, 3, RB, CAUSAL>(tens, tile_begin, T, ntiles, tile_shift, max_ctas, scales, partials, status, st, out_stride);
        default: return cudaErrorInvalidValue;
    }
}

template <int DT>
static cudaError_t launch_score_dt(int rb, int causal, const Tensor* tens, const long long* tile_begin, int T,
                                   long long ntiles, int tile_shift, int max_ctas, int fmask, const float* scales,
                                   double* partials, LaunchStatus* status, cudaStream_t st, int out_stride) {
    if (causal) {  // causal operands are per-sample operands: one sample per read
        if (rb != 1) return cudaErrorInvalidValue;
        return launch_score_rb<DT, 1, true>(tens, tile_begin, T, ntiles, tile_shift, max_ctas, fmask, scales, partials, status, st, out_stride);
    }
    switch (rb) {
        case 1: return launch_score_rb<DT, 1, false>(tens, tile_begin, T, ntiles, tile_shift, max_ctas, fmask, scales, partials, status, st, out_stride);
        case 2: return launch_score_rb<DT, 2, false>(tens, tile_begin, T, ntiles, tile_shift, max_ctas, fmask, scales, partials, status, st, out_stride);
        case 3: return launch_score_rb<DT, 3, false>(tens, tile_begin, T, ntiles, tile_shift, max_ctas, fmask, scales, partials, status, st, out_stride);
        case 4: return launch_score_rb<DT, 4, false>(tens, tile_begin, T, ntiles, tile_shift, max_ctas, fmask, scales, partials, status, st, out_stride);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_score(int dtype, int rb, const Tensor* tens, const long long* tile_begin, int T, long long ntiles,
                         int tile_shift, int max_ctas, int fmask, const float* scales, double* partials,
                         LaunchStatus* status, cudaStream_t st, int causal, int out_stride) {
    if (ntiles <= 0) return cudaSuccess;
    if (max_ctas < 1 || tile_shift < kMinTileShift || tile_shift > kMaxTileShift) return cudaErrorInvalidValue;
    if (dtype == 0)
        return launch_score_dt<0>(rb, causal, tens, tile_begin, T, ntiles, tile_shift, max_ctas, fmask, scales, partials, status, st, out_stride);
    if (dtype == 1)
        return launch_score_dt<1>(rb, causal, tens, tile_begin, T, ntiles, tile_shift, max_ctas, fmask, scales, partials, status, st, out_stride);
    return cudaErrorInvalidValue;
}

cudaError_t launch_finalize(const Segment* segs, int nseg, int nacc, const double* partials, double* seg_out,
                            cudaStream_t st, const CombineArgs& tail) {
    if (nseg <= 0) return cudaSuccess;
    const int warps_per_block = 8;
    finalize_kernel<<<(nseg + warps_per_block - 1) / warps_per_block, warps_per_block * 32, 0, st>>>(
        segs, nseg, nacc, partials, seg_out, tail);
    return cudaGetLastError();
}

cudaError_t launch_combine(const Layer* layers, int L, int F, const CombineParams& prm, const double* seg_out,
                           double* layer_out, cudaStream_t st) {
    if (L <= 0) return cudaSuccess;
    combine_kernel<<<(L + 127) / 128, 128, 0, st>>>(layers, L, F, prm, seg_out, layer_out);
    return cudaGetLastError();
}

cudaError_t launch_job_prepare(SegmentJob* job, const void* values, const void* grads, long long n, int dtype,
                               float amax_preset, long long ntiles, long long namax, int fmask, int pow2,
                               LaunchStatus* status, cudaStream_t st) {
    job_prepare_kernel<<<1, 32, 0, st>>>(job, values, grads, n, dtype, amax_preset, ntiles, namax, fmask, pow2, status);
    return cudaGetLastError();
}

cudaError_t launch_job_finish(const SegmentJob* job, int nacc, const double* partials, double* seg_out, int tensor,
                              unsigned* amax_bits, int* flags, float* scales, cudaStream_t st) {
    job_finish_kernel<<<1, 32, 0, st>>>(job, nacc, partials, seg_out, tensor, amax_bits, flags, scales);
    return cudaGetLastError();
}

cudaError_t launch_fake_quant(int dtype, int fmt_mask, const void* values, long long n, const float* scale_pair,
                              void* out, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    long long blocks = ((n + 1) / 2 + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    const unsigned grid = (unsigned)blocks;
    if (dtype == 0 && fmt_mask == kMaskE4M3) fake_quant_kernel<0, kMaskE4M3><<<grid, 256, 0, st>>>(values, n, scale_pair, out);
    else if (dtype == 0) fake_quant_kernel<0, kMaskE5M2><<<grid, 256, 0, st>>>(values, n, scale_pair, out);
    else if (fmt_mask == kMaskE4M3) fake_quant_kernel<1, kMaskE4M3><<<grid, 256, 0, st>>>(values, n, scale_pair, out);
    else fake_quant_kernel<1, kMaskE5M2><<<grid, 256, 0, st>>>(values, n, scale_pair, out);
    return cudaGetLastError();
}

cudaError_t launch_codes(int dtype, int fmt_mask, const void* values, long long n, const float* scale_pair,
                         unsigned char* out, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    long long blocks = ((n + 1) / 2 + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    const unsigned grid = (unsigned)blocks;
    if (dtype == 0 && fmt_mask == kMaskE4M3) codes_kernel<0, kMaskE4M3><<<grid, 256, 0, st>>>(values, n, scale_pair, out);
    else if (dtype == 0) codes_kernel<0, kMaskE5M2><<<grid, 256, 0, st>>>(values, n, scale_pair, out);
    else if (fmt_mask == kMaskE4M3) codes_kernel<1, kMaskE4M3><<<grid, 256, 0, st>>>(values, n, scale_pair, out);
    else codes_kernel<1, kMaskE5M2><<<grid, 256, 0, st>>>(values, n, scale_pair, out);
    return cudaGetLastError();
}

}  // namespace ampq

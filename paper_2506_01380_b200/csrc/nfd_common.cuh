// Shared device-side types and helpers of libnfd (CUDA, sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "nfd.h"

typedef __nv_bfloat16 bf16;

// One frame of a forward pass.
struct FrameDesc {
    int stream;      // batch slot
    int frame;       // absolute frame index (RoPE position, ring slot = frame % R)
    int win_first;   // first frame this one attends to (>= 0, >= frame - W)
    int cond_row;    // slot of the modulation cache that holds this frame's adaLN modulation
    int first_new;   // first frame of this stream whose K/V the current pass writes (earlier pages are final)
    int src;         // which input set of the pass this frame's latent comes from (0 or 1)
    int src_index;   // frame slot inside that input set
    int out_index;   // frame slot of v_out this frame's velocity goes to, or -1 (no output wanted)
};

// One (FM time, action) pair whose modulation this pass has to compute: the pairs
// of a pass that are not in the modulation cache yet.
struct CondDesc {
    float t;
    int action;
    int slot;        // cache slot the result goes to
};

// Everything that changes from pass to pass.  Written to device memory by the
// first kernel of every pass so that a captured graph can be replayed with new
// values (cache position, timestep, action, I/O pointers).
struct StepParams {
    int nf;                 // frames in this pass (tokens = nf * T)
    int nc;                 // conditioning rows to compute in this pass (0: every pair is cached)
    int kind;               // 0 denoise (all layers + velocity head), 1 commit (K/V only)
    int layer_for_attn;     // nfd_attention: which layer's pages hold the data
    // Two input sets: a frame's model input is alpha[s] * x_a[s] + beta[s] * x_b[s] with s = its `src`.
    // Set 0 feeds the frames being denoised (or committed), set 1 the frames whose commit was deferred
    // and rides along with this pass.
    const float *x_a[2];
    const float *x_b[2];    // may be NULL
    float alpha[2], beta[2];
    float *v_out;           // [frames with out_index >= 0, C,H,W]
    FrameDesc fr[NFD_MAX_PASS_FRAMES];
    CondDesc cd[NFD_MAX_PASS_FRAMES];
};

// Static model dimensions, passed by value to kernels.
struct Dims {
    int L, d, H, dh;
    int dm;                 // MLP width as stored: the configured width rounded up to a multiple of 8
    int n1;                 // output columns of the first MLP projection: dm, or 2*dm for the gated form
    int act;                // 0 GELU, 1 gated (SiLU(gate) * up; gate and up columns interleaved)
    int C, Hl, Wl, p, th, tw, T, P;
    int R, W, n_streams;
    int norm;
    float eps, t_scale;
    size_t page_elems;      // H*T*dh
};

#define NFD_MAX_HALF_DH 64
// RoPE table: for pair i of the head dimension, the axis it rotates with
// (0 frame, 1 row, 2 col) and its frequency.
struct RopeTab {
    float freq[NFD_MAX_HALF_DH];
    int axis[NFD_MAX_HALF_DH];
};

// ---- programmatic dependent launch ------------------------------------------
// Every kernel of a pass is launched with programmatic stream serialisation: it
// may start while its predecessor is still running.  pdl_wait() blocks until the
// predecessor grids have completed and their writes are visible; anything that
// does not depend on them (barrier set-up, tensor-memory allocation, weight
// prefetch) goes before it.  pdl_launch() lets the successor start its own
// prologue.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Pull a byte range towards L2 (addr 16-byte aligned, bytes a multiple of 16).
__device__ __forceinline__ void bulk_prefetch_l2(const void *addr, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(addr), "r"(bytes) : "memory");
}

// ---- timeline instrumentation (compiled out unless NFD_TRACE is defined) ------
// With -DNFD_TRACE every CTA of the instrumented kernels appends one record
// (kernel kind, SM, start and end on the global nanosecond timer) to a buffer
// that nfd_trace_read() copies out; the default build contains none of it.
#ifdef NFD_TRACE
#define NFD_TRACE_CAP (1 << 20)
struct NfdTraceRec {
    unsigned long long t0, t1;
    int kind, sm;
};
__device__ NfdTraceRec g_trace[NFD_TRACE_CAP];
__device__ unsigned int g_trace_n;
__device__ __forceinline__ unsigned long long nfd_trace_now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Point events inside a kernel (NFD_TRACE_MARK*) are kept in shared memory and written out together with
// the CTA's record at NFD_TRACE_END, so that taking a mark costs one shared-memory store and does not
// disturb what it measures.  A mark must not be taken before the kernel's first __syncthreads().
#define NFD_TRACE_MARKS 24
__device__ __forceinline__ void nfd_trace_flush(int kind, unsigned long long t0, const unsigned long long *marks) {
    int n = 1;
    for (int i = 0; i < NFD_TRACE_MARKS; ++i) n += marks[i] != 0;
    unsigned int at = atomicAdd(&g_trace_n, (unsigned int)n);
    unsigned int sm;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
    sm |= (blockIdx.x & 0xfffu) << 8 | (blockIdx.y & 0xfffu) << 20;      // SM in bits 0-7, then blockIdx.x, .y
    if (at < NFD_TRACE_CAP) g_trace[at].t0 = t0, g_trace[at].t1 = nfd_trace_now(), g_trace[at].kind = kind, g_trace[at].sm = (int)sm;
    for (int i = 0; i < NFD_TRACE_MARKS; ++i) {
        if (!marks[i]) continue;
        ++at;
        if (at < NFD_TRACE_CAP) g_trace[at].t0 = g_trace[at].t1 = marks[i], g_trace[at].kind = i, g_trace[at].sm = (int)sm;
    }
}
#define NFD_TRACE_T0()                                               \
    const unsigned long long nfd_t0_ = nfd_trace_now();              \
    __shared__ unsigned long long nfd_marks_[NFD_TRACE_MARKS];       \
    if (threadIdx.x < NFD_TRACE_MARKS) nfd_marks_[threadIdx.x] = 0
#define NFD_TRACE_END(kind)                          \
    do {                                             \
        if (threadIdx.x == 0) nfd_trace_flush((kind), nfd_t0_, nfd_marks_); \
    } while (0)
#define NFD_TRACE_MARK(kind)                                  \
    do {                                                      \
        if (threadIdx.x == 0) nfd_marks_[(kind) % NFD_TRACE_MARKS] = nfd_trace_now(); \
    } while (0)
#define NFD_TRACE_MARK_T(kind, tid)                           \
    do {                                                      \
        if (threadIdx.x == (tid)) nfd_marks_[(kind) % NFD_TRACE_MARKS] = nfd_trace_now(); \
    } while (0)
#else
#define NFD_TRACE_T0() do { } while (0)
#define NFD_TRACE_END(kind) do { } while (0)
#define NFD_TRACE_MARK(kind) do { } while (0)
#define NFD_TRACE_MARK_T(kind, tid) do { } while (0)
#endif
enum { TRK_PARAMS = 0, TRK_GEMV, TRK_PATCH, TRK_ADALN, TRK_GEMM, TRK_ATTN, TRK_OTHER };

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<bf16>(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ size_t kv_page_offset(const Dims &D, int stream, int layer, int frame) {
    return ((size_t)(stream * D.L + layer) * D.R + (size_t)(frame % D.R)) * D.page_elems;
}

__device__ __forceinline__ float silu_f(float x) { return x / (1.0f + expf(-x)); }
// for values that are rounded to bf16 afterwards
__device__ __forceinline__ float silu_fast_f(float x) { return __fdividef(x, 1.0f + __expf(-x)); }
__device__ __forceinline__ float gelu_erf_f(float x) { return 0.5f * x * (1.0f + erff(x * 0.70710678118654752440f)); }

// Two fp32 lanes per instruction (sm_100 f32x2 forms): d = a * b + c and d = a + b on register pairs.
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
    unsigned long long ra, rb, rc, rd;
    asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a.x), "f"(a.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b.x), "f"(b.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(rc) : "f"(c.x), "f"(c.y));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(rd) : "l"(ra), "l"(rb), "l"(rc));
    float2 d;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d.x), "=f"(d.y) : "l"(rd));
    return d;
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
    unsigned long long ra, rb, rd;
    asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a.x), "f"(a.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b.x), "f"(b.y));
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(rd) : "l"(ra), "l"(rb));
    float2 d;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d.x), "=f"(d.y) : "l"(rd));
    return d;
}

__device__ __forceinline__ float2 fmul2(float2 a, float2 b) {
    unsigned long long ra, rb, rd;
    asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a.x), "f"(a.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b.x), "f"(b.y));
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(rd) : "l"(ra), "l"(rb));
    float2 d;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d.x), "=f"(d.y) : "l"(rd));
    return d;
}

// GELU (erf form), x/2 (1 + erf(x / sqrt 2)), for values that are rounded to bf16 afterwards, two at a time on
// the two-lane fp32 instructions and without the special-function unit: with z = x / sqrt 2 clamped to
// [-3, 3], erf(z) = z P(z^2) with a degree-8 polynomial fitted to erf on that interval (least squares on
// Chebyshev nodes, reweighted towards equal ripple).  Largest absolute error of the GELU value over all x,
// evaluated in fp32 as here: 5.4e-5; the bf16 rounding step of a value of size one is 3.9e-3.
__device__ __forceinline__ float2 gelu_erf_bf16_f2(float2 x) {
    const float Z = 3.0f;
    const float2 zr = fmul2(x, make_float2(0.70710678118654752440f, 0.70710678118654752440f));
    const float2 z = make_float2(fminf(fmaxf(zr.x, -Z), Z), fminf(fmaxf(zr.y, -Z), Z));
    const float2 t = fmul2(z, z);
    auto k2 = [](float c) { return make_float2(c, c); };
    float2 p = ffma2(k2(4.074211901183844e-08f), t, k2(-1.9448232251306763e-06f));
    p = ffma2(p, t, k2(4.106053529540077e-05f));
    p = ffma2(p, t, k2(-0.000511036952957511f));
    p = ffma2(p, t, k2(0.00423542782664299f));
    p = ffma2(p, t, k2(-0.02510286308825016f));
    p = ffma2(p, t, k2(0.11107934266328812f));
    p = ffma2(p, t, k2(-0.3753148913383484f));
    p = ffma2(p, t, k2(1.1282684803009033f));
    const float2 e = fmul2(z, p);
    const float2 h = fmul2(x, k2(0.5f));
    return ffma2(h, e, h);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Folded LayerNorm (see k_modw and the GEMM epilogues): what a GEMM that follows an adaLN needs in order to
// apply the normalisation in its epilogue.
struct LnFold {
    const float2 *uv;       // (u, v) of this layer's projection: uv[slot * row_stride + n]; nullptr = not folded
    size_t row_stride;
    const float2 *stats;    // [rows][npart] (sum z, sum z^2) per 32 columns
    int npart;              // d / 32
    int norm;               // 0 LayerNorm, 1 RMSNorm
    float eps;
    const StepParams *sp;   // frame -> cache slot
    int T;                  // rows per frame
    static constexpr int kMaxFrames = 16;   // frames that a 128-row tile may span (the caller guarantees it)
    __device__ __forceinline__ bool on() const { return uv != nullptr; }
    // (u, v) of columns n, n+1 for the rows of frame j of the pass
    __device__ __forceinline__ float4 uv_pair(int j, int n) const {
        return *reinterpret_cast<const float4 *>(uv + (size_t)sp->fr[j].cond_row * row_stride + n);
    }
    // Row statistics are gathered by 8 adjacent lanes per row: lane `sub` takes partials sub, sub+8, ...
    // (part), the lanes' sums are combined by a fixed shuffle tree and finished by finish().  The order of
    // the additions depends on npart only, not on how the producer or the consumer tiled the rows.
    __device__ __forceinline__ float2 part(int m, int i) const {
        return (m >= 0 && i < npart) ? stats[(size_t)m * npart + i] : make_float2(0.f, 0.f);
    }
    __device__ __forceinline__ float2 finish(float s, float q) const {
        const float inv_d = 1.0f / (float)(npart * 32);
        const float mean = norm == 0 ? s * inv_d : 0.f;
        const float var = fmaxf(q * inv_d - mean * mean, 0.f);
        return make_float2(mean, rsqrtf(var + eps));
    }
};
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

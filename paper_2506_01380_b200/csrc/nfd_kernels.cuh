// Plain CUDA kernels of libnfd: conditioning, patch embedding, adaLN norm,
// epilogue functors shared by every GEMM, a straightforward tiled GEMM and a
// straightforward attention kernel (both used in fp32 validation mode and as
// the "fast = 0" path in bf16 mode), sampler glue, cache digest / read-out.
#pragma once
#include "nfd_common.cuh"

// ---------------------------------------------------------------------------
// Pass parameters: first kernel of every pass.
// ---------------------------------------------------------------------------
// Every index that the kernels of a pass derive from the descriptor (cache page,
// modulation row, input and output frame slots) is checked here, once, against
// the limits of the context before the descriptor reaches device memory.  A
// frame that fails is recorded (NFD_E_DEVICE in the status latch) and replaced
// by a harmless one -- batch slot 0, frame j of the pass, seeing only itself, no
// output -- so that nothing downstream leaves its buffers; the caller learns of
// it from nfd_status and must treat the cache as lost.
struct DescLimits {
    int n_streams, W, n_slots, n_actions, max_frames, pend_slots;
};
// It does not release its dependents early: a kernel that starts after this one
// may read the descriptor before its own wait on the predecessor grid.
__global__ void k_set_params(StepParams p, StepParams *dst, DescLimits lim, int *status) {
    NFD_TRACE_T0();
    __shared__ int s_bad;
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    const int t = threadIdx.x;
    bool bad = false;
    if (t == 0) bad = p.nf < 0 || p.nf > lim.max_frames || p.nc < 0 || p.nc > lim.max_frames;
    if (t < NFD_MAX_PASS_FRAMES && t < p.nf) {
        const FrameDesc &f = p.fr[t];
        bad = bad || f.stream < 0 || f.stream >= lim.n_streams || f.frame < 0 || f.win_first < 0 ||
              f.win_first > f.frame || f.frame - f.win_first > lim.W || f.first_new < 0 || f.first_new > f.frame ||
              f.cond_row < 0 || f.cond_row >= lim.n_slots || f.src < 0 || f.src > 1 || f.src_index < 0 ||
              f.src_index >= (f.src ? lim.pend_slots : lim.max_frames) || f.out_index < -1 ||
              f.out_index >= lim.max_frames;
    }
    if (t >= 64 && t - 64 < NFD_MAX_PASS_FRAMES && t - 64 < p.nc) {
        const CondDesc &cd = p.cd[t - 64];
        bad = bad || cd.slot < 0 || cd.slot >= lim.n_slots || cd.action < 0 || cd.action >= lim.n_actions;
    }
    if (bad) s_bad = 1;
    __syncthreads();
    const bool any_bad = s_bad != 0;
    pdl_wait();
    const int n_words = sizeof(StepParams) / 4;
    const int *src = reinterpret_cast<const int *>(&p);
    int *d = reinterpret_cast<int *>(dst);
    for (int i = threadIdx.x; i < n_words; i += blockDim.x) d[i] = src[i];
    if (any_bad) {
        __syncthreads();
        if (t == 0) {
            atomicCAS(status, 0, NFD_E_DEVICE);
            int nf = p.nf;
            nf = nf < 0 ? 0 : (nf > lim.max_frames ? lim.max_frames : nf);
            dst->nf = nf;
            dst->nc = 0;
        }
        if (t < NFD_MAX_PASS_FRAMES) {
            FrameDesc f;
            f.stream = 0, f.frame = t, f.win_first = t, f.cond_row = 0, f.first_new = 0;
            f.src = 0, f.src_index = 0, f.out_index = -1;
            dst->fr[t] = f;
        }
    }
    NFD_TRACE_END(TRK_PARAMS);
}

// ---------------------------------------------------------------------------
// Conditioning (adaLN-zero on timestep + action, Section 3.1 "Action
// Conditioning"): sinusoidal embedding of t_scale * t, MLP with SiLU, plus the
// action embedding row; then per-layer modulation W_mod * SiLU(c) + b.
// ---------------------------------------------------------------------------
__global__ void k_temb(const StepParams *sp, float t_scale, float *emb /*[rows][256]*/) {
    pdl_wait();
    pdl_launch();
    int c = blockIdx.x;
    if (c >= sp->nc) return;
    int i = threadIdx.x;              // 0..127
    if (i >= 128) return;
    // double precision: the argument reaches ~1e3 rad
    double f = exp(-9.210340371976184 /* ln 1e4 */ * (double)i / 128.0);
    double a = (double)t_scale * (double)sp->cd[c].t * f;
    double s, co;
    sincos(a, &s, &co);
    emb[c * 256 + i] = (float)co;
    emb[c * 256 + 128 + i] = (float)s;
}

enum { GEMV_T1 = 0, GEMV_T2 = 1, GEMV_MOD = 2 };

// y[c][o] = f( sum_i Wt[o][i] * x[c][i] + b[o] ), one warp per output o, all
// conditioning rows c (four at a time, so a weight row is read once for up to
// four rows).  Weights are read 16 bytes per lane.  blockIdx.y selects the
// layer for GEMV_MOD.  n_in must be a multiple of 8.
template <typename TS> struct WVec;
template <> struct WVec<bf16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void load(const bf16 *p, float *f) {
        const uint4 u = *reinterpret_cast<const uint4 *>(p);
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 t = __bfloat1622float2(h[i]);
            f[2 * i] = t.x, f[2 * i + 1] = t.y;
        }
    }
};
template <> struct WVec<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void load(const float *p, float *f) {
        const float4 u = *reinterpret_cast<const float4 *>(p);
        f[0] = u.x, f[1] = u.y, f[2] = u.z, f[3] = u.w;
    }
};

template <typename TS, int MODE>
__global__ void __launch_bounds__(256) k_gemv(const StepParams *sp, const TS *const *Wt_l, const TS *const *b_l,
                                              const TS *a_emb, const float *x, float *y, int n_in, int n_out,
                                              size_t y_row_stride, size_t y_layer_stride) {
    NFD_TRACE_T0();
    pdl_wait();
    pdl_launch();
    constexpr int NV = WVec<TS>::N;
    const int layer = blockIdx.y;
    const TS *Wt = Wt_l[layer];
    const TS *b = b_l[layer];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int o = blockIdx.x * (blockDim.x >> 5) + warp;
    if (o >= n_out) return;
    const int nc = sp->nc;
    const TS *wrow = Wt + (size_t)o * n_in;
    for (int c0 = 0; c0 < nc; c0 += 4) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int i = lane * NV; i < n_in; i += 32 * NV) {
            float w[NV];
            WVec<TS>::load(wrow + i, w);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (c0 + u < nc) {
                    const float *xc = x + (size_t)(c0 + u) * n_in + i;
#pragma unroll
                    for (int e = 0; e < NV; e += 4) {
                        const float4 xv = *reinterpret_cast<const float4 *>(xc + e);
                        acc[u] = fmaf(w[e], xv.x, acc[u]);
                        acc[u] = fmaf(w[e + 1], xv.y, acc[u]);
                        acc[u] = fmaf(w[e + 2], xv.z, acc[u]);
                        acc[u] = fmaf(w[e + 3], xv.w, acc[u]);
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int c = c0 + u;
            if (c >= nc) break;
            const float r = warp_sum(acc[u]);
            if (lane == 0) {
                float v = r + to_f(b[o]);
                if (MODE == GEMV_T1) v = silu_f(v);
                if (MODE == GEMV_T2) v = silu_f(v + to_f(a_emb[(size_t)sp->cd[c].action * n_out + o]));
                const int out_row = MODE == GEMV_MOD ? sp->cd[c].slot : c;     // modulation goes to its cache slot
                y[(size_t)out_row * y_row_stride + (size_t)layer * y_layer_stride + o] = v;
            }
        }
    }
    NFD_TRACE_END(TRK_GEMV);
}

// ---------------------------------------------------------------------------
// Folded LayerNorm, weight side.  A projection that follows an adaLN,
//     y[n] = sum_k ((z[k] - mean) * rstd * (1 + scale[k]) + shift[k]) * W[n][k] + b[n],
// equals
//     y[n] = rstd * (sum_k z[k] (1 + scale[k]) W[n][k]  -  mean * u[n]) + v[n],
//     u[n] = sum_k (1 + scale[k]) W[n][k],      v[n] = sum_k shift[k] W[n][k] + b[n],
// so the GEMM can run on z*(1+scale), written by the kernel that produces z,
// and apply mean and rstd per row in its epilogue.  u and v depend on the
// conditioning row only and are kept in the modulation cache next to shift and
// scale.  This kernel fills (u, v) for the QKV projection (outputs 0..3d) and
// the first MLP projection (outputs 3d..3d+dm) of layer blockIdx.y: 64 outputs
// per CTA (one warp per output, eight in turn), four conditioning rows at a time.
// ---------------------------------------------------------------------------
#define MODW_OUT 64          // outputs per CTA of k_modw (8 per warp)
template <typename TS>
__global__ void __launch_bounds__(256) k_modw(const StepParams *sp, const TS *const *Wqkv_l, const TS *const *bqkv_l,
                                              const TS *const *Wfc1_l, const TS *const *bfc1_l, const float *mod,
                                              size_t mod_row_stride, float2 *uv, size_t uv_row_stride, int d, int dm) {
    // (1 + scale) and shift of up to four conditioning rows, 1024 columns at a time: every warp of the CTA
    // works on the same layer and projection, so they are fetched once per CTA
    __shared__ __align__(16) float s_sc[4][1024];
    __shared__ __align__(16) float s_sh[4][1024];
    NFD_TRACE_T0();
    pdl_wait();
    pdl_launch();
    constexpr int NV = WVec<TS>::N;
    const int layer = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int o_cta = blockIdx.x * MODW_OUT;                   // 3d is a multiple of the outputs of a CTA
    const bool mlp = o_cta >= 3 * d;
    const TS *W = mlp ? Wfc1_l[layer] : Wqkv_l[layer];
    const TS *B = mlp ? bfc1_l[layer] : bqkv_l[layer];
    const size_t off_shift = (size_t)layer * 6 * d + (mlp ? 3 * d : 0);
    const size_t off_scale = off_shift + d;
    const int nc = sp->nc;
    for (int c0 = 0; c0 < nc; c0 += 4) {
        for (int i0 = 0; i0 < d; i0 += 1024) {
            const int span = d - i0 < 1024 ? d - i0 : 1024;
            __syncthreads();
            for (int idx = threadIdx.x * 4; idx < 4 * span; idx += blockDim.x * 4) {
                const int r = idx / span, i = idx - r * span;
                if (c0 + r < nc) {
                    const float *mrow = mod + (size_t)sp->cd[c0 + r].slot * mod_row_stride;
                    const float4 sc = *reinterpret_cast<const float4 *>(mrow + off_scale + i0 + i);
                    *reinterpret_cast<float4 *>(&s_sc[r][i]) = make_float4(1.0f + sc.x, 1.0f + sc.y, 1.0f + sc.z, 1.0f + sc.w);
                    *reinterpret_cast<float4 *>(&s_sh[r][i]) = *reinterpret_cast<const float4 *>(mrow + off_shift + i0 + i);
                }
            }
            __syncthreads();
            // every warp takes MODW_OUT / 8 outputs; a row wider than 1024 is summed in parts (kept in uv itself)
            for (int oi = 0; oi < MODW_OUT / 8; ++oi) {
                const int o = o_cta + warp * (MODW_OUT / 8) + oi;
                if (o >= 3 * d + dm) break;
                const int oo = mlp ? o - 3 * d : o;
                const TS *wrow = W + (size_t)oo * d + i0;
                float au[4] = {0.f, 0.f, 0.f, 0.f}, av[4] = {0.f, 0.f, 0.f, 0.f};
                for (int i = lane * NV; i < span; i += 32 * NV) {
                    float w[NV];
                    WVec<TS>::load(wrow + i, w);
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        if (c0 + r < nc) {
#pragma unroll
                            for (int e = 0; e < NV; e += 4) {
                                const float4 sc = *reinterpret_cast<const float4 *>(&s_sc[r][i + e]);
                                const float4 sh = *reinterpret_cast<const float4 *>(&s_sh[r][i + e]);
                                au[r] = fmaf(w[e], sc.x, au[r]), av[r] = fmaf(w[e], sh.x, av[r]);
                                au[r] = fmaf(w[e + 1], sc.y, au[r]), av[r] = fmaf(w[e + 1], sh.y, av[r]);
                                au[r] = fmaf(w[e + 2], sc.z, au[r]), av[r] = fmaf(w[e + 2], sh.z, av[r]);
                                au[r] = fmaf(w[e + 3], sc.w, au[r]), av[r] = fmaf(w[e + 3], sh.w, av[r]);
                            }
                        }
                    }
                }
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    if (c0 + r >= nc) break;
                    float su = warp_sum(au[r]), sv = warp_sum(av[r]);
                    float2 *dst = uv + (size_t)sp->cd[c0 + r].slot * uv_row_stride + (size_t)layer * (3 * d + dm) + o;
                    if (lane == 0) {
                        if (i0 > 0) su += dst->x, sv += dst->y;          // this thread wrote the earlier part itself
                        if (i0 + span >= d) sv += to_f(B[oo]);
                        *dst = make_float2(su, sv);
                    }
                }
            }
        }
    }
    NFD_TRACE_END(TRK_GEMV);
}

// ---------------------------------------------------------------------------
// Patchify + embed: z[tok][o] = sum_p (alpha*x_a + beta*x_b)[patch p of tok] * W_pe[p][o] + b[o].
// A CTA takes PE_TOK tokens (blockIdx.x) and 256 output columns (blockIdx.y).
// Each thread owns one output column: it loads 64 rows of its W_pe column at a
// time into registers (independent loads, all in flight together) and reuses
// them for all tokens of the CTA.  W_pe is used in its [P][d] layout so that
// adjacent threads read adjacent columns.
// With a_out set (folded LayerNorm, see the GEMM epilogues below; d a multiple of
// 32) it also writes the first layer's GEMM operand z*(1+scale) and the row-sum
// partials of z per 32 columns.
// ---------------------------------------------------------------------------
#define PE_TOK 8
template <typename TS>
__global__ void __launch_bounds__(256) k_patch_embed(const StepParams *sp, Dims D, const TS *W_pe, const TS *b_pe,
                                                     float *z, TS *a_out, float2 *stats, const float *scale0,
                                                     size_t mod_row_stride, const RopeTab *rt, float2 *rope_tab) {
    extern __shared__ float s_patch[];          // [PE_TOK][P]
    NFD_TRACE_T0();
    pdl_wait();
    pdl_launch();
    const int M = sp->nf * D.T;
    const int m0 = blockIdx.x * PE_TOK;
    if (m0 >= M) return;
    if (rope_tab && blockIdx.y == 0) {
        // the per-pass rotary table (cos, sin) of this CTA's tokens: [token][pair of the head dimension]
        const int half = D.dh >> 1;
        for (int idx = threadIdx.x; idx < PE_TOK * half; idx += blockDim.x) {
            const int m = m0 + idx / half, pi = idx % half;
            if (m < M) {
                const int tok = m % D.T;
                const int ax = rt->axis[pi];
                const float pos = (float)(ax == 0 ? sp->fr[m / D.T].frame : (ax == 1 ? tok / D.tw : tok % D.tw));
                float sn, cs;
                sincosf(pos * rt->freq[pi], &sn, &cs);
                rope_tab[(size_t)m * half + pi] = make_float2(cs, sn);
            }
        }
    }
    for (int i = threadIdx.x; i < PE_TOK * D.P; i += blockDim.x) {
        const int t = i / D.P, p = i - t * D.P, m = m0 + t;
        float v = 0.f;
        if (m < M) {
            const int j = m / D.T, tok = m % D.T;
            const int r = tok / D.tw, c = tok % D.tw;
            const int ch = p / (D.p * D.p), py = (p / D.p) % D.p, px = p % D.p;
            const int set = sp->fr[j].src, fj = sp->fr[j].src_index;
            const float *xa = sp->x_a[set], *xb = sp->x_b[set];
            const size_t idx = (((size_t)fj * D.C + ch) * D.Hl + (r * D.p + py)) * D.Wl + (c * D.p + px);
            v = sp->alpha[set] * xa[idx];
            if (xb) v = fmaf(sp->beta[set], xb[idx], v);
        }
        s_patch[i] = v;
    }
    __syncthreads();
    const int o = blockIdx.y * blockDim.x + threadIdx.x;
    if (o >= D.d) return;
    float acc[PE_TOK];
#pragma unroll
    for (int t = 0; t < PE_TOK; ++t) acc[t] = 0.f;
    if (D.P % 64 == 0) {
        for (int p0 = 0; p0 < D.P; p0 += 64) {
            TS wr[64];
#pragma unroll
            for (int u = 0; u < 64; ++u) wr[u] = W_pe[(size_t)(p0 + u) * D.d + o];      // 64 independent loads
#pragma unroll
            for (int t = 0; t < PE_TOK; ++t) {
                const float4 *sp_t = reinterpret_cast<const float4 *>(s_patch + t * D.P + p0);
#pragma unroll
                for (int u = 0; u < 16; ++u) {
                    const float4 x = sp_t[u];
                    acc[t] = fmaf(x.x, to_f(wr[4 * u]), acc[t]);
                    acc[t] = fmaf(x.y, to_f(wr[4 * u + 1]), acc[t]);
                    acc[t] = fmaf(x.z, to_f(wr[4 * u + 2]), acc[t]);
                    acc[t] = fmaf(x.w, to_f(wr[4 * u + 3]), acc[t]);
                }
            }
        }
    } else {
        for (int p = 0; p < D.P; ++p) {
            const float w = to_f(W_pe[(size_t)p * D.d + o]);
#pragma unroll
            for (int t = 0; t < PE_TOK; ++t) acc[t] = fmaf(s_patch[t * D.P + p], w, acc[t]);
        }
    }
    const float bo = to_f(b_pe[o]);
#pragma unroll
    for (int t = 0; t < PE_TOK; ++t) {
        if (m0 + t >= M) break;
        const int m = m0 + t;
        const float zv = acc[t] + bo;
        z[(size_t)m * D.d + o] = zv;
        if (a_out) {
            const float sc = scale0[(size_t)sp->fr[m / D.T].cond_row * mod_row_stride + o];
            a_out[(size_t)m * D.d + o] = from_f<TS>(zv * (1.0f + sc));
            const float s1 = warp_sum(zv), s2 = warp_sum(zv * zv);
            if ((threadIdx.x & 31) == 0) stats[(size_t)m * (D.d >> 5) + (o >> 5)] = make_float2(s1, s2);
        }
    }
    NFD_TRACE_END(TRK_PATCH);
}

// ---------------------------------------------------------------------------
// adaLN: out = norm(z) * (1 + scale_f) + shift_f, one warp per token.  Rows of
// up to 1024 elements are held in registers (one read of z); longer rows are
// re-read from L1/L2.
// ---------------------------------------------------------------------------
template <typename TS> __device__ __forceinline__ void store4(TS *o, float a, float b, float c, float d);
template <> __device__ __forceinline__ void store4<float>(float *o, float a, float b, float c, float d) {
    *reinterpret_cast<float4 *>(o) = make_float4(a, b, c, d);
}
template <> __device__ __forceinline__ void store4<bf16>(bf16 *o, float a, float b, float c, float d) {
    uint2 u;
    __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&u);
    h[0] = __floats2bfloat162_rn(a, b);
    h[1] = __floats2bfloat162_rn(c, d);
    *reinterpret_cast<uint2 *>(o) = u;
}

template <typename TS>
__global__ void __launch_bounds__(128) k_adaln(const StepParams *sp, Dims D, const float *z, TS *out,
                                               const float *mod, size_t row_stride, size_t off_shift,
                                               size_t off_scale) {
    NFD_TRACE_T0();
    pdl_wait();
    NFD_TRACE_MARK(TRK_OTHER);
    pdl_launch();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m = blockIdx.x * (blockDim.x >> 5) + warp;
    if (m >= sp->nf * D.T) return;
    const int row = sp->fr[m / D.T].cond_row;
    const float *zr = z + (size_t)m * D.d;
    const float *sh = mod + (size_t)row * row_stride + off_shift;
    const float *sc = mod + (size_t)row * row_stride + off_scale;
    const float inv_d = 1.0f / (float)D.d;
    if (D.d <= 1024) {
        // every load of the row is issued before anything is consumed or stored: z, then shift and scale
        float4 v[8], a[8], b[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = u * 128 + lane * 4;
            v[u] = i < D.d ? *reinterpret_cast<const float4 *>(zr + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = u * 128 + lane * 4;
            if (i < D.d) {
                a[u] = *reinterpret_cast<const float4 *>(sh + i);
                b[u] = *reinterpret_cast<const float4 *>(sc + i);
            }
        }
        float s = 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u) s += (v[u].x + v[u].y) + (v[u].z + v[u].w);
        const float mean = (D.norm == 0) ? warp_sum(s) * inv_d : 0.f;
        float q = 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (u * 128 + lane * 4 < D.d) {
                const float c0 = v[u].x - mean, c1 = v[u].y - mean, c2 = v[u].z - mean, c3 = v[u].w - mean;
                q += (c0 * c0 + c1 * c1) + (c2 * c2 + c3 * c3);
            }
        }
        const float rstd = rsqrtf(warp_sum(q) * inv_d + D.eps);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = u * 128 + lane * 4;
            if (i < D.d)
                store4<TS>(out + (size_t)m * D.d + i, fmaf((v[u].x - mean) * rstd, 1.0f + b[u].x, a[u].x),
                           fmaf((v[u].y - mean) * rstd, 1.0f + b[u].y, a[u].y),
                           fmaf((v[u].z - mean) * rstd, 1.0f + b[u].z, a[u].z),
                           fmaf((v[u].w - mean) * rstd, 1.0f + b[u].w, a[u].w));
        }
        NFD_TRACE_END(TRK_ADALN);
        return;
    }
    float s = 0.f;
    for (int i = lane * 4; i < D.d; i += 128) {
        float4 v = *reinterpret_cast<const float4 *>(zr + i);
        s += (v.x + v.y) + (v.z + v.w);
    }
    float mean = (D.norm == 0) ? warp_sum(s) * inv_d : 0.f;
    float q = 0.f;
    for (int i = lane * 4; i < D.d; i += 128) {
        float4 v = *reinterpret_cast<const float4 *>(zr + i);
        float a = v.x - mean, b = v.y - mean, c = v.z - mean, e = v.w - mean;
        q += (a * a + b * b) + (c * c + e * e);
    }
    const float rstd = rsqrtf(warp_sum(q) * inv_d + D.eps);
    for (int i = lane * 4; i < D.d; i += 128) {
        float4 v = *reinterpret_cast<const float4 *>(zr + i);
        float4 a = *reinterpret_cast<const float4 *>(sh + i);
        float4 b = *reinterpret_cast<const float4 *>(sc + i);
        store4<TS>(out + (size_t)m * D.d + i, fmaf((v.x - mean) * rstd, 1.0f + b.x, a.x),
                   fmaf((v.y - mean) * rstd, 1.0f + b.y, a.y), fmaf((v.z - mean) * rstd, 1.0f + b.z, a.z),
                   fmaf((v.w - mean) * rstd, 1.0f + b.w, a.w));
    }
}

__device__ __forceinline__ void unpack_bf16x8(const uint4 &u, float *f) {
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 t = __bfloat1622float2(h[i]);
        f[2 * i] = t.x;
        f[2 * i + 1] = t.y;
    }
}
__device__ __forceinline__ uint4 pack_bf16x8(const float *f) {
    uint4 u;
    __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    return u;
}

// ---------------------------------------------------------------------------
// GEMM epilogues.  operator() takes one output row m and two adjacent columns
// (n, n+1), n even, holding the fp32 accumulators (plain GEMM).  The tensor-core
// GEMM (bf16 storage only) works on eight adjacent columns n..n+7, n a multiple
// of 8, 16 bytes at a time, in two steps: load() fetches everything the item
// needs besides the accumulators (bias, gate, residual, rotary table) into a
// Side record, so that the fetch can be issued while the UMMAs still run;
// apply() combines it with the accumulators and stores.  apply() also gets the
// (mean, rstd) of the item's row and the (u, v) pairs of its 8 columns (in shared
// memory) when the functor asks for row statistics (kRowStats) and the
// LayerNorm is folded, and the mask of the warp's lanes that hold a valid item; four
// adjacent lanes always hold the four 8-column items of one 32-column group.
//
// Folded LayerNorm (tensor-core path only, see k_modw): the functors that update
// the residual stream z also write the next GEMM's operand z*(1+scale) and the
// (sum z, sum z^2) partials of every 32 columns of the row; the functors of the
// GEMMs that follow an adaLN turn those partials into (mean, rstd) and apply
// rstd*(acc - mean*u[n]) + v[n].
// ---------------------------------------------------------------------------
// uv: (u, v, u, v) of columns 2i, 2i+1 of the item at uv[i * stride]
__device__ __forceinline__ void ln_fold_apply(float *a, const float4 *uv, int stride, float2 ms) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float4 w = uv[i * stride];
        a[2 * i] = fmaf(ms.y, fmaf(-ms.x, w.x, a[2 * i]), w.y);
        a[2 * i + 1] = fmaf(ms.y, fmaf(-ms.x, w.z, a[2 * i + 1]), w.w);
    }
}
__device__ __forceinline__ void bias_add(float *a, const uint4 &bits) {
    float b[8];
    unpack_bf16x8(bits, b);
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] += b[i];
}
// QKV: + bias, 3D RoPE on q and k (Section 3.1 "3D Positional Embedding":
// adjacent pairs, per-axis frequencies), q -> [H][Nq][dh], k/v -> cache pages.
template <typename TS> struct EpiQKV {
    const StepParams *sp;
    const TS *bias;
    TS *q, *kc, *vc;
    const RopeTab *rt;
    Dims D;
    int layer;
    const float2 *rope_cs;      // [nf*T][dh/2] (cos, sin), used by the tensor-core path
    int n_rows;                 // nf*T: rows of the pass (q is [H][n_rows][dh])
    LnFold ln;                  // folded adaLN in front of this projection (tensor-core path only)
    int kv_prefetch = 1;        // 0: leave the cached pages alone (option "l2_prefetch")
    // Pull the cached K/V pages that the attention kernel of this layer is about to read towards L2 (the
    // pages of frames before this pass are final); each CTA of the launch takes a slice of every page.
    __device__ __forceinline__ void prefetch(unsigned int cta, unsigned int n_cta) const {
        if (sizeof(TS) != 2 || !kv_prefetch) return;
        const FrameDesc fr = sp->fr[0];
        const size_t page_bytes = D.page_elems * sizeof(TS);
        const size_t per = ((page_bytes / n_cta + 15) / 16) * 16;
        const size_t b = (size_t)cta * per;
        if (b >= page_bytes) return;
        const unsigned int n = (unsigned int)(page_bytes - b < per ? page_bytes - b : per);
        for (int g = fr.win_first; g < fr.first_new; ++g) {
            const size_t off = kv_page_offset(D, fr.stream, layer, g);
            bulk_prefetch_l2(reinterpret_cast<const unsigned char *>(kc + off) + b, n);
            bulk_prefetch_l2(reinterpret_cast<const unsigned char *>(vc + off) + b, n);
        }
    }
    static constexpr int kBatch = 4;        // epilogue items a thread keeps in flight together
    static constexpr bool kRowStats = true;
    // Where a row (token) and an 8-column chunk of the output go, worked out once per tile row and tile
    // column chunk and kept in shared memory, so that an item needs no division.
    static constexpr bool kTables = true;
    struct Row {
        long long q_off;        // m * dh
        long long kv_off;       // page of the token's frame + tok * dh
    };
    struct Col {
        int which, pad;         // 0 q, 1 k, 2 v
        long long q_off;        // head * n_rows * dh + e
        long long kv_off;       // head * T * dh + e
    };
    __device__ __forceinline__ Row row_info(int m) const {
        const int j = m / D.T, tok = m - j * D.T;
        const FrameDesc &f = sp->fr[j];
        Row r;
        r.q_off = (long long)m * D.dh;
        r.kv_off = (long long)kv_page_offset(D, f.stream, layer, f.frame) + (long long)tok * D.dh;
        return r;
    }
    __device__ __forceinline__ Col col_info(int n) const {
        Col c;
        c.which = n / D.d;
        const int col = n - c.which * D.d;
        const int head = col / D.dh, e = col - head * D.dh;
        c.pad = 0;
        c.q_off = ((long long)head * n_rows) * D.dh + e;
        c.kv_off = ((long long)head * D.T) * D.dh + e;
        return c;
    }
    struct Side {
        uint4 bias;             // unused with the folded LayerNorm (v carries the bias)
        float4 c01, c23;        // (cos, sin) of four adjacent pairs
    };
    __device__ __forceinline__ void load(int m, int n, Side &s) const {
        if (!ln.on()) s.bias = *reinterpret_cast<const uint4 *>(bias + n);
        const int which = n / D.d, col = n - which * D.d;
        const int e = col % D.dh;
        if (which < 2) {
            const float4 *cs = reinterpret_cast<const float4 *>(rope_cs + (size_t)m * (D.dh >> 1) + (e >> 1));
            s.c01 = cs[0], s.c23 = cs[1];
        }
    }
    __device__ __forceinline__ void apply(int, int, float *a, const Side &s, float2 ms, const float4 *uv, int uv_stride,
                                          unsigned, const Row &row, const Col &col) const {
        const int which = col.which;
        if (ln.on())
            ln_fold_apply(a, uv, uv_stride, ms);
        else
            bias_add(a, s.bias);
        TS *dst;
        if (which < 2) {
            const float cv[4] = {s.c01.x, s.c01.z, s.c23.x, s.c23.z}, sv[4] = {s.c01.y, s.c01.w, s.c23.y, s.c23.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float r0 = a[2 * i] * cv[i] - a[2 * i + 1] * sv[i];
                const float r1 = a[2 * i] * sv[i] + a[2 * i + 1] * cv[i];
                a[2 * i] = r0;
                a[2 * i + 1] = r1;
            }
        }
        if (which == 0)
            dst = q + (row.q_off + col.q_off);
        else
            dst = ((which == 1) ? kc : vc) + (row.kv_off + col.kv_off);
        *reinterpret_cast<uint4 *>(dst) = pack_bf16x8(a);
    }
    __device__ __forceinline__ void operator()(int m, int n, float a0, float a1) const {
        a0 += to_f(bias[n]);
        a1 += to_f(bias[n + 1]);
        const int which = n / D.d, col = n % D.d;
        const int head = col / D.dh, e = col % D.dh;
        const int j = m / D.T, tok = m % D.T;
        const FrameDesc fr = sp->fr[j];
        if (which < 2) {
            const int pi = e >> 1;
            const int ax = rt->axis[pi];
            const float pos = (float)(ax == 0 ? fr.frame : (ax == 1 ? tok / D.tw : tok % D.tw));
            float sn, cs;
            sincosf(pos * rt->freq[pi], &sn, &cs);
            const float r0 = a0 * cs - a1 * sn, r1 = a0 * sn + a1 * cs;
            a0 = r0;
            a1 = r1;
        }
        TS *dst;
        if (which == 0) {
            dst = q + ((size_t)head * n_rows + m) * D.dh + e;
        } else {
            TS *base = (which == 1) ? kc : vc;
            dst = base + kv_page_offset(D, fr.stream, layer, fr.frame) + ((size_t)head * D.T + tok) * D.dh + e;
        }
        dst[0] = from_f<TS>(a0);
        dst[1] = from_f<TS>(a1);
    }
};

// z += gate_f * (acc + bias): residual update of the fp32 stream.  With stats set
// (folded LayerNorm) it also writes the row-sum partials of the new z and, with
// a_out set, the next GEMM's operand z*(1+scale_next).
template <typename TS> struct EpiGateRes {
    const StepParams *sp;
    const TS *bias;
    float *z;
    const float *gate;      // mod + layer offset + chunk offset
    size_t row_stride;
    Dims D;
    TS *a_out;              // [rows][d] or nullptr
    const float *scale_next;// mod + layer offset + chunk offset of the adaLN scale that follows (with a_out)
    float2 *stats;          // [rows][d/32] or nullptr
    __device__ __forceinline__ void prefetch(unsigned int, unsigned int) const {}
    static constexpr int kBatch = 2;        // epilogue items a thread keeps in flight together
    static constexpr bool kRowStats = false;
    static constexpr bool kTables = false;
    struct Row {};
    struct Col {};
    struct Side {
        uint4 bias;
        float4 g0, g1, z0, z1, s0, s1;
    };
    __device__ __forceinline__ void load(int m, int n, Side &s) const {
        s.bias = *reinterpret_cast<const uint4 *>(bias + n);
        const int row = sp->fr[m / D.T].cond_row;
        const float4 *g = reinterpret_cast<const float4 *>(gate + (size_t)row * row_stride + n);
        const float4 *zp = reinterpret_cast<const float4 *>(z + (size_t)m * D.d + n);
        s.g0 = g[0], s.g1 = g[1];
        s.z0 = zp[0], s.z1 = zp[1];
        if (a_out) {
            const float4 *sc = reinterpret_cast<const float4 *>(scale_next + (size_t)row * row_stride + n);
            s.s0 = sc[0], s.s1 = sc[1];
        }
    }
    __device__ __forceinline__ void apply(int m, int n, float *a, const Side &s, float2, const float4 *, int,
                                          unsigned mask, const Row &, const Col &) const {
        float b[8];
        unpack_bf16x8(s.bias, b);
        float4 z0 = s.z0, z1 = s.z1;
        z0.x = fmaf(s.g0.x, a[0] + b[0], z0.x);
        z0.y = fmaf(s.g0.y, a[1] + b[1], z0.y);
        z0.z = fmaf(s.g0.z, a[2] + b[2], z0.z);
        z0.w = fmaf(s.g0.w, a[3] + b[3], z0.w);
        z1.x = fmaf(s.g1.x, a[4] + b[4], z1.x);
        z1.y = fmaf(s.g1.y, a[5] + b[5], z1.y);
        z1.z = fmaf(s.g1.z, a[6] + b[6], z1.z);
        z1.w = fmaf(s.g1.w, a[7] + b[7], z1.w);
        float4 *zp = reinterpret_cast<float4 *>(z + (size_t)m * D.d + n);
        zp[0] = z0;
        zp[1] = z1;
        if (stats) {
            if (a_out) {
                float o[8] = {z0.x * (1.0f + s.s0.x), z0.y * (1.0f + s.s0.y), z0.z * (1.0f + s.s0.z),
                              z0.w * (1.0f + s.s0.w), z1.x * (1.0f + s.s1.x), z1.y * (1.0f + s.s1.y),
                              z1.z * (1.0f + s.s1.z), z1.w * (1.0f + s.s1.w)};
                *reinterpret_cast<uint4 *>(a_out + (size_t)m * D.d + n) = pack_bf16x8(o);
            }
            // the four lanes of a 32-column group hold the same row and are valid together
            float s1 = ((z0.x + z0.y) + (z0.z + z0.w)) + ((z1.x + z1.y) + (z1.z + z1.w));
            float s2 = ((z0.x * z0.x + z0.y * z0.y) + (z0.z * z0.z + z0.w * z0.w)) +
                       ((z1.x * z1.x + z1.y * z1.y) + (z1.z * z1.z + z1.w * z1.w));
            s1 += __shfl_xor_sync(mask, s1, 1), s2 += __shfl_xor_sync(mask, s2, 1);
            s1 += __shfl_xor_sync(mask, s1, 2), s2 += __shfl_xor_sync(mask, s2, 2);
            if ((n & 31) == 0) stats[(size_t)m * (D.d >> 5) + (n >> 5)] = make_float2(s1, s2);
        }
    }
    __device__ __forceinline__ void operator()(int m, int n, float a0, float a1) const {
        const int row = sp->fr[m / D.T].cond_row;
        const float *g = gate + (size_t)row * row_stride + n;
        float *zp = z + (size_t)m * D.d + n;
        zp[0] = fmaf(g[0], a0 + to_f(bias[n]), zp[0]);
        zp[1] = fmaf(g[1], a1 + to_f(bias[n + 1]), zp[1]);
    }
};

// out = GELU(acc + bias), exact erf form.
template <typename TS> struct EpiGelu {
    const TS *bias;
    TS *out;
    int N;                  // columns of the GEMM (n1)
    int act;                // 0: out[m][n] = GELU(.); 1: out[m][n/2] = SiLU(gate) * up, (gate, up) = columns (n, n+1)
    LnFold ln;              // folded adaLN in front of this projection (tensor-core path only)
    __device__ __forceinline__ void prefetch(unsigned int, unsigned int) const {}
    static constexpr int kBatch = 8;        // epilogue items a thread keeps in flight together
    static constexpr bool kRowStats = true;
    static constexpr bool kTables = false;
    struct Row {};
    struct Col {};
    struct Side {
        uint4 bias;         // unused with the folded LayerNorm (v carries the bias)
    };
    __device__ __forceinline__ void load(int m, int n, Side &s) const {
        (void)m;
        if (!ln.on()) s.bias = *reinterpret_cast<const uint4 *>(bias + n);
    }
    __device__ __forceinline__ void apply(int m, int n, float *a, const Side &s, float2 ms, const float4 *uv,
                                          int uv_stride, unsigned, const Row &, const Col &) const {
        if (ln.on())
            ln_fold_apply(a, uv, uv_stride, ms);
        else
            bias_add(a, s.bias);
        if (act == 0) {
#pragma unroll
            for (int i = 0; i < 8; i += 2) {
                const float2 g = gelu_erf_bf16_f2(make_float2(a[i], a[i + 1]));
                a[i] = g.x, a[i + 1] = g.y;
            }
            *reinterpret_cast<uint4 *>(out + (size_t)m * N + n) = pack_bf16x8(a);
        } else {
            uint2 o;
            __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&o);
            h[0] = __floats2bfloat162_rn(silu_fast_f(a[0]) * a[1], silu_fast_f(a[2]) * a[3]);
            h[1] = __floats2bfloat162_rn(silu_fast_f(a[4]) * a[5], silu_fast_f(a[6]) * a[7]);
            *reinterpret_cast<uint2 *>(out + (size_t)m * (N >> 1) + (n >> 1)) = o;
        }
    }
    __device__ __forceinline__ void operator()(int m, int n, float a0, float a1) const {
        if (act) {
            out[(size_t)m * (N >> 1) + (n >> 1)] = from_f<TS>(silu_f(a0 + to_f(bias[n])) * (a1 + to_f(bias[n + 1])));
            return;
        }
        TS *o = out + (size_t)m * N + n;
        o[0] = from_f<TS>(gelu_erf_f(a0 + to_f(bias[n])));
        o[1] = from_f<TS>(gelu_erf_f(a1 + to_f(bias[n + 1])));
    }
};

// Velocity head: + bias, unpatchify into v_out [nf,C,H,W].
template <typename TS> struct EpiFinal {
    const StepParams *sp;
    const TS *bias;
    Dims D;
    __device__ __forceinline__ void prefetch(unsigned int, unsigned int) const {}
    static constexpr int kBatch = 4;        // epilogue items a thread keeps in flight together
    static constexpr bool kRowStats = false;
    static constexpr bool kTables = false;
    struct Row {};
    struct Col {};
    struct Side {
        int unused;
    };
    __device__ __forceinline__ void load(int, int, Side &) const {}
    __device__ __forceinline__ void apply(int m, int n, float *a, const Side &, float2, const float4 *, int,
                                          unsigned, const Row &, const Col &) const {
#pragma unroll
        for (int i = 0; i < 8; i += 2) (*this)(m, n + i, a[i], a[i + 1]);
    }
    __device__ __forceinline__ void operator()(int m, int n, float a0, float a1) const {
        const int jp = m / D.T, tok = m % D.T;
        const int j = sp->fr[jp].out_index;        // frames that only ride along for their K/V have no output
        if (j < 0) return;
        const int r = tok / D.tw, c = tok % D.tw;
        float av[2] = {a0 + to_f(bias[n]), a1 + to_f(bias[n + 1])};
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            int p = n + u;
            int ch = p / (D.p * D.p), py = (p / D.p) % D.p, px = p % D.p;
            size_t idx = (((size_t)j * D.C + ch) * D.Hl + (r * D.p + py)) * D.Wl + (c * D.p + px);
            sp->v_out[idx] = av[u];
        }
    }
};

// ---------------------------------------------------------------------------
// Straightforward GEMM: C[m][n] = sum_k A[m][k] * Wt[n][k], fp32 accumulation,
// 64x64 tile, 16-deep k slices.  M = sp->nf * T (read on the device).
// ---------------------------------------------------------------------------
template <typename TS, typename Epi>
__global__ void __launch_bounds__(256) k_gemm_simple(const StepParams *sp, int T, const TS *__restrict__ A,
                                                     const TS *__restrict__ Wt, int N, int K, Epi epi) {
    __shared__ float As[16][64];
    __shared__ float Bs[16][64];
    pdl_wait();
    pdl_launch();
    const int M = sp->nf * T;
    const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    if (m0 >= M) return;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int lr = tid >> 2, lk = (tid & 3) * 4;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int k0 = 0; k0 < K; k0 += 16) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            int k = k0 + lk + u;
            int m = m0 + lr, n = n0 + lr;
            As[lk + u][lr] = (m < M && k < K) ? to_f(A[(size_t)m * K + k]) : 0.f;
            Bs[lk + u][lr] = (n < N && k < K) ? to_f(Wt[(size_t)n * K + k]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            float4 a = *reinterpret_cast<const float4 *>(&As[kk][ty * 4]);
            float4 b = *reinterpret_cast<const float4 *>(&Bs[kk][tx * 4]);
            float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; j += 2) {
            int n = n0 + tx * 4 + j;
            if (n + 1 < N) epi(m, n, acc[i][j], acc[i][j + 1]);
        }
    }
}

// ---------------------------------------------------------------------------
// Straightforward block-wise causal attention (Section 3.1): one warp per
// (query token, head); keys are walked frame page by frame page over the
// query frame's window, so the mask is a page range and never a matrix.
// Lanes split the head dimension; online softmax in fp32.
// ---------------------------------------------------------------------------
template <typename TS, int DH>
__global__ void __launch_bounds__(128) k_attn_simple(const StepParams *sp, Dims D, int layer, const TS *q,
                                                     const TS *kc, const TS *vc, TS *out) {
    constexpr int R = DH / 32;
    pdl_wait();
    pdl_launch();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int Nq = sp->nf * D.T;
    const long long w = (long long)blockIdx.x * (blockDim.x >> 5) + warp;
    if (w >= (long long)Nq * D.H) return;
    const int m = (int)(w / D.H), h = (int)(w % D.H);
    const FrameDesc fr = sp->fr[m / D.T];
    float qv[R], acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        qv[r] = to_f(q[((size_t)h * Nq + m) * DH + lane + 32 * r]);
        acc[r] = 0.f;
    }
    const float scale = rsqrtf((float)DH);
    float mx = -INFINITY, l = 0.f;
    for (int g = fr.win_first; g <= fr.frame; ++g) {
        const size_t off = kv_page_offset(D, fr.stream, layer, g) + (size_t)h * D.T * DH;
        const TS *kp = kc + off, *vp = vc + off;
        for (int j = 0; j < D.T; ++j) {
            float s = 0.f;
#pragma unroll
            for (int r = 0; r < R; ++r) s = fmaf(qv[r], to_f(kp[(size_t)j * DH + lane + 32 * r]), s);
            s = warp_sum(s) * scale;
            const float mn = fmaxf(mx, s);
            const float corr = expf(mx - mn), p = expf(s - mn);
            l = l * corr + p;
#pragma unroll
            for (int r = 0; r < R; ++r) acc[r] = fmaf(p, to_f(vp[(size_t)j * DH + lane + 32 * r]), acc[r] * corr);
            mx = mn;
        }
    }
    const float inv = 1.0f / l;
#pragma unroll
    for (int r = 0; r < R; ++r) out[(size_t)m * D.d + h * DH + lane + 32 * r] = from_f<TS>(acc[r] * inv);
}

// ---------------------------------------------------------------------------
// Sampler glue (Section 4.1): elementwise.
// ---------------------------------------------------------------------------
// out = a*x + b*y (y may be NULL)
__global__ void k_axpby(float *out, float a, const float *x, float b, const float *y, size_t n) {
    pdl_wait();
    pdl_launch();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float v = a * x[i];
    if (y) v = fmaf(b, y[i], v);
    out[i] = v;
}

// x0 = a*x' + b*v  (= sigma_d (x_in - t v));  if z: x' <- c*x0 + s*z  (re-noise to the next timestep)
__global__ void k_sampler_post(float *xp, const float *v, const float *z, float *x0, float a, float b, float c,
                               float s, size_t n) {
    pdl_wait();
    pdl_launch();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float e = fmaf(b, v[i], a * xp[i]);
    x0[i] = e;
    if (z) xp[i] = fmaf(s, z[i], c * e);
}

// One step of DPM-Solver++(2M) on the Flow-Matching path (Section 3.2 "Sampling" names the solver; the update
// is the published multistep form with data prediction x0 = x - t v):
//     x <- a x + b ((1 + c) x0 - c x0_prev),   x0_prev <- x0;   out = scale * x  when out is given (last step).
__global__ void k_dpmpp_update(float *x, const float *v, float *x0_prev, float t, float a, float b, float c,
                               float *out, float scale, size_t n) {
    pdl_wait();
    pdl_launch();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const float xi = x[i];
    const float x0 = fmaf(-t, v[i], xi);
    float D = x0;
    if (c != 0.f) D = fmaf(c, x0 - x0_prev[i], x0);
    const float xn = fmaf(b, D, a * xi);
    x[i] = xn;
    x0_prev[i] = x0;
    if (out) out[i] = scale * xn;
}

// ---------------------------------------------------------------------------
// Cache read-out, fill and digest.
// ---------------------------------------------------------------------------
template <typename TS>
__global__ void k_kv_read(Dims D, const TS *cache, int stream, int layer, int frame, float *out) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= D.page_elems) return;
    out[i] = to_f(cache[kv_page_offset(D, stream, layer, frame) + i]);
}

template <typename TS> __global__ void k_to_f32(const TS *src, float *out, size_t n) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = to_f(src[i]);
}

// copy [H][n_frames*T][dh] (storage type) into pages of (stream 0, layer) frames 0..n_frames-1
template <typename TS>
__global__ void k_kv_fill(Dims D, TS *cache, int layer, const TS *src, int n_frames) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    size_t total = (size_t)n_frames * D.page_elems;
    if (i >= total) return;
    int e = (int)(i % D.dh);
    size_t r = i / D.dh;
    int tok_all = (int)(r % ((size_t)n_frames * D.T));
    int h = (int)(r / ((size_t)n_frames * D.T));
    int f = tok_all / D.T, tok = tok_all % D.T;
    cache[kv_page_offset(D, 0, layer, f) + ((size_t)h * D.T + tok) * D.dh + e] = src[i];
}

__device__ __forceinline__ unsigned long long mix64(unsigned long long x) {
    x ^= x >> 33;
    x *= 0xff51afd7ed558ccdULL;
    x ^= x >> 33;
    x *= 0xc4ceb9fe1a85ec53ULL;
    x ^= x >> 33;
    return x;
}

// Order-independent digest: sum over elements of mix(logical position, raw bits).
// The logical position is (layer, absolute frame, K or V, offset in page), so
// the digest does not depend on which ring slot holds a frame.
template <typename TS>
__global__ void k_kv_hash(Dims D, const TS *kc, const TS *vc, int stream, int first, int count,
                          unsigned long long *acc) {
    const size_t per_layer = (size_t)count * D.page_elems;
    const size_t total = per_layer * D.L;
    unsigned long long local = 0;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        int layer = (int)(i / per_layer);
        size_t r = i % per_layer;
        int f = first + (int)(r / D.page_elems);
        size_t e = r % D.page_elems;
        size_t off = kv_page_offset(D, stream, layer, f) + e;
        unsigned long long kb, vb;
        if (sizeof(TS) == 2) {
            kb = *reinterpret_cast<const unsigned short *>(kc + off);
            vb = *reinterpret_cast<const unsigned short *>(vc + off);
        } else {
            kb = *reinterpret_cast<const unsigned int *>(kc + off);
            vb = *reinterpret_cast<const unsigned int *>(vc + off);
        }
        unsigned long long pos = (((unsigned long long)layer * 0x100000ULL + (unsigned long long)f) << 32) ^ e;
        local += mix64(pos * 2 + 0 + (kb << 40) + 0x9e3779b97f4a7c15ULL) + mix64((pos * 2 + 1) ^ (vb << 36));
    }
    atomicAdd(acc, local);
}

// transpose [rows][cols] -> [cols][rows]
// First MLP projection, repacked as [n1][d] (one row per output column): row r is column r of the caller's
// [d][dm] matrix (act 0) or, for the gated form ([d][2 dm], gate columns first), rows 2i and 2i+1 are the gate
// and the up column of hidden unit i, so that a GEMM epilogue finds both in adjacent accumulators.  Rows of
// the padding (hidden units dm .. dmp-1) are zero.  n_in = 1 repacks the bias the same way.
template <typename TS>
__global__ void k_repack_fc1(const TS *src, TS *dst, int n_in, int dm, int dmp, int act) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int n1 = act ? 2 * dmp : dmp;
    if (idx >= (size_t)n1 * n_in) return;
    const int r = (int)(idx / n_in), i = (int)(idx % n_in);
    const int unit = act ? r >> 1 : r;
    const int col = act ? ((r & 1) ? dm + unit : unit) : r;
    dst[idx] = unit < dm ? src[(size_t)i * (act ? 2 * dm : dm) + col] : from_f<TS>(0.f);
}
// Second MLP projection, repacked as [d][dmp] with zero columns for the padding.
template <typename TS>
__global__ void k_repack_fc2(const TS *src, TS *dst, int d, int dm, int dmp) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)d * dmp) return;
    const int o = (int)(idx / dmp), k = (int)(idx % dmp);
    dst[idx] = k < dm ? src[(size_t)k * d + o] : from_f<TS>(0.f);
}

template <typename TS>
__global__ void k_transpose(const TS *in, TS *out, int rows, int cols) {
    __shared__ TS tile[32][33];
    int c = blockIdx.x * 32 + threadIdx.x, r0 = blockIdx.y * 32;
    for (int i = threadIdx.y; i < 32; i += blockDim.y)
        if (r0 + i < rows && c < cols) tile[i][threadIdx.x] = in[(size_t)(r0 + i) * cols + c];
    __syncthreads();
    int r = r0 + threadIdx.x, c0 = blockIdx.x * 32;
    for (int i = threadIdx.y; i < 32; i += blockDim.y)
        if (c0 + i < cols && r < rows) out[(size_t)(c0 + i) * rows + r] = tile[threadIdx.x][i];
}

// Block-wise causal flash attention on tcgen05 / TMEM (bf16, head_dim 64).
//
// Work item = (frame of the pass, head, 128-row query tile, split of the key
// range).  The keys of a query frame are the frame pages win_first..frame of the
// ring cache, walked in blocks of KB keys (KB divides the tokens per frame, so a
// block never straddles a page and the frame-granular mask needs no per-element
// test at all).  Per block:
//     S  = Q K^T          UMMA 128 x KB x 64, operands in shared memory (TMA),
//                         accumulator in tensor memory
//     P  = exp2(S*c - m)  one thread per query row: TMEM -> registers, running
//                         max / sum, bf16 P written to shared memory
//     O += P V            UMMA 128 x 64 x KB, V used straight from its page
//                         (MN-major B operand), accumulated in tensor memory
// The reference maximum m of a row is raised only when a block's maximum exceeds
// it by more than 2^8; only then is the row's O accumulator rescaled (in tensor
// memory), so that in the steady state O is never read back.  The final
// normalisation by the running sum makes the result independent of that choice.
// Warp 0 = TMA producer, warp 1 = UMMA issuer, warps 2-5 and 6-9 = two softmax
// groups.  Group g takes the key blocks b with b % 2 == g and keeps its own
// (max, sum, O) state, S accumulator and P tile, so that one group's
// exponentials overlap the other's tensor-memory traffic and UMMAs.
// At the end the two groups' states are merged in shared memory.  A key range
// longer than CH blocks is split over several CTAs; each writes its unnormalised
// (O, m, l) state, and the CTA that finishes last (a counter per query tile)
// merges the states in split order and writes the output.
// CH depends only on the configuration, so a frame's result does not depend on
// which other frames share its pass.
#pragma once
#include "nfd_sm100.cuh"

struct AttnPlan {
    int KB = 0;          // keys per block
    int BPF = 0;         // blocks per frame page
    int QT = 0;          // 128-row query tiles per frame
    int CH = 0;          // key blocks per split
    int MAXSPLIT = 0;    // splits of the longest window
};

#ifndef ATTN_POLY_PAIR
#define ATTN_POLY_PAIR (-1)     // which of the 4 column pairs of an 8-column group uses ex2_poly (-1: none)
#endif

template <int KB> struct AttnCfg {
    static constexpr int NST = 4;                          // K/V ring stages
    static constexpr int Q_BYTES = 128 * 128;
    static constexpr int P_BYTES = 2 * 128 * 128;          // one group's P tile: two 64-key atoms
    static constexpr int KV_BYTES = KB * 128;              // one K (or V) block
    static constexpr int RING_BYTES = NST * 2 * KV_BYTES;
    static constexpr int OROW = 68;                        // floats per parked O row (64 + pad)
    static constexpr int PARK_BYTES = 128 * OROW * 4 + 128 * 8;           // group 1's state: O rows, then (m, l)
    static constexpr int SMEM = Q_BYTES + 2 * P_BYTES + RING_BYTES + 1024 + 256;
    static constexpr int TMEM_COLS = 512;                  // S0 @0, S1 @128, O0 @256, O1 @320
    static constexpr int THREADS = 320;
    static_assert(PARK_BYTES <= 2 * P_BYTES, "group 1's parked state must fit the P tiles");
};

__host__ __device__ constexpr uint32_t umma_idesc_bf16_bmn(int M, int N) {
    return umma_idesc_bf16(M, N) | (1u << 16);             // B operand MN-major
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 2^y on the FMA and integer pipes, for a share of the softmax's exponentials: the special-function unit
// (16 ex2 per clock and SM) is what bounds the softmax at head dimension 64.  Round-to-nearest split
// y = n + f by the magic-number addition, a cubic for 2^f on [-0.5, 0.5] (relative error 7.5e-5, far below
// the bf16 rounding of P), n added to the exponent field.  y <= 127; results below 2^-125 are clamped there.
__device__ __forceinline__ float ex2_poly(float y) {
    y = fmaxf(y, -125.0f);
    const float t = y + 12582912.0f;               // 1.5 * 2^23: round(y) lands in the low mantissa bits
    const float f = y - (t - 12582912.0f);
    float p = fmaf(0.05517220f, f, 0.24261118f);
    p = fmaf(p, f, 0.69326091f);
    p = fmaf(p, f, 0.99992806f);
    return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}

__device__ __forceinline__ void named_bar_sync(int id, int n_threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n_threads) : "memory");
}

template <int KB>
__global__ void __launch_bounds__(AttnCfg<KB>::THREADS, 1)
k_attn_tc(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
          const __grid_constant__ CUtensorMap tmV, const StepParams *sp, Dims D, int layer, AttnPlan pl, bf16 *out,
          float *part_o, float2 *part_ml, unsigned int *counters, int *status) {
    using A = AttnCfg<KB>;
    extern __shared__ uint8_t smem_raw[];
    NFD_TRACE_T0();
    const int z = blockIdx.z, j = z / D.H, h = z % D.H;
    const int qt = blockIdx.y, split = blockIdx.x;
    // the pass descriptor was written by the first kernel of the pass, which completed long ago
    const FrameDesc fr = sp->fr[j];
    const int nbt = (fr.frame - fr.win_first + 1) * pl.BPF;      // key blocks of this frame's window
    const int nsplit = (nbt + pl.CH - 1) / pl.CH;
    if (split >= nsplit) return;                                  // uniform for the CTA, before any barrier or allocation
    const int b0 = split * pl.CH;
    const int nb = min(nbt, b0 + pl.CH) - b0;                     // >= 1
    const int Nq = sp->nf * D.T;

    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *sQ = smem, *sP = smem + A::Q_BYTES, *sKV = sP + 2 * A::P_BYTES;
    uint64_t *bars = reinterpret_cast<uint64_t *>(sKV + A::RING_BYTES);
    const uint32_t q_full = smem_u32(bars), kv_full = smem_u32(bars + 1), kv_empty = smem_u32(bars + 1 + A::NST),
                   s_full = smem_u32(bars + 1 + 2 * A::NST), p_full = s_full + 16, pv_done = s_full + 32;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 1 + 2 * A::NST + 6);
    int *last_flag = reinterpret_cast<int *>(tmem_slot + 1);
    // group 1 parks its state here after the main loop (the P tiles are free by then)
    float *parkO = reinterpret_cast<float *>(sP);
    float2 *parkML = reinterpret_cast<float2 *>(sP + 128 * A::OROW * 4);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
        mbar_init(q_full, 1);
        for (int s = 0; s < A::NST; ++s) {
            mbar_init(kv_full + 8 * s, 1);
            mbar_init(kv_empty + 8 * s, 1);
        }
        for (int g = 0; g < 2; ++g) {
            mbar_init(s_full + 8 * g, 1);
            mbar_init(p_full + 8 * g, 128);
            mbar_init(pv_done + 8 * g, 1);
        }
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), A::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            const int page_rows = D.H * D.T;
            bool waited = false;
            for (int b = 0; b < nb; ++b) {
                const int s = b % A::NST;
                const int blk = b0 + b;
                const int g = fr.win_first + blk / pl.BPF, kb = blk % pl.BPF;
                // pages of frames written earlier than this pass may be fetched before the predecessor finishes
                if (!waited && (g >= fr.first_new || b >= A::NST)) {
                    pdl_wait();
                    waited = true;
                    mbar_expect_tx(q_full, A::Q_BYTES);
                    tma_load_2d(smem_u32(sQ), &tmQ, q_full, 0, h * Nq + j * D.T + qt * 128);
                }
                if (b >= A::NST && !mbar_wait(kv_empty + 8 * s, ((b / A::NST) - 1) & 1, status)) break;
                const int row = ((fr.stream * D.L + layer) * D.R + (g % D.R)) * page_rows + h * D.T + kb * KB;
                mbar_expect_tx(kv_full + 8 * s, 2 * A::KV_BYTES);
                tma_load_2d(smem_u32(sKV + s * 2 * A::KV_BYTES), &tmK, kv_full + 8 * s, 0, row);
                tma_load_2d(smem_u32(sKV + s * 2 * A::KV_BYTES + A::KV_BYTES), &tmV, kv_full + 8 * s, 0, row);
            }
            if (!waited) {
                pdl_wait();
                mbar_expect_tx(q_full, A::Q_BYTES);
                tma_load_2d(smem_u32(sQ), &tmQ, q_full, 0, h * Nq + j * D.T + qt * 128);
            }
        }
    } else if (warp == 1) {
        // ---------------- UMMA issuer ----------------
        if (lane == 0) {
            pdl_launch();
            constexpr uint32_t idesc_s = umma_idesc_bf16(128, KB);
            constexpr uint32_t idesc_pv = umma_idesc_bf16_bmn(128, 64);
            const uint64_t qd = umma_desc_k128(smem_u32(sQ));
            bool ok = mbar_wait(q_full, 0, status);
            auto issue_s = [&](int b) {          // S(b) = Q K(b)^T into group (b & 1)'s accumulator
                const int s = b % A::NST, g = b & 1;
                if (!mbar_wait(kv_full + 8 * s, (b / A::NST) & 1, status)) return false;
                tc_fence_after();
                const uint64_t kd = umma_desc_k128(smem_u32(sKV + s * 2 * A::KV_BYTES));
#pragma unroll
                for (int k4 = 0; k4 < 4; ++k4) umma_bf16_ss(tmem + 128 * g, qd + 2 * k4, kd + 2 * k4, idesc_s, k4 != 0);
                umma_commit(s_full + 8 * g);
                return true;
            };
            if (ok) ok = issue_s(0);
            if (ok && nb > 1) ok = issue_s(1);
            for (int b = 0; b < nb && ok; ++b) {
                const int g = b & 1, s = b % A::NST;
                ok = mbar_wait(p_full + 8 * g, (b >> 1) & 1, status);
                if (!ok) break;
                // the group has consumed S(b): its next S goes first, so that it is ready as early as possible
                if (b + 2 < nb) ok = issue_s(b + 2);
                if (!ok) break;
                tc_fence_after();
                const uint64_t pd = umma_desc_k128(smem_u32(sP + g * A::P_BYTES));
                const uint64_t vd = umma_desc_k128(smem_u32(sKV + s * 2 * A::KV_BYTES + A::KV_BYTES));
#pragma unroll
                for (int i = 0; i < KB / 16; ++i) {
                    // P: K-major, 64-key atoms of 16 KiB; V: MN-major, 16 keys = 2 KiB per step
                    const uint64_t pa = pd + (uint64_t)((i >> 2) * (16384 >> 4) + (i & 3) * 2);
                    umma_bf16_ss(tmem + 256 + 64 * g, pa, vd + (uint64_t)(i * (2048 >> 4)), idesc_pv,
                                 (uint32_t)((b >> 1) != 0 || i != 0));
                }
                umma_commit(pv_done + 8 * g);
                umma_commit(kv_empty + 8 * s);
            }
        }
    } else {
        // ---------------- softmax: one thread per query row, two groups ----------------
        const int g = (warp - 2) >> 2;                     // group: blocks b with (b & 1) == g
        const int quad = warp & 3;
        const int trow = quad * 32 + lane;
        const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
        const uint32_t tS = tmem + 128 * g + lane_off, tO = tmem + 256 + 64 * g + lane_off;
        const float c = (1.0f / sqrtf((float)D.dh)) * 1.4426950408889634f;   // softmax scale in the log2 domain
        float m_run = -INFINITY, l_run = 0.f;
        uint8_t *prow = sP + g * A::P_BYTES + trow * 128;
        bool ok = true;
        int i = 0;
        for (int b = g; b < nb; b += 2, ++i) {
            ok = mbar_wait(s_full + 8 * g, i & 1, status);
            if (!ok) break;
            tc_fence_after();
            // pass 1 over S: row maximum (all loads in flight together; the values die right after)
            float mx;
            {
                uint32_t sr[KB];
#pragma unroll
                for (int cc = 0; cc < KB; cc += 32) {
                    if (cc + 32 <= KB)
                        tmem_ld32(tS + cc, sr + cc);
                    else
                        tmem_ld16(tS + cc, sr + cc);
                }
                tmem_ld_wait();
                float m4[4] = {__uint_as_float(sr[0]), __uint_as_float(sr[1]), __uint_as_float(sr[2]),
                               __uint_as_float(sr[3])};
#pragma unroll
                for (int e = 4; e < KB; ++e) m4[e & 3] = fmaxf(m4[e & 3], __uint_as_float(sr[e]));
                mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
            }
            const float m_blk = mx * c;
            if (i > 0) {
                // the previous P V product of this group is complete: its P tile is free, O is at rest
                ok = mbar_wait(pv_done + 8 * g, (i - 1) & 1, status);
                if (!ok) break;
                tc_fence_after();
            }
            const bool raise = m_blk > m_run + 8.0f;       // always true for the first block (m_run = -inf)
            if (__any_sync(0xffffffffu, raise)) {
                const float m_new = raise ? m_blk : m_run;
                const float f = ex2_approx(m_run - m_new);  // 1 for rows that keep their reference maximum
                if (i > 0) {
#pragma unroll
                    for (int cc = 0; cc < 64; cc += 32) {
                        uint32_t r[32];
                        tmem_ld32(tO + cc, r);
                        tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * f);
                        tmem_st32(tO + cc, r);
                    }
                    tmem_st_wait();
                }
                l_run *= f;
                m_run = m_new;
            }
            // pass 2 over S, 16 columns at a time with the next load in flight:
            // P = exp2(S c - m) as bf16 into shared memory (128-byte-swizzled K-major layout)
            float2 ls2[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
            uint32_t sa[16], sb[16];
            tmem_ld16(tS, sa);
#pragma unroll
            for (int cc = 0; cc < KB; cc += 16) {
                uint32_t *cur = ((cc >> 4) & 1) ? sb : sa, *nxt = ((cc >> 4) & 1) ? sa : sb;
                tmem_ld_wait();
                if (cc + 16 < KB) tmem_ld16(tS + cc + 16, nxt);
#pragma unroll
                for (int u2 = 0; u2 < 2; ++u2) {
                    uint32_t pk[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        // one pair in four goes to the FMA pipes (ex2_poly)
                        const float2 y = ffma2(make_float2(__uint_as_float(cur[8 * u2 + 2 * u]),
                                                           __uint_as_float(cur[8 * u2 + 2 * u + 1])),
                                               make_float2(c, c), make_float2(-m_run, -m_run));
                        const float p0 = (u == ATTN_POLY_PAIR) ? ex2_poly(y.x) : ex2_approx(y.x);
                        const float p1 = (u == ATTN_POLY_PAIR) ? ex2_poly(y.y) : ex2_approx(y.y);
                        ls2[u] = fadd2(ls2[u], make_float2(p0, p1));
                        const __nv_bfloat162 hp = __floats2bfloat162_rn(p0, p1);
                        pk[u] = *reinterpret_cast<const uint32_t *>(&hp);
                    }
                    const int ch = (cc >> 3) + u2;
                    uint8_t *dst = prow + (ch >> 3) * 16384 + (((ch & 7) ^ (trow & 7)) << 4);
                    *reinterpret_cast<uint4 *>(dst) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
            }
            l_run += ((ls2[0].x + ls2[0].y) + (ls2[1].x + ls2[1].y)) + ((ls2[2].x + ls2[2].y) + (ls2[3].x + ls2[3].y));
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(p_full + 8 * g);
        }
        // this group's O accumulator (unnormalised, relative to m_run)
        float O[64];
#pragma unroll
        for (int e = 0; e < 64; ++e) O[e] = 0.f;
        if (ok && i > 0) {
            ok = mbar_wait(pv_done + 8 * g, (i - 1) & 1, status);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int cc = 0; cc < 64; cc += 32) {
                    uint32_t r[32];
                    tmem_ld32(tO + cc, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) O[cc + e] = __uint_as_float(r[e]);
                }
            }
        }
        if (!ok || i == 0) {                               // no block or a failed wait: this state counts for nothing
            m_run = -INFINITY, l_run = 0.f;
#pragma unroll
            for (int e = 0; e < 64; ++e) O[e] = 0.f;
        }
        const int row = qt * 128 + trow;
        const size_t item_q = (size_t)z * pl.QT + qt;      // (frame, head, query tile)
        // ---- the two groups of this CTA first: group 1 parks its state, group 0 folds it in ----
        named_bar_sync(1, 256);                            // both groups are past their last UMMA: the P tiles are free
        if (g == 1) {
            float4 *po = reinterpret_cast<float4 *>(parkO + (size_t)trow * A::OROW);
#pragma unroll
            for (int e = 0; e < 64; e += 4) po[e >> 2] = make_float4(O[e], O[e + 1], O[e + 2], O[e + 3]);
            parkML[trow] = make_float2(m_run, l_run);
        }
        named_bar_sync(1, 256);
        float m_cta = m_run, l_cta = l_run;
        if (g == 0) {
            const float2 ml1 = parkML[trow];
            m_cta = fmaxf(m_run, ml1.x);
            const float w0 = ex2_approx(m_run - m_cta), w1 = ex2_approx(ml1.x - m_cta);
            l_cta = l_run * w0 + ml1.y * w1;
            const float4 *po = reinterpret_cast<const float4 *>(parkO + (size_t)trow * A::OROW);
#pragma unroll
            for (int e = 0; e < 64; e += 4) {
                const float4 v = po[e >> 2];
                O[e] = fmaf(O[e], w0, v.x * w1), O[e + 1] = fmaf(O[e + 1], w0, v.y * w1);
                O[e + 2] = fmaf(O[e + 2], w0, v.z * w1), O[e + 3] = fmaf(O[e + 3], w0, v.w * w1);
            }
        }
        if (nsplit == 1) {
            if (g == 0 && row < D.T) {
                const float inv = 1.0f / l_cta;
                bf16 *o = out + (size_t)(j * D.T + row) * D.d + h * 64;
#pragma unroll
                for (int e = 0; e < 64; e += 8) {
                    float t[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) t[u] = O[e + u] * inv;
                    *reinterpret_cast<uint4 *>(o + e) = pack_bf16x8(t);
                }
            }
        } else {
            // ---- publish this CTA's state; the CTA that finishes last merges the splits in split order ----
            const size_t st0 = item_q * pl.MAXSPLIT * 128;                           // first state row of this query tile
            if (g == 0) {
                const size_t item = st0 + (size_t)split * 128 + trow;
                float4 *po4 = reinterpret_cast<float4 *>(part_o + item * 64);
                float4 *ps4 = reinterpret_cast<float4 *>(parkO + (size_t)trow * A::OROW);     // own copy for the merge
#pragma unroll
                for (int e = 0; e < 64; e += 4) {
                    const float4 v = make_float4(O[e], O[e + 1], O[e + 2], O[e + 3]);
                    po4[e >> 2] = v;
                    ps4[e >> 2] = v;
                }
                part_ml[item] = make_float2(m_cta, l_cta);
                parkML[trow] = make_float2(m_cta, l_cta);
                __threadfence();
            }
            named_bar_sync(1, 256);
            if (threadIdx.x == 64) {
                const unsigned int prev = atomicAdd(counters + item_q, 1u);
                const int last = prev == (unsigned int)(nsplit - 1);
                if (last) counters[item_q] = 0;            // ready for the next launch
                *last_flag = last;
            }
            named_bar_sync(1, 256);
            if (*last_flag) {
                __threadfence();
                // an item = 8 adjacent output columns of a row; two items per thread and round, so that the
                // loads of both (all splits, four at a time) are in flight together
                for (int it0 = (int)threadIdx.x - 64; it0 < 128 * 8; it0 += 512) {
                    int r[2], ch[2];
                    bool live[2];
                    float acc[2][8], l[2], mx[2];
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        const int it = it0 + q * 256;
                        r[q] = it >> 3, ch[q] = it & 7;
                        live[q] = it < 128 * 8 && qt * 128 + r[q] < D.T;
                        l[q] = 0.f, mx[q] = -INFINITY;
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[q][e] = 0.f;
                    }
                    for (int s0 = 0; s0 < nsplit; s0 += 4) {
                        // this CTA's own state comes from shared memory (same values as its published copy)
                        float2 ml[2][4];
                        float4 v0[2][4], v1[2][4];
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            if (!live[q]) continue;
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                const int sidx = s0 + u < nsplit ? s0 + u : nsplit - 1;
                                if (sidx == split) {
                                    ml[q][u] = parkML[r[q]];
                                    const float4 *po =
                                        reinterpret_cast<const float4 *>(parkO + (size_t)r[q] * A::OROW + ch[q] * 8);
                                    v0[q][u] = po[0], v1[q][u] = po[1];
                                } else {
                                    const size_t item = st0 + (size_t)sidx * 128 + r[q];
                                    ml[q][u] = __ldcg(&part_ml[item]);
                                    const float4 *po = reinterpret_cast<const float4 *>(part_o + item * 64 + ch[q] * 8);
                                    v0[q][u] = __ldcg(po), v1[q][u] = __ldcg(po + 1);
                                }
                            }
                        }
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            if (!live[q]) continue;
                            float mb = mx[q];
#pragma unroll
                            for (int u = 0; u < 4; ++u)
                                if (s0 + u < nsplit) mb = fmaxf(mb, ml[q][u].x);
                            const float fo = ex2_approx(mx[q] - mb);   // rescale of what was merged so far (0 at first)
                            l[q] *= fo;
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc[q][e] *= fo;
                            mx[q] = mb;
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                if (s0 + u < nsplit) {
                                    const float w = ex2_approx(ml[q][u].x - mb);
                                    l[q] = fmaf(ml[q][u].y, w, l[q]);
                                    acc[q][0] = fmaf(v0[q][u].x, w, acc[q][0]), acc[q][1] = fmaf(v0[q][u].y, w, acc[q][1]);
                                    acc[q][2] = fmaf(v0[q][u].z, w, acc[q][2]), acc[q][3] = fmaf(v0[q][u].w, w, acc[q][3]);
                                    acc[q][4] = fmaf(v1[q][u].x, w, acc[q][4]), acc[q][5] = fmaf(v1[q][u].y, w, acc[q][5]);
                                    acc[q][6] = fmaf(v1[q][u].z, w, acc[q][6]), acc[q][7] = fmaf(v1[q][u].w, w, acc[q][7]);
                                }
                            }
                        }
                    }
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        if (!live[q]) continue;
                        const float inv = 1.0f / l[q];
#pragma unroll
                        for (int u = 0; u < 8; ++u) acc[q][u] *= inv;
                        *reinterpret_cast<uint4 *>(out + (size_t)(j * D.T + qt * 128 + r[q]) * D.d + h * 64 + ch[q] * 8) =
                            pack_bf16x8(acc[q]);
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, A::TMEM_COLS);
    NFD_TRACE_END(TRK_ATTN);
}

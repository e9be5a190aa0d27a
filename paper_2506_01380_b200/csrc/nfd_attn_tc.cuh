// Block-wise causal flash attention on tcgen05 / TMEM (bf16, head_dim 64).
//
// Work item = (frame of the pass, head, 128-row query tile, split of the key
// range).  The keys of a query frame are the frame pages win_first..frame of the
// ring cache, walked in blocks of KB keys (KB divides the tokens per frame, so a
// block never straddles a page and the frame-granular mask needs no per-element
// test at all).  Per block:
//     S  = Q K^T          UMMA 128 x KB x 64, operands in shared memory (TMA),
//                         accumulator in tensor memory (double buffered)
//     P  = exp2(S*c - m)  one thread per query row: TMEM -> registers, running
//                         max / sum, bf16 P written to shared memory
//     PV = P V            UMMA 128 x 64 x KB, V used straight from its page
//                         (MN-major B operand), accumulator in tensor memory
//     O  = O*corr + PV    in registers
// Warp 0 = TMA producer, warp 1 = UMMA issuer, warps 2-5 = softmax.
// A key range longer than CH blocks is split over several CTAs which write
// unnormalised (O, m, l) partials; k_attn_combine merges them in split order.
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

template <int KB> struct AttnCfg {
    static constexpr int NST = 4;                          // K/V ring stages
    static constexpr int Q_BYTES = 128 * 128;
    static constexpr int P_BYTES = 2 * 128 * 128;          // two 64-key atoms
    static constexpr int KV_BYTES = KB * 128;              // one K (or V) block
    static constexpr int SMEM = Q_BYTES + P_BYTES + NST * 2 * KV_BYTES + 1024 + 256;
    static constexpr int TMEM_COLS = 512;                  // S0 @0, S1 @128, PV @256
};

__host__ __device__ constexpr uint32_t umma_idesc_bf16_bmn(int M, int N) {
    return umma_idesc_bf16(M, N) | (1u << 16);             // B operand MN-major
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int KB>
__global__ void __launch_bounds__(192, 1)
k_attn_tc(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
          const __grid_constant__ CUtensorMap tmV, const StepParams *sp, Dims D, int layer, AttnPlan pl, bf16 *out,
          float *part_o, float2 *part_ml, int *status) {
    using A = AttnCfg<KB>;
    extern __shared__ uint8_t smem_raw[];
    const int z = blockIdx.z, j = z / D.H, h = z % D.H;
    const int qt = blockIdx.y, split = blockIdx.x;
    const FrameDesc fr = sp->fr[j];
    const int nbt = (fr.frame - fr.win_first + 1) * pl.BPF;      // key blocks of this frame's window
    const int nsplit = (nbt + pl.CH - 1) / pl.CH;
    if (split >= nsplit) return;                                  // uniform for the CTA
    const int b0 = split * pl.CH;
    const int nb = min(nbt, b0 + pl.CH) - b0;
    const int Nq = sp->nf * D.T;

    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *sQ = smem, *sP = smem + A::Q_BYTES, *sKV = sP + A::P_BYTES;
    uint64_t *bars = reinterpret_cast<uint64_t *>(sKV + A::NST * 2 * A::KV_BYTES);
    const uint32_t q_full = smem_u32(bars), kv_full = smem_u32(bars + 1), kv_empty = smem_u32(bars + 1 + A::NST),
                   s_full = smem_u32(bars + 1 + 2 * A::NST), s_empty = s_full + 16, p_full = s_full + 32,
                   pv_full = s_full + 40;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 1 + 2 * A::NST + 6);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (warp == 0 && lane == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < A::NST; ++s) {
            mbar_init(kv_full + 8 * s, 1);
            mbar_init(kv_empty + 8 * s, 1);
        }
        mbar_init(s_full, 1);
        mbar_init(s_full + 8, 1);
        mbar_init(s_empty, 128);
        mbar_init(s_empty + 8, 128);
        mbar_init(p_full, 128);
        mbar_init(pv_full, 1);
        fence_mbar_init();
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), A::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tS0 = tmem, tPV = tmem + 256;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            mbar_expect_tx(q_full, A::Q_BYTES);
            tma_load_2d(smem_u32(sQ), &tmQ, q_full, 0, h * Nq + j * D.T + qt * 128);
            const int page_rows = D.H * D.T;
            for (int b = 0; b < nb; ++b) {
                const int s = b % A::NST;
                if (b >= A::NST && !mbar_wait(kv_empty + 8 * s, ((b / A::NST) - 1) & 1, status)) break;
                const int blk = b0 + b;
                const int g = fr.win_first + blk / pl.BPF, kb = blk % pl.BPF;
                const int row = ((fr.stream * D.L + layer) * D.R + (g % D.R)) * page_rows + h * D.T + kb * KB;
                mbar_expect_tx(kv_full + 8 * s, 2 * A::KV_BYTES);
                tma_load_2d(smem_u32(sKV + s * 2 * A::KV_BYTES), &tmK, kv_full + 8 * s, 0, row);
                tma_load_2d(smem_u32(sKV + s * 2 * A::KV_BYTES + A::KV_BYTES), &tmV, kv_full + 8 * s, 0, row);
            }
        }
    } else if (warp == 1) {
        // ---------------- UMMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t idesc_s = umma_idesc_bf16(128, KB);
            constexpr uint32_t idesc_pv = umma_idesc_bf16_bmn(128, 64);
            const uint64_t qd = umma_desc_k128(smem_u32(sQ));
            const uint64_t pd = umma_desc_k128(smem_u32(sP));
            bool ok = mbar_wait(q_full, 0, status) && mbar_wait(kv_full, 0, status);
            if (ok) {
                tc_fence_after();
                const uint64_t kd = umma_desc_k128(smem_u32(sKV));
#pragma unroll
                for (int k4 = 0; k4 < 4; ++k4) umma_bf16_ss(tS0, qd + 2 * k4, kd + 2 * k4, idesc_s, k4 != 0);
                umma_commit(s_full);
            }
            for (int b = 0; b < nb && ok; ++b) {
                if (b + 1 < nb) {
                    const int b1 = b + 1, s1 = b1 % A::NST;
                    ok = mbar_wait(kv_full + 8 * s1, (b1 / A::NST) & 1, status);
                    if (ok && b1 >= 2) ok = mbar_wait(s_empty + 8 * (b1 & 1), ((b1 >> 1) - 1) & 1, status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t kd = umma_desc_k128(smem_u32(sKV + s1 * 2 * A::KV_BYTES));
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4)
                        umma_bf16_ss(tS0 + 128 * (b1 & 1), qd + 2 * k4, kd + 2 * k4, idesc_s, k4 != 0);
                    umma_commit(s_full + 8 * (b1 & 1));
                }
                ok = mbar_wait(p_full, b & 1, status);
                if (!ok) break;
                tc_fence_after();
                const uint64_t vd = umma_desc_k128(smem_u32(sKV + (b % A::NST) * 2 * A::KV_BYTES + A::KV_BYTES));
#pragma unroll
                for (int i = 0; i < KB / 16; ++i) {
                    // P: K-major, 64-key atoms of 16 KiB; V: MN-major, 16 keys = 2 KiB per step
                    const uint64_t pa = pd + (uint64_t)((i >> 2) * (16384 >> 4) + (i & 3) * 2);
                    umma_bf16_ss(tPV, pa, vd + (uint64_t)(i * (2048 >> 4)), idesc_pv, i != 0);
                }
                umma_commit(pv_full);
                umma_commit(kv_empty + 8 * (b % A::NST));
            }
        }
    } else {
        // ---------------- softmax: one thread per query row ----------------
        const int quad = warp & 3;
        const int trow = quad * 32 + lane;
        const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
        const float c = (1.0f / sqrtf((float)D.dh)) * 1.4426950408889634f;   // softmax scale in the log2 domain
        float m_run = -INFINITY, l_run = 0.f;
        float O[64];
#pragma unroll
        for (int e = 0; e < 64; ++e) O[e] = 0.f;
        uint8_t *prow = sP + trow * 128;
        bool ok = true;
        for (int b = 0; b < nb; ++b) {
            ok = mbar_wait(s_full + 8 * (b & 1), (b >> 1) & 1, status);
            if (!ok) break;
            tc_fence_after();
            uint32_t sr[KB];
            const uint32_t ts = tS0 + 128 * (b & 1) + lane_off;
#pragma unroll
            for (int cc = 0; cc < KB; cc += 32) {
                if (cc + 32 <= KB)
                    tmem_ld32(ts + cc, sr + cc);
                else
                    tmem_ld16(ts + cc, sr + cc);
            }
            tmem_ld_wait();
            tc_fence_before();
            mbar_arrive(s_empty + 8 * (b & 1));
            float mx = __uint_as_float(sr[0]);
#pragma unroll
            for (int i = 1; i < KB; ++i) mx = fmaxf(mx, __uint_as_float(sr[i]));
            const float m_new = fmaxf(m_run, mx * c);
            const float corr = ex2_approx(m_run - m_new);
            float ls = 0.f;
            uint32_t pk[KB / 2];
#pragma unroll
            for (int i = 0; i < KB; i += 2) {
                const float p0 = ex2_approx(fmaf(__uint_as_float(sr[i]), c, -m_new));
                const float p1 = ex2_approx(fmaf(__uint_as_float(sr[i + 1]), c, -m_new));
                // the row sum uses the bf16-rounded probabilities that the P V product sees
                const __nv_bfloat162 hp = __floats2bfloat162_rn(p0, p1);
                const float2 pf = __bfloat1622float2(hp);
                ls += pf.x + pf.y;
                pk[i >> 1] = *reinterpret_cast<const uint32_t *>(&hp);
            }
            l_run = fmaf(l_run, corr, ls);
            m_run = m_new;
            if (b > 0) {
                ok = mbar_wait(pv_full, (b - 1) & 1, status);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int cc = 0; cc < 64; cc += 32) {
                    uint32_t r[32];
                    tmem_ld32(tPV + lane_off + cc, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) O[cc + e] += __uint_as_float(r[e]);
                }
            }
#pragma unroll
            for (int e = 0; e < 64; ++e) O[e] *= corr;
            // P (bf16) into shared memory in the 128-byte-swizzled K-major layout
#pragma unroll
            for (int ch = 0; ch < KB / 8; ++ch) {
                uint8_t *dst = prow + (ch >> 3) * 16384 + (((ch & 7) ^ (trow & 7)) << 4);
                *reinterpret_cast<uint4 *>(dst) = make_uint4(pk[4 * ch], pk[4 * ch + 1], pk[4 * ch + 2], pk[4 * ch + 3]);
            }
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(p_full);
        }
        if (ok && nb > 0) {
            ok = mbar_wait(pv_full, (nb - 1) & 1, status);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int cc = 0; cc < 64; cc += 32) {
                    uint32_t r[32];
                    tmem_ld32(tPV + lane_off + cc, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) O[cc + e] += __uint_as_float(r[e]);
                }
            }
        }
        const int row = qt * 128 + trow;
        if (ok && row < D.T) {
            if (nsplit == 1) {
                const float inv = 1.0f / l_run;
                bf16 *o = out + (size_t)(j * D.T + row) * D.d + h * 64;
#pragma unroll
                for (int e = 0; e < 64; e += 8) {
                    float t[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) t[u] = O[e + u] * inv;
                    *reinterpret_cast<uint4 *>(o + e) = pack_bf16x8(t);
                }
            } else {
                const size_t item = ((size_t)(z * pl.QT + qt) * pl.MAXSPLIT + split) * 128 + trow;
                float4 *po = reinterpret_cast<float4 *>(part_o + item * 64);
#pragma unroll
                for (int e = 0; e < 64; e += 4) po[e >> 2] = make_float4(O[e], O[e + 1], O[e + 2], O[e + 3]);
                part_ml[item] = make_float2(m_run, l_run);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, A::TMEM_COLS);
}

// Merge the split partials of one (frame, head, query tile): thread = query row.
__global__ void __launch_bounds__(128) k_attn_combine(const StepParams *sp, Dims D, AttnPlan pl, const float *part_o,
                                                      const float2 *part_ml, bf16 *out) {
    const int z = blockIdx.y, j = z / D.H, h = z % D.H, qt = blockIdx.x;
    const FrameDesc fr = sp->fr[j];
    const int nbt = (fr.frame - fr.win_first + 1) * pl.BPF;
    const int nsplit = (nbt + pl.CH - 1) / pl.CH;
    if (nsplit == 1) return;                      // the attention kernel already wrote the result
    const int trow = threadIdx.x, row = qt * 128 + trow;
    if (row >= D.T) return;
    const size_t item0 = ((size_t)(z * pl.QT + qt) * pl.MAXSPLIT) * 128 + trow;
    float mx = -INFINITY;
    for (int s = 0; s < nsplit; ++s) mx = fmaxf(mx, part_ml[item0 + (size_t)s * 128].x);
    float acc[64];
#pragma unroll
    for (int e = 0; e < 64; ++e) acc[e] = 0.f;
    float l = 0.f;
    for (int s = 0; s < nsplit; ++s) {
        const float2 ml = part_ml[item0 + (size_t)s * 128];
        const float w = ex2_approx(ml.x - mx);
        l = fmaf(ml.y, w, l);
        const float4 *po = reinterpret_cast<const float4 *>(part_o + (item0 + (size_t)s * 128) * 64);
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            const float4 v = po[e];
            acc[4 * e] = fmaf(v.x, w, acc[4 * e]);
            acc[4 * e + 1] = fmaf(v.y, w, acc[4 * e + 1]);
            acc[4 * e + 2] = fmaf(v.z, w, acc[4 * e + 2]);
            acc[4 * e + 3] = fmaf(v.w, w, acc[4 * e + 3]);
        }
    }
    const float inv = 1.0f / l;
    bf16 *o = out + (size_t)(j * D.T + row) * D.d + h * 64;
#pragma unroll
    for (int e = 0; e < 64; e += 8) {
        float t[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) t[u] = acc[e + u] * inv;
        *reinterpret_cast<uint4 *>(o + e) = pack_bf16x8(t);
    }
}

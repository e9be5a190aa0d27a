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
//                         max / sum, bf16 P written back to tensor memory over
//                         the first half of the S columns it came from
//     O += P V            UMMA 128 x 64 x KB, P read from tensor memory, V used
//                         straight from its page (MN-major B operand in shared
//                         memory), accumulated in tensor memory
// The reference maximum m of a row is raised only when a block's maximum exceeds
// it by more than 2^8; only then is the row's O accumulator rescaled (in tensor
// memory), so that in the steady state O is never read back.  The final
// normalisation by the running sum makes the result independent of that choice.
// Warp 0 = TMA producer, warp 1 = UMMA issuer, warps 2-5 and 6-9 = two softmax
// groups.  Group g takes the key blocks b with b % 2 == g and keeps its own
// (max, sum, O) state and P tile, so that one group's exponentials overlap the
// other's tensor-memory traffic and UMMAs.  S has three accumulators in tensor
// memory, block b using number b % 3, and S(b + 3) is issued right behind
// P V(b), which reads P(b) from that accumulator (the tensor pipe takes its
// instructions in order): a group finds its next S ready when it comes back for
// it, instead of waiting for the issue, the product and the completion signal
// each time.  P never passes through shared memory: the kernel is bound by the
// rate at which the tensor pipe gets its operands out of shared memory, and a
// P tile there would be written once and read once more per block.
// K blocks go through a ring of three stages (stage b % 3; a stage is free again
// when S(b) is complete, which the barrier of accumulator b % 3 tells), V blocks
// through a ring of four (free when P V of its block is complete).  Two
// completion signals per block are all the issuing thread sends, and that
// thread is the busiest of the kernel.
// At the end the two groups' states are merged in shared memory.  A key range
// longer than CH blocks is split over several CTAs; each leaves its unnormalised
// (O, m, l) state in a tile of shared memory and publishes it with one bulk copy;
// the CTA that finishes last (a counter per query tile) pulls the other tiles in
// with bulk copies, merges the states in split order and writes the output.
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
    static constexpr int NK = 3;                           // K ring stages = S accumulators
    static constexpr int NV = 4;                           // V ring stages
    static constexpr int Q_BYTES = 128 * 128;
    static constexpr int P_BYTES = 2 * 128 * 128;          // one group's P tile: two 64-key atoms
    static constexpr int KV_BYTES = KB * 128;              // one K (or V) block
    static constexpr int RING_BYTES = (NK + NV) * KV_BYTES;
    // A parked state: 128 rows of 64 floats (256 bytes per row; the 16-byte words of row r are stored at
    // word index c ^ (r & 15), so that one thread per row writes without bank conflicts), then 128 x (m, l).
    static constexpr int PARK_O_BYTES = 128 * 256;
    static constexpr int PARK_BYTES = PARK_O_BYTES + 128 * 8;
    static constexpr int N_IN = RING_BYTES / PARK_BYTES;   // other splits' states that the K/V ring holds at once
    static constexpr int SMEM = Q_BYTES + 2 * P_BYTES + RING_BYTES + 1024 + 256;
    static constexpr int TMEM_COLS = 512;                  // S0 @0, S1 @128, S2 @256, O0 @384, O1 @448
    static constexpr int THREADS = 320;
    static_assert(PARK_BYTES <= 2 * P_BYTES, "the parked state must fit the P tiles");
    static_assert(N_IN >= 1, "the K/V ring must hold one incoming state");
};

__host__ __device__ constexpr uint32_t umma_idesc_bf16_bmn(int M, int N) {
    return umma_idesc_bf16(M, N) | (1u << 16);             // B operand MN-major
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void named_bar_sync(int id, int n_threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n_threads) : "memory");
}

template <int KB>
__global__ void __launch_bounds__(AttnCfg<KB>::THREADS, 1)
k_attn_tc(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
          const __grid_constant__ CUtensorMap tmV, const StepParams *sp, Dims D, int layer, AttnPlan pl, bf16 *out,
          float *part_o, unsigned int *counters, int *status) {
    using A = AttnCfg<KB>;
    extern __shared__ uint8_t smem_raw[];
    NFD_TRACE_T0();
    const int z = blockIdx.z, j = z / D.H, h = z % D.H;
    const int qt = blockIdx.y, split = blockIdx.x;
    // the pass descriptor was written by the first kernel of the pass, which completed long ago; the loads
    // are issued here and first used after the set-up below, which hides their latency
    const FrameDesc fr = sp->fr[j];
    const int nf_pass = sp->nf;

    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *sQ = smem, *sP = smem + A::Q_BYTES, *sKV = sP + 2 * A::P_BYTES;
    uint64_t *bars = reinterpret_cast<uint64_t *>(sKV + A::RING_BYTES);
    // barriers: q_full | k_full[NK] | s_full[NK] | v_full[NV] | v_empty[NV] | p_full[2] | in_full
    const uint32_t q_full = smem_u32(bars), k_full = q_full + 8, s_full = k_full + 8 * A::NK,
                   v_full = s_full + 8 * A::NK, v_empty = v_full + 8 * A::NV, p_full = v_empty + 8 * A::NV,
                   in_full = p_full + 16;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 1 + 2 * A::NK + 2 * A::NV + 3);
    int *last_flag = reinterpret_cast<int *>(tmem_slot + 1);
    // states are parked here after the main loop (the P tiles are free by then)
    uint8_t *parkO = sP;
    float2 *parkML = reinterpret_cast<float2 *>(sP + A::PARK_O_BYTES);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
        mbar_init(q_full, 1);
        for (int s = 0; s < A::NK; ++s) {
            mbar_init(k_full + 8 * s, 1);
            mbar_init(s_full + 8 * s, 1);
        }
        for (int s = 0; s < A::NV; ++s) {
            mbar_init(v_full + 8 * s, 1);
            mbar_init(v_empty + 8 * s, 1);
        }
        for (int g = 0; g < 2; ++g) mbar_init(p_full + 8 * g, 128);
        mbar_init(in_full, 1);
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

    const int nbt = (fr.frame - fr.win_first + 1) * pl.BPF;      // key blocks of this frame's window
    const int nsplit = (nbt + pl.CH - 1) / pl.CH;
    // a CTA beyond the splits of its frame's window has nothing to do (uniform for the CTA): it skips the
    // roles below and leaves by the common exit
    const bool idle = split >= nsplit;
    const int b0 = split * pl.CH;
    const int nb = idle ? 0 : min(nbt, b0 + pl.CH) - b0;          // >= 1 unless idle
    const int Nq = nf_pass * D.T;

    if (idle) {
        // nothing
    } else if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            const int page_rows = D.H * D.T;
            uint8_t *sK = sKV, *sV = sKV + A::NK * A::KV_BYTES;
            bool waited = false, ok = true;
            auto need_q = [&]() {                // from here on the predecessor's output is needed
                if (waited) return;
                pdl_wait();
                NFD_TRACE_MARK(TRK_OTHER + 10);
                waited = true;
                mbar_expect_tx(q_full, A::Q_BYTES);
                tma_load_2d(smem_u32(sQ), &tmQ, q_full, 0, h * Nq + j * D.T + qt * 128);
            };
            auto row_of = [&](int b, bool &is_new) {
                const int blk = b0 + b;
                const int g = fr.win_first + blk / pl.BPF, kb = blk % pl.BPF;
                is_new = g >= fr.first_new;      // pages written by this pass; earlier ones are final already
                return ((fr.stream * D.L + layer) * D.R + (g % D.R)) * page_rows + h * D.T + kb * KB;
            };
            auto load_k = [&](int b) {
                bool is_new;
                const int row = row_of(b, is_new), st = b % A::NK;
                if (is_new || b >= A::NK) need_q();      // a stage is freed by an S product, which needs Q
                if (b >= A::NK && !mbar_wait(s_full + 8 * st, ((b / A::NK) - 1) & 1, status)) return false;
                mbar_expect_tx(k_full + 8 * st, A::KV_BYTES);
                tma_load_2d(smem_u32(sK + st * A::KV_BYTES), &tmK, k_full + 8 * st, 0, row);
                return true;
            };
            auto load_v = [&](int b) {
                bool is_new;
                const int row = row_of(b, is_new), st = b % A::NV;
                if (is_new || b >= A::NV) need_q();
                if (b >= A::NV && !mbar_wait(v_empty + 8 * st, ((b / A::NV) - 1) & 1, status)) return false;
                mbar_expect_tx(v_full + 8 * st, A::KV_BYTES);
                tma_load_2d(smem_u32(sV + st * A::KV_BYTES), &tmV, v_full + 8 * st, 0, row);
                return true;
            };
            // K runs ahead of V: K(b) is used three blocks before V(b)
            for (int b = 0; b < A::NK && b < nb && ok; ++b) ok = load_k(b);
            for (int b = 0; b < nb && ok; ++b) {
                ok = load_v(b);
                if (ok && b + A::NK < nb) ok = load_k(b + A::NK);
            }
            need_q();
        }
    } else if (warp == 1) {
        // ---------------- UMMA issuer ----------------
        if (lane == 0) {
            pdl_launch();
            constexpr uint32_t idesc_s = umma_idesc_bf16(128, KB);
            constexpr uint32_t idesc_pv = umma_idesc_bf16_bmn(128, 64);
            const uint64_t qd = umma_desc_k128(smem_u32(sQ));
            const uint32_t sK = smem_u32(sKV), sV = sK + A::NK * A::KV_BYTES;
            bool ok = mbar_wait(q_full, 0, status);
            auto issue_s = [&](int b) {          // S(b) = Q K(b)^T into accumulator b % 3
                const int st = b % A::NK;
                if (!mbar_wait(k_full + 8 * st, (b / A::NK) & 1, status)) return false;
                tc_fence_after();
                const uint64_t kd = umma_desc_k128(sK + st * A::KV_BYTES);
#pragma unroll
                for (int k4 = 0; k4 < 4; ++k4) umma_bf16_ss(tmem + 128 * st, qd + 2 * k4, kd + 2 * k4, idesc_s, k4 != 0);
                umma_commit(s_full + 8 * st);    // S(b) is ready; K's stage is free
                return true;
            };
            for (int b = 0; b < A::NK && b < nb && ok; ++b) ok = issue_s(b);
            for (int b = 0; b < nb && ok; ++b) {
                const int g = b & 1, sv = b % A::NV;
                ok = mbar_wait(p_full + 8 * g, (b >> 1) & 1, status) && mbar_wait(v_full + 8 * sv, (b / A::NV) & 1, status);
                if (!ok) break;
                if (b == 4) NFD_TRACE_MARK_T(TRK_OTHER + 6, 32);
                tc_fence_after();
                const uint64_t vd = umma_desc_k128(sV + sv * A::KV_BYTES);
                const uint32_t tP = tmem + 128 * (b % A::NK);
#pragma unroll
                for (int i = 0; i < KB / 16; ++i) {
                    // P: 16 keys = 8 columns of packed bf16 pairs; V: MN-major, 16 keys = 2 KiB per step
                    umma_bf16_ts(tmem + 384 + 64 * g, tP + 8 * i, vd + (uint64_t)(i * (2048 >> 4)), idesc_pv,
                                 (uint32_t)((b >> 1) != 0 || i != 0));
                }
                umma_commit(v_empty + 8 * sv);   // P V(b) is complete: V's stage is free, the group's O at rest
                if (b == 4) NFD_TRACE_MARK_T(TRK_OTHER + 7, 32);
                // the group has read S(b): its accumulator takes the block three ahead
                if (b + A::NK < nb) ok = issue_s(b + A::NK);
                if (b == 4) NFD_TRACE_MARK_T(TRK_OTHER + 8, 32);
            }
        }
    } else {
        // ---------------- softmax: one thread per query row, two groups ----------------
        const int g = (warp - 2) >> 2;                     // group: blocks b with (b & 1) == g
        const int quad = warp & 3;
        const int trow = quad * 32 + lane;
        const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
        const uint32_t tO = tmem + 384 + 64 * g + lane_off;
        const float c = (1.0f / sqrtf((float)D.dh)) * 1.4426950408889634f;   // softmax scale in the log2 domain
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        int i = 0;
        for (int b = g; b < nb; b += 2, ++i) {
            const uint32_t tS = tmem + 128 * (b % A::NK) + lane_off;
            ok = mbar_wait(s_full + 8 * (b % A::NK), (b / A::NK) & 1, status);
            if (!ok) break;
            tc_fence_after();
            if (i == 0) NFD_TRACE_MARK_T(TRK_OTHER + 11, 64);
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
            const bool raise = m_blk > m_run + 8.0f;       // always true for the first block (m_run = -inf)
            if (__any_sync(0xffffffffu, raise)) {
                const float m_new = raise ? m_blk : m_run;
                const float f = ex2_approx(m_run - m_new);  // 1 for rows that keep their reference maximum
                if (i > 0) {
                    // the previous P V product of this group must be complete before O is touched
                    ok = mbar_wait(v_empty + 8 * ((b - 2) % A::NV), ((b - 2) / A::NV) & 1, status);
                    if (!ok) break;
                    tc_fence_after();
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
            // pass 2 over S, 16 columns at a time with the next load in flight: P = exp2(S c - m) as packed bf16
            // pairs, written over the columns of S that have been read already (keys k .. k+15 go to columns
            // k/2 .. k/2+7, which never reach ahead of the columns still to be read)
            float2 ls2[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
            uint32_t sa[16], sb[16];
            tmem_ld16(tS, sa);
#pragma unroll
            for (int cc = 0; cc < KB; cc += 16) {
                uint32_t *cur = ((cc >> 4) & 1) ? sb : sa, *nxt = ((cc >> 4) & 1) ? sa : sb;
                tmem_ld_wait();
                if (cc + 16 < KB) tmem_ld16(tS + cc + 16, nxt);
                uint32_t pk[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const float2 y = ffma2(make_float2(__uint_as_float(cur[2 * u]), __uint_as_float(cur[2 * u + 1])),
                                           make_float2(c, c), make_float2(-m_run, -m_run));
                    const float p0 = ex2_approx(y.x), p1 = ex2_approx(y.y);
                    ls2[u & 3] = fadd2(ls2[u & 3], make_float2(p0, p1));
                    const __nv_bfloat162 hp = __floats2bfloat162_rn(p0, p1);
                    pk[u] = *reinterpret_cast<const uint32_t *>(&hp);
                }
                tmem_st8(tS + (cc >> 1), pk);
            }
            l_run += ((ls2[0].x + ls2[0].y) + (ls2[1].x + ls2[1].y)) + ((ls2[2].x + ls2[2].y) + (ls2[3].x + ls2[3].y));
            tmem_st_wait();                                // P is in tensor memory
            tc_fence_before();
            mbar_arrive(p_full + 8 * g);
        }
        NFD_TRACE_MARK_T(TRK_OTHER + 12, 64);
        // this group's O accumulator (unnormalised, relative to m_run)
        float O[64];
#pragma unroll
        for (int e = 0; e < 64; ++e) O[e] = 0.f;
        if (ok && i > 0) {
            const int bl = g + 2 * (i - 1);                  // this group's last block
            ok = mbar_wait(v_empty + 8 * (bl % A::NV), (bl / A::NV) & 1, status);
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
        // 16-byte word c of row r of a parked state
        auto park_word = [](uint8_t *base, int r, int c) { return reinterpret_cast<float4 *>(base + r * 256 + ((c ^ (r & 15)) << 4)); };
        // ---- the two groups of this CTA first: group 1 parks its state, group 0 folds it in ----
        named_bar_sync(1, 256);                            // both groups are past their last UMMA: P tiles and ring are free
        if (g == 1) {
#pragma unroll
            for (int e = 0; e < 64; e += 4) *park_word(parkO, trow, e >> 2) = make_float4(O[e], O[e + 1], O[e + 2], O[e + 3]);
            parkML[trow] = make_float2(m_run, l_run);
        }
        named_bar_sync(1, 256);
        float m_cta = m_run, l_cta = l_run;
        if (g == 0) {
            const float2 ml1 = parkML[trow];
            m_cta = fmaxf(m_run, ml1.x);
            const float w0 = ex2_approx(m_run - m_cta), w1 = ex2_approx(ml1.x - m_cta);
            l_cta = l_run * w0 + ml1.y * w1;
#pragma unroll
            for (int e = 0; e < 64; e += 4) {
                const float4 v = *park_word(parkO, trow, e >> 2);
                O[e] = fmaf(O[e], w0, v.x * w1), O[e + 1] = fmaf(O[e + 1], w0, v.y * w1);
                O[e + 2] = fmaf(O[e + 2], w0, v.z * w1), O[e + 3] = fmaf(O[e + 3], w0, v.w * w1);
            }
        }
        NFD_TRACE_MARK_T(TRK_OTHER + 13, 64);
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
            // state tiles in global memory: [query tile][split] x PARK_BYTES, laid out like the parked tile
            uint8_t *gstates = reinterpret_cast<uint8_t *>(part_o);
            const size_t st0 = item_q * pl.MAXSPLIT;
            if (g == 0) {
                // (each thread rewrites only the row it has just read)
#pragma unroll
                for (int e = 0; e < 64; e += 4) *park_word(parkO, trow, e >> 2) = make_float4(O[e], O[e + 1], O[e + 2], O[e + 3]);
                parkML[trow] = make_float2(m_cta, l_cta);
                fence_proxy_async_smem();                  // the bulk copy below reads what this thread wrote
            }
            named_bar_sync(1, 256);
            if (threadIdx.x == 64) {
                bulk_store_s2g(gstates + (st0 + split) * A::PARK_BYTES, smem_u32(parkO), A::PARK_BYTES);
                bulk_commit();
                bulk_wait_all();                           // the tile has been written
                __threadfence();
                const unsigned int prev = atomicAdd(counters + item_q, 1u);
                const int last = prev == (unsigned int)(nsplit - 1);
                if (last) {
                    counters[item_q] = 0;                  // ready for the next launch
                    __threadfence();
                }
                *last_flag = last;
            }
            NFD_TRACE_MARK_T(TRK_OTHER + 14, 64);
            named_bar_sync(1, 256);
            if (*last_flag) {
                // an item = 8 adjacent output columns of a row; four items per thread (256 threads, 128 x 8 items).
                // The other splits' states come in through the K/V ring, N_IN at a time; every item keeps a
                // running (max, sum, accumulator) and takes the splits in split order whatever N_IN is.
                const int et = (int)threadIdx.x - 64;
                float acc[4][8], l[4], mx[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    l[q] = 0.f, mx[q] = -INFINITY;
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[q][e] = 0.f;
                }
                uint32_t in_phase = 0;
                bool ok_in = true;
                for (int s0 = 0, s1 = 0; s0 < nsplit && ok_in; s0 = s1) {
                    // this round: splits s0 .. s1-1; the own split (if in range) is read from the parked tile
                    int n_in = 0;
                    while (s1 < nsplit && (n_in < A::N_IN || s1 == split)) n_in += (s1 != split), ++s1;
                    if (s0 > 0) named_bar_sync(1, 256);    // everyone is done reading the ring's previous contents
                    if (threadIdx.x == 64 && n_in > 0) {
                        fence_proxy_async_all();
                        mbar_expect_tx(in_full, (uint32_t)n_in * A::PARK_BYTES);
                        int slot = 0;
                        for (int sidx = s0; sidx < s1; ++sidx)
                            if (sidx != split)
                                bulk_load_g2s(smem_u32(sKV + (slot++) * A::PARK_BYTES), gstates + (st0 + sidx) * A::PARK_BYTES,
                                              A::PARK_BYTES, in_full);
                    }
                    if (n_in > 0) {
                        ok_in = mbar_wait(in_full, in_phase, status);
                        in_phase ^= 1;
                        if (!ok_in) break;
                    }
                    int slot = 0;
                    for (int sidx = s0; sidx < s1; ++sidx) {
                        uint8_t *base = sidx == split ? parkO : sKV + (slot++) * A::PARK_BYTES;
                        const float2 *bml = reinterpret_cast<const float2 *>(base + A::PARK_O_BYTES);
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const int it = et + q * 256, r = it >> 3, ch = it & 7;
                            const float2 ml = bml[r];
                            const float4 v0 = *park_word(base, r, 2 * ch), v1 = *park_word(base, r, 2 * ch + 1);
                            const float mb = fmaxf(mx[q], ml.x);
                            // (a state without any key has m = -inf, l = 0: it must count for nothing)
                            const float fo = mx[q] == mb ? 1.0f : ex2_approx(mx[q] - mb);
                            const float w = ml.x == -INFINITY ? 0.f : ex2_approx(ml.x - mb);
                            mx[q] = mb;
                            l[q] = fmaf(ml.y, w, l[q] * fo);
                            acc[q][0] = fmaf(v0.x, w, acc[q][0] * fo), acc[q][1] = fmaf(v0.y, w, acc[q][1] * fo);
                            acc[q][2] = fmaf(v0.z, w, acc[q][2] * fo), acc[q][3] = fmaf(v0.w, w, acc[q][3] * fo);
                            acc[q][4] = fmaf(v1.x, w, acc[q][4] * fo), acc[q][5] = fmaf(v1.y, w, acc[q][5] * fo);
                            acc[q][6] = fmaf(v1.z, w, acc[q][6] * fo), acc[q][7] = fmaf(v1.w, w, acc[q][7] * fo);
                        }
                    }
                }
                if (ok_in) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int it = et + q * 256, r = it >> 3, ch = it & 7;
                        if (qt * 128 + r < D.T) {
                            const float inv = 1.0f / l[q];
#pragma unroll
                            for (int u = 0; u < 8; ++u) acc[q][u] *= inv;
                            *reinterpret_cast<uint4 *>(out + (size_t)(j * D.T + qt * 128 + r) * D.d + h * 64 + ch * 8) =
                                pack_bf16x8(acc[q]);
                        }
                    }
                }
            }
        }
    }
    NFD_TRACE_MARK_T(TRK_OTHER + 16, 64);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, A::TMEM_COLS);
    NFD_TRACE_END(TRK_ATTN);
}

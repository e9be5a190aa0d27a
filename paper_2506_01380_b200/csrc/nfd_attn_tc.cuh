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
    static constexpr int NST = 4;                          // K/V ring stages
    static constexpr int Q_BYTES = 128 * 128;
    static constexpr int P_BYTES = 2 * 128 * 128;          // one group's P tile: two 64-key atoms
    static constexpr int KV_BYTES = KB * 128;              // one K (or V) block
    static constexpr int RING_BYTES = NST * 2 * KV_BYTES;
    // A parked state: 128 rows of 64 floats (256 bytes per row; the 16-byte words of row r are stored at
    // word index c ^ (r & 15), so that one thread per row writes without bank conflicts), then 128 x (m, l).
    static constexpr int PARK_O_BYTES = 128 * 256;
    static constexpr int PARK_BYTES = PARK_O_BYTES + 128 * 8;
    static constexpr int N_IN = RING_BYTES / PARK_BYTES;   // other splits' states that the K/V ring holds at once
    static constexpr int SMEM = Q_BYTES + 2 * P_BYTES + RING_BYTES + 1024 + 256;
    static constexpr int TMEM_COLS = 512;                  // S0 @0, S1 @128, O0 @256, O1 @320
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
    const uint32_t q_full = smem_u32(bars), kv_full = smem_u32(bars + 1), kv_empty = smem_u32(bars + 1 + A::NST),
                   s_full = smem_u32(bars + 1 + 2 * A::NST), p_full = s_full + 16, pv_done = s_full + 32,
                   in_full = s_full + 48, stagger = s_full + 56;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 1 + 2 * A::NST + 8);
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
        for (int s = 0; s < A::NST; ++s) {
            mbar_init(kv_full + 8 * s, 1);
            mbar_init(kv_empty + 8 * s, 1);
        }
        for (int g = 0; g < 2; ++g) {
            mbar_init(s_full + 8 * g, 1);
            mbar_init(p_full + 8 * g, 128);
            mbar_init(pv_done + 8 * g, 1);
        }
        mbar_init(in_full, 1);
        mbar_init(stagger, 128);
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
            bool waited = false;
            for (int b = 0; b < nb; ++b) {
                const int s = b % A::NST;
                const int blk = b0 + b;
                const int g = fr.win_first + blk / pl.BPF, kb = blk % pl.BPF;
                // pages of frames written earlier than this pass may be fetched before the predecessor finishes
                if (!waited && (g >= fr.first_new || b >= A::NST)) {
                    pdl_wait();
                    NFD_TRACE_MARK(TRK_OTHER + 10);
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
            // The two groups share each scheduler's special-function unit.  Started together they stay in step:
            // both wait for their S at the same time and both exponentiate at the same time, at half the
            // rate each.  Group 1's first S is therefore issued only when group 0 is half way through its
            // first block, which puts the groups in opposite phases: one exponentiates while the other waits.
            if (ok) ok = issue_s(0);
            if (ok && nb > 1) ok = mbar_wait(stagger, 0, status) && issue_s(1);
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
                if (cc == (KB / 32) * 16 && g == 0 && i == 0) mbar_arrive(stagger);     // see the UMMA issuer
#pragma unroll
                for (int u2 = 0; u2 < 2; ++u2) {
                    uint32_t pk[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float2 y = ffma2(make_float2(__uint_as_float(cur[8 * u2 + 2 * u]),
                                                           __uint_as_float(cur[8 * u2 + 2 * u + 1])),
                                               make_float2(c, c), make_float2(-m_run, -m_run));
                        const float p0 = ex2_approx(y.x), p1 = ex2_approx(y.y);
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
        NFD_TRACE_MARK_T(TRK_OTHER + 12, 64);
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

// Tensor-core GEMM of libnfd (bf16 operands, fp32 accumulation in tensor memory).
//
//   C[M,N] = A[M,K] * Wt[N,K]^T  followed by a fused epilogue functor.
//
// The projections of one forward pass have M = (frames in the pass) x (tokens per
// frame): 336 rows at batch 1.  Such a GEMM is a few microseconds of work and is
// bound by the rate and latency with which operand tiles reach an SM, so the
// kernel is built around latency:
//   - one CTA per 128 x BN output tile and K range; the K range of a tile is
//     split over the S CTAs of a thread-block cluster (S = 1, 2 or 4), which
//     keeps 148 SMs busy with 3 row tiles and shortens every CTA's chain of
//     dependent loads;
//   - each CTA parks its partial accumulator in its own shared memory; after a
//     cluster barrier CTA r reads rows [r*128/S, (r+1)*128/S) of all S partials
//     through distributed shared memory, sums them in split order
//     (deterministic) and runs the epilogue for those rows;
//   - warp 0 = TMA producer, warp 1 = tensor-memory allocation + UMMA issue,
//     warps 2-9 = accumulator read-out and epilogue (two warps per TMEM lane
//     quadrant, each taking half of the columns);
//   - programmatic dependent launch: barrier set-up, tensor-memory allocation and
//     the first weight tiles (which never depend on the previous kernel) are
//     issued before the wait on the predecessor grid; the epilogue's side inputs
//     (bias, gate, residual, rotary table) are fetched while the UMMAs run;
//   - every CTA also pulls a slice of the NEXT GEMM's weights towards L2, so that
//     the weight stream from HBM runs one kernel ahead of its use.
// One CTA fills an SM (its operand ring is sized for that): with programmatic
// dependent launch CTAs are placed wherever there is room at that moment, and
// two small CTAs piling onto one SM while others stay empty costs more than it
// gains.
#pragma once
#include "nfd_sm100.cuh"

template <int BN> struct GemmCfg {
    // ring deep enough that one CTA owns an SM; the wide tiles (passes of several frames) keep about the same
    // number of bytes in flight with fewer, larger stages
    static constexpr int STAGES = BN <= 32 ? 7 : (BN <= 128 ? 6 : (BN <= 192 ? 4 : 3));
    static constexpr int A_BYTES = 128 * 128;                  // 128 rows x 64 bf16
    static constexpr int B_BYTES = BN * 128;
    static constexpr int RING_BYTES = STAGES * (A_BYTES + B_BYTES);
    static constexpr int SROW = BN + 4;                        // staging row stride (floats)
    static constexpr int STAGE_BYTES = 128 * SROW * 4;         // partial accumulator tile; reuses the ring
    static constexpr int TMEM_COLS = BN <= 32 ? 32 : (BN <= 64 ? 64 : (BN <= 128 ? 128 : 256));
    static constexpr int UV_BYTES = LnFold::kMaxFrames * BN * 8;   // folded LayerNorm: (u, v) per frame and column
    static constexpr int TAB_BYTES = 128 * 16 + (BN / 8) * 32 + 128;   // epilogue row and column tables, row -> frame
    static constexpr int SMEM = RING_BYTES + 1024 /*align*/ + 256 /*barriers*/ + 1024 /*row statistics*/ + UV_BYTES +
                                TAB_BYTES;
    static constexpr int THREADS = 320;
    static constexpr int EPI_THREADS = 256;
    static constexpr int MAX_S = 4;                            // largest cluster split
    static constexpr int MIN_CTAS = 1;
    static_assert(STAGE_BYTES <= RING_BYTES, "staging tile must fit the operand ring");
};

// A byte range that the CTAs of a launch pull towards L2 (the next GEMM's weights).
struct L2Prefetch {
    const void *ptr;
    unsigned long long bytes;      // multiple of 16; 0 = nothing
};

// SC: the split factor when it is known at compile time (1: no cluster; the epilogue then works on four items at
// a time instead of two, which gives its dependent instruction chains more to overlap with), 0: run-time S.
template <int BN, typename Epi, int SC = 0>
__global__ void __launch_bounds__(GemmCfg<BN>::THREADS, GemmCfg<BN>::MIN_CTAS)
k_gemm_tc(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, int M, int N, int K,
          int S_rt, Epi epi, L2Prefetch pf, int *status) {
    using G = GemmCfg<BN>;
    const int S = SC ? SC : S_rt;
    constexpr int GRP = SC == 1 ? 4 : 2;                     // epilogue items finished together
    constexpr int NS = SC == 1 ? 1 : G::MAX_S;               // partials kept per item
    constexpr int MAX_ITEMS = Epi::kBatch;                   // epilogue items in flight together per thread
    extern __shared__ uint8_t smem_raw[];
    NFD_TRACE_T0();
    // blockIdx.x = n_tile * S + split; the S splits of a tile form one cluster
    const int split = blockIdx.x % S, n_tile = blockIdx.x / S;
    const int m0 = blockIdx.y * 128, n0 = n_tile * BN;
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *sA = smem, *sB = smem + G::STAGES * G::A_BYTES;
    float *stage = reinterpret_cast<float *>(smem);          // reuses the ring once the UMMAs are done
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + G::RING_BYTES);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + G::STAGES),
                   accf = smem_u32(bars + 2 * G::STAGES);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * G::STAGES + 1);
    float2 *rowstat = reinterpret_cast<float2 *>(smem + G::RING_BYTES + 256);   // (mean, rstd) of the tile's rows
    float4 *uvs = reinterpret_cast<float4 *>(smem + G::RING_BYTES + 256 + 1024); // (u, v): [frame of the tile][BN]
    static_assert(sizeof(typename Epi::Row) <= 16 && sizeof(typename Epi::Col) <= 32, "epilogue tables");
    uint8_t *tab_raw = smem + G::RING_BYTES + 256 + 1024 + G::UV_BYTES;
    // rows at a stride of 16 bytes from tab_raw, column chunks at a stride of 32 bytes after them
    uint8_t *rowfr = tab_raw + 128 * 16 + (BN / 8) * 32;     // frame of a tile row, relative to the tile's first frame
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nkb_all = (K + 63) / 64;
    const int kb0 = (int)((long long)nkb_all * split / S), kb1 = (int)((long long)nkb_all * (split + 1) / S);
    const int nkb = kb1 - kb0;
    const int rows_per = 128 / S;                            // rows of the tile this CTA finishes

    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
        for (int s = 0; s < G::STAGES; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(accf, 1);
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), G::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // epilogue state that lives across the cluster barrier (used by warps 2-9 only)
    constexpr int CPR = BN / 8;                              // 8-column chunks per row
    const int et = (int)threadIdx.x - 64;                    // 0..255 for the epilogue warps
    const int n_items = rows_per * CPR;                      // items of this CTA's row slice
    const int r_base = (S > 1 ? (int)cluster_ctarank() : 0) * rows_per;   // first tile row of the slice
    typename Epi::Side side[MAX_ITEMS];
    int uv_f0 = 0;                                           // first frame of the tile (folded LayerNorm)
    if constexpr (Epi::kRowStats) uv_f0 = m0 / epi.ln.T;

    if (warp == 0) {
        if (lane == 0) {
            // weights never depend on the previous kernel: fill the ring's weight halves first
            const int pre = nkb < G::STAGES ? nkb : G::STAGES;
            for (int kb = 0; kb < pre; ++kb) {
                mbar_expect_tx(full0 + 8 * kb, G::A_BYTES + G::B_BYTES);
                tma_load_2d(smem_u32(sB + kb * G::B_BYTES), &tmB, full0 + 8 * kb, (kb0 + kb) * 64, n0);
            }
            // test switch (see nfd_sm100.cuh): leave out the last stage, so that the wait for it runs out
            const int skip_last = *reinterpret_cast<volatile int *>(status + 2);
            pdl_wait();
            NFD_TRACE_MARK(TRK_OTHER + 1);
            for (int kb = 0; kb < pre; ++kb) {
                if (skip_last && kb == nkb - 1) continue;      // its weight half has landed; the stage stays incomplete
                tma_load_2d(smem_u32(sA + kb * G::A_BYTES), &tmA, full0 + 8 * kb, (kb0 + kb) * 64, m0);
            }
            for (int kb = pre; kb < nkb; ++kb) {
                if (skip_last && kb == nkb - 1) break;
                const int s = kb % G::STAGES;
                if (!mbar_wait(empty0 + 8 * s, ((kb / G::STAGES) - 1) & 1, status)) break;
                mbar_expect_tx(full0 + 8 * s, G::A_BYTES + G::B_BYTES);
                tma_load_2d(smem_u32(sA + s * G::A_BYTES), &tmA, full0 + 8 * s, (kb0 + kb) * 64, m0);
                tma_load_2d(smem_u32(sB + s * G::B_BYTES), &tmB, full0 + 8 * s, (kb0 + kb) * 64, n0);
            }
        } else if (lane == 1) {
            // this CTA's slice of the next GEMM's weights, towards L2 in 8 KiB pieces, and whatever the
            // epilogue functor knows the next kernel will read
            const unsigned long long n_cta = (unsigned long long)gridDim.x * gridDim.y;
            const unsigned long long cta = (unsigned long long)blockIdx.y * gridDim.x + blockIdx.x;
            epi.prefetch((unsigned int)cta, (unsigned int)n_cta);
            const unsigned long long per = ((pf.bytes / n_cta + 15) / 16 + 1) * 16;
            unsigned long long b = cta * per, e = b + per;
            if (e > pf.bytes) e = pf.bytes;
            if (!pf.bytes) b = e = 0;
            for (; b < e; b += 8192) {
                const unsigned long long n = e - b < 8192 ? e - b : 8192;
                bulk_prefetch_l2(reinterpret_cast<const uint8_t *>(pf.ptr) + b, (uint32_t)n);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            pdl_launch();
            constexpr uint32_t idesc = umma_idesc_bf16(128, BN);
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % G::STAGES;
                if (!mbar_wait(full0 + 8 * s, (kb / G::STAGES) & 1, status)) break;
                tc_fence_after();
                if (kb == 0) NFD_TRACE_MARK_T(TRK_OTHER + 5, 32);
                if (kb == nkb - 1) NFD_TRACE_MARK_T(TRK_OTHER + 6, 32);
                const uint64_t ad = umma_desc_k128(smem_u32(sA + s * G::A_BYTES));
                const uint64_t bd = umma_desc_k128(smem_u32(sB + s * G::B_BYTES));
#pragma unroll
                for (int k4 = 0; k4 < 4; ++k4)
                    umma_bf16_ss(tmem_base, ad + 2 * k4, bd + 2 * k4, idesc, (kb | k4) != 0);
                umma_commit(empty0 + 8 * s);
            }
            umma_commit(accf);          // arrives when every UMMA above has completed
        }
    } else {
        pdl_wait();
        // side inputs of the first items (bias, gate, residual, rotary table), fetched while the UMMAs run
#pragma unroll
        for (int i = 0; i < MAX_ITEMS; ++i) {
            const int it = et + i * G::EPI_THREADS;
            if (it < n_items) {
                const int m = m0 + r_base + it / CPR, n = n0 + (it % CPR) * 8;
                if (m < M && n < N) epi.load(m, n, side[i]);
            }
        }
        if constexpr (Epi::kTables) {
            // where the rows and the column chunks of this CTA's slice go
            if (et < rows_per && m0 + r_base + et < M)
                *reinterpret_cast<typename Epi::Row *>(tab_raw + (r_base + et) * 16) = epi.row_info(m0 + r_base + et);
            if (et >= 128 && et < 128 + CPR && n0 + (et - 128) * 8 < N)
                *reinterpret_cast<typename Epi::Col *>(tab_raw + 128 * 16 + (et - 128) * 32) =
                    epi.col_info(n0 + (et - 128) * 8);
        }
        if constexpr (Epi::kRowStats) {
            if (epi.ln.on()) {
                // folded LayerNorm: (u, v) of the tile's columns for every frame the tile's rows belong to, and
                // (mean, rstd) of the rows this CTA finishes, from the producer's partial sums
                const int m_last = (m0 + 127 < M ? m0 + 127 : M - 1);
                const int n_fr = m_last / epi.ln.T - uv_f0 + 1;
                // layout [frame][pair of columns within a chunk][chunk]: the lanes of a warp, which hold adjacent
                // chunks, read adjacent 16-byte words
                for (int idx = et; idx < n_fr * (BN / 2); idx += G::EPI_THREADS) {
                    const int fr = idx / (BN / 2), c2 = idx - fr * (BN / 2);
                    if (n0 + 2 * c2 < N)
                        uvs[(fr * 4 + (c2 & 3)) * CPR + (c2 >> 2)] = epi.ln.uv_pair(uv_f0 + fr, n0 + 2 * c2);
                }
                if (et < rows_per) {
                    const int m = m0 + r_base + et;
                    rowfr[r_base + et] = (uint8_t)((m < M ? m : M - 1) / epi.ln.T - uv_f0);
                }
                // 8 lanes per row, 32 rows per sweep; every load is issued before the first sum
                constexpr int SWEEPS = 128 / (G::EPI_THREADS / 8);
                const int sub = et & 7;
                float2 pv[SWEEPS][4];
#pragma unroll
                for (int w = 0; w < SWEEPS; ++w) {
                    const int r = (et >> 3) + w * (G::EPI_THREADS / 8);
                    const int m = (r < rows_per && m0 + r_base + r < M) ? m0 + r_base + r : -1;
#pragma unroll
                    for (int u = 0; u < 4; ++u) pv[w][u] = epi.ln.part(m, sub + 8 * u);
                }
#pragma unroll
                for (int w = 0; w < SWEEPS; ++w) {
                    const int r = (et >> 3) + w * (G::EPI_THREADS / 8);
                    float s1 = 0.f, s2 = 0.f;
#pragma unroll
                    for (int u = 0; u < 4; ++u) s1 += pv[w][u].x, s2 += pv[w][u].y;
                    if (epi.ln.npart > 32) {              // rows wider than 1024
                        const int m = (r < rows_per && m0 + r_base + r < M) ? m0 + r_base + r : -1;
                        for (int i = sub + 32; i < epi.ln.npart; i += 8) {
                            const float2 t = epi.ln.part(m, i);
                            s1 += t.x, s2 += t.y;
                        }
                    }
#pragma unroll
                    for (int o = 1; o < 8; o <<= 1) {
                        s1 += __shfl_xor_sync(0xffffffffu, s1, o);
                        s2 += __shfl_xor_sync(0xffffffffu, s2, o);
                    }
                    if (sub == 0 && r < rows_per) rowstat[r_base + r] = epi.ln.finish(s1, s2);
                }
            }
        }
        // partial accumulator: tensor memory -> this CTA's staging tile (the ring is free by now)
        const int quad = warp & 3;                           // TMEM lane quadrant this warp may read
        const int half = (warp - 2) >> 2;                    // which half of the columns
        const int row = quad * 32 + lane;                    // tile row held by this thread
        if (mbar_wait(accf, 0, status)) {
            tc_fence_after();
            NFD_TRACE_MARK_T(TRK_OTHER + 2, 64);
            float *srow = stage + (size_t)row * G::SROW;
            constexpr int HC = BN / 2;                       // columns per half
#pragma unroll
            for (int c = 0; c < HC; c += 16) {
                uint32_t r[16];
                tmem_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + half * HC + c, r);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 16; j += 4)
                    *reinterpret_cast<uint4 *>(srow + half * HC + c + j) = make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]);
            }
        }
    }
    tc_fence_before();
    __syncwarp();
    if (S > 1)
        cluster_sync_all();              // every CTA of the cluster has parked its partial tile
    else
        __syncthreads();
    NFD_TRACE_MARK_T(TRK_OTHER + 3, 64);
    if (warp >= 2) {
        // Items in batches of MAX_ITEMS: first every side input of the batch is requested, then the items are
        // finished two at a time: all loads of the S partials of the pair (remote ones come through distributed
        // shared memory and take long), the sum in split order, the fused epilogue (8 adjacent columns per item).
        const uint32_t stage_u32 = smem_u32(stage);
        for (int i0 = 0; i0 * G::EPI_THREADS < n_items; i0 += MAX_ITEMS) {
            int mm[MAX_ITEMS], nn[MAX_ITEMS], tr[MAX_ITEMS];
            unsigned vmask[MAX_ITEMS];
#pragma unroll
            for (int i = 0; i < MAX_ITEMS; ++i) {
                const int it = et + (i0 + i) * G::EPI_THREADS;
                tr[i] = r_base + it / CPR;
                mm[i] = m0 + tr[i], nn[i] = n0 + (it % CPR) * 8;
                if (it >= n_items || mm[i] >= M || nn[i] >= N)
                    mm[i] = -1;
                else if (i0 > 0)
                    epi.load(mm[i], nn[i], side[i]);
                vmask[i] = __ballot_sync(0xffffffffu, mm[i] >= 0);
            }
#pragma unroll
            for (int j0 = 0; j0 < MAX_ITEMS; j0 += GRP) {
                float4 u0[GRP][NS], u1[GRP][NS];
#pragma unroll
                for (int jj = 0; jj < GRP; ++jj) {
                    const int i = j0 + jj;
                    if (i >= MAX_ITEMS || mm[i] < 0) continue;
                    const uint32_t off = (uint32_t)(tr[i] * G::SROW + (nn[i] - n0)) * 4;
                    if (S == 1) {
                        const float *p = stage + (size_t)tr[i] * G::SROW + (nn[i] - n0);
                        u0[jj][0] = *reinterpret_cast<const float4 *>(p), u1[jj][0] = *reinterpret_cast<const float4 *>(p + 4);
                    } else {
#pragma unroll
                        for (int sp_ = 0; sp_ < NS; ++sp_) {
                            if (sp_ < S) {
                                const uint32_t ra = cluster_map(stage_u32 + off, (uint32_t)sp_);
                                u0[jj][sp_] = ld_cluster_f4(ra), u1[jj][sp_] = ld_cluster_f4(ra + 16);
                            }
                        }
                    }
                }
#pragma unroll
                for (int jj = 0; jj < GRP; ++jj) {
                    const int i = j0 + jj;
                    if (i >= MAX_ITEMS || mm[i] < 0) continue;
                    float4 v0 = u0[jj][0], v1 = u1[jj][0];
#pragma unroll
                    for (int sp_ = 1; sp_ < NS; ++sp_) {
                        if (sp_ < S) {
                            v0.x += u0[jj][sp_].x, v0.y += u0[jj][sp_].y, v0.z += u0[jj][sp_].z, v0.w += u0[jj][sp_].w;
                            v1.x += u1[jj][sp_].x, v1.y += u1[jj][sp_].y, v1.z += u1[jj][sp_].z, v1.w += u1[jj][sp_].w;
                        }
                    }
                    float a[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
                    float2 ms = make_float2(0.f, 1.f);
                    const float4 *uvp = nullptr;
                    if constexpr (Epi::kRowStats) {
                        if (epi.ln.on()) {
                            ms = rowstat[tr[i]];
                            uvp = uvs + (int)rowfr[tr[i]] * 4 * CPR + ((nn[i] - n0) >> 3);   // planes CPR words apart
                        }
                    }
                    typename Epi::Row rinfo{};
                    typename Epi::Col cinfo{};
                    if constexpr (Epi::kTables) {
                        rinfo = *reinterpret_cast<const typename Epi::Row *>(tab_raw + tr[i] * 16);
                        cinfo = *reinterpret_cast<const typename Epi::Col *>(tab_raw + 128 * 16 + ((nn[i] - n0) >> 3) * 32);
                    }
                    epi.apply(mm[i], nn[i], a, side[i], ms, uvp, CPR, vmask[i], rinfo, cinfo);
                }
                if (i0 == 0 && j0 == 0) NFD_TRACE_MARK_T(TRK_OTHER + 7, 64);
            }
        }
    }
    NFD_TRACE_MARK_T(TRK_OTHER + 4, 64);
    tc_fence_before();
    if (S > 1) {
        cluster_arrive_relaxed();        // no CTA leaves while a peer may still read its partial tile
        cluster_wait();
    } else {
        __syncthreads();
    }
    if (warp == 1) tmem_dealloc(tmem_base, G::TMEM_COLS);
    NFD_TRACE_END(TRK_GEMM + 16 * (int)(K > 2048) + 32 * (int)(N / 1024));
}

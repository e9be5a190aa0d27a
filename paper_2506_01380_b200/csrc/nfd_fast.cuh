// Tensor-core path of libnfd (bf16 only): tcgen05/TMEM GEMM fed by TMA with the
// fused epilogues of nfd_kernels.cuh, and the dispatch hooks used by
// nfd_api.cu.  fast_gemm / fast_attention return false when they do not handle
// a case; the caller then launches the plain kernels.
#pragma once
#include <map>
#include <tuple>

#include "nfd_sm100.cuh"
#include "nfd_attn_tc.cuh"

enum { TC_NONE = 0, TC_QKV = 1, TC_RES = 2, TC_GELU = 3 };

typedef CUresult (*PFN_encodeTiled)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct FastState {
    bool ready = false;
    PFN_encodeTiled encode = nullptr;
    int *d_status = nullptr;
    int n_sm = 148;
    size_t a_rows = 0;     // rows of every activation buffer (NFD_MAX_PASS_FRAMES * T)
    AttnPlan plan;         // KB == 0: tensor-core attention not available for this shape
    float *part_o = nullptr;
    float2 *part_ml = nullptr;
    size_t cache_rows = 0;
    std::map<std::tuple<const void *, int, int, int>, CUtensorMap> maps;   // (ptr, rows, cols, box_rows)
};

static int fast_create(FastState &fs, const Dims &D, bool bf16_mode, cudaStream_t st, int *d_status) {
    (void)st;
    fs.ready = false;
    fs.d_status = d_status;
    fs.a_rows = (size_t)NFD_MAX_PASS_FRAMES * D.T;
    if (!bf16_mode) return NFD_OK;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess) {
        cudaGetLastError();
        fprintf(stderr, "libnfd: cuTensorMapEncodeTiled is unavailable; tensor-core path disabled\n");
        return NFD_OK;
    }
    fs.encode = (PFN_encodeTiled)fn;
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&fs.n_sm, cudaDevAttrMultiProcessorCount, dev);
    fs.ready = true;
    // attention plan: head_dim 64, key blocks that divide the tokens per frame
    AttnPlan pl;
    const int KB = D.T % 128 == 0 ? 128 : (D.T % 112 == 0 ? 112 : (D.T % 64 == 0 ? 64 : 0));
    fs.cache_rows = (size_t)D.n_streams * D.L * D.R * D.H * D.T;
    if (D.dh == 64 && KB && D.H * D.T >= 128 && fs.cache_rows < 0x7fffffffull) {
        pl.KB = KB;
        pl.BPF = D.T / KB;
        pl.QT = (D.T + 127) / 128;
        const int target = fs.n_sm / (D.H * pl.QT) > 1 ? fs.n_sm / (D.H * pl.QT) : 1;
        pl.CH = ((D.W + 1) * pl.BPF + target - 1) / target;
        pl.MAXSPLIT = (D.R * pl.BPF + pl.CH - 1) / pl.CH;
        const size_t items = (size_t)NFD_MAX_PASS_FRAMES * D.H * pl.QT * pl.MAXSPLIT * 128;
        if (cudaMalloc((void **)&fs.part_o, items * 64 * sizeof(float)) != cudaSuccess ||
            cudaMalloc((void **)&fs.part_ml, items * sizeof(float2)) != cudaSuccess) {
            cudaGetLastError();
            return NFD_E_NOMEM;
        }
        fs.plan = pl;
    }
    return NFD_OK;
}

static void fast_destroy(FastState &fs) {
    fs.maps.clear();
    if (fs.part_o) cudaFree(fs.part_o);
    if (fs.part_ml) cudaFree(fs.part_ml);
    fs.part_o = nullptr, fs.part_ml = nullptr;
    fs.ready = false;
}

// 2D bf16 tensor map [rows][cols], box = 64 columns (128 bytes) x box_rows, 128-byte swizzle.
static const CUtensorMap *get_map_2d(FastState &fs, const void *ptr, int rows, int cols, int box_rows) {
    auto key = std::make_tuple(ptr, rows, cols, box_rows);
    auto it = fs.maps.find(key);
    if (it != fs.maps.end()) return &it->second;
    CUtensorMap m;
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstr[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fs.encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), gdim, gstr, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        fprintf(stderr, "libnfd: cuTensorMapEncodeTiled failed (%d) for [%d x %d] box %d\n", (int)r, rows, cols,
                box_rows);
        return nullptr;
    }
    return &fs.maps.emplace(key, m).first->second;
}

// ---------------------------------------------------------------------------
// C[M,N] = A[M,K] * Wt[N,K]^T, bf16 in, fp32 accumulation in tensor memory.
// One CTA per 128 x BN output tile.  Warp 0: TMA producer; warp 1: TMEM
// allocation and UMMA issue; warps 2-5: epilogue (TMEM -> registers -> fused
// epilogue functor).  K is walked in 64-element blocks through a STAGES-deep
// shared-memory ring guarded by full/empty mbarriers.
// ---------------------------------------------------------------------------
template <int BN> struct GemmCfg {
    static constexpr int STAGES = BN <= 32 ? 8 : (BN <= 128 ? 6 : 4);
    static constexpr int A_BYTES = 128 * 128;
    static constexpr int B_BYTES = BN * 128;
    static constexpr int TMEM_COLS = BN < 32 ? 32 : BN;
    static constexpr int SMEM = STAGES * (A_BYTES + B_BYTES) + 1024 /*align*/ + 256 /*barriers*/;
};

template <int BN, typename Epi>
__global__ void __launch_bounds__(192, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const StepParams *sp,
          int T, int N, int K, Epi epi, int *status) {
    using G = GemmCfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    const int M = sp->nf * T;
    const int m0 = blockIdx.y * 128, n0 = blockIdx.x * BN;
    if (m0 >= M) return;                                    // uniform for the CTA, before any barrier or allocation
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *sA = smem, *sB = smem + G::STAGES * G::A_BYTES;
    uint64_t *bars = reinterpret_cast<uint64_t *>(sB + G::STAGES * G::B_BYTES);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + G::STAGES),
                   accf = smem_u32(bars + 2 * G::STAGES);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * G::STAGES + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nkb = (K + 63) / 64;
    constexpr int SROW = BN + 4;                         // staging row stride in floats
    float *stage = reinterpret_cast<float *>(smem);      // 128 x SROW floats, reuses the operand ring
    static_assert(128 * (BN + 4) * 4 <= G::STAGES * (G::A_BYTES + G::B_BYTES), "staging tile must fit the ring");

    if (warp == 0 && lane == 0) {
        for (int s = 0; s < G::STAGES; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(accf, 1);
        fence_mbar_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), G::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % G::STAGES;
                if (kb >= G::STAGES && !mbar_wait(empty0 + 8 * s, ((kb / G::STAGES) - 1) & 1, status)) break;
                mbar_expect_tx(full0 + 8 * s, G::A_BYTES + G::B_BYTES);
                tma_load_2d(smem_u32(sA + s * G::A_BYTES), &tmA, full0 + 8 * s, kb * 64, m0);
                tma_load_2d(smem_u32(sB + s * G::B_BYTES), &tmB, full0 + 8 * s, kb * 64, n0);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, BN);
            bool ok = true;
            for (int kb = 0; kb < nkb && ok; ++kb) {
                const int s = kb % G::STAGES;
                ok = mbar_wait(full0 + 8 * s, (kb / G::STAGES) & 1, status);
                if (!ok) break;
                tc_fence_after();
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
        // accumulators: TMEM -> registers -> shared memory (the operand ring is free by now)
        const int quad = warp & 3;      // TMEM lane quadrant this warp may read
        const int row = quad * 32 + lane;
        if (mbar_wait(accf, 0, status)) {
            tc_fence_after();
            float *srow = stage + (size_t)row * SROW;
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                uint32_t r[32];
                tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + c, r);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                    *reinterpret_cast<uint4 *>(srow + c + j) = make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    // fused epilogue from shared memory: 8 adjacent columns per thread, rows coalesced
    {
        constexpr int CPR = BN / 8;     // chunks per row
        for (int ch = threadIdx.x; ch < 128 * CPR; ch += 192) {
            const int row = ch / CPR, cc = ch % CPR;
            const int m = m0 + row, n = n0 + cc * 8;
            if (m < M && n < N) {
                const float4 *sp4 = reinterpret_cast<const float4 *>(stage + (size_t)row * SROW + cc * 8);
                const float4 v0 = sp4[0], v1 = sp4[1];
                float a[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
                epi.vec8(m, n, a);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, G::TMEM_COLS);
}

template <int BN, typename Epi>
static bool launch_gemm_tc(FastState &fs, cudaStream_t st, const StepParams *sp, int T, const bf16 *A, const bf16 *Wt,
                           int M, int N, int K, Epi epi) {
    using G = GemmCfg<BN>;
    static bool attr_set = false;
    auto kern = k_gemm_tc<BN, Epi>;
    if (!attr_set) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM) != cudaSuccess) {
            cudaGetLastError();
            return false;
        }
        attr_set = true;
    }
    const CUtensorMap *ma = get_map_2d(fs, A, (int)fs.a_rows, K, 128);
    const CUtensorMap *mb = get_map_2d(fs, Wt, N, K, BN);
    if (!ma || !mb) return false;
    dim3 grid((N + BN - 1) / BN, (M + 127) / 128);
    kern<<<grid, 192, G::SMEM, st>>>(*ma, *mb, sp, T, N, K, epi, fs.d_status);
    return true;
}

template <typename TS, typename Epi>
static bool fast_gemm(bool enabled, FastState &fs, cudaStream_t st, const StepParams *sp, int T, const TS *A,
                      const TS *Wt, int M, int N, int K, Epi epi, int tc_kind) {
    (void)tc_kind;
    if constexpr (!std::is_same<TS, bf16>::value) {
        return false;
    } else {
        if (!enabled || !fs.ready) return false;
        if (K % 8 || K < 64 || N < 32 || (N & 7)) return false;
        if (((uintptr_t)A & 15) || ((uintptr_t)Wt & 15)) return false;
        // largest tile that still gives every SM (about) one CTA
        const int mt = (M + 127) / 128;
        const int want = fs.n_sm * 4 / 5;
        if (N >= 256 && mt * ((N + 255) / 256) >= want) return launch_gemm_tc<256, Epi>(fs, st, sp, T, A, Wt, M, N, K, epi);
        if (N >= 128 && mt * ((N + 127) / 128) >= want) return launch_gemm_tc<128, Epi>(fs, st, sp, T, A, Wt, M, N, K, epi);
        if (N >= 64 && mt * ((N + 63) / 64) >= want) return launch_gemm_tc<64, Epi>(fs, st, sp, T, A, Wt, M, N, K, epi);
        return launch_gemm_tc<32, Epi>(fs, st, sp, T, A, Wt, M, N, K, epi);
    }
}

template <int KB>
static int launch_attn_tc(FastState &fs, cudaStream_t st, const StepParams *sp, const Dims &D, int nf, int layer,
                          const bf16 *q, const bf16 *kc, const bf16 *vc, bf16 *out) {
    using A = AttnCfg<KB>;
    static bool attr_set = false;
    auto kern = k_attn_tc<KB>;
    if (!attr_set) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, A::SMEM) != cudaSuccess) {
            cudaGetLastError();
            return 0;
        }
        attr_set = true;
    }
    const CUtensorMap *mq = get_map_2d(fs, q, D.H * nf * D.T, 64, 128);
    const CUtensorMap *mk = get_map_2d(fs, kc, (int)fs.cache_rows, 64, KB);
    const CUtensorMap *mv = get_map_2d(fs, vc, (int)fs.cache_rows, 64, KB);
    if (!mq || !mk || !mv) return 0;
    const AttnPlan &pl = fs.plan;
    dim3 grid(pl.MAXSPLIT, pl.QT, nf * D.H);
    kern<<<grid, 192, A::SMEM, st>>>(*mq, *mk, *mv, sp, D, layer, pl, out, fs.part_o, fs.part_ml, fs.d_status);
    if (pl.MAXSPLIT == 1) return 1;
    k_attn_combine<<<dim3(pl.QT, nf * D.H), 128, 0, st>>>(sp, D, pl, fs.part_o, fs.part_ml, out);
    return 2;
}

// Returns the number of kernels launched (0: not handled, use the plain kernel).
template <typename TS>
static int fast_attention(bool enabled, FastState &fs, cudaStream_t st, const StepParams *sp, const Dims &D, int nf,
                          int layer, const TS *q, const TS *kc, const TS *vc, TS *out) {
    if constexpr (!std::is_same<TS, bf16>::value) {
        return 0;
    } else {
        if (!enabled || !fs.ready || fs.plan.KB == 0) return 0;
        if (fs.plan.KB == 128) return launch_attn_tc<128>(fs, st, sp, D, nf, layer, q, kc, vc, out);
        if (fs.plan.KB == 112) return launch_attn_tc<112>(fs, st, sp, D, nf, layer, q, kc, vc, out);
        return launch_attn_tc<64>(fs, st, sp, D, nf, layer, q, kc, vc, out);
    }
}

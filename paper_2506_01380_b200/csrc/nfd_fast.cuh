// Tensor-core path of libnfd (bf16 only): tcgen05/TMEM GEMM fed by TMA with the
// fused epilogues of nfd_kernels.cuh, and the dispatch hooks used by
// nfd_api.cu.  fast_gemm / fast_attention return false when they do not handle
// a case; the caller then launches the plain kernels.
#pragma once
#include <map>
#include <tuple>
#include <utility>

#include "nfd_sm100.cuh"
#include "nfd_gemm_tc.cuh"
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
    float *part_o = nullptr;           // per-split states of the attention kernel: [query tile][split] x PARK_BYTES
    unsigned int *attn_counters = nullptr;   // one per (frame, head, query tile); zero between launches
    size_t cache_rows = 0;
    std::map<std::tuple<const void *, int, int, int>, CUtensorMap> maps;   // (ptr, rows, cols, box_rows)
    int force_BN = 0, force_S = 0;     // set while candidates are being timed
    int slots[5] = {0, 0, 0, 0, 0};    // CTAs of a GEMM that can be resident at once, by cluster size (1, 2, 4)
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
        // no silent change of path: without tensor maps a bf16 context would run the plain validation kernels
        cudaGetLastError();
        fprintf(stderr, "libnfd: the driver does not provide cuTensorMapEncodeTiled; a bf16 context needs it\n");
        return NFD_E_CUDA;
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
        // split the longest window (a frame sees at most W + 1 pages) so that streams x heads x query tiles x
        // splits fills the SMs once: a context made for several streams is run with batched passes, which bring
        // enough (frame, head, query tile) items by themselves, and long unsplit key ranges amortise the
        // start and the merge of a CTA.  The split depends on the configuration only, never on the pass.
        const int items_per_pass = D.n_streams * D.H * pl.QT;
        const int target = fs.n_sm / items_per_pass > 1 ? fs.n_sm / items_per_pass : 1;
        pl.CH = ((D.W + 1) * pl.BPF + target - 1) / target;
        pl.MAXSPLIT = ((D.W + 1) * pl.BPF + pl.CH - 1) / pl.CH;
        if (pl.MAXSPLIT > 1) {
            const size_t tiles = (size_t)NFD_MAX_PASS_FRAMES * D.H * pl.QT;
            if (cudaMalloc((void **)&fs.part_o, tiles * pl.MAXSPLIT * (size_t)AttnCfg<64>::PARK_BYTES) != cudaSuccess ||
                cudaMalloc((void **)&fs.attn_counters, tiles * sizeof(unsigned int)) != cudaSuccess ||
                cudaMemset(fs.attn_counters, 0, tiles * sizeof(unsigned int)) != cudaSuccess) {
                cudaGetLastError();
                return NFD_E_NOMEM;
            }
        }
        fs.plan = pl;
    }
    return NFD_OK;
}

static void fast_destroy(FastState &fs) {
    fs.maps.clear();
    if (fs.part_o) cudaFree(fs.part_o);
    if (fs.attn_counters) cudaFree(fs.attn_counters);
    fs.part_o = nullptr, fs.attn_counters = nullptr;
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
// Kernel launch with programmatic stream serialisation (and an optional cluster
// along x).  Works the same under stream capture.
// ---------------------------------------------------------------------------
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              int cluster_x, Args &&...args) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid, cfg.blockDim = block, cfg.dynamicSmemBytes = smem, cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int na = 0;
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
    if (cluster_x > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = (unsigned)cluster_x, attr[na].val.clusterDim.y = 1, attr[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.attrs = attr, cfg.numAttrs = (unsigned)na;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

// ---------------------------------------------------------------------------
// Tile width BN and cluster split S of a GEMM [M x N x K].
// ---------------------------------------------------------------------------
struct GemmPlan {
    int BN, S;
};
// Plans found by timing (nfd_create), shared by every context of the process so that two contexts of the same
// shape always sum in the same order: (kind, N, K, n_sm) -> S, and (kind, N, K, n_sm, M) -> BN.
static std::map<std::tuple<int, int, int, int>, int> g_tuned_S;
static std::map<std::tuple<int, int, int, int, int>, int> g_tuned_BN;

// CTAs that can be resident at once: one per SM, less what clusters cannot use (a cluster lives inside one
// GPC).  Asked of the runtime at create (on a 148-SM B200: 148 for clusters of 1 and 2, 132 for clusters of
// 4); the fallback figures are those.
static int gemm_slots(const FastState &fs, int S) {
    if (S >= 1 && S <= 4 && fs.slots[S] > 0) return fs.slots[S];
    if (S >= 4) return (fs.n_sm / 4 - 4) * 4;
    return fs.n_sm;
}
template <typename Kern> static void query_gemm_slots(FastState &fs, Kern kern, int smem, int threads) {
    for (int cs = 1; cs <= 4; cs *= 2) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(fs.n_sm / cs * cs), cfg.blockDim = dim3(threads), cfg.dynamicSmemBytes = (size_t)smem;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = cs, at[0].val.clusterDim.y = 1, at[0].val.clusterDim.z = 1;
        cfg.attrs = at, cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) == cudaSuccess && n > 0)
            fs.slots[cs] = n * cs < fs.n_sm ? n * cs : fs.n_sm;
        else
            cudaGetLastError();
    }
}

static GemmPlan plan_gemm(const FastState &fs, int M, int N, int K, int tc_kind) {
    if (fs.force_BN) return {fs.force_BN, fs.force_S};
    const int kind_key = tc_kind + (K > 2048 ? 10 : 0);
    {
        auto is = g_tuned_S.find(std::make_tuple(kind_key, N, K, fs.n_sm));
        auto ib = g_tuned_BN.find(std::make_tuple(kind_key, N, K, fs.n_sm, M));
        if (is != g_tuned_S.end() && ib != g_tuned_BN.end()) return {ib->second, is->second};
    }
    // Cost in SM cycles, fitted to measurements on B200: an SM takes in operand tiles at about
    // 55 bytes per cycle whatever the ring depth; CTAs that share an SM share that rate.
    // The split S is chosen for a one-frame pass (M = tokens per frame) and then kept for every M:
    // the order in which the K range is summed, and with it every bit of the result, must not
    // depend on how many frames share a pass.  Only the tile width follows M.
    const int nkb = (K + 63) / 64;
    auto cost_of = [&](int m_rows, int BN, int S) {
        const int mt = (m_rows + 127) / 128, nt = (N + BN - 1) / BN;
        const long long ctas = (long long)mt * nt * S;
        const int slots = gemm_slots(fs, S);
        const double waves = (double)((ctas + slots - 1) / slots);
        const double share = 1.0;
        const double kb = (double)((nkb + S - 1) / S);
        const double load = kb * (16384.0 + BN * 128.0) / 55.0 * share;
        const double items = (128.0 / S) * (BN / 8.0) / 256.0;                 // epilogue items per thread
        // with S > 1 every pair of items waits for the partials of the S - 1 other CTAs (distributed shared
        // memory: a slow round trip per pair, longer the more peers are asked)
        const double pairs = (double)(((int)(items + 0.999) + 1) / 2);
        const double epi = 400.0 + items * 350.0 + (S - 1) * (pairs * 1000.0 + 300.0) + BN * 4.0;
        const double fixed = 3200.0 + (S > 1 ? 500.0 : 0.0);
        return waves * (fixed + load + epi);
    };
    const int bns[4] = {32, 64, 96, 128};
    const int T = (int)(fs.a_rows / NFD_MAX_PASS_FRAMES);
    int S_best = 1;
    double best_cost = 1e30;
    for (int bi = 0; bi < 4; ++bi) {
        if (bns[bi] > 32 && bns[bi] > N) continue;
        for (int S = 1; S <= GemmCfg<64>::MAX_S; S *= 2) {
            if (S > 1 && nkb / S < 2) break;
            const double c = cost_of(T, bns[bi], S);
            if (c < best_cost) best_cost = c, S_best = S;
        }
    }
    {
        // a split found by timing binds the model too (sizes of M that were not timed)
        auto is = g_tuned_S.find(std::make_tuple(kind_key, N, K, fs.n_sm));
        if (is != g_tuned_S.end()) S_best = is->second;
    }
    GemmPlan best{32, S_best};
    best_cost = 1e30;
    // the tile width follows M; passes of several frames may take the wide tiles
    const int bnw[6] = {32, 64, 96, 128, 192, 256};
    for (int bi = 0; bi < 6; ++bi) {
        if (bnw[bi] > 32 && bnw[bi] > N) continue;
        const double c = cost_of(M, bnw[bi], S_best);
        if (c < best_cost) best_cost = c, best.BN = bnw[bi];
    }
    return best;
}

template <int BN, typename Epi, int SC>
static bool launch_gemm_tc_sc(FastState &fs, cudaStream_t st, const bf16 *A, const bf16 *Wt, int M, int N, int K, int S,
                              Epi epi, L2Prefetch pf) {
    using G = GemmCfg<BN>;
    static bool attr_set = false;
    auto kern = k_gemm_tc<BN, Epi, SC>;
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
    dim3 grid(((N + BN - 1) / BN) * S, (M + 127) / 128);
    cudaError_t e = launch_pdl(kern, grid, dim3(G::THREADS), (size_t)G::SMEM, st, S, *ma, *mb, M, N, K, S, epi, pf,
                               fs.d_status);
    if (e != cudaSuccess) {
        fprintf(stderr, "libnfd: tensor-core GEMM launch failed (BN %d, S %d): %s\n", BN, S, cudaGetErrorString(e));
        cudaGetLastError();
        return false;
    }
    return true;
}

// the unsplit case has a kernel of its own (see k_gemm_tc)
template <int BN, typename Epi>
static bool launch_gemm_tc(FastState &fs, cudaStream_t st, const bf16 *A, const bf16 *Wt, int M, int N, int K, int S,
                           Epi epi, L2Prefetch pf) {
    if (S == 1) return launch_gemm_tc_sc<BN, Epi, 1>(fs, st, A, Wt, M, N, K, S, epi, pf);
    return launch_gemm_tc_sc<BN, Epi, 0>(fs, st, A, Wt, M, N, K, S, epi, pf);
}

template <typename TS, typename Epi>
static bool fast_gemm(bool enabled, FastState &fs, cudaStream_t st, const TS *A, const TS *Wt, int M, int N, int K,
                      Epi epi, int tc_kind, L2Prefetch pf) {
    if constexpr (!std::is_same<TS, bf16>::value) {
        return false;
    } else {
        if (!enabled || !fs.ready) return false;
        if (K % 8 || K < 64 || N < 32 || (N & 7)) return false;
        if (((uintptr_t)A & 15) || ((uintptr_t)Wt & 15)) return false;
        const GemmPlan pl = plan_gemm(fs, M, N, K, tc_kind);
        switch (pl.BN) {
            case 256: return launch_gemm_tc<256, Epi>(fs, st, A, Wt, M, N, K, pl.S, epi, pf);
            case 192: return launch_gemm_tc<192, Epi>(fs, st, A, Wt, M, N, K, pl.S, epi, pf);
            case 128: return launch_gemm_tc<128, Epi>(fs, st, A, Wt, M, N, K, pl.S, epi, pf);
            case 96: return launch_gemm_tc<96, Epi>(fs, st, A, Wt, M, N, K, pl.S, epi, pf);
            case 64: return launch_gemm_tc<64, Epi>(fs, st, A, Wt, M, N, K, pl.S, epi, pf);
            default: return launch_gemm_tc<32, Epi>(fs, st, A, Wt, M, N, K, pl.S, epi, pf);
        }
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
    cudaError_t e = launch_pdl(kern, grid, dim3(A::THREADS), (size_t)A::SMEM, st, 1, *mq, *mk, *mv, sp, D, layer, pl, out,
                               fs.part_o, fs.attn_counters, fs.d_status);
    if (e != cudaSuccess) {
        fprintf(stderr, "libnfd: tensor-core attention launch failed: %s\n", cudaGetErrorString(e));
        cudaGetLastError();
        return 0;
    }
    return 1;
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

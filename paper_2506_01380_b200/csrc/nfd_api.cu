// libnfd host side: context, weight repacking, frame-paged KV cache bookkeeping,
// pass construction, CUDA-graph capture / replay and the C ABI of include/nfd.h.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <map>
#include <new>
#include <vector>

#include "nfd_kernels.cuh"
#include "nfd_fast.cuh"

#define CK(call)                                                                                   \
    do {                                                                                           \
        cudaError_t e_ = (call);                                                                   \
        if (e_ != cudaSuccess) {                                                                   \
            fprintf(stderr, "libnfd: %s failed: %s (%s:%d)\n", #call, cudaGetErrorString(e_),      \
                    __FILE__, __LINE__);                                                           \
            return NFD_E_CUDA;                                                                     \
        }                                                                                          \
    } while (0)

#define RET(expr)                  \
    do {                           \
        int r_ = (expr);           \
        if (r_ != NFD_OK) return r_; \
    } while (0)

struct GraphEntry {
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    cudaGraphNode_t param_node = nullptr;
    long long launches = 0;
};

struct nfd_ctx {
    nfd_cfg cfg;
    Dims D;
    cudaStream_t st = nullptr;
    bool bf16_mode = false;
    size_t esz = 4;
    bool use_graph = true, fast = true;
    long long launches = 0;
    cudaError_t launch_err = cudaSuccess;    // first failed launch since the last take_launch_err()
    // test switches (nfd_set_option "test_*"): each acts on the next call only
    bool test_fail_launch = false;           // the next sampler launch gets a block size the runtime refuses
    bool test_corrupt_desc = false;          // the next pass descriptor names a batch slot that does not exist
    int test_words[4] = {0, 0, 0, 0};        // host copies of the status block's test words (sources of async copies)
    bool l2_prefetch = true;                 // GEMMs pull the next GEMM's weights towards L2
    bool kv_prefetch = false;                // the QKV GEMM pulls the layer's cached K/V pages towards L2
    std::vector<void *> allocs;

    // repacked weights: matrices [out][in], storage type
    void *w_pe_io = nullptr;                    // patch embedding in its [P][d] layout
    void *w_pe = nullptr, *b_pe = nullptr, *w_t1 = nullptr, *b_t1 = nullptr, *w_t2 = nullptr, *b_t2 = nullptr;
    void *a_emb = nullptr, *w_fmod = nullptr, *b_fmod = nullptr, *w_out = nullptr, *b_out = nullptr;
    std::vector<void *> w_mod, b_mod, w_qkv, b_qkv, w_o, b_o, w_fc1, b_fc1, w_fc2, b_fc2;
    // device arrays of pointers for the GEMV kernels
    void **dp_wmod = nullptr, **dp_bmod = nullptr, **dp_t1 = nullptr, **dp_t2 = nullptr, **dp_fmod = nullptr;
    void **dp_wqkv = nullptr, **dp_bqkv = nullptr, **dp_wfc1 = nullptr, **dp_bfc1 = nullptr;
    RopeTab *d_rope = nullptr;

    void *kc = nullptr, *vc = nullptr;          // [n_streams][L][R][H][T][dh]
    float *z = nullptr;                         // residual stream [Nq_max][d]
    void *hbuf = nullptr, *qbuf = nullptr, *abuf = nullptr, *mbuf = nullptr;
    float *emb = nullptr, *h1 = nullptr, *sc = nullptr, *mod = nullptr, *fmod = nullptr;
    float *xp = nullptr, *vbuf = nullptr;       // sampler state, velocity
    float *x0_prev = nullptr;                   // previous data prediction of the multistep ODE sampler
    float2 *rope_cs = nullptr;                  // per-pass RoPE table [Nq_max][dh/2]
    StepParams *d_sp = nullptr;
    StepParams h_sp;
    unsigned long long *d_hash = nullptr;
    int *d_status = nullptr;                // status block of four ints (see nfd_sm100.cuh)
    DescLimits lim;
    FastState fs;

    std::vector<int> n_committed, n_tentative;
    // Deferred commits: the newest n_pending[s] frames of stream s are counted above but their K/V pages are
    // not written yet; their clean latents, context noise and actions wait in pend_* until the next
    // speculation carries them along in its first pass (or until something needs the pages).
    bool lazy = true;
    std::vector<int> n_pending;
    std::vector<std::vector<int>> pend_act;
    float *pend_x0 = nullptr, *pend_cz = nullptr;     // [n_streams][k_max][C,H,W]
    // Modulation cache: the adaLN modulation depends on (FM time, action) only, so each pair is computed
    // once and kept in one of n_slots rows of `mod` / `fmod`; least recently used rows are replaced.
    struct CondSlot {
        unsigned t_bits = 0;
        int action = -1;
        long long last_use = -1;
    };
    std::vector<CondSlot> cond_slots;
    // Folded LayerNorm (tensor-core path): the in-layer adaLN kernels are replaced by work in the epilogues
    // of the neighbouring GEMMs.  uvtab holds, per cache slot and layer, the (u, v) pairs of the QKV and
    // first MLP projections; ln_stats the row-sum partials of z.
    bool fuse_ln = true;
    float2 *uvtab = nullptr;                    // [n_slots][L][3d + n1]
    float2 *ln_stats = nullptr;                 // [Nq_max][d / 32]
    bool fold_active() const {
        const int d = D.d, dm = D.dm;
        // (a 128-row GEMM tile must not span more frames than the kernel keeps (u, v) rows for)
        return fuse_ln && fast && bf16_mode && fs.ready && d % 32 == 0 && d >= 64 && dm % 8 == 0 && dm >= 64 &&
               127 / D.T + 2 <= LnFold::kMaxFrames;
    }
    long long pass_no = 0, cond_hits = 0, cond_misses = 0;
    std::map<int, GraphEntry> graphs;

    // per-kernel-class timing (nfd_profile_begin / nfd_profile_end)
    bool prof = false;
    int cls = 0;
    std::vector<cudaEvent_t> prof_ev;       // pairs: start, stop
    std::vector<int> prof_cls;
    size_t prof_used = 0;

    size_t frame_elems() const { return (size_t)cfg.latent_c * cfg.latent_h * cfg.latent_w; }
    int n_total(int s) const { return n_committed[s] + n_tentative[s]; }
};

// ---------------------------------------------------------------------------
static int dev_alloc(nfd_ctx *c, void **p, size_t bytes) {
    *p = nullptr;
    if (bytes == 0) bytes = 16;
    cudaError_t e = cudaMalloc(p, bytes);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return NFD_E_NOMEM;
    }
    c->allocs.push_back(*p);
    return NFD_OK;
}

template <typename TS>
static int repack_matrix(nfd_ctx *c, const void *src, int n_in, int n_out, void **dst, bool transpose) {
    if (!src) return NFD_E_NULLPTR;
    RET(dev_alloc(c, dst, (size_t)n_in * n_out * sizeof(TS)));
    if (transpose) {
        dim3 grid((n_out + 31) / 32, (n_in + 31) / 32), block(32, 8);
        k_transpose<TS><<<grid, block, 0, c->st>>>((const TS *)src, (TS *)*dst, n_in, n_out);
        CK(cudaGetLastError());
    } else {
        CK(cudaMemcpyAsync(*dst, src, (size_t)n_in * n_out * sizeof(TS), cudaMemcpyDeviceToDevice, c->st));
    }
    return NFD_OK;
}

template <typename TS> static int repack_all(nfd_ctx *c, const nfd_weights *w) {
    const nfd_cfg &g = c->cfg;
    const int d = g.d_model, P = c->D.P, L = g.n_layers, dm = g.d_mlp;
    const int dmp = c->D.dm, n1 = c->D.n1, act = c->D.act;
    RET(repack_matrix<TS>(c, w->w_pe, P, d, &c->w_pe, true));
    RET(repack_matrix<TS>(c, w->w_pe, P, d, &c->w_pe_io, false));
    RET(repack_matrix<TS>(c, w->b_pe, 1, d, &c->b_pe, false));
    RET(repack_matrix<TS>(c, w->w_t1, 256, d, &c->w_t1, true));
    RET(repack_matrix<TS>(c, w->b_t1, 1, d, &c->b_t1, false));
    RET(repack_matrix<TS>(c, w->w_t2, d, d, &c->w_t2, true));
    RET(repack_matrix<TS>(c, w->b_t2, 1, d, &c->b_t2, false));
    RET(repack_matrix<TS>(c, w->a_emb, g.n_actions, d, &c->a_emb, false));
    RET(repack_matrix<TS>(c, w->w_fmod, d, 2 * d, &c->w_fmod, true));
    RET(repack_matrix<TS>(c, w->b_fmod, 1, 2 * d, &c->b_fmod, false));
    RET(repack_matrix<TS>(c, w->w_out, d, P, &c->w_out, true));
    RET(repack_matrix<TS>(c, w->b_out, 1, P, &c->b_out, false));
    if (!w->w_mod || !w->b_mod || !w->w_qkv || !w->b_qkv || !w->w_o || !w->b_o || !w->w_fc1 || !w->b_fc1 ||
        !w->w_fc2 || !w->b_fc2)
        return NFD_E_NULLPTR;
    c->w_mod.resize(L), c->b_mod.resize(L), c->w_qkv.resize(L), c->b_qkv.resize(L), c->w_o.resize(L);
    c->b_o.resize(L), c->w_fc1.resize(L), c->b_fc1.resize(L), c->w_fc2.resize(L), c->b_fc2.resize(L);
    for (int l = 0; l < L; ++l) {
        RET(repack_matrix<TS>(c, w->w_mod[l], d, 6 * d, &c->w_mod[l], true));
        RET(repack_matrix<TS>(c, w->b_mod[l], 1, 6 * d, &c->b_mod[l], false));
        RET(repack_matrix<TS>(c, w->w_qkv[l], d, 3 * d, &c->w_qkv[l], true));
        RET(repack_matrix<TS>(c, w->b_qkv[l], 1, 3 * d, &c->b_qkv[l], false));
        RET(repack_matrix<TS>(c, w->w_o[l], d, d, &c->w_o[l], true));
        RET(repack_matrix<TS>(c, w->b_o[l], 1, d, &c->b_o[l], false));
        // MLP: hidden width padded to dmp with zero weights; gate and up columns of the gated form interleaved
        if (!w->w_fc1[l] || !w->b_fc1[l] || !w->w_fc2[l]) return NFD_E_NULLPTR;
        RET(dev_alloc(c, &c->w_fc1[l], (size_t)n1 * d * sizeof(TS)));
        RET(dev_alloc(c, &c->b_fc1[l], (size_t)n1 * sizeof(TS)));
        RET(dev_alloc(c, &c->w_fc2[l], (size_t)d * dmp * sizeof(TS)));
        k_repack_fc1<TS><<<(unsigned)(((size_t)n1 * d + 255) / 256), 256, 0, c->st>>>((const TS *)w->w_fc1[l],
                                                                                      (TS *)c->w_fc1[l], d, dm, dmp, act);
        k_repack_fc1<TS><<<(n1 + 255) / 256, 256, 0, c->st>>>((const TS *)w->b_fc1[l], (TS *)c->b_fc1[l], 1, dm, dmp, act);
        k_repack_fc2<TS><<<(unsigned)(((size_t)d * dmp + 255) / 256), 256, 0, c->st>>>((const TS *)w->w_fc2[l],
                                                                                       (TS *)c->w_fc2[l], d, dm, dmp);
        CK(cudaGetLastError());
        RET(repack_matrix<TS>(c, w->b_fc2[l], 1, d, &c->b_fc2[l], false));
    }
    return NFD_OK;
}

static int upload_ptrs(nfd_ctx *c, const std::vector<void *> &v, void ***dst) {
    RET(dev_alloc(c, (void **)dst, v.size() * sizeof(void *)));
    CK(cudaMemcpyAsync(*dst, v.data(), v.size() * sizeof(void *), cudaMemcpyHostToDevice, c->st));
    CK(cudaStreamSynchronize(c->st));
    return NFD_OK;
}

static int validate_cfg(const nfd_cfg &g) {
    if (g.n_layers < 1 || g.d_model < 128 || g.d_model > 8192 || g.d_model % 128) return NFD_E_BADCFG;
    if (g.n_heads < 1 || g.n_heads * g.head_dim != g.d_model) return NFD_E_BADCFG;
    if (g.head_dim != 32 && g.head_dim != 64 && g.head_dim != 128) return NFD_E_BADCFG;
    if (g.d_mlp < 2 || g.d_mlp % 2) return NFD_E_BADCFG;
    if (g.latent_c < 1 || g.latent_h < 1 || g.latent_w < 1 || g.patch < 1) return NFD_E_BADCFG;
    if (g.latent_h % g.patch || g.latent_w % g.patch) return NFD_E_BADCFG;
    int P = g.latent_c * g.patch * g.patch;
    if (P % 2 || P > 512) return NFD_E_BADCFG;
    if ((size_t)g.latent_c * g.latent_h * g.latent_w % 4) return NFD_E_BADCFG;
    if (g.n_actions < 1 || g.ctx_frames < 0 || g.ctx_frames > 4096) return NFD_E_BADCFG;
    if (g.max_spec < 1 || g.max_spec > 8) return NFD_E_BADCFG;
    if (g.n_streams < 1 || g.n_streams > 1024) return NFD_E_BADCFG;
    if (g.dtype != NFD_DTYPE_FP32 && g.dtype != NFD_DTYPE_BF16) return NFD_E_BADCFG;
    if (g.norm != 0 && g.norm != 1) return NFD_E_BADCFG;
    if (g.act != 0 && g.act != 1) return NFD_E_BADCFG;
    if (g.rope_t < 0 || g.rope_h < 0 || g.rope_w < 0 || (g.rope_t | g.rope_h | g.rope_w) & 1) return NFD_E_BADCFG;
    if (g.rope_t + g.rope_h + g.rope_w != g.head_dim) return NFD_E_BADCFG;
    if (!(g.rope_theta > 0.f) || !(g.norm_eps > 0.f) || !(g.sigma_d > 0.f)) return NFD_E_BADCFG;
    if (!(g.t_ctx_trig >= 0.f) || !(g.t_ctx_trig < 1.5707963f)) return NFD_E_BADCFG;
    if (g.n_steps < 1 || g.n_steps > 64) return NFD_E_BADCFG;
    return NFD_OK;
}

static bool aligned16(const void *p) { return ((uintptr_t)p & 15) == 0; }

// ---------------------------------------------------------------------------
// One forward pass, enqueued on the context's stream.
// ---------------------------------------------------------------------------
#define NFD_COND_SLOTS 256      // rows of the modulation cache (> NFD_MAX_PASS_FRAMES)

enum { CLS_PARAMS = 0, CLS_COND, CLS_PATCH, CLS_ADALN, CLS_GEMM_QKV, CLS_ATTN, CLS_GEMM_O, CLS_GEMM_FC1,
       CLS_GEMM_FC2, CLS_HEAD, CLS_SAMPLER, CLS_CACHE, CLS_COUNT };
static const char *const kClassNames[CLS_COUNT] = {"params", "conditioning", "patch_embed", "adaln_norm",
                                                   "gemm_qkv_rope_kvstore", "attention", "gemm_out_gate_res",
                                                   "gemm_fc1_gelu", "gemm_fc2_gate_res", "velocity_head",
                                                   "sampler", "cache_util"};

static void prof_mark(nfd_ctx *c, bool stop) {
    if (!c->prof) return;
    if (!stop) {
        if (c->prof_used + 2 > c->prof_ev.size()) {
            for (int i = 0; i < 2; ++i) {
                cudaEvent_t e;
                cudaEventCreate(&e);
                c->prof_ev.push_back(e);
            }
        }
        c->prof_cls.resize(c->prof_ev.size() / 2);
        c->prof_cls[c->prof_used / 2] = c->cls;
        cudaEventRecord(c->prof_ev[c->prof_used], c->st);
    } else {
        cudaEventRecord(c->prof_ev[c->prof_used + 1], c->st);
        c->prof_used += 2;
    }
}

#define LAUNCH(c, kern, grid, block, smem, ...)                 \
    do {                                                        \
        prof_mark((c), false);                                  \
        kern<<<grid, block, smem, (c)->st>>>(__VA_ARGS__);      \
        prof_mark((c), true);                                   \
        (c)->launches++;                                        \
    } while (0)

// Kernels of a forward pass: launched with programmatic stream serialisation, so
// that each one's prologue overlaps the tail of its predecessor.  Every such
// kernel calls pdl_wait() before it touches global memory.
#define PLAUNCH(c, kern, grid, block, smem, ...)                                                    \
    do {                                                                                            \
        prof_mark((c), false);                                                                      \
        cudaError_t le_ = launch_pdl(kern, dim3(grid), dim3(block), (size_t)(smem), (c)->st, 1, __VA_ARGS__); \
        if (le_ != cudaSuccess && !(c)->launch_err) (c)->launch_err = le_;                          \
        prof_mark((c), true);                                                                       \
        (c)->launches++;                                                                            \
    } while (0)

// The first launch error recorded since the last call of this function; the record is cleared, so that one
// refused launch fails the call it belongs to and nothing after it.
static cudaError_t take_launch_err(nfd_ctx *c) {
    cudaError_t e = c->launch_err;
    c->launch_err = cudaSuccess;
    if (e == cudaSuccess) e = cudaGetLastError();
    else cudaGetLastError();
    return e;
}

template <typename TS, typename Epi>
static void launch_gemm(nfd_ctx *c, const TS *A, const TS *Wt, int M, int N, int K, Epi epi, int tc_kind,
                        const void *next_w = nullptr, size_t next_elems = 0, bool folded = false) {
    prof_mark(c, false);
    // the next GEMM's weights, pulled towards L2 by this launch
    const L2Prefetch pf{next_w, next_w && c->l2_prefetch ? (unsigned long long)(next_elems * sizeof(TS)) & ~15ull : 0ull};
    if (fast_gemm<TS, Epi>(c->fast && c->bf16_mode, c->fs, c->st, A, Wt, M, N, K, epi, tc_kind, pf)) {
        prof_mark(c, true);
        c->launches++;
        return;
    }
    if (folded) {
        // the plain kernel knows nothing of the folded LayerNorm: fail the pass rather than compute garbage
        fprintf(stderr, "libnfd: tensor-core GEMM unavailable for a pass with folded LayerNorm\n");
        if (!c->launch_err) c->launch_err = cudaErrorNotSupported;
        return;
    }
    dim3 grid((N + 63) / 64, (M + 63) / 64);
    PLAUNCH(c, (k_gemm_simple<TS, Epi>), grid, 256, 0, (const StepParams *)c->d_sp, c->D.T, A, Wt, N, K, epi);
}

template <typename TS> static void launch_attention(nfd_ctx *c, int nf, int layer) {
    const Dims &D = c->D;
    c->cls = CLS_ATTN;
    prof_mark(c, false);
    const int n_fast = fast_attention<TS>(c->fast && c->bf16_mode, c->fs, c->st, c->d_sp, D, nf, layer,
                                          (const TS *)c->qbuf, (const TS *)c->kc, (const TS *)c->vc, (TS *)c->abuf);
    if (n_fast > 0) {
        prof_mark(c, true);
        c->launches += n_fast;
        return;
    }
    long long warps = (long long)nf * D.T * D.H;
    int grid = (int)((warps + 3) / 4);
    if (D.dh == 32)
        PLAUNCH(c, (k_attn_simple<TS, 32>), grid, 128, 0, (const StepParams *)c->d_sp, D, layer, (const TS *)c->qbuf,
                (const TS *)c->kc, (const TS *)c->vc, (TS *)c->abuf);
    else if (D.dh == 64)
        PLAUNCH(c, (k_attn_simple<TS, 64>), grid, 128, 0, (const StepParams *)c->d_sp, D, layer, (const TS *)c->qbuf,
                (const TS *)c->kc, (const TS *)c->vc, (TS *)c->abuf);
    else
        PLAUNCH(c, (k_attn_simple<TS, 128>), grid, 128, 0, (const StepParams *)c->d_sp, D, layer, (const TS *)c->qbuf,
                (const TS *)c->kc, (const TS *)c->vc, (TS *)c->abuf);
}

// Conditioning kernels for the c->h_sp.nc (time, action) pairs that the pass found missing in the
// modulation cache; `rows` bounds their number (grid of the embedding kernel).
template <typename TS> static void enqueue_conditioning(nfd_ctx *c, int rows) {
    const Dims &D = c->D;
    const int d = D.d, L = D.L, nf = rows;
    const StepParams *sp = c->d_sp;
    const size_t mod_row = (size_t)L * 6 * d;
    const size_t uv_row = (size_t)L * (3 * d + D.n1);
    const bool fold = c->fold_active();
    c->cls = CLS_COND;
    {
        PLAUNCH(c, k_temb, nf, 128, 0, sp, D.t_scale, c->emb);
        PLAUNCH(c, (k_gemv<TS, GEMV_T1>), dim3((d + 7) / 8, 1), 256, 0, sp, (const TS *const *)c->dp_t1,
                (const TS *const *)(c->dp_t1 + 1), (const TS *)nullptr, (const float *)c->emb, c->h1, 256, d, (size_t)d,
                (size_t)0);
        PLAUNCH(c, (k_gemv<TS, GEMV_T2>), dim3((d + 7) / 8, 1), 256, 0, sp, (const TS *const *)c->dp_t2,
                (const TS *const *)(c->dp_t2 + 1), (const TS *)c->a_emb, (const float *)c->h1, c->sc, d, d, (size_t)d,
                (size_t)0);
        PLAUNCH(c, (k_gemv<TS, GEMV_MOD>), dim3((6 * d + 7) / 8, L), 256, 0, sp, (const TS *const *)c->dp_wmod,
                (const TS *const *)c->dp_bmod, (const TS *)nullptr, (const float *)c->sc, c->mod, d, 6 * d, mod_row,
                (size_t)6 * d);
        PLAUNCH(c, (k_gemv<TS, GEMV_MOD>), dim3((2 * d + 7) / 8, 1), 256, 0, sp, (const TS *const *)c->dp_fmod,
                (const TS *const *)(c->dp_fmod + 1), (const TS *)nullptr, (const float *)c->sc, c->fmod, d, 2 * d,
                (size_t)2 * d, (size_t)0);
        if (fold)
            PLAUNCH(c, (k_modw<TS>), dim3((3 * d + D.n1 + MODW_OUT - 1) / MODW_OUT, L), 256, 0, sp, (const TS *const *)c->dp_wqkv,
                    (const TS *const *)c->dp_bqkv, (const TS *const *)c->dp_wfc1, (const TS *const *)c->dp_bfc1,
                    (const float *)c->mod, mod_row, c->uvtab, uv_row, d, D.n1);
    }
}

// Kernels after k_set_params.  nf and kind are fixed per captured graph.
template <typename TS> static void enqueue_body(nfd_ctx *c, int nf, int kind) {
    const Dims &D = c->D;
    const int d = D.d, L = D.L, M = nf * D.T;
    const StepParams *sp = c->d_sp;
    const size_t mod_row = (size_t)L * 6 * d;
    const size_t uv_row = (size_t)L * (3 * d + D.n1);
    const bool fold = c->fold_active();
    // conditioning: only for the (t, action) pairs that are not in the modulation cache
    if (c->h_sp.nc > 0) enqueue_conditioning<TS>(c, nf);
    // tokens
    c->cls = CLS_PATCH;
    // (the tensor-core QKV epilogue reads the rotary table that the patch embedding writes on the side)
    PLAUNCH(c, (k_patch_embed<TS>), dim3((M + PE_TOK - 1) / PE_TOK, (d + 255) / 256), 256, PE_TOK * D.P * sizeof(float), sp, D,
            (const TS *)c->w_pe_io, (const TS *)c->b_pe, c->z, fold ? (TS *)c->hbuf : (TS *)nullptr, c->ln_stats,
            (const float *)c->mod + d, mod_row, (const RopeTab *)c->d_rope,
            (c->bf16_mode && c->fast) ? c->rope_cs : (float2 *)nullptr);
    const int ln_grid = (M + 3) / 4;
    for (int l = 0; l < L; ++l) {
        const float *modl = c->mod + (size_t)l * 6 * d;
        // with the folded LayerNorm hbuf already holds z*(1+scale) and ln_stats the row sums of z
        LnFold lq{nullptr, uv_row, c->ln_stats, d / 32, D.norm, D.eps, sp, D.T}, lm = lq;
        if (fold) {
            lq.uv = c->uvtab + (size_t)l * (3 * d + D.n1);
            lm.uv = lq.uv + 3 * d;
        } else {
            c->cls = CLS_ADALN;
            PLAUNCH(c, (k_adaln<TS>), ln_grid, 128, 0, sp, D, (const float *)c->z, (TS *)c->hbuf, modl, mod_row,
                    (size_t)0, (size_t)d);
        }
        EpiQKV<TS> eq{sp, (const TS *)c->b_qkv[l], (TS *)c->qbuf, (TS *)c->kc, (TS *)c->vc, c->d_rope, D, l,
                      c->rope_cs, M, lq, c->kv_prefetch ? 1 : 0};
        c->cls = CLS_GEMM_QKV;
        launch_gemm<TS>(c, (const TS *)c->hbuf, (const TS *)c->w_qkv[l], M, 3 * d, d, eq, TC_QKV, c->w_o[l],
                        (size_t)d * d, fold);
        if (kind == 1 && l == L - 1) break;      // a commit only needs the K/V of every layer
        launch_attention<TS>(c, nf, l);
        EpiGateRes<TS> eo{sp, (const TS *)c->b_o[l], c->z, modl + 2 * d, mod_row, D,
                          fold ? (TS *)c->hbuf : (TS *)nullptr, modl + 4 * d, fold ? c->ln_stats : (float2 *)nullptr};
        c->cls = CLS_GEMM_O;
        launch_gemm<TS>(c, (const TS *)c->abuf, (const TS *)c->w_o[l], M, d, d, eo, TC_RES, c->w_fc1[l],
                        (size_t)d * D.n1, fold);
        if (!fold) {
            c->cls = CLS_ADALN;
            PLAUNCH(c, (k_adaln<TS>), ln_grid, 128, 0, sp, D, (const float *)c->z, (TS *)c->hbuf, modl, mod_row,
                    (size_t)3 * d, (size_t)4 * d);
        }
        EpiGelu<TS> eg{(const TS *)c->b_fc1[l], (TS *)c->mbuf, D.n1, D.act, lm};
        c->cls = CLS_GEMM_FC1;
        launch_gemm<TS>(c, (const TS *)c->hbuf, (const TS *)c->w_fc1[l], M, D.n1, d, eg, TC_GELU, c->w_fc2[l],
                        (size_t)d * D.dm, fold);
        // the last layer's output goes to the final adaLN kernel, which reads z itself
        const bool more = fold && l + 1 < L;
        EpiGateRes<TS> e2{sp, (const TS *)c->b_fc2[l], c->z, modl + 5 * d, mod_row, D,
                          more ? (TS *)c->hbuf : (TS *)nullptr, modl + 6 * d + d, more ? c->ln_stats : (float2 *)nullptr};
        c->cls = CLS_GEMM_FC2;
        launch_gemm<TS>(c, (const TS *)c->mbuf, (const TS *)c->w_fc2[l], M, d, D.dm, e2, TC_RES,
                        l + 1 < L ? c->w_qkv[l + 1] : nullptr, (size_t)3 * d * d, fold);
    }
    if (kind == 0) {
        c->cls = CLS_HEAD;
        PLAUNCH(c, (k_adaln<TS>), ln_grid, 128, 0, sp, D, (const float *)c->z, (TS *)c->hbuf, (const float *)c->fmod,
                (size_t)2 * d, (size_t)0, (size_t)d);
        EpiFinal<TS> ef{sp, (const TS *)c->b_out, D};
        launch_gemm<TS>(c, (const TS *)c->hbuf, (const TS *)c->w_out, M, D.P, d, ef, TC_NONE);
    }
}

// ---------------------------------------------------------------------------
// Tile width and split of the four GEMMs of a block, found by timing at create.  For a pass of one frame
// every (width, split) pair is timed and the best split is kept for good (the order in which the K range is
// summed must not depend on the pass); for passes of more frames only the width is timed.  Results are kept
// per process (nfd_fast.cuh), so a second context of the same shape does not time anything and sums in the
// same order.  The timed launches run the real epilogues on scratch frames 0..nf-1 of stream 0 with whatever
// the modulation tables hold; the caller clears the cache afterwards.
// ---------------------------------------------------------------------------
static int tune_gemms(nfd_ctx *c) {
    const Dims &D = c->D;
    const int d = D.d, T = D.T;
    FastState &fs = c->fs;
    if (!c->bf16_mode || !c->fast || !fs.ready || getenv("NFD_NO_TUNE")) return NFD_OK;
    const bool fold = c->fold_active();
    const size_t mod_row = (size_t)D.L * 6 * d, uv_row = (size_t)D.L * (3 * d + D.n1);
    struct Kind { int tc, N, K; };
    const Kind kinds[4] = {{TC_QKV, 3 * d, d}, {TC_RES, d, d}, {TC_GELU, D.n1, d}, {TC_RES, d, D.dm}};
    cudaEvent_t e0, e1;
    CK(cudaEventCreate(&e0));
    CK(cudaEventCreate(&e1));
    const StepParams *sp = c->d_sp;
    auto launch = [&](int ki, int M) -> bool {        // one launch of GEMM `ki` of layer 0 with the forced plan
        const L2Prefetch pf{nullptr, 0};
        const float *modl = c->mod;
        LnFold ln{nullptr, uv_row, c->ln_stats, d / 32, D.norm, D.eps, sp, T};
        if (ki == 0) {
            if (fold) ln.uv = c->uvtab;
            EpiQKV<bf16> e{sp, (const bf16 *)c->b_qkv[0], (bf16 *)c->qbuf, (bf16 *)c->kc, (bf16 *)c->vc, c->d_rope, D, 0,
                           c->rope_cs, M, ln};
            return fast_gemm<bf16>(true, fs, c->st, (const bf16 *)c->hbuf, (const bf16 *)c->w_qkv[0], M, 3 * d, d, e, TC_QKV, pf);
        }
        if (ki == 1) {
            EpiGateRes<bf16> e{sp, (const bf16 *)c->b_o[0], c->z, modl + 2 * d, mod_row, D,
                               fold ? (bf16 *)c->hbuf : (bf16 *)nullptr, modl + 4 * d, fold ? c->ln_stats : (float2 *)nullptr};
            return fast_gemm<bf16>(true, fs, c->st, (const bf16 *)c->abuf, (const bf16 *)c->w_o[0], M, d, d, e, TC_RES, pf);
        }
        if (ki == 2) {
            if (fold) ln.uv = c->uvtab + 3 * d;
            EpiGelu<bf16> e{(const bf16 *)c->b_fc1[0], (bf16 *)c->mbuf, D.n1, D.act, ln};
            return fast_gemm<bf16>(true, fs, c->st, (const bf16 *)c->hbuf, (const bf16 *)c->w_fc1[0], M, D.n1, d, e, TC_GELU, pf);
        }
        EpiGateRes<bf16> e{sp, (const bf16 *)c->b_fc2[0], c->z, modl + 5 * d, mod_row, D,
                           fold ? (bf16 *)c->hbuf : (bf16 *)nullptr, modl + 7 * d, fold ? c->ln_stats : (float2 *)nullptr};
        return fast_gemm<bf16>(true, fs, c->st, (const bf16 *)c->mbuf, (const bf16 *)c->w_fc2[0], M, d, D.dm, e, TC_RES, pf);
    };
    auto time_of = [&](int ki, int M, int BN, int S, float *us) -> bool {
        fs.force_BN = BN, fs.force_S = S;
        bool ok = true;
        for (int i = 0; i < 3 && ok; ++i) ok = launch(ki, M);
        float best = 1e30f;
        for (int rep = 0; rep < 3 && ok; ++rep) {
            cudaEventRecord(e0, c->st);
            for (int i = 0; i < 8 && ok; ++i) ok = launch(ki, M);
            cudaEventRecord(e1, c->st);
            if (cudaEventSynchronize(e1) != cudaSuccess) ok = false;
            float ms = 0.f;
            if (ok && cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess && ms < best) best = ms;
        }
        fs.force_BN = fs.force_S = 0;
        if (!ok) cudaGetLastError();
        *us = best * 1000.f / 8.f;
        return ok;
    };
    const int nfs[] = {1, 2, 3, 4, 5, 6, 8, 12, 16, 24, 32};
    const int widths[] = {32, 64, 96, 128, 192, 256};
    bool touched = false;
    // the largest pass this context can build: per stream a speculation plus the deferred frames of the last one
    const int nf_max = D.n_streams * 2 * c->cfg.max_spec;
    for (int nf : nfs) {
        if (nf > NFD_MAX_PASS_FRAMES || nf > nf_max) break;
        const int M = nf * T;
        bool need = false;
        for (const Kind &k : kinds)
            if (!g_tuned_BN.count(std::make_tuple(k.tc + (k.K > 2048 ? 10 : 0), k.N, k.K, fs.n_sm, M))) need = true;
        if (!need) continue;
        // a pass descriptor for nf scratch frames of stream 0
        StepParams &p = c->h_sp;
        memset(&p, 0, sizeof(p));
        p.nf = nf;
        for (int j = 0; j < nf; ++j) {
            p.fr[j].stream = 0, p.fr[j].frame = j, p.fr[j].win_first = 0, p.fr[j].cond_row = 0, p.fr[j].first_new = 0;
            p.fr[j].src = 0, p.fr[j].src_index = j, p.fr[j].out_index = -1;
        }
        k_set_params<<<1, 256, 0, c->st>>>(p, c->d_sp, c->lim, c->d_status);
        CK(cudaGetLastError());
        touched = true;
        for (int ki = 0; ki < 4; ++ki) {
            const Kind &k = kinds[ki];
            const int kk = k.tc + (k.K > 2048 ? 10 : 0);
            const auto skey = std::make_tuple(kk, k.N, k.K, fs.n_sm);
            const auto bkey = std::make_tuple(kk, k.N, k.K, fs.n_sm, M);
            if (g_tuned_BN.count(bkey)) continue;
            const bool s_open = !g_tuned_S.count(skey);
            if (s_open && nf != 1) continue;                 // the split is decided by the one-frame pass
            const int nkb = (k.K + 63) / 64;
            // the cost model's plan is the incumbent: another one must beat it by 3 % (timing noise must not
            // flip plans between processes without need)
            const GemmPlan model = plan_gemm(fs, M, k.N, k.K, k.tc);
            float t_best = 1e30f;
            GemmPlan best = model;
            if (!time_of(ki, M, model.BN, model.S, &t_best)) t_best = 1e30f;
            t_best *= 0.97f;
            for (int S = 1; S <= 4; S *= 2) {
                if (!s_open && S != g_tuned_S[skey]) continue;
                if (S > 1 && nkb / S < 2) continue;
                for (int BN : widths) {
                    if (BN > 32 && BN > k.N) continue;
                    if (nf == 1 && BN > 128) continue;
                    if (BN == model.BN && S == model.S) continue;
                    const long long ctas = (long long)((M + 127) / 128) * ((k.N + BN - 1) / BN) * S;
                    if (ctas > 3LL * fs.n_sm) continue;          // hopeless: several waves
                    float t;
                    const bool ok_t = time_of(ki, M, BN, S, &t);
                    if (ok_t && t < t_best) t_best = t, best = GemmPlan{BN, S};
                }
            }
            if (s_open) g_tuned_S[skey] = best.S;
            g_tuned_BN[bkey] = best.BN;
        }
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (touched) {
        // the timed epilogues wrote into scratch pages of stream 0 and into the activation buffers
        const size_t cache_bytes = (size_t)D.n_streams * D.L * D.R * D.page_elems * c->esz;
        CK(cudaMemsetAsync(c->kc, 0, cache_bytes, c->st));
        CK(cudaMemsetAsync(c->vc, 0, cache_bytes, c->st));
        CK(cudaMemsetAsync(c->d_status, 0, 16, c->st));
        CK(cudaStreamSynchronize(c->st));
        memset(&c->h_sp, 0, sizeof(c->h_sp));
    }
    return NFD_OK;
}

static void enqueue_body_any(nfd_ctx *c, int nf, int kind) {
    if (c->bf16_mode)
        enqueue_body<bf16>(c, nf, kind);
    else
        enqueue_body<float>(c, nf, kind);
}

static int run_pass_inner(nfd_ctx *c);

// Run the pass described by c->h_sp.  If it cannot be enqueued, the cache slots that it was to fill are
// given up again.
static int run_pass(nfd_ctx *c) {
    if (c->test_corrupt_desc) {
        // test switch: a batch slot that does not exist; the first kernel of the pass must catch it
        c->test_corrupt_desc = false;
        c->h_sp.fr[0].stream = c->cfg.n_streams + 7;
    }
    const int rc = run_pass_inner(c);
    if (rc != NFD_OK)
        for (int r = 0; r < c->h_sp.nc; ++r) c->cond_slots[c->h_sp.cd[r].slot] = nfd_ctx::CondSlot();
    return rc;
}

static int run_pass_inner(nfd_ctx *c) {
    const int nf = c->h_sp.nf, kind = c->h_sp.kind;
    if (!c->use_graph || c->st == nullptr || c->prof) {
        c->cls = CLS_PARAMS;
        PLAUNCH(c, k_set_params, 1, 256, 0, c->h_sp, c->d_sp, c->lim, c->d_status);
        enqueue_body_any(c, nf, kind);
        CK(take_launch_err(c));
        return NFD_OK;
    }
    // (no conditioning kernels when all pairs are cached)
    const int key = kind * 64 + nf + (c->fast ? 0 : 4096) + (c->h_sp.nc > 0 ? 0 : 8192) + (c->fuse_ln ? 0 : 16384) +
                    (c->l2_prefetch ? 0 : 32768) + (c->kv_prefetch ? 0 : 65536);
    auto it = c->graphs.find(key);
    if (it == c->graphs.end()) {
        GraphEntry ge;
        long long before = c->launches;
        CK(cudaStreamBeginCapture(c->st, cudaStreamCaptureModeThreadLocal));
        PLAUNCH(c, k_set_params, 1, 256, 0, c->h_sp, c->d_sp, c->lim, c->d_status);
        enqueue_body_any(c, nf, kind);
        cudaError_t e = cudaStreamEndCapture(c->st, &ge.graph);
        ge.launches = c->launches - before;
        c->launches = before;
        const cudaError_t le = take_launch_err(c);
        if (e == cudaSuccess) e = le;
        if (e != cudaSuccess || !ge.graph) {
            fprintf(stderr, "libnfd: graph capture failed: %s\n", cudaGetErrorString(e));
            cudaGetLastError();
            return NFD_E_CUDA;
        }
        size_t n_roots = 0;
        CK(cudaGraphGetRootNodes(ge.graph, nullptr, &n_roots));
        if (n_roots != 1) {
            fprintf(stderr, "libnfd: captured graph has %zu root nodes, expected 1\n", n_roots);
            cudaGraphDestroy(ge.graph);
            return NFD_E_CUDA;
        }
        CK(cudaGraphGetRootNodes(ge.graph, &ge.param_node, &n_roots));
        CK(cudaGraphInstantiate(&ge.exec, ge.graph, 0));
        it = c->graphs.emplace(key, ge).first;
    }
    GraphEntry &ge = it->second;
    void *args[4] = {(void *)&c->h_sp, (void *)&c->d_sp, (void *)&c->lim, (void *)&c->d_status};
    cudaKernelNodeParams kp;
    memset(&kp, 0, sizeof(kp));
    kp.func = (void *)k_set_params;
    kp.gridDim = dim3(1, 1, 1);
    kp.blockDim = dim3(256, 1, 1);
    kp.sharedMemBytes = 0;
    kp.kernelParams = args;
    kp.extra = nullptr;
    CK(cudaGraphExecKernelNodeSetParams(ge.exec, ge.param_node, &kp));
    CK(cudaGraphLaunch(ge.exec, c->st));
    c->launches += ge.launches;
    return NFD_OK;
}

// One frame of a pass as the host describes it.
struct PassFrame {
    int stream, frame;       // batch slot, absolute frame index
    float t;                 // FM time
    int action;
    int first_new;           // first frame of the stream whose K/V this pass writes
    int src, src_index;      // input set and frame slot in it
    int out_index;           // v_out slot or -1
};

struct PassInputs {
    const float *x_a[2] = {nullptr, nullptr}, *x_b[2] = {nullptr, nullptr};
    float alpha[2] = {0.f, 0.f}, beta[2] = {0.f, 0.f};
    float *v_out = nullptr;
};

// Fill c->h_sp for a pass over the given frames.  Nothing is changed if it fails.
static int build_pass_frames(nfd_ctx *c, const std::vector<PassFrame> &fr, int kind, const PassInputs &in) {
    const nfd_cfg &g = c->cfg;
    const int nf = (int)fr.size();
    if (nf < 1 || nf > NFD_MAX_PASS_FRAMES) return NFD_E_RANGE;
    // validate everything before the modulation cache is touched
    for (const PassFrame &f : fr) {
        if (f.stream < 0 || f.stream >= g.n_streams) return NFD_E_RANGE;
        if (!(f.t >= 0.f) || !(f.t <= 1.f)) return NFD_E_RANGE;
        if (f.action < 0 || f.action >= g.n_actions) return NFD_E_RANGE;
    }
    StepParams &p = c->h_sp;
    memset(&p, 0, sizeof(p));
    ++c->pass_no;
    p.nf = nf;
    p.kind = kind;
    for (int s = 0; s < 2; ++s) p.x_a[s] = in.x_a[s], p.x_b[s] = in.x_b[s], p.alpha[s] = in.alpha[s], p.beta[s] = in.beta[s];
    p.v_out = in.v_out;
    int nc = 0;
    for (int j = 0; j < nf; ++j) {
        const PassFrame &pf = fr[j];
        // modulation cache: reuse the slot of this (t, action) pair, else take the least recently used one
        unsigned tb;
        memcpy(&tb, &pf.t, 4);
        int row = -1, lru = -1;
        for (int r = 0; r < (int)c->cond_slots.size(); ++r) {
            const nfd_ctx::CondSlot &cs = c->cond_slots[r];
            if (cs.action == pf.action && cs.t_bits == tb) row = r;
            if (cs.last_use != c->pass_no && (lru < 0 || cs.last_use < c->cond_slots[lru].last_use)) lru = r;
        }
        if (row < 0) {
            if (lru < 0 || nc >= NFD_MAX_PASS_FRAMES) return NFD_E_RANGE;      // cannot happen: slots > frames per pass
            row = lru;
            c->cond_slots[row].t_bits = tb, c->cond_slots[row].action = pf.action;
            p.cd[nc].t = pf.t, p.cd[nc].action = pf.action, p.cd[nc].slot = row;
            ++nc;
            ++c->cond_misses;
        } else if (c->cond_slots[row].last_use != c->pass_no) {
            ++c->cond_hits;
        }
        c->cond_slots[row].last_use = c->pass_no;
        FrameDesc &f = p.fr[j];
        f.stream = pf.stream;
        f.frame = pf.frame;
        f.win_first = pf.frame - g.ctx_frames > 0 ? pf.frame - g.ctx_frames : 0;
        f.cond_row = row;
        f.first_new = pf.first_new;
        f.src = pf.src, f.src_index = pf.src_index, f.out_index = pf.out_index;
    }
    p.nc = nc;
    return NFD_OK;
}

// A pass over n streams x k frames that follow the frames counted so far (plus `offset`).
//   actions: per stream (per_frame_actions = false) or per frame.
static int build_pass(nfd_ctx *c, int n, const int *streams, int k, int offset, const float *t, const int *actions,
                      bool per_frame_actions, int kind, const float *x_a, float alpha, const float *x_b, float beta,
                      float *v_out) {
    const nfd_cfg &g = c->cfg;
    if (n < 1 || k < 1 || offset < 0 || offset + k > g.max_spec) return NFD_E_RANGE;
    if ((long long)n * k > NFD_MAX_PASS_FRAMES) return NFD_E_RANGE;
    for (int i = 0; i < n; ++i) {
        if (streams[i] < 0 || streams[i] >= g.n_streams) return NFD_E_RANGE;
        for (int j = 0; j < i; ++j)
            if (streams[j] == streams[i]) return NFD_E_RANGE;
    }
    std::vector<PassFrame> fr;
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < k; ++j) {
            PassFrame f;
            f.stream = streams[i];
            f.frame = c->n_total(streams[i]) + offset + j;
            f.t = t[i];
            f.action = per_frame_actions ? actions[i * k + j] : actions[i];
            f.first_new = c->n_total(streams[i]) + offset;
            f.src = 0, f.src_index = i * k + j, f.out_index = i * k + j;
            fr.push_back(f);
        }
    PassInputs in;
    in.x_a[0] = x_a, in.x_b[0] = x_b, in.alpha[0] = alpha, in.beta[0] = beta, in.v_out = v_out;
    return build_pass_frames(c, fr, kind, in);
}

// ---------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------
extern "C" {

const char *nfd_strerror(int code) {
    switch (code) {
        case NFD_OK: return "ok";
        case NFD_E_BADCFG: return "bad configuration";
        case NFD_E_NULLPTR: return "null pointer";
        case NFD_E_ALIGN: return "pointer not 16-byte aligned";
        case NFD_E_RANGE: return "argument out of range";
        case NFD_E_STATE: return "call not allowed in this cache state";
        case NFD_E_NOMEM: return "out of memory";
        case NFD_E_CUDA: return "CUDA error";
        case NFD_E_TIMEOUT: return "device-side wait timed out";
        case NFD_E_DEVICE: return "device-side check failed";
        default: return "unknown error";
    }
}

int nfd_destroy(nfd_ctx *c) {
    if (!c) return NFD_E_NULLPTR;
    cudaStreamSynchronize(c->st);
    for (auto &kv : c->graphs) {
        if (kv.second.exec) cudaGraphExecDestroy(kv.second.exec);
        if (kv.second.graph) cudaGraphDestroy(kv.second.graph);
    }
    fast_destroy(c->fs);
    for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
    for (void *p : c->allocs) cudaFree(p);
    delete c;
    return NFD_OK;
}

int nfd_create(nfd_ctx **out, const nfd_weights *w, const nfd_cfg *cfg, void *cuda_stream) {
    if (!out || !w || !cfg) return NFD_E_NULLPTR;
    *out = nullptr;
    RET(validate_cfg(*cfg));
    nfd_ctx *c = new (std::nothrow) nfd_ctx();
    if (!c) return NFD_E_NOMEM;
    c->cfg = *cfg;
    c->st = (cudaStream_t)cuda_stream;
    c->bf16_mode = cfg->dtype == NFD_DTYPE_BF16;
    c->esz = c->bf16_mode ? 2 : 4;
    Dims &D = c->D;
    D.L = cfg->n_layers, D.d = cfg->d_model, D.H = cfg->n_heads, D.dh = cfg->head_dim;
    D.dm = (cfg->d_mlp + 7) / 8 * 8, D.act = cfg->act, D.n1 = D.act ? 2 * D.dm : D.dm;
    D.C = cfg->latent_c, D.Hl = cfg->latent_h, D.Wl = cfg->latent_w, D.p = cfg->patch;
    D.th = D.Hl / D.p, D.tw = D.Wl / D.p, D.T = D.th * D.tw, D.P = D.C * D.p * D.p;
    // ring pages per layer: the window, the frames of a speculation and the deferred frames that may ride along
    D.R = cfg->ctx_frames + 2 * cfg->max_spec, D.W = cfg->ctx_frames, D.n_streams = cfg->n_streams;
    D.norm = cfg->norm, D.eps = cfg->norm_eps, D.t_scale = cfg->t_scale;
    D.page_elems = (size_t)D.H * D.T * D.dh;
    c->lim.n_streams = cfg->n_streams, c->lim.W = cfg->ctx_frames, c->lim.n_slots = NFD_COND_SLOTS;
    c->lim.n_actions = cfg->n_actions, c->lim.max_frames = NFD_MAX_PASS_FRAMES;
    c->lim.pend_slots = cfg->n_streams * cfg->max_spec;
    c->n_committed.assign(cfg->n_streams, 0);
    c->n_tentative.assign(cfg->n_streams, 0);
    c->n_pending.assign(cfg->n_streams, 0);
    c->pend_act.assign(cfg->n_streams, std::vector<int>());
    if (getenv("NFD_NO_GRAPH")) c->use_graph = false;
    if (getenv("NFD_NO_FAST")) c->fast = false;
    if (getenv("NFD_NO_FUSE_LN")) c->fuse_ln = false;

    int rc = c->bf16_mode ? repack_all<bf16>(c, w) : repack_all<float>(c, w);
    const int NF = NFD_MAX_PASS_FRAMES;
    const size_t Mmax = (size_t)NF * D.T;
    auto A = [&](void **p, size_t bytes) { if (rc == NFD_OK) rc = dev_alloc(c, p, bytes); };
    const size_t cache_elems = (size_t)D.n_streams * D.L * D.R * D.page_elems;
    A(&c->kc, cache_elems * c->esz);
    A(&c->vc, cache_elems * c->esz);
    A((void **)&c->z, Mmax * D.d * 4);
    A(&c->hbuf, Mmax * D.d * c->esz);
    A(&c->qbuf, Mmax * D.d * c->esz);
    A(&c->abuf, Mmax * D.d * c->esz);
    A(&c->mbuf, Mmax * D.dm * c->esz);
    A((void **)&c->emb, (size_t)NF * 256 * 4);
    A((void **)&c->h1, (size_t)NF * D.d * 4);
    A((void **)&c->sc, (size_t)NF * D.d * 4);
    const int n_slots = NFD_COND_SLOTS;
    c->cond_slots.assign(n_slots, nfd_ctx::CondSlot());
    A((void **)&c->mod, (size_t)n_slots * D.L * 6 * D.d * 4);
    A((void **)&c->fmod, (size_t)n_slots * 2 * D.d * 4);
    if (c->bf16_mode) {
        A((void **)&c->uvtab, (size_t)n_slots * D.L * (3 * D.d + D.n1) * sizeof(float2));
        A((void **)&c->ln_stats, Mmax * ((D.d + 31) / 32) * sizeof(float2));
    }
    A((void **)&c->pend_x0, (size_t)cfg->n_streams * cfg->max_spec * c->frame_elems() * 4);
    A((void **)&c->pend_cz, (size_t)cfg->n_streams * cfg->max_spec * c->frame_elems() * 4);
    A((void **)&c->xp, (size_t)NF * c->frame_elems() * 4);
    A((void **)&c->vbuf, (size_t)NF * c->frame_elems() * 4);
    A((void **)&c->x0_prev, (size_t)NF * c->frame_elems() * 4);
    A((void **)&c->d_sp, sizeof(StepParams));
    A((void **)&c->d_hash, 8);
    A((void **)&c->d_status, 16);
    A((void **)&c->d_rope, sizeof(RopeTab));
    A((void **)&c->rope_cs, Mmax * (D.dh / 2) * sizeof(float2));
    if (rc == NFD_OK) {
        std::vector<void *> v;
        v = c->w_mod; rc = upload_ptrs(c, v, &c->dp_wmod);
        if (rc == NFD_OK) { v = c->b_mod; rc = upload_ptrs(c, v, &c->dp_bmod); }
        if (rc == NFD_OK) { v = {c->w_t1, c->b_t1}; rc = upload_ptrs(c, v, &c->dp_t1); }
        if (rc == NFD_OK) { v = {c->w_t2, c->b_t2}; rc = upload_ptrs(c, v, &c->dp_t2); }
        if (rc == NFD_OK) { v = {c->w_fmod, c->b_fmod}; rc = upload_ptrs(c, v, &c->dp_fmod); }
        if (rc == NFD_OK) { v = c->w_qkv; rc = upload_ptrs(c, v, &c->dp_wqkv); }
        if (rc == NFD_OK) { v = c->b_qkv; rc = upload_ptrs(c, v, &c->dp_bqkv); }
        if (rc == NFD_OK) { v = c->w_fc1; rc = upload_ptrs(c, v, &c->dp_wfc1); }
        if (rc == NFD_OK) { v = c->b_fc1; rc = upload_ptrs(c, v, &c->dp_bfc1); }
    }
    if (rc == NFD_OK) {
        RopeTab rt;
        memset(&rt, 0, sizeof(rt));
        int pi = 0;
        const int dims[3] = {cfg->rope_t, cfg->rope_h, cfg->rope_w};
        for (int ax = 0; ax < 3; ++ax)
            for (int i = 0; i < dims[ax] / 2; ++i, ++pi) {
                rt.axis[pi] = ax;
                rt.freq[pi] = (float)pow((double)cfg->rope_theta, -2.0 * i / (double)dims[ax]);
            }
        cudaError_t e = cudaMemcpyAsync(c->d_rope, &rt, sizeof(rt), cudaMemcpyHostToDevice, c->st);
        if (e == cudaSuccess) e = cudaMemsetAsync(c->kc, 0, cache_elems * c->esz, c->st);
        if (e == cudaSuccess) e = cudaMemsetAsync(c->vc, 0, cache_elems * c->esz, c->st);
        if (e == cudaSuccess) e = cudaMemsetAsync(c->d_status, 0, 16, c->st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(c->st);
        if (e != cudaSuccess) {
            fprintf(stderr, "libnfd: create: %s\n", cudaGetErrorString(e));
            rc = NFD_E_CUDA;
        }
    }
    if (rc == NFD_OK) rc = fast_create(c->fs, D, c->bf16_mode, c->st, c->d_status);
    if (rc == NFD_OK && c->fs.ready) {
        // how many CTAs of a GEMM fit at once, per cluster size (any instantiation: one CTA fills an SM)
        auto kern = k_gemm_tc<96, EpiGateRes<bf16>, 0>;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, GemmCfg<96>::SMEM) == cudaSuccess)
            query_gemm_slots(c->fs, kern, GemmCfg<96>::SMEM, GemmCfg<96>::THREADS);
        else
            cudaGetLastError();
    }
    if (rc == NFD_OK) rc = tune_gemms(c);
    if (rc != NFD_OK) {
        nfd_destroy(c);
        return rc;
    }
    *out = c;
    return NFD_OK;
}

int nfd_reset(nfd_ctx *c, int stream) {
    if (!c) return NFD_E_NULLPTR;
    if (stream < 0 || stream >= c->cfg.n_streams) return NFD_E_RANGE;
    c->n_committed[stream] = 0;
    c->n_tentative[stream] = 0;
    c->n_pending[stream] = 0;
    return NFD_OK;
}

static int flush_pending(nfd_ctx *c, int s);

static int check_io(const void *a, const void *b) {
    if (!a || !b) return NFD_E_NULLPTR;
    if (!aligned16(a) || !aligned16(b)) return NFD_E_ALIGN;
    return NFD_OK;
}

int nfd_denoise_step_batched(nfd_ctx *c, int n, const int *streams, const float *x_t, int k, const float *t,
                             const int *actions, float *v_out) {
    if (!c || !streams || !t || !actions) return NFD_E_NULLPTR;
    RET(check_io(x_t, v_out));
    for (int i = 0; i < n; ++i) {
        if (streams[i] < 0 || streams[i] >= c->cfg.n_streams) return NFD_E_RANGE;
        RET(flush_pending(c, streams[i]));
    }
    RET(build_pass(c, n, streams, k, 0, t, actions, false, 0, x_t, 1.0f, nullptr, 0.f, v_out));
    return run_pass(c);
}

int nfd_denoise_step_at(nfd_ctx *c, int stream, int offset, const float *x_t, int k, float t, int action,
                        float *v_out) {
    if (!c) return NFD_E_NULLPTR;
    RET(check_io(x_t, v_out));
    if (stream < 0 || stream >= c->cfg.n_streams) return NFD_E_RANGE;
    if (!(t >= 0.f) || !(t <= 1.f) || action < 0 || action >= c->cfg.n_actions) return NFD_E_RANGE;
    RET(flush_pending(c, stream));
    RET(build_pass(c, 1, &stream, k, offset, &t, &action, false, 0, x_t, 1.0f, nullptr, 0.f, v_out));
    return run_pass(c);
}

int nfd_denoise_step(nfd_ctx *c, int stream, const float *x_t, int k, float t, int action, float *v_out) {
    return nfd_denoise_step_at(c, stream, 0, x_t, k, t, action, v_out);
}

// Input scaling of a commit (Section 4.3): x' = cos(t_ctx) x0 + sin(t_ctx) sigma_d z at the constant context
// timestep, then brought to Flow-Matching scale; returns the FM time and the two coefficients.
static void commit_coeffs(const nfd_ctx *c, float *t_fm, float *a, float *b) {
    const double tc = c->cfg.t_ctx_trig, sd = c->cfg.sigma_d;
    const double sn = sin(tc), cs = cos(tc);
    const double t = sn / (sn + cs);
    const double scale = sqrt(t * t + (1 - t) * (1 - t));
    *t_fm = (float)t, *a = (float)(cs * scale / sd), *b = (float)(sn * scale);
}

// FM time of sampler step s (Section 4.1 "Sampling": t' from pi/2 down in S equal steps).
static double sampler_fm_time(int S, int s) {
    const double tp = 0.5 * M_PI * (double)(S - s) / (double)S;
    const double sn = sin(tp), cs = cos(tp);
    return sn / (sn + cs);
}

// Fill the modulation cache for every (time, action) pair that nfd_speculate and the commits can ask for:
// the S sampler times and the context time, for each action.  Pairs that are cached already are left alone.
int nfd_warm_modulation(nfd_ctx *c) {
    if (!c) return NFD_E_NULLPTR;
    const int S = c->cfg.n_steps, A = c->cfg.n_actions;
    std::vector<float> ts;
    for (int s = 0; s < S; ++s) ts.push_back((float)sampler_fm_time(S, s));
    float t_fm, ca, cb;
    commit_coeffs(c, &t_fm, &ca, &cb);
    ts.push_back(t_fm);
    if ((long long)ts.size() * A > (long long)c->cond_slots.size()) return NFD_E_RANGE;
    int filled = 0;
    std::vector<std::pair<float, int>> todo;
    for (float t : ts)
        for (int a = 0; a < A; ++a) todo.push_back(std::make_pair(t, a));
    for (size_t i0 = 0; i0 < todo.size(); i0 += NFD_MAX_PASS_FRAMES) {
        // a conditioning-only pass: the frame list is only used to look the pairs up
        std::vector<PassFrame> fr;
        for (size_t i = i0; i < todo.size() && i < i0 + NFD_MAX_PASS_FRAMES; ++i) {
            PassFrame f;
            f.stream = 0, f.frame = 0, f.t = todo[i].first, f.action = todo[i].second, f.first_new = 0;
            f.src = 0, f.src_index = 0, f.out_index = -1;
            fr.push_back(f);
        }
        RET(build_pass_frames(c, fr, 2, PassInputs()));
        const int nc = c->h_sp.nc;
        if (nc == 0) continue;
        c->cls = CLS_PARAMS;
        PLAUNCH(c, k_set_params, 1, 256, 0, c->h_sp, c->d_sp, c->lim, c->d_status);
        if (c->bf16_mode)
            enqueue_conditioning<bf16>(c, (int)fr.size());
        else
            enqueue_conditioning<float>(c, (int)fr.size());
        const cudaError_t e = take_launch_err(c);
        if (e != cudaSuccess) {
            for (int r = 0; r < nc; ++r) c->cond_slots[c->h_sp.cd[r].slot] = nfd_ctx::CondSlot();
            fprintf(stderr, "libnfd: %s\n", cudaGetErrorString(e));
            return NFD_E_CUDA;
        }
        filled += nc;
    }
    return filled;
}

// Commit pass over n streams x k frames; actions per frame.
static int commit_pass(nfd_ctx *c, int n, const int *streams, int k, const int *actions, const float *x0,
                       const float *ctx_noise, bool tentative) {
    float t_fm, ca, cb;
    commit_coeffs(c, &t_fm, &ca, &cb);
    std::vector<float> t(n, t_fm);
    RET(build_pass(c, n, streams, k, 0, t.data(), actions, true, 1, x0, ca, ctx_noise, cb, nullptr));
    RET(run_pass(c));
    for (int i = 0; i < n; ++i) (tentative ? c->n_tentative : c->n_committed)[streams[i]] += k;
    return NFD_OK;
}

// Frames of stream s whose commit was deferred, as frames of a pass (input set `set`, K/V only).
static void pending_frames(const nfd_ctx *c, int s, int set, std::vector<PassFrame> &fr) {
    float t_fm, ca, cb;
    commit_coeffs(c, &t_fm, &ca, &cb);
    const int P = c->n_pending[s], total = c->n_total(s);
    for (int j = 0; j < P; ++j) {
        PassFrame f;
        f.stream = s, f.frame = total - P + j, f.t = t_fm, f.action = c->pend_act[s][j];
        f.first_new = total - P;
        f.src = set, f.src_index = s * c->cfg.max_spec + j, f.out_index = -1;
        fr.push_back(f);
    }
}

// Write the K/V pages of the deferred frames of one stream now (a commit pass of their own).
static int flush_pending(nfd_ctx *c, int s) {
    if (c->n_pending[s] == 0) return NFD_OK;
    std::vector<PassFrame> fr;
    pending_frames(c, s, 0, fr);
    PassInputs in;
    float t_fm;
    commit_coeffs(c, &t_fm, &in.alpha[0], &in.beta[0]);
    in.x_a[0] = c->pend_x0, in.x_b[0] = c->pend_cz;
    RET(build_pass_frames(c, fr, 1, in));
    RET(run_pass(c));
    c->n_pending[s] = 0;
    return NFD_OK;
}

int nfd_commit_frame(nfd_ctx *c, int stream, const float *x0, int n, const int *actions, const float *ctx_noise) {
    if (!c || !x0 || !actions) return NFD_E_NULLPTR;
    if (!aligned16(x0) || !aligned16(ctx_noise)) return NFD_E_ALIGN;
    if (stream < 0 || stream >= c->cfg.n_streams) return NFD_E_RANGE;
    if (c->n_tentative[stream] != 0) return NFD_E_STATE;
    if (n < 1 || n > c->cfg.max_spec) return NFD_E_RANGE;
    for (int j = 0; j < n; ++j)
        if (actions[j] < 0 || actions[j] >= c->cfg.n_actions) return NFD_E_RANGE;
    RET(flush_pending(c, stream));
    return commit_pass(c, 1, &stream, n, actions, x0, ctx_noise, false);
}

int nfd_speculate_batched(nfd_ctx *c, int n, const int *streams, int k, const int *actions, const float *noise,
                          const float *ctx_noise, float *x0_out) {
    if (!c || !streams || !actions) return NFD_E_NULLPTR;
    RET(check_io(noise, x0_out));
    if (!aligned16(ctx_noise)) return NFD_E_ALIGN;
    if (n < 1 || k < 1 || k > c->cfg.max_spec || (long long)n * k > NFD_MAX_PASS_FRAMES) return NFD_E_RANGE;
    int n_pend = 0;
    for (int i = 0; i < n; ++i) {
        if (streams[i] < 0 || streams[i] >= c->cfg.n_streams) return NFD_E_RANGE;
        for (int j = 0; j < i; ++j)
            if (streams[j] == streams[i]) return NFD_E_RANGE;
        if (actions[i] < 0 || actions[i] >= c->cfg.n_actions) return NFD_E_RANGE;
        if (c->n_tentative[streams[i]] != 0) return NFD_E_STATE;
        n_pend += c->n_pending[streams[i]];
    }
    // deferred frames ride along with the first denoising pass if the pass can hold them
    const bool carry = c->lazy && n_pend > 0 && n * k + n_pend <= NFD_MAX_PASS_FRAMES;
    if (!carry)
        for (int i = 0; i < n; ++i) RET(flush_pending(c, streams[i]));
    const int S = c->cfg.n_steps;
    const double sd = c->cfg.sigma_d;
    const size_t fe = c->frame_elems();
    const size_t ne = (size_t)n * k * fe;
    const int eg = (int)((ne + 255) / 256);
    // Section 4.1 "Sampling": start from pure noise at t' = pi/2
    c->cls = CLS_SAMPLER;
    // (test switch: a block size beyond the device's limit, which the runtime refuses on the host)
    const int blk0 = c->test_fail_launch ? 4096 : 256;
    c->test_fail_launch = false;
    PLAUNCH(c, k_axpby, eg, blk0, 0, c->xp, (float)sd, noise, 0.f, (const float *)nullptr, ne);
    std::vector<float> tv(n);
    for (int s = 0; s < S; ++s) {
        const double tp = 0.5 * M_PI * (double)(S - s) / (double)S;
        const double sn = sin(tp), cs = cos(tp);
        const double t = sn / (sn + cs);
        const double alpha = sqrt(t * t + (1 - t) * (1 - t)) / sd;
        for (int i = 0; i < n; ++i) tv[i] = (float)t;
        if (s == 0 && carry) {
            // one block-causal pass: per stream its deferred frames (K/V only), then the k new frames
            std::vector<PassFrame> fr;
            for (int i = 0; i < n; ++i) {
                const int st = streams[i], total = c->n_total(st), P = c->n_pending[st];
                pending_frames(c, st, 1, fr);
                for (int j = 0; j < k; ++j) {
                    PassFrame f;
                    f.stream = st, f.frame = total + j, f.t = (float)t, f.action = actions[i];
                    f.first_new = total - P;
                    f.src = 0, f.src_index = i * k + j, f.out_index = i * k + j;
                    fr.push_back(f);
                }
            }
            PassInputs in;
            float t_fm;
            commit_coeffs(c, &t_fm, &in.alpha[1], &in.beta[1]);
            in.x_a[1] = c->pend_x0, in.x_b[1] = c->pend_cz;
            in.x_a[0] = c->xp, in.alpha[0] = (float)alpha, in.v_out = c->vbuf;
            RET(build_pass_frames(c, fr, 0, in));
            RET(run_pass(c));
            for (int i = 0; i < n; ++i) c->n_pending[streams[i]] = 0;
        } else {
            RET(build_pass(c, n, streams, k, 0, tv.data(), actions, false, 0, c->xp, (float)alpha, nullptr, 0.f,
                           c->vbuf));
            RET(run_pass(c));
        }
        // clean estimate sigma_d (x_in - t v), then re-noise to the next timestep
        const float *z = nullptr;
        double cn = 0, sn_next = 0;
        if (s + 1 < S) {
            const double tpn = 0.5 * M_PI * (double)(S - s - 1) / (double)S;
            z = noise + (size_t)(s + 1) * ne;
            cn = cos(tpn), sn_next = sin(tpn) * sd;
        }
        c->cls = CLS_SAMPLER;
        PLAUNCH(c, k_sampler_post, eg, 256, 0, c->xp, (const float *)c->vbuf, z, x0_out, (float)(sd * alpha),
                (float)(-sd * t), (float)cn, (float)sn_next, ne);
    }
    CK(take_launch_err(c));
    if (!c->lazy) {
        std::vector<int> fa((size_t)n * k);
        for (int i = 0; i < n; ++i)
            for (int j = 0; j < k; ++j) fa[i * k + j] = actions[i];
        return commit_pass(c, n, streams, k, fa.data(), x0_out, ctx_noise, true);
    }
    // defer the commit: keep what it needs; the frames count as tentative from now on
    for (int i = 0; i < n; ++i) {
        const int st = streams[i];
        const size_t off = (size_t)st * c->cfg.max_spec * fe;
        CK(cudaMemcpyAsync(c->pend_x0 + off, x0_out + (size_t)i * k * fe, (size_t)k * fe * 4, cudaMemcpyDeviceToDevice,
                           c->st));
        if (ctx_noise)
            CK(cudaMemcpyAsync(c->pend_cz + off, ctx_noise + (size_t)i * k * fe, (size_t)k * fe * 4,
                               cudaMemcpyDeviceToDevice, c->st));
        else
            CK(cudaMemsetAsync(c->pend_cz + off, 0, (size_t)k * fe * 4, c->st));
        c->pend_act[st].assign(k, actions[i]);
        c->n_pending[st] = k;
        c->n_tentative[st] += k;
    }
    return NFD_OK;
}

// The undistilled sampler (Section 3.2 "Sampling"): DPM-Solver++(2M) over n_evals equal steps of FM time from
// t = 1 (pure noise) to t = 0; first order where no finite previous step exists (the first two steps) and at
// the last step.  Coefficients as in the published algorithm, with alpha_t = 1 - t, sigma_t = t.
int nfd_sample_dpmpp(nfd_ctx *c, int stream, int k, int action, int n_evals, const float *noise,
                     const float *ctx_noise, float *x0_out) {
    if (!c) return NFD_E_NULLPTR;
    RET(check_io(noise, x0_out));
    if (!aligned16(ctx_noise)) return NFD_E_ALIGN;
    if (stream < 0 || stream >= c->cfg.n_streams) return NFD_E_RANGE;
    if (k < 1 || k > c->cfg.max_spec || n_evals < 1 || n_evals > 1000) return NFD_E_RANGE;
    if (action < 0 || action >= c->cfg.n_actions) return NFD_E_RANGE;
    if (c->n_tentative[stream] != 0) return NFD_E_STATE;
    RET(flush_pending(c, stream));
    const size_t ne = (size_t)k * c->frame_elems();
    const int eg = (int)((ne + 255) / 256);
    c->cls = CLS_SAMPLER;
    PLAUNCH(c, k_axpby, eg, 256, 0, c->xp, 1.0f, noise, 0.f, (const float *)nullptr, ne);
    const int M = n_evals;
    auto tgrid = [M](int i) { return 1.0 - (double)i / (double)M; };
    auto lam = [](double u) { return log((1.0 - u) / u); };
    for (int i = 1; i <= M; ++i) {
        const double tp = tgrid(i - 1), tn = tgrid(i);
        const float tf = (float)tp;
        RET(build_pass(c, 1, &stream, k, 0, &tf, &action, false, 0, c->xp, 1.0f, nullptr, 0.f, c->vbuf));
        RET(run_pass(c));
        const double a = tn / tp;
        const double b = (1.0 - tn) - (1.0 - tp) * tn / tp;
        double cc = 0.0;
        if (i >= 3 && i < M) {                // a finite previous step exists and this is not the last step
            const double tpp = tgrid(i - 2);
            cc = (lam(tn) - lam(tp)) / (2.0 * (lam(tp) - lam(tpp)));
        }
        c->cls = CLS_SAMPLER;
        PLAUNCH(c, k_dpmpp_update, eg, 256, 0, c->xp, (const float *)c->vbuf, c->x0_prev, tf, (float)a, (float)b,
                (float)cc, i == M ? x0_out : (float *)nullptr, c->cfg.sigma_d, ne);
    }
    CK(take_launch_err(c));
    std::vector<int> fa(k, action);
    return commit_pass(c, 1, &stream, k, fa.data(), x0_out, ctx_noise, true);
}

int nfd_speculate(nfd_ctx *c, int stream, int k, int action, const float *noise, const float *ctx_noise,
                  float *x0_out) {
    return nfd_speculate_batched(c, 1, &stream, k, &action, noise, ctx_noise, x0_out);
}

int nfd_rollback(nfd_ctx *c, int stream, int n_accept) {
    if (!c) return NFD_E_NULLPTR;
    if (stream < 0 || stream >= c->cfg.n_streams) return NFD_E_RANGE;
    if (n_accept < 0 || n_accept > c->n_tentative[stream]) return NFD_E_RANGE;
    c->n_committed[stream] += n_accept;
    c->n_tentative[stream] = 0;
    if (c->n_pending[stream] > n_accept) c->n_pending[stream] = n_accept;     // rejected frames were never written
    return NFD_OK;
}

int nfd_kv_state(nfd_ctx *c, int stream, int *n_committed, int *n_tentative, int *window_first) {
    if (!c) return NFD_E_NULLPTR;
    if (stream < 0 || stream >= c->cfg.n_streams) return NFD_E_RANGE;
    if (n_committed) *n_committed = c->n_committed[stream];
    if (n_tentative) *n_tentative = c->n_tentative[stream];
    int wf = c->n_total(stream) - c->cfg.ctx_frames;
    if (window_first) *window_first = wf > 0 ? wf : 0;
    return NFD_OK;
}

int nfd_kv_hash(nfd_ctx *c, int stream, unsigned long long *h) {
    if (!c || !h) return NFD_E_NULLPTR;
    if (stream < 0 || stream >= c->cfg.n_streams) return NFD_E_RANGE;
    RET(flush_pending(c, stream));
    const int total = c->n_total(stream);
    const int first = total - c->cfg.ctx_frames > 0 ? total - c->cfg.ctx_frames : 0;
    const int count = total - first;
    CK(cudaMemsetAsync(c->d_hash, 0, 8, c->st));
    c->cls = CLS_CACHE;
    if (count > 0) {
        if (c->bf16_mode)
            LAUNCH(c, (k_kv_hash<bf16>), 592, 256, 0, c->D, (const bf16 *)c->kc, (const bf16 *)c->vc, stream, first,
                   count, c->d_hash);
        else
            LAUNCH(c, (k_kv_hash<float>), 592, 256, 0, c->D, (const float *)c->kc, (const float *)c->vc, stream,
                   first, count, c->d_hash);
        CK(cudaGetLastError());
    }
    unsigned long long v = 0;
    CK(cudaMemcpyAsync(&v, c->d_hash, 8, cudaMemcpyDeviceToHost, c->st));
    CK(cudaStreamSynchronize(c->st));
    v ^= 0x9e3779b97f4a7c15ULL * (unsigned long long)(c->n_committed[stream] + 1);
    v ^= 0xc2b2ae3d27d4eb4fULL * (unsigned long long)(c->n_tentative[stream] + 1);
    *h = v;
    return NFD_OK;
}

int nfd_kv_read(nfd_ctx *c, int stream, int layer, int frame, float *k_out, float *v_out) {
    if (!c) return NFD_E_NULLPTR;
    if (stream < 0 || stream >= c->cfg.n_streams || layer < 0 || layer >= c->cfg.n_layers) return NFD_E_RANGE;
    RET(flush_pending(c, stream));
    const int total = c->n_total(stream);
    if (frame < 0 || frame >= total + c->cfg.max_spec || frame < total + c->cfg.max_spec - c->D.R) return NFD_E_RANGE;
    const int grid = (int)((c->D.page_elems + 255) / 256);
    c->cls = CLS_CACHE;
    for (int which = 0; which < 2; ++which) {
        float *o = which ? v_out : k_out;
        const void *cache = which ? c->vc : c->kc;
        if (!o) continue;
        if (c->bf16_mode)
            LAUNCH(c, (k_kv_read<bf16>), grid, 256, 0, c->D, (const bf16 *)cache, stream, layer, frame, o);
        else
            LAUNCH(c, (k_kv_read<float>), grid, 256, 0, c->D, (const float *)cache, stream, layer, frame, o);
    }
    CK(cudaGetLastError());
    return NFD_OK;
}

int nfd_attention(nfd_ctx *c, const void *q, const void *k, const void *v, int n_q, int n_kv, int window,
                  void *out) {
    if (!c || !q || !out) return NFD_E_NULLPTR;
    if ((k == nullptr) != (v == nullptr)) return NFD_E_NULLPTR;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return NFD_E_ALIGN;
    if (n_q < 1 || n_q > c->cfg.max_spec || n_kv < n_q || n_kv > c->D.R || window < 0 || window > c->D.W)
        return NFD_E_RANGE;
    const Dims &D = c->D;
    c->n_committed[0] = 0;
    c->n_tentative[0] = 0;
    c->n_pending[0] = 0;
    const size_t fill = (size_t)n_kv * D.page_elems;
    c->cls = CLS_CACHE;
    if (k) {
        const int grid = (int)((fill + 255) / 256);
        if (c->bf16_mode) {
            LAUNCH(c, (k_kv_fill<bf16>), grid, 256, 0, D, (bf16 *)c->kc, 0, (const bf16 *)k, n_kv);
            LAUNCH(c, (k_kv_fill<bf16>), grid, 256, 0, D, (bf16 *)c->vc, 0, (const bf16 *)v, n_kv);
        } else {
            LAUNCH(c, (k_kv_fill<float>), grid, 256, 0, D, (float *)c->kc, 0, (const float *)k, n_kv);
            LAUNCH(c, (k_kv_fill<float>), grid, 256, 0, D, (float *)c->vc, 0, (const float *)v, n_kv);
        }
    }
    const size_t qbytes = (size_t)n_q * D.T * D.d * c->esz;
    CK(cudaMemcpyAsync(c->qbuf, q, qbytes, cudaMemcpyDeviceToDevice, c->st));
    StepParams &p = c->h_sp;
    memset(&p, 0, sizeof(p));
    p.nf = n_q;
    p.nc = 1;
    for (int j = 0; j < n_q; ++j) {
        p.fr[j].stream = 0;
        p.fr[j].frame = n_kv - n_q + j;
        p.fr[j].win_first = p.fr[j].frame - window > 0 ? p.fr[j].frame - window : 0;
        p.fr[j].first_new = n_kv - n_q;
    }
    c->cls = CLS_PARAMS;
    PLAUNCH(c, k_set_params, 1, 256, 0, p, c->d_sp, c->lim, c->d_status);
    if (c->bf16_mode)
        launch_attention<bf16>(c, n_q, 0);
    else
        launch_attention<float>(c, n_q, 0);
    CK(take_launch_err(c));
    CK(cudaMemcpyAsync(out, c->abuf, qbytes, cudaMemcpyDeviceToDevice, c->st));
    return NFD_OK;
}

// Section 4.2: frames i .. i+k-1 were generated under actions[i]; the leading frames whose true action equals
// it are verified, the first mismatch and everything after it are discarded.  Frame i itself used its true
// action, so the count is at least 1.
int nfd_accepted_count(const int *actions, int n, int i, int k) {
    if (!actions) return NFD_E_NULLPTR;
    if (n < 1 || i < 0 || i >= n || k < 1) return NFD_E_RANGE;
    int m = 1;
    while (m < k && i + m < n && actions[i + m] == actions[i]) ++m;
    return m;
}

int nfd_debug_read(nfd_ctx *c, const char *name, float *out, long long n_elems) {
    if (!c || !name || !out) return NFD_E_NULLPTR;
    if (!aligned16(out)) return NFD_E_ALIGN;
    const size_t rows = (size_t)NFD_MAX_PASS_FRAMES * c->D.T;
    const void *src = nullptr;
    size_t cap = 0;
    bool is_f32 = !c->bf16_mode;
    if (!strcmp(name, "z")) src = c->z, cap = rows * c->D.d, is_f32 = true;
    else if (!strcmp(name, "hbuf")) src = c->hbuf, cap = rows * c->D.d;
    else if (!strcmp(name, "qbuf")) src = c->qbuf, cap = rows * c->D.d;
    else if (!strcmp(name, "abuf")) src = c->abuf, cap = rows * c->D.d;
    else if (!strcmp(name, "mbuf")) src = c->mbuf, cap = rows * c->D.dm;
    else return NFD_E_RANGE;
    if (n_elems < 1 || (size_t)n_elems > cap) return NFD_E_RANGE;
    c->cls = CLS_CACHE;
    const int grid = (int)(((size_t)n_elems + 255) / 256);
    if (is_f32)
        LAUNCH(c, (k_to_f32<float>), grid, 256, 0, (const float *)src, out, (size_t)n_elems);
    else
        LAUNCH(c, (k_to_f32<bf16>), grid, 256, 0, (const bf16 *)src, out, (size_t)n_elems);
    CK(cudaGetLastError());
    return NFD_OK;
}

int nfd_status(nfd_ctx *c) {
    if (!c) return NFD_E_NULLPTR;
    int s = 0;
    CK(cudaMemcpyAsync(&s, c->d_status, 4, cudaMemcpyDeviceToHost, c->st));
    CK(cudaStreamSynchronize(c->st));
    return s;
}

long long nfd_launch_count(nfd_ctx *c) { return c ? c->launches : 0; }

int nfd_cond_cache_stats(nfd_ctx *c, long long *hits, long long *misses) {
    if (!c) return NFD_E_NULLPTR;
    if (hits) *hits = c->cond_hits;
    if (misses) *misses = c->cond_misses;
    return NFD_OK;
}

int nfd_profile_begin(nfd_ctx *c) {
    if (!c) return NFD_E_NULLPTR;
    CK(cudaStreamSynchronize(c->st));
    c->prof = true;
    c->prof_used = 0;
    return NFD_OK;
}

int nfd_profile_end(nfd_ctx *c, int n_classes, long long *n_launches, float *total_ms) {
    if (!c || !n_launches || !total_ms) return NFD_E_NULLPTR;
    if (!c->prof) return NFD_E_STATE;
    c->prof = false;
    CK(cudaStreamSynchronize(c->st));
    for (int i = 0; i < n_classes; ++i) n_launches[i] = 0, total_ms[i] = 0.f;
    for (size_t i = 0; i + 1 < c->prof_used; i += 2) {
        float ms = 0.f;
        CK(cudaEventElapsedTime(&ms, c->prof_ev[i], c->prof_ev[i + 1]));
        int k = c->prof_cls[i / 2];
        if (k >= 0 && k < n_classes) n_launches[k]++, total_ms[k] += ms;
    }
    c->prof_used = 0;
    return NFD_OK;
}

int nfd_profile_class_count(void) { return CLS_COUNT; }

const char *nfd_profile_class_name(int id) { return (id >= 0 && id < CLS_COUNT) ? kClassNames[id] : ""; }

int nfd_set_option(nfd_ctx *c, const char *name, int value) {
    if (!c || !name) return NFD_E_NULLPTR;
    if (!strcmp(name, "graph")) {
        c->use_graph = value != 0;
        return NFD_OK;
    }
    if (!strcmp(name, "fast") || !strcmp(name, "fuse_ln")) {
        // cached modulation rows carry the folded-LayerNorm vectors only if they were filled while the
        // fold was active: start the cache afresh
        (name[1] == 'a' ? c->fast : c->fuse_ln) = value != 0;
        for (auto &cs : c->cond_slots) cs = nfd_ctx::CondSlot();
        return NFD_OK;
    }
    if (!strcmp(name, "l2_prefetch")) {
        c->l2_prefetch = value != 0;
        return NFD_OK;
    }
    if (!strcmp(name, "kv_prefetch")) {
        c->kv_prefetch = value != 0;
        return NFD_OK;
    }
    if (!strcmp(name, "clear_status")) {
        CK(cudaMemsetAsync(c->d_status, 0, 4, c->st));
        return NFD_OK;
    }
    if (!strcmp(name, "test_wait_limit_us") || !strcmp(name, "test_skip_stage")) {
        // words 1 and 2 of the status block (see nfd_sm100.cuh); 0 restores normal operation
        if (value < 0) return NFD_E_RANGE;
        const int word = name[5] == 'w' ? 1 : 2;
        c->test_words[word] = value;
        CK(cudaMemcpyAsync(c->d_status + word, &c->test_words[word], 4, cudaMemcpyHostToDevice, c->st));
        return NFD_OK;
    }
    if (!strcmp(name, "test_fail_launch")) {
        c->test_fail_launch = value != 0;
        return NFD_OK;
    }
    if (!strcmp(name, "test_corrupt_desc")) {
        c->test_corrupt_desc = value != 0;
        return NFD_OK;
    }
    if (!strcmp(name, "lazy_commit")) {
        if (!value)
            for (int s = 0; s < c->cfg.n_streams; ++s) RET(flush_pending(c, s));
        c->lazy = value != 0;
        return NFD_OK;
    }
    return NFD_E_RANGE;
}


#ifdef NFD_TRACE
// Timeline instrumentation (only in builds with -DNFD_TRACE): copy out the records gathered so far
// (host buffer of `cap` records of 24 bytes: t0, t1, kind, sm), reset the buffer, return their number.
int nfd_trace_read(nfd_ctx *c, void *host_buf, int cap) {
    if (!c || !host_buf) return NFD_E_NULLPTR;
    CK(cudaStreamSynchronize(c->st));
    unsigned int n = 0;
    CK(cudaMemcpyFromSymbol(&n, g_trace_n, sizeof(n)));
    if (n > NFD_TRACE_CAP) n = NFD_TRACE_CAP;
    if ((int)n > cap) n = (unsigned int)cap;
    CK(cudaMemcpyFromSymbol(host_buf, g_trace, (size_t)n * sizeof(NfdTraceRec)));
    const unsigned int zero = 0;
    CK(cudaMemcpyToSymbol(g_trace_n, &zero, sizeof(zero)));
    return (int)n;
}
#endif

}  // extern "C"

// ---------------------------------------------------------------------------
// Allocation-free attention entry point.
//
// The pass descriptor that the attention kernel reads (which frames are
// queried, which page window each may see) normally lives in memory the
// context allocated with cudaMalloc.  Here it lives in a fixed array that is
// part of the library image, so the call needs no allocator at all.
// ---------------------------------------------------------------------------
#define NFD_NOALLOC_SCRATCH_BYTES 4096
static __device__ __align__(256) unsigned char g_noalloc_scratch[NFD_NOALLOC_SCRATCH_BYTES];
#define NFD_NOALLOC_STATUS_OFFSET 3072       // four status ints behind the descriptor
static_assert(sizeof(StepParams) <= NFD_NOALLOC_STATUS_OFFSET, "pass descriptor must fit the static scratch");

#define NFD_NOALLOC_MAX_DEVICES 64
// Device address of g_noalloc_scratch per device ordinal.  In host code the
// symbol itself is only a stand-in, so its address is looked up once per device.
static void *g_noalloc_dev_ptr[NFD_NOALLOC_MAX_DEVICES] = {nullptr};

template <typename TS>
static int noalloc_launch(cudaStream_t st, const StepParams *d_sp, const Dims &D, int n_q, const void *q,
                          const void *k_pages, const void *v_pages, void *out) {
    const long long warps = (long long)n_q * D.T * D.H;
    const int grid = (int)((warps + 3) / 4);
    if (D.dh == 32)
        k_attn_simple<TS, 32><<<grid, 128, 0, st>>>(d_sp, D, 0, (const TS *)q, (const TS *)k_pages,
                                                    (const TS *)v_pages, (TS *)out);
    else if (D.dh == 64)
        k_attn_simple<TS, 64><<<grid, 128, 0, st>>>(d_sp, D, 0, (const TS *)q, (const TS *)k_pages,
                                                    (const TS *)v_pages, (TS *)out);
    else
        k_attn_simple<TS, 128><<<grid, 128, 0, st>>>(d_sp, D, 0, (const TS *)q, (const TS *)k_pages,
                                                     (const TS *)v_pages, (TS *)out);
    CK(cudaGetLastError());
    return NFD_OK;
}

extern "C" int nfd_attention_noalloc(const void *q, const void *k_pages, const void *v_pages, int dtype, int n_heads,
                          int head_dim, int tokens_per_frame, int n_q_frames, int n_kv_frames, int window,
                          void *out, void *cuda_stream) {
    if (!q || !k_pages || !v_pages || !out) return NFD_E_NULLPTR;
    if (!aligned16(q) || !aligned16(k_pages) || !aligned16(v_pages) || !aligned16(out)) return NFD_E_ALIGN;
    if (dtype != NFD_DTYPE_FP32 && dtype != NFD_DTYPE_BF16) return NFD_E_BADCFG;
    if (head_dim != 32 && head_dim != 64 && head_dim != 128) return NFD_E_BADCFG;
    if (n_heads < 1 || tokens_per_frame < 1 || window < 0) return NFD_E_RANGE;
    if (n_q_frames < 1 || n_q_frames > NFD_MAX_PASS_FRAMES) {
        fprintf(stderr, "libnfd: nfd_attention_noalloc: n_q_frames = %d, but the static scratch holds the "
                        "descriptors of at most %d query frames\n", n_q_frames, NFD_MAX_PASS_FRAMES);
        return NFD_E_RANGE;
    }
    if (n_kv_frames < n_q_frames || n_kv_frames > 65536) return NFD_E_RANGE;
    // sizes whose products the kernel forms in 32-bit integers (model width, rows of the pass, grid)
    if (n_heads > 1024 || tokens_per_frame > (1 << 20)) return NFD_E_RANGE;
    const long long rows_ll = (long long)n_q_frames * tokens_per_frame;
    const long long warps_ll = rows_ll * n_heads;
    if (rows_ll > 0x7fffffffLL / 4 || (warps_ll + 3) / 4 > 0x7fffffffLL) return NFD_E_RANGE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int dev = -1;
    CK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= NFD_NOALLOC_MAX_DEVICES) return NFD_E_RANGE;
    if (!g_noalloc_dev_ptr[dev]) {
        // one-time set-up for the current device: turn the symbol into a device address
        void *p = nullptr;
        CK(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        if (!p) return NFD_E_CUDA;
        g_noalloc_dev_ptr[dev] = p;
    }
    StepParams *d_sp = (StepParams *)g_noalloc_dev_ptr[dev];
    // the descriptor check of k_set_params records a failure in a status word; it lives in the same array
    int *d_stat = (int *)((unsigned char *)g_noalloc_dev_ptr[dev] + NFD_NOALLOC_STATUS_OFFSET);
    Dims D;
    memset(&D, 0, sizeof(D));
    D.L = 1, D.H = n_heads, D.dh = head_dim, D.d = n_heads * head_dim, D.T = tokens_per_frame;
    D.R = n_kv_frames, D.W = window, D.n_streams = 1;
    D.page_elems = (size_t)n_heads * tokens_per_frame * head_dim;
    StepParams p;
    memset(&p, 0, sizeof(p));
    p.nf = n_q_frames;
    p.nc = 1;
    for (int j = 0; j < n_q_frames; ++j) {
        p.fr[j].stream = 0;
        p.fr[j].frame = n_kv_frames - n_q_frames + j;
        p.fr[j].win_first = p.fr[j].frame - window > 0 ? p.fr[j].frame - window : 0;
        p.fr[j].first_new = n_kv_frames - n_q_frames;
    }
    DescLimits lim;
    lim.n_streams = 1, lim.W = window, lim.n_slots = 1, lim.n_actions = 1, lim.max_frames = NFD_MAX_PASS_FRAMES;
    lim.pend_slots = 1;
    // the descriptor is rewritten in full on every call; nothing of the previous call survives
    k_set_params<<<1, 256, 0, st>>>(p, d_sp, lim, d_stat);
    CK(cudaGetLastError());
    if (dtype == NFD_DTYPE_BF16) return noalloc_launch<bf16>(st, d_sp, D, n_q_frames, q, k_pages, v_pages, out);
    return noalloc_launch<float>(st, d_sp, D, n_q_frames, q, k_pages, v_pages, out);
}

/*
 * nfd.h -- C ABI of libnfd: the few-step denoising forward pass of a block-wise
 * causal diffusion transformer with a frame-paged KV cache and k-frame
 * speculative decoding (Next-Frame Diffusion, arxiv 2506.01380), for one
 * NVIDIA B200 (sm_100a).
 *
 * Conventions
 *   - "dev" pointers are CUDA device pointers, "host" pointers ordinary host
 *     memory.  The caller owns every pointer it passes.  The library owns the
 *     context, its repacked weights, the KV cache, activations and graphs.
 *   - All device work is enqueued on the CUDA stream given to nfd_create.
 *     Calls are asynchronous with respect to the host unless stated otherwise.
 *   - Every function returns 0 on success or a negative NFD_E_* code.  A failed
 *     call leaves the cache and its counters unchanged.  Nothing throws or
 *     aborts across this boundary.
 *   - A frame is a latent [C, H, W] (row-major, fp32).  It is cut into
 *     (H/p)*(W/p) tokens in row-major order over (row, col); a token's patch
 *     vector is ordered (channel, py, px).
 *   - "stream" (int) below is a batch slot: an independent generation stream
 *     with its own cache, 0 <= stream < cfg.n_streams.
 *   - Frames are numbered 0,1,2,... per stream since the last nfd_reset.  A
 *     frame f attends to frames max(0, f - W) .. f  (W = cfg.ctx_frames):
 *     bidirectionally inside f, causally to the earlier ones.
 */
#ifndef NFD_H_
#define NFD_H_

#ifdef __cplusplus
extern "C" {
#endif

#define NFD_OK          0
#define NFD_E_BADCFG   -1   /* inconsistent or unsupported configuration          */
#define NFD_E_NULLPTR  -2   /* a required pointer is NULL                          */
#define NFD_E_ALIGN    -3   /* a device pointer is not 16-byte aligned             */
#define NFD_E_RANGE    -4   /* an index / count argument is out of range           */
#define NFD_E_STATE    -5   /* call not allowed in the cache's current state       */
#define NFD_E_NOMEM    -6   /* device or host allocation failed                    */
#define NFD_E_CUDA     -7   /* a CUDA runtime call failed                          */
#define NFD_E_TIMEOUT  -8   /* a bounded device-side wait gave up                  */
#define NFD_E_DEVICE   -9   /* a device-side consistency check failed              */

#define NFD_DTYPE_FP32 0    /* validation mode: fp32 storage and arithmetic        */
#define NFD_DTYPE_BF16 1    /* bf16 operands / cache, fp32 accumulation & residual */

#define NFD_MAX_PASS_FRAMES 32   /* frames one forward pass can carry (streams x k) */

typedef struct nfd_ctx nfd_ctx;

/* Model and cache configuration.  Architecture: Section 3.1 of the paper (DiT
 * with block-wise causal attention, adaLN-zero conditioning on timestep +
 * action, 3D rotary embedding); sampler constants: Section 4.1. */
typedef struct {
    int n_layers, d_model, n_heads, head_dim, d_mlp;   /* n_heads*head_dim == d_model; head_dim in {32,64,128} */
    int latent_c, latent_h, latent_w, patch;            /* tokens/frame T = (h/p)*(w/p); patch vector P = c*p*p  */
    int n_actions;                                      /* one categorical action per frame                      */
    int ctx_frames;                                     /* W: earlier frames a frame attends to                  */
    int max_spec;                                       /* k_max: frames decoded together, 1..8                  */
    int n_streams;                                      /* independent batch slots                               */
    int dtype;                                          /* NFD_DTYPE_*                                           */
    int norm;                                           /* 0 LayerNorm (no affine), 1 RMSNorm                    */
    int act;                                            /* 0 exact (erf) GELU; 1 gated: SiLU(gate) * up          */
    int rope_t, rope_h, rope_w;                         /* even, sum == head_dim (Section 3.1, 3D pos. emb.)     */
    float rope_theta, norm_eps, t_scale;                /* t_scale multiplies the FM time before the sinusoid    */
    float sigma_d;                                      /* TrigFlow data scale (Section 4.1)                     */
    float t_ctx_trig;                                   /* TrigFlow time of the context-noise level (Sec. 4.3)   */
    int n_steps;                                        /* sampling steps S (Section 4.1 "Sampling": 4)          */
} nfd_cfg;

/* Weights: dev pointers, each matrix row-major [in, out], element type given by
 * cfg.dtype (float or bf16).  Per-layer arrays are host arrays of n_layers dev
 * pointers.  nfd_create copies and repacks them; the caller may free its
 * copies afterwards. */
typedef struct {
    const void *w_pe, *b_pe;                 /* [P,d], [d]      patch embedding                          */
    const void *w_t1, *b_t1, *w_t2, *b_t2;   /* [256,d],[d],[d,d],[d]  timestep-embedding MLP (SiLU)     */
    const void *a_emb;                       /* [n_actions,d]   action embedding (linear on one-hot)     */
    const void *const *w_mod, *const *b_mod; /* [d,6d],[6d]     adaLN: shift,scale,gate (attn), same (mlp) */
    const void *const *w_qkv, *const *b_qkv; /* [d,3d],[3d]     columns: q | k | v, each head-major      */
    const void *const *w_o,   *const *b_o;   /* [d,d],[d]                                                */
    const void *const *w_fc1, *const *b_fc1; /* [d,d_mlp],[d_mlp]; act 1: [d,2 d_mlp],[2 d_mlp], gate first */
    const void *const *w_fc2, *const *b_fc2; /* [d_mlp,d],[d]                                            */
    const void *w_fmod, *b_fmod;             /* [d,2d],[2d]     final adaLN: shift, scale                */
    const void *w_out, *b_out;               /* [d,P],[P]       velocity head                            */
} nfd_weights;

/* Create a context.  `cuda_stream` is a cudaStream_t (NULL = legacy default
 * stream).  Validates cfg (NFD_E_BADCFG), copies/repacks the weights, allocates
 * the cache: n_streams x n_layers x (W + 2 k_max) frame pages of K and of V.
 * In bf16 mode the first context of a shape in the process also times its GEMM
 * tile plans on scratch data (about half a second; the environment variable
 * NFD_NO_TUNE=1 skips it and keeps the built-in cost model's plans); the cache is
 * cleared afterwards.  The plan found fixes, among other things, over how many
 * thread blocks the K range of a projection is split, hence the order in which
 * its products are summed: all contexts of one process share the plans and give
 * bitwise equal results for equal inputs, two processes may differ in the last
 * bits (NFD_NO_TUNE=1 makes the plans, and with them the bits, the same
 * everywhere).  A bf16 context needs the driver's cuTensorMapEncodeTiled entry
 * point; without it the call fails with NFD_E_CUDA rather than run the plain
 * validation kernels unasked.  Synchronises the stream before returning. */
int nfd_create(nfd_ctx **out, const nfd_weights *w, const nfd_cfg *cfg, void *cuda_stream);
int nfd_destroy(nfd_ctx *ctx);

/* Empty one batch slot's cache and restart its frame numbering at 0. */
int nfd_reset(nfd_ctx *ctx, int stream);

/* One forward pass v_theta(x_t | cached frames, t, action) (Section 3.2, the
 * argument of the Flow-Matching loss) over k frames decoded together: they
 * follow the cached frames, share the FM time t and the action, and are
 * block-causal among themselves (Section 4.2).  x_t: dev fp32 [k,C,H,W], the
 * model input (already in Flow-Matching scale).  v_out: dev fp32 [k,C,H,W].
 * The k frames' K/V are left in scratch pages after the cached frames; they are
 * not counted by the cache until a commit.  1 <= k <= k_max. */
int nfd_denoise_step(nfd_ctx *ctx, int stream, const float *x_t, int k, float t, int action, float *v_out);

/* As nfd_denoise_step, but the k frames start `offset` frames after the cached
 * ones and the scratch K/V that earlier calls left for those `offset` frames
 * serve as context (offset + k <= k_max).  A joint k-frame pass equals k
 * single-frame calls with offset = 0..k-1. */
int nfd_denoise_step_at(nfd_ctx *ctx, int stream, int offset, const float *x_t, int k, float t, int action,
                        float *v_out);

/* The same pass for n batch slots at once (independent streams, one launch):
 * streams[n] host, x_t dev [n,k,C,H,W], t[n] host, actions[n] host,
 * v_out dev [n,k,C,H,W].  n*k <= NFD_MAX_PASS_FRAMES. */
int nfd_denoise_step_batched(nfd_ctx *ctx, int n, const int *streams, const float *x_t, int k, const float *t,
                             const int *actions, float *v_out);

/* Append n clean frames to the cache (Appendix "KV caching": the K/V of the
 * noisy versions of generated frames are computed once and reused).  Each frame
 * is perturbed to the context-noise level, x' = cos(t_ctx) x0 + sin(t_ctx)
 * sigma_d z (Section 4.3), fed at that constant timestep with the action that
 * produced it, and its K/V written to the next pages.  x0 dev fp32 [n,C,H,W];
 * actions host [n]; ctx_noise dev fp32 [n,C,H,W] or NULL (z = 0).
 * Requires no tentative frames (NFD_E_STATE).  1 <= n <= k_max. */
int nfd_commit_frame(nfd_ctx *ctx, int stream, const float *x0, int n, const int *actions, const float *ctx_noise);

/* Generate k frames speculatively under `action` (Section 4.2): S sampling
 * steps (Section 4.1 "Sampling": denoise, then re-noise to the next timestep)
 * over the k frames decoded together, then append the k clean frames as
 * TENTATIVE.  noise dev fp32 [S,k,C,H,W] (N(0,1): step 0 is the initial sample,
 * step s>0 the re-noising draw); ctx_noise dev [k,C,H,W] or NULL; x0_out dev
 * fp32 [k,C,H,W] receives the clean frames.  Requires no tentative frames.
 *
 * The K/V pages of the k frames are not written by this call: the library keeps
 * a copy of the clean frames, their context noise and the action, counts the
 * frames as tentative, and lets them ride along (K/V only) in the first
 * denoising pass of the next nfd_speculate on this batch slot, which is where
 * the paper's appendix on KV caching places that computation.  Any call that needs the pages earlier (nfd_kv_hash,
 * nfd_kv_read, nfd_denoise_step*, nfd_commit_frame) writes them first.  Results
 * are bitwise those of committing at once (option "lazy_commit" = 0). */
int nfd_speculate(nfd_ctx *ctx, int stream, int k, int action, const float *noise, const float *ctx_noise,
                  float *x0_out);

/* nfd_speculate for n batch slots at once: streams[n], actions[n] host;
 * noise dev [S,n,k,C,H,W]; ctx_noise dev [n,k,C,H,W] or NULL; x0_out dev [n,k,C,H,W]. */
int nfd_speculate_batched(nfd_ctx *ctx, int n, const int *streams, int k, const int *actions, const float *noise,
                          const float *ctx_noise, float *x0_out);

/* Resolve a speculation (Section 4.2: frames after the first action mismatch are
 * discarded, generation resumes from the last verified frame): the first
 * n_accept tentative frames become committed, the rest are dropped (frames whose
 * commit was still deferred are simply forgotten).  Counters only; no data
 * moves.  0 <= n_accept <= n_tentative. */
int nfd_rollback(nfd_ctx *ctx, int stream, int n_accept);

/* Cache counters (host ints, any may be NULL): committed frames, tentative
 * frames, and the first frame the next new frame can see. */
int nfd_kv_state(nfd_ctx *ctx, int stream, int *n_committed, int *n_tentative, int *window_first);

/* 64-bit digest of the counters and of the raw K/V bits of the visible cached
 * frames (the last W), in frame order.  Synchronises the stream. */
int nfd_kv_hash(nfd_ctx *ctx, int stream, unsigned long long *h);

/* Copy one frame's K and V of one layer to dev fp32 buffers [n_heads, T, head_dim]
 * (either may be NULL).  `frame` is absolute; it must be a cached frame still in
 * the ring or one of the scratch frames of the last pass. */
int nfd_kv_read(nfd_ctx *ctx, int stream, int layer, int frame, float *k_out, float *v_out);

/* Block-wise causal attention alone (Section 3.1), for kernel-level tests and
 * timing.  q dev [n_heads, n_q_frames*T, head_dim]; k, v dev
 * [n_heads, n_kv_frames*T, head_dim] in the context's storage type (bf16 or
 * fp32).  Query frame j is frame number (n_kv_frames - n_q_frames + j) of the
 * key sequence and sees key frames max(0, that - window) .. that.  out: dev,
 * storage type, [n_q_frames*T, n_heads*head_dim].  The data are first copied
 * into cache pages of batch slot 0 (which is reset), then the same attention
 * kernel the forward pass uses runs on them.
 * n_kv_frames <= W + 2 k_max, n_q_frames <= k_max, window <= W. */
int nfd_attention(nfd_ctx *ctx, const void *q, const void *k, const void *v, int n_q_frames, int n_kv_frames,
                  int window, void *out);

/* Block-wise causal attention for callers that must not allocate.  (The paper
 * has no counterpart of this call; it exists for integration reasons only.)
 *
 * Some hosts of this library cannot call cudaMalloc at the point where they
 * need attention: code running while a CUDA graph is being captured, a
 * real-time frame loop that forbids allocator calls after start-up, a process
 * whose device memory is handed out by an arena owned by someone else.  This
 * call creates no context and calls no cudaMalloc / cudaFree and no allocating
 * library routine.  Its only working memory, the descriptor of the query frames
 * that the kernel reads, is a fixed 4 KiB array inside the library image; every
 * GPU that loads the library holds those 4 KiB until the process exits.
 *
 *   q        dev [n_heads, n_q_frames*T, head_dim]
 *   k_pages  dev [n_kv_frames, n_heads, T, head_dim]   (frame pages, as the cache stores them)
 *   v_pages  dev [n_kv_frames, n_heads, T, head_dim]
 *   out      dev [n_q_frames*T, n_heads*head_dim]
 *   dtype    NFD_DTYPE_FP32 or NFD_DTYPE_BF16: element type of all four
 *   T = tokens_per_frame.  Query frame j is key frame (n_kv_frames - n_q_frames + j)
 *   and sees key frames max(0, that - window) .. that.
 *
 * Limit: n_q_frames <= NFD_MAX_PASS_FRAMES (32) -- more descriptors do not fit
 * the fixed array; larger values return NFD_E_RANGE and print the reason.
 * The first call on each device looks up the array's device address (with that
 * device current); make that first call outside any stream capture.
 * All calls on a device share the one array: it is rewritten in full by every
 * call, so nothing needs clearing, but two calls whose kernels overlap on the
 * GPU (different streams) race on it -- serialise them.
 * Runs the plain attention kernel on `cuda_stream` (a cudaStream_t). */
int nfd_attention_noalloc(const void *q, const void *k_pages, const void *v_pages, int dtype, int n_heads,
                          int head_dim, int tokens_per_frame, int n_q_frames, int n_kv_frames, int window,
                          void *out, void *cuda_stream);

/* Device-side status latch: 0, or the first NFD_E_* a kernel recorded.
 * NFD_E_TIMEOUT: a bounded wait inside a kernel (on an mbarrier that a TMA copy or
 * a tensor-core operation completes) ran out after 0.4 s; the kernel skipped the
 * rest of its work and left by its normal exit, so the context still runs, but
 * the results of that pass are void.  NFD_E_DEVICE: the first kernel of a pass
 * found an index in the pass descriptor outside the context's limits (batch slot,
 * window, modulation row, frame slots); the frames of that pass were redirected
 * to batch slot 0 so that no kernel left its buffers: treat every cache of the
 * context as lost (nfd_reset).  The latch keeps the first code until
 * nfd_set_option("clear_status", 1).  Synchronises the stream. */
int nfd_status(nfd_ctx *ctx);

/* Verification of a speculation (Section 4.2 and the control flow of the
 * appendix listing): frames i .. i+k-1 were generated under actions[i]
 * (host array of the n true actions).  Returns how many leading frames were
 * generated under their own true action -- at least 1, at most k and n - i --
 * which is the n_accept to pass to nfd_rollback; or a negative code. */
int nfd_accepted_count(const int *actions, int n, int i, int k);

/* Copy the first n_elems elements of one activation buffer of the last pass to
 * dev fp32 memory, for kernel-level tests: "z" the residual stream [rows, d]
 * (fp32), "hbuf" the operand of the QKV / first MLP projection [rows, d], "qbuf"
 * the rotated queries [n_heads, rows, head_dim], "abuf" the attention output
 * [rows, d], "mbuf" the MLP hidden activation [rows, d_mlp rounded up to a
 * multiple of 8].  rows = frames of the pass x T.  Buffers are reused by every
 * layer, so what is read belongs to the last layer that wrote it.
 * NFD_E_RANGE for another name or more elements than the buffer holds. */
int nfd_debug_read(nfd_ctx *ctx, const char *name, float *out, long long n_elems);

/* Number of kernels the library launched (or replayed inside graphs) since
 * creation. */
long long nfd_launch_count(nfd_ctx *ctx);

/* The adaLN modulation of a frame (Section 3.1, "Action Conditioning") depends on
 * its (FM time, action) pair only.  The library keeps the modulation of the most
 * recently used pairs (256 of them) and computes a pair's modulation only when it
 * is not there.  Returns how many pairs were found (hits) and how many had to be
 * computed (misses) since creation; either pointer may be NULL. */
int nfd_cond_cache_stats(nfd_ctx *ctx, long long *hits, long long *misses);

/* Per-kernel timing.  Between nfd_profile_begin and nfd_profile_end every
 * kernel is launched directly (no graph replay) with a CUDA event before and
 * after it on the context's stream.  nfd_profile_end synchronises and returns,
 * per kernel class id < n_classes, the number of launches and their summed
 * device time in milliseconds (host arrays of n_classes entries).  Class ids
 * run 0 .. nfd_profile_class_count()-1 and are named by
 * nfd_profile_class_name. */
int nfd_profile_begin(nfd_ctx *ctx);
int nfd_profile_end(nfd_ctx *ctx, int n_classes, long long *n_launches, float *total_ms);
int nfd_profile_class_count(void);
const char *nfd_profile_class_name(int id);

/* The undistilled sampler of Section 3.2 "Sampling": the Flow-Matching model integrated from pure noise with
 * DPM-Solver++ (the multistep second-order solver for data-prediction models; data prediction x0 = x_t - t v)
 * in n_evals function evaluations (18 in the paper's experiments) for k frames decoded together under
 * `action`.  The paper gives neither grid nor order: equal steps of FM time from 1 to 0, second order except
 * for the first two steps (no finite previous step: lambda is infinite at t = 1) and the last one.
 * noise dev [k,C,H,W] (unit variance), ctx_noise dev [k,C,H,W] or NULL, x0_out dev [k,C,H,W].  Like
 * nfd_speculate it leaves the k frames in the cache as tentative (committed at once, not deferred); pending
 * frames of the stream are written first.  Errors as nfd_speculate; n_evals outside 1..1000: NFD_E_RANGE. */
int nfd_sample_dpmpp(nfd_ctx *ctx, int stream, int k, int action, int n_evals, const float *noise,
                     const float *ctx_noise, float *x0_out);

/* Fills the modulation cache for every (time, action) pair that nfd_speculate
 * and the commits can ask for: the n_steps sampler times (Section 4.1
 * "Sampling") and the context time (Section 4.3), each with every action.  The
 * adaLN modulation depends on nothing else (Section 3.1 "Action Conditioning"),
 * so after this call a generation loop runs no conditioning kernels at all.
 * Returns the number of pairs computed (pairs already cached are left alone),
 * NFD_E_RANGE if (n_steps + 1) * n_actions exceeds the cache's 256 rows (nothing
 * is done then: the cache keeps working on demand), or another negative code.
 * Asynchronous on the context's stream. */
int nfd_warm_modulation(nfd_ctx *ctx);

/* Run-time switches, for tests and profiling: "graph" 0/1 (replay CUDA graphs
 * or launch kernels directly), "fast" 0/1 (tensor-core kernels or the plain
 * validation kernels; bf16 only), "lazy_commit" 0/1 (defer the commit of
 * speculated frames into the next speculation's first pass, or commit them at
 * once), "fuse_ln" 0/1 (bf16 tensor-core path: fold the two adaLN LayerNorms of
 * every block into the epilogues of the neighbouring GEMMs, or run them as
 * kernels of their own; the two differ by bf16 rounding of the GEMM operand
 * only), "l2_prefetch" 0/1 (each GEMM pulls the next GEMM's weights towards
 * L2; on by default), "kv_prefetch" 0/1 (the QKV GEMM pulls the layer's cached
 * K/V pages towards L2 ahead of the attention kernel; off by default, it was
 * measured slower), "clear_status" (reset the device-side status latch).  Changing "fast" or "fuse_ln" empties the
 * modulation cache.
 * Switches that exist for the tests of the error paths; each makes a fault on
 * the host or lets a bounded wait expire, none makes the device fault:
 * "test_fail_launch" 1: the next nfd_speculate's first launch asks for a block
 * size the runtime refuses, so the call returns NFD_E_CUDA; "test_corrupt_desc"
 * 1: the next pass descriptor names a batch slot that does not exist, which the
 * pass's first kernel must catch (NFD_E_DEVICE); "test_skip_stage" 1/0: the TMA
 * producer of every tensor-core GEMM leaves out its last pipeline stage, so that
 * the consumer's wait for it expires (NFD_E_TIMEOUT); "test_wait_limit_us" n:
 * bounded waits give up after n microseconds instead of 0.4 s (0 = default).
 * Returns NFD_E_RANGE for unknown names. */
int nfd_set_option(nfd_ctx *ctx, const char *name, int value);

const char *nfd_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* NFD_H_ */

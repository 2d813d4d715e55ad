/*
 * cpe.h - C ABI of the centroid-positional-encoding decoder for NVIDIA B200 (sm_100a).
 *
 * The library turns a dense per-pixel sinusoidal encoding of instance centroids into instance
 * masks: every participating pixel's embedding is decoded to a centroid estimate, the estimates
 * vote into an integer centroid map, local maxima of that map become instance centres, and every
 * participating pixel is assigned to the centre whose encoding is nearest.
 *
 * Notation follows the paper: F harmonics per axis (the paper's L), D = 4F channels,
 * gamma(p) = (sin(2^l pi p), cos(2^l pi p)), l = 0..F-1 (Eq. 2); palettes P_n hold gamma at the bin
 * positions -1 + 2i/(n+1), i = 1..n (Eq. 9); the vote map has B_w x B_h bins (Sec. 3.2).
 *
 * Conventions
 *   emb       planar [B][4F][H][W], contiguous, element type given by cpe_params.dtype.
 *             channel c = axis*2F + 2l + t; axis 0 = x (width), 1 = y (height); t = 0 sin, 1 cos
 *             (Eq. 1-3: concat(gamma(x), gamma(y)), each gamma as (sin, cos) per harmonic).
 *   fg_mask   [B][H][W] bytes; a pixel participates iff its byte is non-zero.  NULL: all pixels
 *             participate (the paper's set S is the whole output grid, Eq. 6).
 *   images of a batch are independent: own vote map, own peak list, labels numbered from 1.
 *
 * All pointers named "device" are device memory owned by the caller; nothing in the stream-taking
 * entry points allocates, frees, synchronises or reads device memory on the host, so they may be
 * called while the stream is being captured into a CUDA graph.  Return value: 0 (CPE_OK) or a
 * negative CPE_ERR_* code, reported before any work is enqueued.  Run-time conditions (more peaks
 * than max_instances, non-finite pixels) are reported in the device status word, never as faults.
 */
#ifndef CPE_H_
#define CPE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* A CUDA stream handle (cudaStream_t / CUstream); 0 is the legacy default stream. */
typedef struct CUstream_st* cpe_stream_t;

enum { CPE_F32 = 0, CPE_F16 = 1 };

enum {
  CPE_OK = 0,
  CPE_ERR_NULL = -1,       /* a required pointer is NULL                                  */
  CPE_ERR_SIZE = -2,       /* B, H, W < 1, F outside [1,16], bins outside [1,4096], ...    */
  CPE_ERR_DTYPE = -3,      /* unknown element type                                         */
  CPE_ERR_ALIGN = -4,      /* emb / outputs not aligned to their element size              */
  CPE_ERR_WORKSPACE = -5,  /* workspace missing, misaligned (256 B) or too small           */
  CPE_ERR_PARAM = -6,      /* struct_size mismatch, negative threshold, max_instances < 1  */
  CPE_ERR_CUDA = -7,       /* a CUDA runtime call failed (see cpe_last_cuda_error)         */
  CPE_ERR_WHICH = -8,      /* unknown intermediate id, or it was not requested by flags    */
  CPE_ERR_NOMEM = -9,      /* host or device allocation failed (context helpers only)      */
  CPE_ERR_STATIC_LIMIT = -10, /* the problem needs more scratch than cpe_decode_static has      */
  CPE_ERR_BUSY = -11       /* host front end: two calls are already in flight (or, for the
                              synchronous call, one is)                                    */
};

/* cpe_params.flags */
enum {
  CPE_FLAG_WRITE_SCORES = 1u, /* also store the best and second-best Eq. 4 distance of every pixel */
  CPE_FLAG_EXACT_ASSIGN = 2u, /* score every (pixel, peak) pair in binary32 on the plain ALUs instead of
                                 filtering with the tensor cores first; same results, for cross-checking */
  CPE_FLAG_FILTER_ASSIGN = 8u,/* use the tensor-core filtered kernel for every image, however few peaks it has
                                 (by default images with few peaks take the all-pairs kernel); same results   */
  CPE_FLAG_KEEP_VOTES = 4u,   /* leave the vote map readable after the decode (CPE_INT_VOTES).  Without it the
                                 last kernel of a decode re-zeroes the map for the next decode, which saves the
                                 clearing pass at the start; with it every decode starts with that pass.       */
  CPE_FLAG_NO_PDL = 32u,      /* launch the kernels of a decode plainly, without programmatic stream serialisation
                                 (A/B timing; same results)                                                    */
  CPE_FLAG_TC_ALL_ROUNDS = 64u,   /* filtered assignment: let the tensor-memory (tcgen05) body take every image whose
                                     peaks fit its shared-memory operand, in rounds of 64, instead of handing images
                                     with more than 128 peaks to the mma.sync body (tests, comparisons; same results) */
  CPE_FLAG_TC_ONE_STAGE = 128u,   /* ... or only images with at most 64 peaks (one tensor-memory stage per tile)     */
  CPE_FLAG_MMA_ASSIGN = 256u,     /* filtered assignment: the mma.sync kernel for every image (comparisons)          */
  CPE_FLAG_NO_PRUNE = 512u,       /* do not prune the candidates of Eq. 7 (see cpe_decode): every image with more peaks
                                     than the all-pairs range goes to the tensor-core filtered kernels; same results  */
  CPE_FLAG_PRUNE_ALL = 1024u,     /* the pruned assignment however small the input is and whatever max_instances is
                                     (it serves every image of a decode, also those with few peaks); same results     */
  CPE_FLAG_PRUNE_ANY_SIZE = 8192u,/* the pruned assignment also for inputs of fewer than 2^19 pixels (by default those
                                     go without it: its extra launches cost more than it saves there); same results    */
  CPE_FLAG_PRUNE_WALK_ONLY = 2048u, /* pruned assignment: the one-thread-per-pixel kernel also where the streaming kernel
                                       would run (tests, comparisons; same results)                                   */
  CPE_FLAG_TEST_STALL = 4096u,    /* tests of the time-out path only: the tensor-memory assignment's producer warps
                                     withhold the arrival of each CTA's first tile, so that the consumers' bounded wait
                                     runs out, the kernel winds down and returns, and CPE_STATUS_TIMEOUT is set (the
                                     label map of that decode is incomplete)                                          */
  CPE_FLAG_FUSE_PEAKS = 32768u,   /* small inputs (at most 2^20 pixels, vote maps of at most 8192 bins, no pruned
                                     assignment): the voting kernel's last CTA of each image also searches the map
                                     for the peaks, one kernel launch fewer per decode; same results.  Off by default:
                                     the hand-over inside the kernel (ticket, fences) measured 2 to 4 us SLOWER per
                                     decode than the separate launch it saves                                          */
  CPE_FLAG_SOFT_VOTE = 16384u,    /* vote as the paper prints it: the map is the real-valued histogram of Eq. 6,
                                     H(a, b) = sum over the participating pixels of exp(-d) with d of Eq. 4 (the sum
                                     that cpe_soft_votes computes, same accuracy), instead of the integer counts of the
                                     hard vote.  A bin is a candidate centroid iff H > soft_threshold and H exceeds
                                     each existing 8-neighbour STRICTLY (Sec. 3.2 as printed: no tie rule; equal
                                     neighbours are both rejected).  Assignment, outputs and counters are as usual;
                                     CPE_INT_VOTES and CPE_INT_PEAK_VOTES then hold binary32 values of H;
                                     vote_threshold and levels are ignored.  Needs emb 16-byte aligned and H*W a
                                     multiple of 8; not combinable with CPE_FLAG_REFINE (CPE_ERR_PARAM).  The candidates
                                     are never pruned in this mode.                                                   */
  CPE_FLAG_REFINE = 16u       /* sub-cell refined centroids (an extension: the paper's candidates of Eq. 7 are the
                                 bin positions of Eq. 9, up to half a bin off the voted centroid).  Next to its
                                 count every bin keeps the sum of the estimates that fell into it, as integers
                                 rint(p * 2^24) so that the sums do not depend on the order of addition
                                 (CPE_INT_VOTE_SUMS).  A peak is then placed at the mean estimate of its 3x3
                                 neighbourhood, mean = (sum of the sums) / (2^24 * sum of the counts) in binary64:
                                 out_centroids holds that mean in pixel units and the peak's candidate embedding
                                 is gamma(mean) of Eq. 2 (binary64 sin/cos, rounded once) instead of the palette
                                 rows.  Peak detection and everything else are unchanged.  Needs a larger
                                 workspace (16 bytes per bin and image); maps of more than 8192 bins, and decodes
                                 with CPE_FLAG_KEEP_VOTES, add one clearing pass per decode.                  */
};

/* bits of the per-image device status words */
enum {
  CPE_STATUS_PEAK_OVERFLOW = 1u, /* an image had more local maxima than max_instances            */
  CPE_STATUS_NONFINITE = 2u,     /* at least one participating pixel had a non-finite channel    */
  CPE_STATUS_INTERNAL = 4u,      /* an index self-check failed (site code in bits 8..15); the access was
                                    skipped.  Never set by a correct build: please report it.      */
  CPE_STATUS_TIMEOUT = 8u        /* a bounded device-side wait (on an mbarrier of the tensor-core pipeline) ran
                                    out; the kernel wound down and returned, the image's label map is
                                    incomplete.  Never set by a correct build on a healthy GPU.    */
};

/* per-image counters, uint32 [B][CPE_CNT_N] */
enum {
  CPE_CNT_VOTING = 0,       /* pixels that cast a vote                                      */
  CPE_CNT_NONFINITE = 1,    /* participating pixels skipped because a channel was not finite */
  CPE_CNT_RAW_PEAKS = 2,    /* local maxima found before truncation to max_instances        */
  CPE_CNT_TRUNCATED = 3,    /* local maxima dropped by the truncation                       */
  CPE_CNT_TAU_REJECTED = 4, /* pixels whose best distance was not below tau (label 0)       */
  CPE_CNT_FILTER_PAIRS = 5, /* (pixel, peak) pairs that survived the tensor-core filter     */
  CPE_CNT_RESCORED = 6,     /* pixels decided by exact re-scoring of several candidates     */
  CPE_CNT_FULL_SCORED = 7,  /* pixels for which every peak was scored exactly               */
  CPE_CNT_N = 8
};

/* ids for cpe_get_intermediate */
enum {
  CPE_INT_VOTES = 0,        /* uint32 [B][bins_h][bins_w]       hard-vote map (CPE_FLAG_KEEP_VOTES)  */
  CPE_INT_PEAK_CELLS = 1,   /* int32  [B][max_instances]        linear bin cy*bins_w+cx, ascending */
  CPE_INT_PEAK_VOTES = 2,   /* uint32 [B][max_instances]        votes of each kept peak         */
  CPE_INT_PEAK_EMB = 3,     /* float  [B][max_instances][4F]    concat(P_w[cx], P_h[cy]); with
                                                                CPE_FLAG_REFINE gamma of the refined position */
  CPE_INT_PALETTE_W = 4,    /* float  [bins_w][2F]              Eq. 9                           */
  CPE_INT_PALETTE_H = 5,    /* float  [bins_h][2F]                                              */
  CPE_INT_BEST_SCORE = 6,   /* float  [B][H][W]  (CPE_FLAG_WRITE_SCORES) +inf where none        */
  CPE_INT_SECOND_SCORE = 7, /* float  [B][H][W]  (CPE_FLAG_WRITE_SCORES) +inf where none        */
  CPE_INT_STATUS = 8,       /* uint32 [B]                       CPE_STATUS_* bits of each image      */
  CPE_INT_COUNTERS = 9,     /* uint32 [B][CPE_CNT_N]                                            */
  CPE_INT_VOTE_SUMS = 10,   /* int64  [B][bins_h][bins_w][2]    fixed-point (2^-24) sums of the x and y
                                                                estimates per bin (CPE_FLAG_REFINE and
                                                                CPE_FLAG_KEEP_VOTES)                 */
  CPE_INT_PRUNE_STATE = 11, /* uint32 [B][12] the pruned assignment's words of each image (only when it is enabled):
                                                [0] pixels visited, [1] pixels whose candidate list did not settle them,
                                                [2] non-zero: the image was handed to the tensor-core filtered kernel,
                                                [3] pixels queued for the exact walk, [4..7] its own counters (folded
                                                into CPE_INT_COUNTERS), [8] pixels queued for the scan of every peak */
  CPE_INT_N = 12
};

/* stages reported by cpe_profile_decode */
enum {
  CPE_STAGE_CLEAR = 0,      /* zeroing of the vote map (only with CPE_FLAG_KEEP_VOTES; else ~0)  */
  CPE_STAGE_DECODE_VOTE = 1,
  CPE_STAGE_PEAKS = 2,      /* local-maximum test, ordered peak list, centroids, peak embeddings */
  CPE_STAGE_LISTS = 3,      /* per-peak candidate lists of the pruned assignment (~0 without it) */
  CPE_STAGE_ASSIGN = 4,     /* assignment and label-map write                                    */
  CPE_STAGE_N = 5
};

typedef struct cpe_params {
  uint32_t struct_size;    /* sizeof(cpe_params)                                               */
  int32_t dtype;           /* CPE_F32 or CPE_F16 (IEEE binary16) element type of emb           */
  int32_t bins_w, bins_h;  /* B_w, B_h: vote-map size (Sec. 3.2); each in [1, 4096]            */
  int32_t levels;          /* harmonics used by the centroid estimate; 0 or >= F means all F   */
  int32_t vote_threshold;  /* T_v >= 0: a peak needs V > T_v ("predefined threshold", Sec. 3.2) */
  float tau;               /* Eq. 8: a pixel keeps its label iff d < tau; +inf keeps every one */
  int32_t max_instances;   /* K_max: capacity per image of the peak / centroid arrays.  Up to 32
                              (16 when F > 8) the decode enqueues one kernel fewer: no image can
                              then need the tensor-core assignment.                            */
  uint32_t flags;          /* CPE_FLAG_*                                                       */
  float soft_threshold;    /* with CPE_FLAG_SOFT_VOTE: a peak needs H > soft_threshold (finite, >= 0);
                              ignored otherwise                                                 */
  void* workspace;         /* device memory, 256-byte aligned, owned by the caller             */
  size_t workspace_bytes;  /* >= cpe_workspace_size(...) for the same B, H, W, F and params    */
} cpe_params;

/*
 * Bytes of device workspace that cpe_decode needs for these sizes (0 on invalid arguments).
 * The workspace holds what the paper keeps resident between stages: the palettes P_w, P_h
 * (Eq. 9, "stored as model parameters preloaded in memory"), the vote map (Eq. 6, hard-vote
 * form), the peak indicator (the map H-bar of the local-maxima search) and the peak list.
 * Only workspace and workspace_bytes of params are ignored.
 */
size_t cpe_workspace_size(int B, int H, int W, int F, const cpe_params* params);

/*
 * One-time set-up of a workspace (Sec. 3.2: palettes are pre-computed once and kept resident):
 * zeroes it and uploads P_w and P_h, evaluated on the host as (float) sin|cos(pi 2^l pos) in double.
 * Enqueues on `stream`; must not be called during stream capture.  The workspace is then valid for
 * cpe_decode calls with the same B, H, W, F, bins, max_instances and flags.
 */
int cpe_init_workspace(cpe_stream_t stream, int B, int H, int W, int F, const cpe_params* params);

/*
 * The decode path ("recover the predicted instance masks from a noisy estimate", Sec. 3.1),
 * enqueued on `stream` without any host synchronisation:
 *   1. per participating pixel and axis, a centroid estimate p in [-1,1) by coarse-to-fine phase
 *      unwrapping of the harmonics; the pixel votes for the nearest Eq. 9 bin (hard-vote form of Eq. 6);
 *   2. bins that exceed vote_threshold and beat their 8 neighbours (ties: lower linear index) are the
 *      candidate centroids, listed by ascending linear bin index (Sec. 3.2, local-maxima search);
 *   3. every participating pixel gets label 1 + argmin_k ||xhat - P_w(a_k)|| + ||yhat - P_h(b_k)||
 *      (Eq. 4, Eq. 7; lowest k on ties) if that distance is below tau (Eq. 8), else 0.
 *
 * How step 3 is computed does not change its result (every pair that is scored is scored in the same fixed order of
 * binary32 operations): on inputs of at least 2^19 pixels whose max_instances exceeds the all-pairs range (32 peaks,
 * 16 for F > 8) the candidates of Eq. 7 are pruned.  Around a reference point g (gamma of the mean estimate of a
 * peak's 3x3 window of bins) the triangle inequality gives |d_k - G_k| <= t, with G_k the Eq. 4 distance from g to
 * candidate k and t the pixel's distance to g; every peak gets the list of its nearest candidates by G, a pixel is
 * looked up through the bin it voted for, and only candidates that the bound cannot exclude are scored (usually one).
 * Images that the bounds cannot prune, or with more than 1024 peaks, are handed to a tensor-core filtered kernel
 * (binary16 contraction with rigorous error bounds, exact re-scoring of what survives), which also serves smaller
 * inputs with more peaks than the all-pairs range; all pairs are scored on the plain ALUs otherwise.  The pruned
 * path needs the larger workspace that cpe_workspace_size reports for it (4 bytes per pixel for the bins, two queues
 * of H*W/4 entries per image, the lists) and F in {4, 8, 16}.
 *
 * emb, fg_mask      device, see Conventions.  emb aligned to its element size (16 bytes and
 *                   H*W a multiple of 16/elemsize select the vectorised kernels).
 * out_labels        device int32 [B][H][W]; every element is written (0 = background / rejected).
 * out_centroids     device float [B][max_instances][2]: (x, y) of each kept peak's bin position in pixel
 *                   units (pixel centres at integers); rows >= out_count[b] are left untouched.
 * out_count         device int32 [B]: number of instances kept, min(found, max_instances).
 */
int cpe_decode(cpe_stream_t stream, const void* emb, const uint8_t* fg_mask, int B, int H, int W, int F,
               const cpe_params* params, int32_t* out_labels, float* out_centroids, int32_t* out_count);

/*
 * Device address and size of an intermediate inside the workspace (CPE_INT_*); host-only arithmetic.
 * The contents are those left by the last cpe_decode on that workspace.
 */
int cpe_get_intermediate(const cpe_params* params, int which, int B, int H, int W, int F, void** device_ptr,
                         size_t* bytes);

/* Human-readable text for a CPE_ERR_* code; never NULL. */
const char* cpe_strerror(int code);

/* The CUDA runtime error number behind the calling thread's last CPE_ERR_CUDA (0 if none). */
int cpe_last_cuda_error(void);

/*
 * Self-test of the voting kernel's division.  For binary16 input the quotient min(|s|,|c|) / max(|s|,|c|) inside the
 * per-pixel estimate (the atan2 of the coarse-to-fine phase unwrapping) is formed by a reciprocal estimate, one Newton
 * step and one residual correction in packed binary32 instead of two IEEE divisions; the estimate's bins are only
 * bit-exact if that quotient is the IEEE one.  This call checks it for EVERY pair of binary16 values 0 <= a <= b
 * (b = 0 is replaced by the kernel's floor 2^-30), about 5 x 10^8 quotients, and stores the number of results whose
 * bits differ from IEEE division in *out_mismatches (device, 8-byte aligned; 0 on a correct build).  Enqueues a memset
 * and one kernel on `stream`.
 */
int cpe_selftest_half_division(cpe_stream_t stream, unsigned long long* out_mismatches);

/* ------------------------------------------------------------------ CUDA-graph helper ------- */

/*
 * "The whole chain on one stream with no host sync between stages": captures one cpe_decode call with
 * these arguments into a CUDA graph and instantiates it.  The pointers are baked into the graph and
 * must stay valid.  cpe_graph_launch replays it on a stream.  The handle is host memory owned by the
 * library until cpe_graph_destroy.
 */
typedef struct cpe_graph cpe_graph;
int cpe_graph_create(cpe_stream_t stream, const void* emb, const uint8_t* fg_mask, int B, int H, int W, int F,
                     const cpe_params* params, int32_t* out_labels, float* out_centroids, int32_t* out_count,
                     cpe_graph** out_graph);
int cpe_graph_launch(cpe_graph* graph, cpe_stream_t stream);
void cpe_graph_destroy(cpe_graph* graph);
/* Number of kernel nodes in the captured graph (memset nodes not counted). */
int cpe_graph_kernel_nodes(const cpe_graph* graph);

/* ------------------------------------------------------------------ per-stage timing -------- */

/*
 * Runs cpe_decode `iters` times on `stream` with CUDA events recorded between the stages, waits for
 * the stream, and returns the mean device time of each stage in milliseconds in stage_ms[CPE_STAGE_N].
 * Synchronises; not capturable.  Same arguments and results as cpe_decode.
 */
int cpe_profile_decode(cpe_stream_t stream, const void* emb, const uint8_t* fg_mask, int B, int H, int W, int F,
                       const cpe_params* params, int32_t* out_labels, float* out_centroids, int32_t* out_count,
                       int iters, float* stage_ms);

/* ------------------------------------------------------------------ host-buffer front end --- */

/*
 * End-to-end calls for callers whose data lives in host memory.  The context owns two slots, each with its
 * device buffers (input, mask, outputs, workspace), a stream and a captured graph for fixed B, H, W, F and
 * params (params->workspace is ignored).
 *   cpe_host_decode  copies emb and fg_mask to the device, replays the graph, copies labels, centroids and
 *                    counts back and returns when they have arrived.
 *   cpe_host_submit  enqueues the same work on the next slot and returns at once; cpe_host_wait returns when
 *                    the OLDEST submission's results have arrived in the host buffers it was given.  Up to two
 *                    submissions may be in flight (a third returns CPE_ERR_BUSY and enqueues nothing), so the
 *                    copy of one step's inputs overlaps the decode and read-back of the step before.  The host
 *                    buffers of a submission must stay valid and untouched until its wait returns.
 * cpe_host_wait with nothing in flight returns CPE_ERR_PARAM; cpe_host_decode while something is in flight
 * returns CPE_ERR_BUSY.  A context is not thread-safe.  Host buffers should be page-locked for full copy
 * bandwidth and for the overlap (pageable memory works, its copies are staged by the driver).  fg_mask_host
 * may be NULL only if the context was created with has_mask = 0.
 */
typedef struct cpe_host_ctx cpe_host_ctx;
int cpe_host_ctx_create(int B, int H, int W, int F, const cpe_params* params, int has_mask, cpe_host_ctx** out_ctx);
int cpe_host_decode(cpe_host_ctx* ctx, const void* emb_host, const uint8_t* fg_mask_host, int32_t* labels_host,
                    float* centroids_host, int32_t* count_host);
int cpe_host_submit(cpe_host_ctx* ctx, const void* emb_host, const uint8_t* fg_mask_host, int32_t* labels_host,
                    float* centroids_host, int32_t* count_host);
int cpe_host_wait(cpe_host_ctx* ctx);
/* Bytes moved per cpe_host_decode call in each direction. */
int cpe_host_ctx_traffic(const cpe_host_ctx* ctx, size_t* h2d_bytes, size_t* d2h_bytes);
void cpe_host_ctx_destroy(cpe_host_ctx* ctx);

/* ------------------------------------------------------------------ decode without any allocation --- */

/*
 * (No counterpart in the paper: an integration variant of cpe_decode.)
 *
 * For callers that cannot give the library a workspace because they must not allocate device memory at
 * all: plug-ins that run inside another engine's enqueue call, code on a real-time path, processes whose
 * memory pool is fixed at start-up.  cpe_decode_static is cpe_decode with the workspace replaced by a
 * scratch array that is part of the library image itself (a file-scope __device__ array of
 * CPE_STATIC_SCRATCH_BYTES bytes; every GPU that loads the library holds it until the process exits).
 * The caller still passes the inputs and the three outputs; params->workspace and workspace_bytes are
 * ignored, CPE_FLAG_WRITE_SCORES is not available, and cpe_get_intermediate does not apply.
 *
 * It calls no cudaMalloc, cudaFree or any other allocating routine, on the host or on the device.
 *
 * Limits and rules
 *   - The scratch needed (what cpe_workspace_size reports for the same arguments) must not exceed
 *     CPE_STATIC_SCRATCH_BYTES, and bins_w, bins_h must not exceed CPE_STATIC_MAX_BINS; otherwise the
 *     call returns CPE_ERR_STATIC_LIMIT and enqueues nothing.
 *   - The first call on a device, and any call whose sizes or parameters (B, F, bins, max_instances) differ
 *     from the previous call on that device, also sets the scratch up: it looks up the array's device address, uploads the palettes
 *     and waits for the stream.  Make such a call before starting a stream capture: inside one it is refused with
 *     CPE_ERR_PARAM and enqueues nothing (a call that needs no set-up only enqueues).  The device that owns
 *     `stream` must be the current device.
 *   - All calls on a device share the one array, which keeps what the last call left in it; every call
 *     clears the parts that must start at zero.  Two calls that overlap on the GPU (different streams)
 *     would race on it: keep them on one stream, or order them yourself.
 */
#define CPE_STATIC_SCRATCH_BYTES (8u << 20)
#define CPE_STATIC_MAX_BINS 1024
int cpe_decode_static(cpe_stream_t stream, const void* emb, const uint8_t* fg_mask, int B, int H, int W, int F,
                      const cpe_params* params, int32_t* out_labels, float* out_centroids, int32_t* out_count);

/*
 * Second vote mode: the paper's soft-vote histogram (Eq. 4, Eq. 5, Eq. 6),
 *     H(a, b) = sum over the participating pixels (i, j) of exp(-(||xhat(i,j) - P_w[a]|| + ||yhat(i,j) - P_h[b]||)),
 * computed in the factorised form H = E_x^T E_y of Eq. 10-11, with E_x and E_y formed tile by tile on the SM and
 * never stored (the paper materialises both and calls a library GEMM).  Same inputs, layout, participating set
 * (mask byte non-zero, all channels finite) and palettes (set up by cpe_init_workspace in params->workspace) as
 * cpe_decode.  out_hist: device memory, float [B][bins_h][bins_w], written completely (zeroed first, then
 * accumulated: the reduction over pixel tiles uses binary32 atomics, so the last bits depend on the schedule).
 * Accuracy: |H - H_exact| <= 1e-4 H per bin for F <= 8 at any image size (measured 1.4e-5 at most, full-size
 * workloads included: the two weights that meet in the second contraction enter it as binary16 high + low parts,
 * only the product of the two low parts is dropped, and the tensor-memory accumulator is added to the histogram and
 * restarted every eight pixel tiles, which keeps its one-sided accumulation loss below 2.3e-5); for F > 8 the
 * weights are single binary16 numbers and the bound is 2e-3 H.  Enqueues on the stream, capturable, no host
 * synchronisation.
 * Errors: as cpe_decode; CPE_ERR_ALIGN also if emb is not 16-byte aligned or H*W is not a multiple of 8 (this
 * entry point has the vectorised path only).
 */
int cpe_soft_votes(cpe_stream_t stream, const void* emb, const uint8_t* fg_mask, int B, int H, int W, int F,
                   const cpe_params* params, float* out_hist);

/*
 * The paper's output form of the assignment (Sec. 3.2 "Mask aggregation", Eq. 8): one binary mask per candidate
 * centroid and a counter of the pixels that went to it, expanded from a label map as cpe_decode writes it
 * (0 = no mask, m + 1 = mask m).  For m < n_planes:
 *   out_planes [B][n_planes][H][W] uint8:  1 where labels == m + 1, else 0   (NULL: not wanted)
 *   out_pixels [B][n_planes] uint32:       the number of such pixels         (NULL: not wanted)
 * labels, out_planes, out_pixels: device memory owned by the caller; labels int32 [B][H][W].  n_planes in
 * [1, 8191] (usually the decode's max_instances or the largest count); labels above n_planes are ignored.  Both
 * outputs are written completely.  Enqueues on the stream (a memset of the counters and one kernel), capturable.
 * Errors: CPE_ERR_NULL (labels, or both outputs NULL), CPE_ERR_SIZE, CPE_ERR_ALIGN (labels / out_pixels not 4-byte
 * aligned), CPE_ERR_CUDA.
 */
int cpe_instance_masks(cpe_stream_t stream, const int32_t* labels, int B, int H, int W, int n_planes,
                       uint8_t* out_planes, uint32_t* out_pixels);

/*
 * Layout variant.  The paper writes the network prediction as H_O x W_O x 4L (Sec. 3.1, Eq. 3); cpe_decode reads
 * planes.  cpe_channels_last_to_planar copies emb_nhwc [B][H][W][4F] into emb_planar [B][4F][H][W] (same element
 * type, dtype = CPE_F32 or CPE_F16; both device memory owned by the caller, not overlapping), one read and one
 * write of the embedding, so that a producer of the paper's layout can feed the decoder.  Enqueues one kernel on
 * the stream; capturable.  Errors: CPE_ERR_NULL, CPE_ERR_SIZE (B, H, W < 1, F outside [1,16]), CPE_ERR_DTYPE,
 * CPE_ERR_ALIGN (pointers not aligned to the element size), CPE_ERR_CUDA.
 */
int cpe_channels_last_to_planar(cpe_stream_t stream, const void* emb_nhwc, void* emb_planar, int B, int H, int W, int F,
                                int dtype);

#ifdef __cplusplus
}
#endif
#endif /* CPE_H_ */

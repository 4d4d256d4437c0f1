/*
 * psd.h — C ABI of the PSD (Parallel Speculative Decoding for diffusion LLMs) per-step hot path
 * for NVIDIA B200 (sm_100a).
 *
 * One decoding step of PSD, seen from the LM head onwards, is four operations:
 *
 *   psd_confidence      x^_i = argmax_v p(v), c_i = max_v p(v) for every row of final hidden
 *                       states, p = softmax(hidden · W_lm^T)            (Sec. 3.1; Sec. 3.2 Stage 3)
 *   psd_verify_accept   hierarchical acceptance of a chain of drafts    (Sec. 3.2 Stage 3; Alg. 1 Stage 3)
 *   psd_select_unmask   transfer policy pi and the state update          (Sec. 3.2 Stage 1; Eq. (1))
 *   psd_build_drafts    speculative ordering sigma and draft assembly    (Sec. 3.2 Stage 2; Eq. (2))
 *
 * Conventions, common to every entry point unless it says otherwise:
 *   - Every array pointer is a DEVICE pointer owned by the caller.  The library allocates no
 *     device memory.  The computing entry points keep no state between calls; the only state the
 *     library holds is a handful of process-wide settings (psd_set_confidence_impl, psd_set_tuning)
 *     and a per-thread profiling hook (psd_set_kernel_events), all listed at the end of this file.
 *     The settings are plain atomics read at the start of a call: changing one while another thread
 *     is inside a call is not supported (PSD_TUNE_COMPACT_ROWS, for one, changes how much workspace
 *     psd_step needs and which entries of tokV / confV it writes), so set them before the threads
 *     that compute are started, or serialise.
 *   - Calls are asynchronous on `cuda_stream` (a cudaStream_t passed as void*; NULL = the
 *     default stream).  Outputs are valid once the stream has reached the end of the call.
 *   - The return value is PSD_OK or a negative psd_status code.  Argument errors are detected
 *     on the host before anything is launched; nothing is written in that case.
 *   - Layouts are row-major and dense.  A "block" is one sequence's active block of M slots.
 *     B = blocks, D = chain nodes per block in the verification batch (root included; the paper's
 *     draft depth d equals D-1), rows of the verification batch are ordered (b, d, i):
 *     row = (b*D + d)*M + i.
 *   - mask arrays hold 1 for a masked slot ([M] in the paper) and 0 for a committed one.
 *   - No exceptions, no output on stdout/stderr, plain C linkage.
 */
#ifndef PSD_H_
#define PSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum psd_status {
    PSD_OK = 0,
    PSD_ERR_NULL = -1,        /* a required pointer is NULL                                        */
    PSD_ERR_SHAPE = -2,       /* a size is out of range (see each call)                            */
    PSD_ERR_ALIGN = -3,       /* a pointer is not aligned as required                              */
    PSD_ERR_WORKSPACE = -4,   /* workspace smaller than psd_workspace_bytes()                      */
    PSD_ERR_POLICY = -5,      /* k_min < 1, 0 < k_max < k_min, depth out of range, stride < 0,
                                 unknown accept_mode, or tau is NaN                                 */
    PSD_ERR_CUDA = -6,        /* a CUDA runtime or driver call failed (launch, tensor-map encode)  */
    PSD_ERR_UNSUPPORTED = -7, /* a reserved argument was used                                      */
    PSD_ERR_TIMEOUT = -8,     /* device side only, via status_dev: a bounded wait inside a kernel
                                 ran out; the kernel returned early and its outputs are invalid    */
    PSD_ERR_INTERNAL = -9     /* device side only, via status_dev, and only from the library's debug
                                 build (compiled with PSD_DEBUG): a bounds or ring-order check inside
                                 a kernel failed; the offending access was skipped                  */
} psd_status;

/*
 * The device status word (`status_dev` of the entry points that take one): a device int32 that the
 * CALLER zeroes.  After the call it holds
 *     < 0   a psd_status code detected on the device (PSD_ERR_TIMEOUT; PSD_ERR_INTERNAL from the debug
 *           build); it is never replaced by a count;
 *     > 0   PSD_ERR_NONFINITE count: the number of scored rows whose logits held a NaN or an infinity,
 *           so that their confidence is NaN (such a row ranks below every number in the policy and
 *           never exceeds tau; nothing faults);
 *       0   neither.
 * Counts of successive calls add up when the word is not zeroed in between.
 */

/* Limits checked by the entry points. */
#define PSD_MAX_M 1024     /* slots per block                        */
#define PSD_MAX_DEPTH 64   /* chain nodes per block, root included   */

/* accept_mode: the form of the acceptance criterion A_pi(x~_{k,i}, x^_{p,i}, c_{p,i}) of
 * Algorithm 1 (the paper gives "sufficient confidence" as its example and leaves the form open). */
#define PSD_ACCEPT_AGREE_AND_CONF 0   /* x~ == x^_p  and  c_p > tau              (default) */
#define PSD_ACCEPT_AGREE_ONLY 1       /* x~ == x^_p                                         */
#define PSD_ACCEPT_AGREE_AND_POLICY 2 /* x~ == x^_p  and  i is in pi(parent's draft, c_p)  */

/*
 * Parameters of the transfer policy and of the draft chain, passed by value.
 *
 * The policy is confidence thresholding (App. B.2: unmask every masked position whose top-1
 * confidence exceeds tau, strictly), clamped to at least k_min positions (so that the decoding
 * loop of Algorithm 1 always progresses) and at most k_max.  k_min = k_max = 1 is greedy decoding,
 * k_min = k_max = k is fixed-k parallel decoding (Sec. 2.1).
 */
typedef struct psd_policy_t {
    float tau;           /* commit / acceptance threshold, compared with '>' in fp32              */
    int32_t k_min;       /* >= 1                                                                  */
    int32_t k_max;       /* >= k_min, or 0 for "no cap"                                           */
    int32_t depth;       /* D, 1 .. PSD_MAX_DEPTH; D = 1 means no speculation                     */
    int32_t stride;      /* slots each further depth speculates; 0 means k_min                    */
    int32_t accept_mode; /* PSD_ACCEPT_*                                                          */
    int32_t mask_id;     /* token id of [M]; written to no output, kept for callers' bookkeeping  */
} psd_policy_t;

/* Text for a psd_status code (static storage, never NULL). */
const char* psd_status_string(int code);

/*
 * Bytes of scratch that psd_confidence needs for n_rows x H x V.  Returns 0 for invalid sizes.
 * The scratch holds the per-row partial (max, sum-exp, argmax) triples of every vocabulary split.
 */
size_t psd_workspace_bytes(int32_t n_rows, int32_t H, int32_t V);

/*
 * Bytes of scratch for the paths that first copy the rows to score into a dense buffer: psd_confidence
 * with a row list, and psd_step / psd_decode_blocks with PSD_TUNE_COMPACT_ROWS on (n_rows = B*D*M).
 * Always >= psd_workspace_bytes.  Returns 0 for invalid sizes.
 */
size_t psd_compact_workspace_bytes(int32_t n_rows, int32_t H, int32_t V);

/*
 * psd_confidence — LM head + softmax max-probability + argmax, without ever storing logits.
 * (Sec. 3.1: x^_i and c_i; used for the single sequence of Stage 1 and for all drafts of the
 *  batched verification pass of Stage 3.)
 *
 * For each row r:  l_v = sum_j hidden[r,j] * w_lm[v,j]  (bf16 inputs, fp32 accumulation),
 *   out_token[r] = the lowest v attaining max_v l_v,
 *   out_conf[r]  = 1 / sum_v exp(l_v - max_v l_v)   ( = max_v softmax(l)_v ),
 *   out_lse[r]   = max_v l_v + ln sum_v exp(l_v - max_v l_v)      (optional).
 *
 *   hidden_bf16  [n_rows, H] bf16, 16-byte aligned, device
 *   w_lm_bf16    [V, H]      bf16, 16-byte aligned, device
 *   row_ids      NULL, or a device list [n_rows] int32 of the rows of hidden_bf16 to score (a gather list:
 *                output r belongs to hidden row row_ids[r]; hidden_bf16 may then have any number of rows;
 *                every id must be a valid row of it, the library does not check).
 *                The workspace must then hold psd_compact_workspace_bytes(n_rows, H, V)
 *   n_rows >= 1;  H >= 64 and a multiple of 64;  1 <= V < 2^31 - 256
 *   out_token    [n_rows] int32;  out_conf [n_rows] fp32;  out_lse [n_rows] fp32 or NULL
 *   workspace    >= psd_workspace_bytes(n_rows, H, V) bytes, 256-byte aligned, device; contents
 *                are overwritten; concurrent calls need distinct workspaces
 *   status_dev   NULL, or the device status word (see above): PSD_ERR_TIMEOUT if a bounded wait inside
 *                the kernel expired (outputs are then invalid), else the number of non-finite rows
 * Rows whose logits contain NaN produce out_conf = NaN and are counted in status_dev.
 */
int psd_confidence(const void* hidden_bf16, const void* w_lm_bf16, const int32_t* row_ids,
                   int32_t n_rows, int32_t H, int32_t V,
                   int32_t* out_token, float* out_conf, float* out_lse,
                   void* workspace, size_t workspace_bytes,
                   int32_t* status_dev, void* cuda_stream);

/*
 * psd_confidence_masked — psd_confidence on the rows whose row_mask is non-zero, without the host
 * knowing how many there are (Sec. 3.2 Stage 3 needs predictions only at "each masked position").
 * row_mask [n_rows] int32, device: typically the mask of the sequences themselves ([B, M] or
 * [B, D, M] flattened).  Outputs of flagged rows are written at the rows' own places; outputs of the
 * other rows are left untouched.  No host synchronisation: the rows are listed and copied into a dense
 * buffer on the device, and the fused kernel reads their number from device memory.
 * workspace >= psd_compact_workspace_bytes(n_rows, H, V).  Other arguments as for psd_confidence.
 */
int psd_confidence_masked(const void* hidden_bf16, const void* w_lm_bf16, const int32_t* row_mask,
                          int32_t n_rows, int32_t H, int32_t V,
                          int32_t* out_token, float* out_conf, float* out_lse,
                          void* workspace, size_t workspace_bytes, int32_t* status_dev, void* cuda_stream);

/*
 * ---- The vocabulary split over several GPUs ----------------------------------------------------------
 * softmax max / argmax over the whole vocabulary is an associative merge of per-range triples
 * (max logit, sum of exp(logit - max), lowest argmax), the same merge that combines the vocabulary
 * tiles inside psd_confidence.  A GPU that holds rows [v_offset, v_offset + V_shard) of W computes its
 * triple per row; the triples of all GPUs (12 bytes per row and GPU) are exchanged by the caller and
 * merged on every GPU.  (Sec. 3.1 defines x^ and c over the whole vocabulary; the split is this
 * library's, for LM heads sharded over GPUs.)
 *
 * psd_confidence_partial: out_max, out_sumexp [n_rows] fp32, out_arg [n_rows] int32 (GLOBAL vocabulary
 *   index); other arguments as for psd_confidence with V = V_shard.
 * psd_merge_partials: max, sumexp, arg are [n_shards, n_rows] (shard-major, e.g. the all-gathered
 *   outputs of psd_confidence_partial); out_token, out_conf, out_lse as for psd_confidence.  Equal
 *   maxima keep the lowest global index, so the result does not depend on the number of shards
 *   beyond the rounding order of the sums.  All its arrays are 4-byte aligned (PSD_ERR_ALIGN otherwise);
 *   it takes no status word (psd_confidence_partial has counted the non-finite rows of its shard).
 */
int psd_confidence_partial(const void* hidden_bf16, const void* w_shard_bf16, int32_t n_rows, int32_t H,
                           int32_t V_shard, int32_t v_offset, float* out_max, float* out_sumexp, int32_t* out_arg,
                           void* workspace, size_t workspace_bytes, int32_t* status_dev, void* cuda_stream);
int psd_merge_partials(const float* max, const float* sumexp, const int32_t* arg, int32_t n_shards, int32_t n_rows,
                       int32_t* out_token, float* out_conf, float* out_lse, void* cuda_stream);

/*
 * psd_select_unmask — the transfer policy T = pi(x, c) and the state update of Eq. (1).
 * (Sec. 3.2 Stage 1; App. B.2 for the threshold rule.)
 *
 * conf, tok are [B, n_nodes, M]; block b reads the rows of node node[b] (node 0 when node is
 * NULL).  Over the masked slots of block b, ranked by (confidence descending, slot ascending; NaN
 * last):  n_thr = #{c_i > tau},  n = min(#masked, k_max or inf, max(n_thr, k_min)),  T = the first
 * n.  Then tokens[b,i] = tok[i] and mask[b,i] = 0 for i in T; every other slot is left untouched.
 *
 *   tokens, mask [B, M] int32, in/out
 *   sel      [B, M] int32 out: 1 where i in T, else 0
 *   n_sel    [B]    int32 out: |T|
 *   sel_pos  [B, M] int32 out: the slots of T in rank order, then -1
 *   1 <= B; 1 <= M <= PSD_MAX_M; 1 <= n_nodes <= PSD_MAX_DEPTH; node values must lie in [0, n_nodes)
 */
int psd_select_unmask(const float* conf, const int32_t* tok, const int32_t* node, int32_t n_nodes,
                      int32_t* tokens, int32_t* mask, int32_t B, int32_t M, psd_policy_t p,
                      int32_t* sel, int32_t* n_sel, int32_t* sel_pos, void* cuda_stream);

/*
 * psd_build_drafts — speculative ordering and draft assembly for a chain of D = p.depth nodes.
 * (Sec. 3.2 Stage 2; Eq. (2); Algorithm 1 Stage 2.)
 *
 * conf, tok [B, n_nodes, M] are the cached predictions the step started from (node selection as in
 * psd_select_unmask); tokens, mask [B, M] are the state AFTER psd_select_unmask.  With m masked
 * slots left, sigma orders them by (cached confidence descending, slot ascending; NaN last);
 * node d fills S_d = {sigma_1 .. sigma_{n_d}}, n_d = min(m, d * s), s = stride or k_min:
 *   draft_tokens[b,d,i] = tok[i] if i in S_d else tokens[b,i];   draft_mask[b,d,i] = mask[b,i] and i not in S_d.
 * Node 0 is the root (S_0 empty).  A block with m = 0 yields D copies of its state and n_fill = 0.
 *
 *   sigma   [B, M] int32 out, -1 after the first m entries
 *   n_fill  [B, D] int32 out
 *   draft_tokens, draft_mask [B, D, M] int32 out
 */
int psd_build_drafts(const float* conf, const int32_t* tok, const int32_t* node, int32_t n_nodes,
                     const int32_t* tokens, const int32_t* mask, int32_t B, int32_t M, psd_policy_t p,
                     int32_t* sigma, int32_t* n_fill, int32_t* draft_tokens, int32_t* draft_mask,
                     void* cuda_stream);

/*
 * psd_verify_accept — hierarchical acceptance over the chain, then the commit.
 * (Sec. 3.2 Stage 3; Algorithm 1 Stage 3.)
 *
 * tokV, confV [B, D, M] are psd_confidence's outputs on the D drafts built by psd_build_drafts
 * (sigma, n_fill, draft_tokens, draft_mask as written there, D = p.depth).  Node 0 is accepted;
 * node d >= 1 is accepted iff node d-1 is and every slot i = sigma_j, n_{d-1} < j <= n_d, passes
 * A_pi against node d-1's predictions (p.accept_mode).  k* is the accepted node that fills the
 * most slots, lowest index among equals.  Then tokens, mask <- draft k*, and every slot still
 * masked in draft k* whose confV[b,k*,i] > tau is committed to tokV[b,k*,i] as well.
 *
 *   tokens, mask     [B, M] int32 out (fully written)
 *   k_star           [B] int32 out
 *   n_spec_accepted  [B] int32 out: n_fill[b, k*]
 *   n_committed      [B] int32 out: n_spec_accepted plus the extra commits
 *   accepted         [B, D] int32 out or NULL: 1 for accepted nodes
 */
int psd_verify_accept(const int32_t* tokV, const float* confV,
                      const int32_t* sigma, const int32_t* n_fill,
                      const int32_t* draft_tokens, const int32_t* draft_mask,
                      int32_t B, int32_t M, psd_policy_t p,
                      int32_t* tokens, int32_t* mask,
                      int32_t* k_star, int32_t* n_spec_accepted, int32_t* n_committed,
                      int32_t* accepted, void* cuda_stream);

/*
 * psd_confidence_static — psd_confidence without a workspace argument and without any allocation.
 * (The paper has no counterpart: this entry point exists for deployment, not for the method.)
 *
 * For callers that cannot allocate device memory at the point of the call — a server whose own
 * pool already owns all free HBM, a plug-in invoked from another runtime's callback where
 * cudaMalloc and its implicit synchronisation are not allowed.  The scratch that psd_confidence
 * takes from its caller lives here in a fixed array inside the library image, of
 * PSD_STATIC_SCRATCH_BYTES; every GPU that loads the library holds that much until the process exits.
 *
 * Same arguments, outputs and numerics as psd_confidence (always the tcgen05 kernel), except:
 *   - no workspace; sizes with psd_workspace_bytes(n_rows, H, V) > PSD_STATIC_SCRATCH_BYTES are
 *     rejected with PSD_ERR_WORKSPACE (e.g. 128 rows x V = 126464 needs 1.5 MB and fits;
 *     8192 rows do not);
 *   - the first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress, with that device current).  CUDA loads a library's device code lazily
 *     by default, so this look-up can be the moment the driver loads the module and reserves the
 *     array's memory: make one call per device at start-up, BEFORE the process hands the rest of
 *     the device memory to its pool and outside of any stream capture.  A first call made after
 *     the memory is gone fails with PSD_ERR_CUDA.  Later calls on that device touch no allocator;
 *   - it calls no cudaMalloc, cudaFree or other allocating routine;
 *   - all calls on a device share the one array, which keeps the previous call's contents.
 *     Nothing in it needs clearing (every entry read is written first by the same call), but two
 *     calls that overlap on the GPU (different streams, or different host threads) race on it:
 *     serialise them.
 */
#define PSD_STATIC_SCRATCH_BYTES (4u << 20)
int psd_confidence_static(const void* hidden_bf16, const void* w_lm_bf16,
                          int32_t n_rows, int32_t H, int32_t V,
                          int32_t* out_token, float* out_conf, float* out_lse,
                          int32_t* status_dev, void* cuda_stream);

/*
 * All pointers of one decoding step over a batch of B blocks.  Device pointers for psd_step,
 * HOST pointers (pinned memory recommended) for psd_step_host, except w_lm_bf16 which is a
 * device pointer in both.
 */
typedef struct psd_step_io_t {
    const void* hidden_bf16;  /* in  [B*D*M, H] final hidden states of the verification batch      */
    const void* w_lm_bf16;    /* in  [V, H] DEVICE                                                 */
    int32_t* sigma;           /* in/out [B, M]    drafts being verified -> drafts for the next step */
    int32_t* n_fill;          /* in/out [B, D]                                                     */
    int32_t* draft_tokens;    /* in/out [B, D, M]                                                  */
    int32_t* draft_mask;      /* in/out [B, D, M]                                                  */
    int32_t* tokV;            /* out [B, D, M] verifier predictions                                */
    float* confV;             /* out [B, D, M] verifier confidences                                */
    int32_t* tokens;          /* out [B, M] state after acceptance and the policy                  */
    int32_t* mask;            /* out [B, M]                                                        */
    int32_t* k_star;          /* out [B]                                                           */
    int32_t* n_spec_accepted; /* out [B]                                                           */
    int32_t* n_committed;     /* out [B] acceptance commits (the policy's are in n_sel)            */
    int32_t* sel;             /* out [B, M]                                                        */
    int32_t* n_sel;           /* out [B]                                                           */
    int32_t* sel_pos;         /* out [B, M]                                                        */
} psd_step_io_t;

/*
 * psd_step — one whole step on device buffers, on one stream, with no host synchronisation:
 *   psd_confidence on all B*D*M rows  ->  psd_verify_accept on the drafts in io
 *   ->  psd_select_unmask on node k*'s predictions  ->  psd_build_drafts for the next step
 * (the verification pass of Algorithm 1 doubles as the model call of the next iteration).
 * Argument rules are those of the four calls; D = p.depth.
 */
int psd_step(const psd_step_io_t* io, int32_t B, int32_t M, int32_t H, int32_t V, psd_policy_t p,
             void* workspace, size_t workspace_bytes, int32_t* status_dev, void* cuda_stream);

/*
 * Bytes of device staging that psd_step_host needs (inputs, outputs and the step's scratch, sized so
 * that PSD_TUNE_COMPACT_ROWS may be on).  Returns 0 for invalid sizes.
 */
size_t psd_step_host_bytes(int32_t B, int32_t M, int32_t H, int32_t V, int32_t D);

/*
 * Layout of ONE host block that holds every per-step array of psd_step_io_t except hidden_bf16 and
 * w_lm_bf16.  Returns the block's size in bytes (0 for invalid sizes) and, if offsets != NULL, the 15
 * byte offsets of sigma, n_fill, draft_tokens, draft_mask, tokV, confV, tokens, mask, k_star,
 * n_spec_accepted, n_committed, sel, n_sel, sel_pos and of a status word, in this order.  When the
 * io passed to psd_step_host points into such a block (pinned memory recommended), the draft state
 * is copied up in one transfer and all outputs come back in one; any other arrangement of host
 * arrays works too, with one transfer per array.
 */
size_t psd_step_host_block(int32_t B, int32_t M, int32_t D, size_t* offsets);

/*
 * psd_step_host — psd_step for callers whose per-step data lives in host memory.
 * Copies hidden and the draft state host->device into `staging`, runs psd_step, copies every
 * output of io back device->host, and waits for the stream.  io holds HOST pointers
 * (w_lm_bf16 excepted).  staging: device, 256-byte aligned, >= psd_step_host_bytes().
 * status_host: NULL, or receives the device status word (see "The device status word").
 * Synchronous: returns after the outputs are in host memory.
 * Batches of 2048 rows or more go up in two pieces (blocks are independent: the step on the first
 * blocks, then on the rest), the second piece's copy running under the first piece's kernels on an
 * internal stream; the first such call on a device creates that stream and three events, host-side
 * objects that live until the process exits.  Results are those of psd_step on the same pieces;
 * confidences can differ from one psd_step over the whole batch in the last bits (another tiling of
 * the rows), nothing else does.  With the one-block host layout the block's status word is
 * written by this call before the copy (the block goes up whole, which zeroes the device's word).
 */
int psd_step_host(const psd_step_io_t* io, int32_t B, int32_t M, int32_t H, int32_t V, psd_policy_t p,
                  void* staging, size_t staging_bytes, int32_t* status_host, void* cuda_stream);

/*
 * ---- General draft graph (multi-parent DAG) ------------------------------------------------------------
 * (Sec. 3.2 Stage 2: nodes k with subsets S_k of {sigma_1..sigma_m}, an edge (p, k) whenever S_p is a
 *  strict subset of S_k, a node may have several parents; Algorithm 1 Stage 3 for the acceptance.)
 *
 * The graph is fixed at inference time and expressed over RANKS of the speculative ordering: bit j of
 * ranks[k] set means that node k speculates sigma_{j+1} (the slot with the (j+1)-th highest cached
 * confidence among the residual masked slots).  Only the 64 best ranks can be speculated.  Node 0 is
 * the root (ranks[0] = 0).  When fewer than 64 residual slots exist, ranks beyond them drop out of
 * every node.  bit p of parents[k] set means that (p, k) is an edge; S_p must be a strict subset of
 * S_k.  The chain of psd_build_drafts is the special case ranks[d] = lowest d*stride bits,
 * parents[d] = {d-1}.
 */
#define PSD_MAX_DAG_NODES 64
typedef struct psd_dag_t {
    int32_t n_nodes;                      /* K, 1 .. PSD_MAX_DAG_NODES */
    int32_t reserved;
    uint64_t ranks[PSD_MAX_DAG_NODES];
    uint64_t parents[PSD_MAX_DAG_NODES];
} psd_dag_t;

/*
 * Fills *g (host memory) from n_nodes rank words and, optionally, parent words.  parents == NULL makes
 * every strict-subset pair an edge (the paper's edge set).  Returns PSD_ERR_SHAPE if node 0 is not the
 * root, n_nodes is out of range, or an edge is not between a strict subset and its superset.
 */
int psd_dag_init(psd_dag_t* g, int32_t n_nodes, const uint64_t* ranks, const uint64_t* parents);

/*
 * psd_build_drafts_dag — psd_build_drafts for a draft graph: sigma as there; node k fills
 * S_k = {sigma_{j+1} : bit j of g->ranks[k], j < m}; Eq. (2).  g is a HOST pointer.
 *   n_fill [B, K] out: |S_k|;  draft_tokens, draft_mask [B, K, M] out.  p is not used (kept for symmetry).
 */
int psd_build_drafts_dag(const float* conf, const int32_t* tok, const int32_t* node, int32_t n_nodes,
                         const int32_t* tokens, const int32_t* mask, int32_t B, int32_t M, psd_policy_t p,
                         const psd_dag_t* g, int32_t* sigma, int32_t* n_fill, int32_t* draft_tokens,
                         int32_t* draft_mask, void* cuda_stream);

/*
 * psd_verify_accept_dag — hierarchical acceptance over the graph, then the commit (Algorithm 1 Stage 3).
 * tokV, confV [B, K, M] are psd_confidence's outputs on the K drafts.  The root is accepted; in
 * topological order (fewer speculated ranks first, lower index among equals) node k is accepted iff
 * some accepted parent p passes A_pi(x~_{k,i}, x^_{p,i}, c_{p,i}) (p.accept_mode) on every slot of
 * S_k \ S_p; an empty difference passes.  k* = the accepted node with the largest |S_k|, lowest index
 * among equals.  Then as psd_verify_accept: tokens, mask <- draft k*, plus node k*'s own predictions
 * above tau.  accepted [B, K] out or NULL.  p.depth and p.stride are not used.
 */
int psd_verify_accept_dag(const int32_t* tokV, const float* confV, const int32_t* sigma,
                          const int32_t* draft_tokens, const int32_t* draft_mask, int32_t B, int32_t M,
                          psd_policy_t p, const psd_dag_t* g, int32_t* tokens, int32_t* mask, int32_t* k_star,
                          int32_t* n_spec_accepted, int32_t* n_committed, int32_t* accepted, void* cuda_stream);

/*
 * psd_step_dag — psd_step with the drafts of a graph: D = g->n_nodes in every shape of io; acceptance is
 * psd_verify_accept_dag, the next drafts psd_build_drafts_dag (p.depth and p.stride are not used).
 * Runs as separate launches (fused kernel, merge, acceptance, policy, drafts) on the stream.
 */
int psd_step_dag(const psd_step_io_t* io, int32_t B, int32_t M, int32_t H, int32_t V, psd_policy_t p,
                 const psd_dag_t* g, void* workspace, size_t workspace_bytes, int32_t* status_dev,
                 void* cuda_stream);

/*
 * ---- The whole decoding loop of Algorithm 1 over a batch of blocks ----------------------------------
 *
 * The transformer body is the caller's: a function that, given token states on the device, writes
 * their final hidden states.  n_seq sequences of M slots each: tokens, mask [n_seq, M] int32 (device),
 * hidden_bf16 [n_seq * M, H] bf16 (device, row (s, i) at s*M + i).  It must enqueue its work on
 * cuda_stream and return 0, or a negative value that psd_decode_blocks passes on.
 */
typedef int (*psd_body_fn)(void* user, const int32_t* tokens, const int32_t* mask, int32_t n_seq, int32_t M,
                           void* hidden_bf16, void* cuda_stream);

/* Order of operations inside one iteration of psd_decode_blocks. */
#define PSD_ORDER_TWO_PASSES 0 /* Algorithm 1 as printed: a pass on the state, policy, drafts, a batched
                                  pass on the D drafts, acceptance                                      */
#define PSD_ORDER_ONE_PASS 1   /* psd_step: the batched pass on the drafts also serves as the next
                                  iteration's pass on the state (acceptance, then policy on node k*)   */

typedef struct psd_decode_stats_t {
    int32_t iterations;     /* iterations of the while loop that ran                                  */
    int32_t forward_passes; /* calls of the body (batched over all blocks)                            */
    int32_t masked_left;    /* masked slots left over all blocks: 0 unless max_iterations ran out     */
} psd_decode_stats_t;

/* Bytes of device scratch psd_decode_blocks needs besides psd_confidence's workspace (0 = bad sizes). */
size_t psd_decode_scratch_bytes(int32_t B, int32_t M);

/*
 * psd_decode_blocks — Algorithm 1: repeat { forward pass, policy, drafts, batched verification pass,
 * hierarchical acceptance } until no block has a masked slot left, or max_iterations.
 * (Sec. 3.2; Algorithm 1, including its early break when Stage 1 resolves the block.)
 *
 * io holds DEVICE pointers.  io->tokens, io->mask [B, M] are the blocks' state, in and out: normally
 * every slot masked on entry (token = p.mask_id, mask = 1), but any state is accepted.  io->hidden_bf16
 * is scratch of [B*D*M, H] bf16 that the body fills (the library writes through the pointer although
 * the field is const).  Every other array of io is scratch/output with the shapes given at
 * psd_step_io_t; after the call they hold the last iteration's values.  D = p.depth; with D = 1
 * nothing is speculated and every iteration is one pass (plain parallel decoding).
 *
 *   g               NULL: the drafts are the chain of p.depth nodes; else a draft graph (HOST pointer),
 *                   and D = g->n_nodes in every shape above (p.depth, p.stride are then not used)
 *   order           PSD_ORDER_TWO_PASSES or PSD_ORDER_ONE_PASS
 *   scratch         device, 256-byte aligned, >= psd_decode_scratch_bytes(B, M)
 *   workspace       as for psd_confidence with n_rows = B*D*M
 *   passes          NULL or device [B] out: forward passes charged to each block (a block is charged
 *                   for a pass only while it still has masked slots) — M / passes[b] is the block's
 *                   tokens per forward pass
 *   done_iteration  NULL or device [B] out: index of the iteration that resolved the block, -1 if none
 *   trace           NULL or device [max_iterations, B, 4] out: per iteration and block
 *                   (n_sel, k_star, n_spec_accepted, n_committed); the last three are 0 in iterations
 *                   that stopped after Stage 1
 *   stats           host, out
 * The call is synchronous: after every state update the host waits for the stream and reads the number
 * of masked slots, which the counting kernel has written straight into a pinned host word, to decide
 * whether to go on.  It allocates no device memory; the first call of a host thread allocates that one
 * 64-byte pinned word, which lives until the process exits (if that fails, the count is copied instead).
 */
int psd_decode_blocks(psd_body_fn body, void* user, const psd_step_io_t* io, int32_t B, int32_t M, int32_t H,
                      int32_t V, psd_policy_t p, const psd_dag_t* g, int32_t order, int32_t max_iterations,
                      void* scratch, size_t scratch_bytes, void* workspace, size_t workspace_bytes,
                      int32_t* status_dev, int32_t* passes, int32_t* done_iteration, int32_t* trace,
                      psd_decode_stats_t* stats, void* cuda_stream);

/*
 * psd_table_body — a stand-in body for tests and benchmarks (the paper's body is a 7-8B transformer,
 * which is outside this library): a table look-up with no arithmetic.  user points to a
 * psd_table_body_t; hidden row (s, i) = table row ((b*M + i)*3 + c), where b = s / (n_seq / B) is the
 * sequence's block and c in {0, 1, 2} counts the committed neighbours of slot i (slots i-1 and i+1 of
 * the same sequence with mask 0).  tokens is not read.
 */
typedef struct psd_table_body_t {
    const void* table_bf16; /* [B, M, 3, H] bf16, device, 16-byte aligned */
    int32_t B;
    int32_t H;              /* multiple of 8 */
} psd_table_body_t;
int psd_table_body(void* user, const int32_t* tokens, const int32_t* mask, int32_t n_seq, int32_t M,
                   void* hidden_bf16, void* cuda_stream);

/*
 * Which kernel psd_confidence uses.  Process-wide; returns the previous value, or PSD_ERR_SHAPE for
 * an unknown value.
 *   0  (default) the tcgen05/TMA kernels, chosen by size: pairs of CTAs on one tile of 256 rows
 *      (cta_group::2) for 129..256 rows, one CTA per tile of 128 rows otherwise
 *   1  a plain CUDA-core kernel kept for cross-checking
 *   2  always the single-CTA tcgen05 kernel;  3  always the CTA-pair tcgen05 kernel (same results up
 *      to summation order)
 */
int psd_set_confidence_impl(int impl);

/*
 * Performance knobs (process-wide; results never depend on them).  Returns PSD_OK,
 * PSD_ERR_UNSUPPORTED for an unknown knob or PSD_ERR_SHAPE for a bad value.
 *   PSD_TUNE_BAND_BYTES  bytes of the operand that one band of the fused kernel's tile order keeps
 *                        in L2 while the other operand streams past it (default 36 MiB)
 */
#define PSD_TUNE_BAND_BYTES 1
/*   PSD_TUNE_PDL         1 (default): consecutive kernels of a step are launched with programmatic stream
 *                        serialization, so a kernel's set-up overlaps the end of the one before it (the
 *                        fused kernel itself starts early only when the batch is a single row tile);
 *                        2: the fused kernel starts early at every size; 0: plain stream order */
#define PSD_TUNE_PDL 2
/*   PSD_TUNE_TILE_ORDER  0 (default): the library picks the tile order with the smaller estimated DRAM
 *                        traffic; 1: bands of vocabulary tiles (W resident, hidden re-read per band);
 *                        2: bands of row tiles (hidden resident, W re-read per band) */
#define PSD_TUNE_TILE_ORDER 3
/*   PSD_TUNE_COMPACT_ROWS  psd_step scores only the rows of slots that are still masked in their draft
 *                        (Sec. 3.2 Stage 3: "each masked position"): 0 (default) off; 1 on when the
 *                        batch has more than 128 rows; 2 always.  With it on, the workspace must hold
 *                        psd_compact_workspace_bytes, and entries of tokV / confV that belong to
 *                        committed slots are left as they were (no stage reads them) */
#define PSD_TUNE_COMPACT_ROWS 4
/*   PSD_TUNE_WAIT_LIMIT  every wait on a barrier inside the tensor-core kernels gives up after this many
 *                        THOUSANDS of SM clock cycles (default 4 000 000: about 2 s); the kernel then reports
 *                        PSD_ERR_TIMEOUT through status_dev, lets its own copies and tensor-core work finish
 *                        (those waits keep the default limit), frees what it holds and returns normally */
#define PSD_TUNE_WAIT_LIMIT 5
/*   PSD_TUNE_SELFTEST_STALL  1: self-test of that give-up path.  In every CTA (in the leading CTA of every
 *                        pair) the loader, after its first K-slice, waits on a barrier that nothing ever
 *                        arrives on, so the wait runs out after PSD_TUNE_WAIT_LIMIT and the call ends with
 *                        PSD_ERR_TIMEOUT in status_dev and invalid outputs; nothing faults and the next call
 *                        (with 0 here) works as usual.  0 (default): off */
#define PSD_TUNE_SELFTEST_STALL 6
/* 1 if PSD_TUNE_COMPACT_ROWS makes a batch of n_rows rows take the compacted path, else 0. */
int psd_compact_rows_enabled(int32_t n_rows);
int psd_set_tuning(int knob, int value);

/*
 * Profiling aid.  When both events (cudaEvent_t passed as void*) are non-NULL, the next
 * psd_confidence call made by this host thread (directly or through psd_step / psd_step_host)
 * records `start_event` immediately before and `stop_event` immediately after its main kernel
 * (the fused LM-head + confidence kernel, not the combine pass) on the call's stream; the hook then
 * clears itself.  Passing NULLs clears it.  Always returns PSD_OK.
 */
int psd_set_kernel_events(void* start_event, void* stop_event);

/*
 * Name of the kernel that psd_confidence (and psd_step) launches for a batch of n_rows rows under the
 * current psd_set_confidence_impl setting: "confidence_tc_kernel", "confidence_tc2_kernel" or
 * "confidence_simt_kernel" (static storage).  For reports: it computes nothing.
 */
const char* psd_confidence_kernel_name(int32_t n_rows);

/* Number of kernel launches the library has issued in this process (all entry points). */
int64_t psd_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* PSD_H_ */

/*
 * gt_attn.h -- C ABI of the B200 (sm_100a) biased graph-attention library.
 *
 * The library implements the single-GPU hot path of graph-transformer training that the
 * MegaGraph paper parallelises: all-to-all node attention with an additive structural
 * bias (the paper's Eq. 1),
 *
 *     Attention(Q,K,V) = Softmax(Q K^T / sqrt(d) + b_attn) V ,
 *
 * where b_attn encodes topology via shortest-path distances (Sec. "Preliminaries: Graph
 * Transformer" and Sec. "Graph-Aware Context Parallelism", item 2).  Here b_attn is never
 * materialised as floats: it is a uint8 shortest-path-distance (SPD) index matrix shared
 * by all heads plus a small per-head table, b_attn[h][i][j] = bias[h][spd[i][j]].
 *
 * Conventions common to all entry points
 * --------------------------------------
 *  - Every pointer is a DEVICE pointer unless marked (host).  The caller owns every
 *    buffer; the library allocates and frees no device memory.  Scratch comes from a
 *    caller-provided workspace whose size is obtained from the matching *_workspace()
 *    query (host function, no GPU work).  Workspace and all tensor base pointers must be
 *    16-byte aligned.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only
 *    enqueue work and return; they never synchronise.  Errors detected on the host are
 *    returned immediately.  Errors detected on the device (a bounded wait that ran out)
 *    are recorded in a status word at the start of the workspace and are reported by
 *    gt_check(), which synchronises the stream.  The first 256 bytes of a workspace (or step
 *    context) hold that status word and a few counters: they must be ZERO when the buffer is
 *    first handed to the library (one cudaMemset after allocation); the calls do not clear the
 *    status themselves, so that one gt_check() after a sequence of calls on the same workspace
 *    reports a failure of any of them, and gt_check() clears it after reporting.  A workspace
 *    with a dirty header makes gt_check() report an error that no kernel raised.
 *  - Node features are packed: a batch of G graphs with n_g nodes each is stored as
 *    T = sum n_g consecutive rows; Q, K, V, O and their gradients are bf16 [T, H, d]
 *    (row-major, d contiguous); graph g owns rows cu_seqlens[g] .. cu_seqlens[g+1]-1 and
 *    attention is block diagonal (nodes attend only within their graph).  With one graph
 *    (n_graphs == 1) cu_seqlens and spd_offsets may be NULL.
 *  - SPD layout: graph g's block starts at byte spd_offsets[g] (int64, device) and holds
 *    n_g rows of pitch ld_g = round_up(n_g, 16) bytes; spd[i*ld_g + j] is the bucket of the
 *    ordered pair (i -> j): min(hops, max_dist), or max_dist+1 if j is unreachable from i.
 *    There are n_buckets = max_dist + 2 buckets.  A value >= n_buckets is invalid input: no kernel
 *    reads out of bounds on it, but WHICH valid bucket it is taken for is unspecified and differs
 *    between kernels (the forward may use the value modulo 32, the backward the last bucket), so
 *    forward and backward need not agree on such a matrix.  gt_spd_build never writes one;
 *    gt_spd_validate checks a matrix that came from elsewhere.  Padding bytes (j >= n_g) are ignored.
 *  - Supported shapes: head_dim in {32, 64}; 1 <= max_dist <= 254; n_heads >= 1;
 *    anything else returns GT_ERR_UNSUPPORTED / GT_ERR_INVALID_ARG without launching.
 */
#ifndef GT_ATTN_H_
#define GT_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum gt_status {
    GT_OK = 0,
    GT_ERR_INVALID_ARG = 1,    /* NULL required pointer, bad size, misaligned pointer          */
    GT_ERR_UNSUPPORTED = 2,    /* head_dim not in {32,64}, chunked call on a multi-graph batch */
    GT_ERR_WORKSPACE = 3,      /* workspace NULL or smaller than the *_workspace() query       */
    GT_ERR_CUDA = 4,           /* a CUDA runtime/driver call failed (launch, descriptor)       */
    GT_ERR_DEVICE_TIMEOUT = 5, /* a bounded device-side wait expired (reported by gt_check)    */
    GT_ERR_NO_DEVICE = 6,      /* no sm_100 device is current                                  */
    GT_ERR_BAD_SPD = 7         /* gt_spd_validate found entries >= max_dist+2 (reported by gt_check) */
} gt_status;

/* Packed batch description (host struct; cu_seqlens is a device pointer). */
typedef struct gt_batch {
    int32_t n_total;           /* T = sum n_g  (N for a single graph), >= 1              */
    int32_t n_graphs;          /* G >= 1                                                 */
    const int32_t* cu_seqlens; /* device int32[G+1], cu[0]=0, cu[G]=T; may be NULL if G==1 */
    int32_t max_seqlen;        /* max_g n_g (host-known; sizes the launch grid)          */
} gt_batch;

const char* gt_status_string(gt_status s);

/* Synchronises `stream`, then returns and clears the device status word held in the first
 * bytes of `workspace` (GT_OK, or GT_ERR_DEVICE_TIMEOUT if a kernel gave up on a wait; the
 * outputs of that call are then undefined).  `workspace` is one that was passed to any of
 * the calls below. */
gt_status gt_check(void* workspace, void* stream);

/* ---------------------------------------------------------------------------------------
 * gt_spd_build -- structural-encoding construction (the paper builds b_attn from batch
 * topology on the CPU during data loading, Sec. "Preliminaries" and the T_stall term of the
 * latency model; this builds its index form on the GPU).
 *
 * Multi-source breadth-first search over a CSR graph.  row_ptr int32[T+1], col_idx
 * int32[nnz]: row i lists the out-neighbours of packed node i as PACKED node ids; edges
 * must stay inside a graph.  Self loops and duplicate entries are tolerated.  Writes the
 * SPD block(s) described above into spd_out (every byte of every row, padding bytes = 255).
 * The traversal runs to exhaustion, so pairs farther than max_dist (bucket max_dist) stay
 * distinct from unreachable pairs (bucket max_dist+1).  Bit-exact and deterministic.
 * Out-of-range col_idx entries are undefined behaviour.
 * Workspace: about 4(G+1) + 4 n_total + 4 G + 1 KB for a packed batch whose graphs have at most 17 066 nodes each and
 * for a single graph below 14 500 nodes (per-graph offsets, and the connected-component label of every node: the search
 * of an undirected graph without a vertex of more than 64 out-edges stops at level max_dist); a single larger graph (it takes a bit-matrix traversal, which is the faster one from there)
 * needs about 7 KB per node for each of min(4, ceil(n/8192)) groups of thread blocks (seven bit
 * matrices of 1 KB rows per group: visited, and one frontier per level up to 5; later levels reuse two of
 * them) plus 1 KB per 33 edges per group (rows for vertices with more than 32 out-edges) and 16 bytes per
 * 32 edges -- 2.0 GB at 65 536 nodes with 786 000 edges -- and a device that supports cooperative
 * launches; a batch that contains a larger graph needs 12 bytes per node of the largest graph for each
 * of up to 2 x (number of SMs) thread blocks.
 * ------------------------------------------------------------------------------------- */
size_t gt_spd_build_workspace(const gt_batch* batch, int64_t nnz, int32_t max_dist);
gt_status gt_spd_build(const int32_t* row_ptr, const int32_t* col_idx, int64_t nnz,
                       const gt_batch* batch, int32_t max_dist,
                       const int64_t* spd_offsets, uint8_t* spd_out,
                       void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------
 * gt_spd_build_static -- gt_spd_build without a workspace argument.  (No counterpart in the
 * paper: it exists for the way this library is embedded, not for the method.)
 *
 * Some callers cannot hand over scratch memory because they may not allocate on the device at
 * all: a plug-in running inside a host application that owns the GPU allocator, a latency-critical
 * loop in which a device allocation would stall every stream, or code that runs after the process
 * has pinned its memory budget.  For them the scratch of the SPD build lives inside the library,
 * in a fixed array of gt_spd_build_static_limit() bytes (1 MiB) that every GPU loading the library
 * holds until the process exits.  The call itself allocates and frees nothing.
 *
 * Same arguments, results and error codes as gt_spd_build, minus the workspace, with these rules:
 *  - Size limit: the batch must satisfy gt_spd_build_workspace(batch, nnz, max_dist) <=
 *    gt_spd_build_static_limit(); in practice a packed batch whose graphs have at most 17 066 nodes each, or a
 *    single graph below 14 500 nodes (larger ones keep their traversal state in the workspace and need far more).  Otherwise
 *    GT_ERR_WORKSPACE is returned and nothing is launched.
 *  - First call per device: the first call made with a given device current looks up the
 *    device address of the built-in array (a one-off set-up step).  Make that first call outside
 *    any stream capture.
 *  - One array per device, shared by all calls: it still holds what the previous call left (the
 *    call clears the words that must start at zero), and two calls whose GPU work overlaps --
 *    different streams, or different host threads -- race on it.  Serialise them, or give the
 *    concurrent ones their own workspace through gt_spd_build.
 *  - No device status: the caller has no workspace pointer to hand to gt_check().  Nothing is lost by
 *    that: the builds that fit the built-in array contain no bounded device-side wait, so the only
 *    errors this call can have are the ones it returns.
 * ------------------------------------------------------------------------------------- */
size_t gt_spd_build_static_limit(void);
gt_status gt_spd_build_static(const int32_t* row_ptr, const int32_t* col_idx, int64_t nnz,
                              const gt_batch* batch, int32_t max_dist,
                              const int64_t* spd_offsets, uint8_t* spd_out, void* stream);

/* ---------------------------------------------------------------------------------------
 * gt_spd_validate -- checks an SPD index matrix that gt_spd_build did not write (the paper's bias
 * matrix is built by the data loader, Sec. "Preliminaries"; a caller may bring its own): counts the
 * entries of the valid n_g x n_g regions that are >= max_dist + 2.  If there are any, the status
 * word of `workspace` (gt_spd_validate_workspace() bytes, header zeroed as for every workspace) is
 * set to GT_ERR_BAD_SPD, which gt_check(workspace, stream) then returns; gt_spd_validate_count
 * synchronises the stream and copies the number of such entries to *count_host (host pointer).
 * ------------------------------------------------------------------------------------- */
size_t gt_spd_validate_workspace(void);
gt_status gt_spd_validate(const uint8_t* spd, const int64_t* spd_offsets, const gt_batch* batch, int32_t max_dist,
                          void* workspace, size_t workspace_bytes, void* stream);
gt_status gt_spd_validate_count(void* workspace, void* stream, int64_t* count_host);

/* ---------------------------------------------------------------------------------------
 * gt_test_hook_barrier_overcount -- test hook of the device-timeout path (no counterpart in the
 * paper).  Every device-side wait of this library is bounded; one that runs out makes its kernel
 * return and gt_check() report GT_ERR_DEVICE_TIMEOUT.  After gt_test_hook_barrier_overcount(k), k > 0,
 * the NEXT bit-matrix build of this process (gt_spd_build on a single graph of 14 500 nodes or more) waits
 * at its grid barriers for k arrivals more than there are thread blocks, with a shortened limit, so the
 * wait runs out within a second; the kernel issues no asynchronous copies, so nothing is in flight when
 * it returns, the context stays usable and the next build is normal.  The output of the hooked build
 * is undefined.  Not thread-safe; meant for tests only.
 * ------------------------------------------------------------------------------------- */
void gt_test_hook_barrier_overcount(int32_t extra);

/* ---------------------------------------------------------------------------------------
 * gt_biased_attn_fwd -- Eq. 1, forward.  For every graph, head h and query row i:
 *     S_ij = (q_i . k_j)/sqrt(head_dim) + bias[h][spd_ij]        (all j of the same graph)
 *     out_i = sum_j softmax_j(S_i)_j v_j,     lse[h][i] = log sum_j exp(S_ij)  (natural log)
 * computed tile by tile with an online softmax in which the bias is added to the score
 * before the running max / sum are updated (Sec. GA-CP, item 3).  bf16 inputs, fp32
 * accumulation and softmax, bf16 `out` [T,H,d], fp32 `lse` [H,T].
 * bias: fp32 [n_heads, max_dist+2].
 * ------------------------------------------------------------------------------------- */
size_t gt_biased_attn_fwd_workspace(const gt_batch* batch, int32_t n_heads, int32_t head_dim);
gt_status gt_biased_attn_fwd(const void* q, const void* k, const void* v,
                             const uint8_t* spd, const int64_t* spd_offsets, const float* bias,
                             const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                             void* out, float* lse,
                             void* workspace, size_t workspace_bytes, void* stream);

/* gt_biased_attn_fwd_ex -- gt_biased_attn_fwd that can also return the output BEFORE its rounding to
 * bf16: out_f32, fp32 [T,H,d], or NULL (then the call is gt_biased_attn_fwd).  It exists for the
 * backward: Delta_i = dout_i . out_i of Eq. 1's gradient is formed from the stored output, and where a
 * few distance buckets hold nearly all pairs (max_dist 1-3, a hub or global node joined to every node,
 * mostly unreachable pairs) dbias is a small residue of large cancelling sums, so the 2^-9 relative
 * rounding of a bf16 `out` alone moves it by several per cent.  Pass the same out_f32 to
 * gt_biased_attn_bwd_ex and dbias keeps the accuracy of the other gradients. */
gt_status gt_biased_attn_fwd_ex(const void* q, const void* k, const void* v,
                                const uint8_t* spd, const int64_t* spd_offsets, const float* bias,
                                const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                void* out, float* lse, float* out_f32,
                                void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------
 * gt_biased_attn_bwd -- gradient of Eq. 1 for upstream gradient `dout` (bf16 [T,H,d]).
 * With P_ij = exp(S_ij - lse_i) recomputed tile by tile:
 *     Delta_i = dout_i . out_i         dP_ij = dout_i . v_j        dS_ij = P_ij (dP_ij - Delta_i)
 *     dv_j = sum_i P_ij dout_i         dq_i = sum_j dS_ij k_j / sqrt(d)
 *     dk_j = sum_i dS_ij q_i / sqrt(d) dbias[h][b] = sum over pairs with spd_ij == b of dS_ij
 * `out` and `lse` are the forward results.  dq, dk, dv (bf16 [T,H,d]) and dbias
 * (fp32 [n_heads, max_dist+2], summed over all graphs of the batch) are OVERWRITTEN.
 * dq and dbias are accumulated with floating-point atomics, so their low-order bits may
 * differ from run to run.
 * ------------------------------------------------------------------------------------- */
size_t gt_biased_attn_bwd_workspace(const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist);
gt_status gt_biased_attn_bwd(const void* q, const void* k, const void* v, const void* out,
                             const void* dout, const float* lse,
                             const uint8_t* spd, const int64_t* spd_offsets, const float* bias,
                             const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                             void* dq, void* dk, void* dv, float* dbias,
                             void* workspace, size_t workspace_bytes, void* stream);
/* gt_biased_attn_bwd_ex -- gt_biased_attn_bwd with Delta_i = dout_i . out_f32_i taken from the fp32
 * forward output of gt_biased_attn_fwd_ex (out_f32 fp32 [T,H,d]; NULL: Delta from the bf16 `out`, i.e.
 * gt_biased_attn_bwd).  Same workspace query.  With the bf16 `out` alone dbias can miss the 2e-2
 * relative-L2 bound on graphs whose pairs sit in very few buckets; with out_f32 it does not. */
gt_status gt_biased_attn_bwd_ex(const void* q, const void* k, const void* v, const void* out,
                                const void* dout, const float* lse,
                                const uint8_t* spd, const int64_t* spd_offsets, const float* bias,
                                const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                void* dq, void* dk, void* dv, float* dbias, const float* out_f32,
                                void* workspace, size_t workspace_bytes, void* stream);

/* gt_profile_bwd_kernel_events -- measurement hook (no counterpart in the paper): `before` and `after` are host
 * arrays of n caller-owned cudaEvent_t handles (passed as void*); the i-th of the next n calls of
 * gt_biased_attn_bwd / _bwd_ex / _bwd_chunked records before[i] and after[i] on its stream around the launches of
 * its main kernel (after the pre-passes, before the final conversion), so that a benchmark can report the kernel's
 * own duration from inside its timed loop.  n = 0 or NULL arrays switch the hook off.  Not thread-safe. */
void gt_profile_bwd_kernel_events(void** before, void** after, int32_t n);

/* ---------------------------------------------------------------------------------------
 * gt_biased_attn_fwd_step -- one ring step of graph-aware context parallelism driven by the caller
 * (Sec. GA-CP, items 1-3): the query rows [q_begin, q_end) of a rank attend to ONE incoming key/value
 * block, which is the union of a regular-node range [kv_begin0, kv_end0) and a super-node range
 * [kv_begin1, kv_end1) (either may be empty); the bias columns are taken at those GLOBAL indices
 * (Eq. 2, the two-part slice of the rank's bias shard) and folded in before the softmax statistics.
 * The online-softmax state of the rows is carried in normalised form: with running max m, running
 * sum l and unnormalised accumulator A, the caller holds  lse_acc = m + log l  (fp32 [H, N]) and
 * o_acc = A / l  (fp32 [N, H, d]); start with lse_acc = -inf and o_acc = 0.  The step updates both
 * for the rows of the range only:  lse' = log(exp lse + sum_r exp lse_r),  o' = the matching convex
 * combination.  After the last step o_acc is the attention output and lse_acc its LSE.
 * q, k, v, spd: the tensors of the whole single graph (n_graphs == 1), as for gt_biased_attn_fwd.
 * out: optional bf16 [N, H, d]; its rows [q_begin, q_end) receive bf16(o_acc) after the step.
 * A non-empty key range must start at a multiple of 16 (else GT_ERR_UNSUPPORTED); ranges of one row's steps
 * must not overlap (a key seen twice is counted twice).
 * ------------------------------------------------------------------------------------- */
size_t gt_biased_attn_fwd_step_workspace(const gt_batch* batch, int32_t n_heads, int32_t head_dim);
gt_status gt_biased_attn_fwd_step(const void* q, const void* k, const void* v,
                                  const uint8_t* spd, const float* bias,
                                  const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                  int32_t q_begin, int32_t q_end,
                                  int32_t kv_begin0, int32_t kv_end0, int32_t kv_begin1, int32_t kv_end1,
                                  float* o_acc, float* lse_acc, void* out,
                                  void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------
 * gt_biased_attn_bwd_chunked -- the backward pass taken one key/value chunk at a time, the view a
 * ring step of graph-aware context parallelism has (Sec. GA-CP; the paper trains through it but
 * does not spell the backward out): a step holds the key rows of one chunk, the queries, and the
 * forward results `out` and `lse` of the WHOLE row.  With the chunks of gt_biased_attn_fwd_chunked
 * (w = round_up(ceil(N / n_kv_chunks), 128) rows, the last may be short or empty) and
 *     P_ij = exp(S_ij - lse_i),  dS_ij = P_ij (dout_i . v_j - dout_i . out_i)      for j in the chunk,
 * a chunk completes dk and dv of its own rows and adds its share to dq and dbias; the chunks run
 * one after the other in stream order.  Results equal gt_biased_attn_bwd up to rounding.
 * Single graph only (n_graphs == 1).  dbias_chunks: optional fp32 [n_kv_chunks, n_heads,
 * max_dist+2] receiving each chunk's share of dbias (zeros for empty chunks), or NULL.
 * ------------------------------------------------------------------------------------- */
size_t gt_biased_attn_bwd_chunked_workspace(const gt_batch* batch, int32_t n_heads, int32_t head_dim,
                                            int32_t max_dist, int32_t n_kv_chunks);
gt_status gt_biased_attn_bwd_chunked(const void* q, const void* k, const void* v, const void* out,
                                     const void* dout, const float* lse,
                                     const uint8_t* spd, const float* bias,
                                     const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                     int32_t n_kv_chunks,
                                     void* dq, void* dk, void* dv, float* dbias, float* dbias_chunks,
                                     void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------
 * gt_biased_attn_bwd_step_* -- the backward of one ring step of graph-aware context parallelism,
 * driven by the caller (Sec. GA-CP; counterpart of gt_biased_attn_fwd_step).  A backward pass is
 *   prepare  once: from the forward results of the whole rows (`out` bf16, `lse`) and `dout` it writes
 *            the per-(query, head) terms and a transposed copy of `spd` into `context`
 *            (gt_biased_attn_bwd_step_context_bytes bytes, device memory, kept until finish);
 *   step     once per (query rows [q_begin, q_end), arriving key/value block = regular range
 *            [kv_begin0, kv_end0) united with super-node range [kv_begin1, kv_end1), either may be
 *            empty): for the pairs (i, j) of that block it ADDS, unscaled and in fp32,
 *                dq_acc[i] += sum_j dS_ij k_j    dk_acc[j] += sum_i dS_ij q_i    dv_acc[j] += sum_i P_ij dout_i
 *            ([N, H, d] each) and dbias_acc[h][b] += sum of dS over the block's pairs in bucket b
 *            (fp64 [n_heads, max_dist+2]); the accumulators start at zero, dk_acc / dv_acc are the ones
 *            that travel with the block, every pair must be visited exactly once;
 *   finish   once: dq = bf16(dq_acc / sqrt(d)), dk = bf16(dk_acc / sqrt(d)), dv = bf16(dv_acc),
 *            dbias = float(dbias_acc).
 * q, k, v, dout: the tensors of the whole single graph (n_graphs == 1) at their global rows.
 * q_begin must be a multiple of 16 (else GT_ERR_UNSUPPORTED).  The status word of the step calls
 * lives in `context` (gt_check(context, stream)).
 * ------------------------------------------------------------------------------------- */
size_t gt_biased_attn_bwd_step_context_bytes(const gt_batch* batch, int32_t n_heads, int32_t head_dim);
gt_status gt_biased_attn_bwd_step_prepare(const void* out, const void* dout, const float* lse, const uint8_t* spd,
                                          const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                          void* context, size_t context_bytes, void* stream);
/* prepare_ex: the same with the fp32 forward output (the o_acc that gt_biased_attn_fwd_step leaves after its
 * last step) for the per-query term dout_i . out_i; `out` (bf16) may then be NULL. */
gt_status gt_biased_attn_bwd_step_prepare_ex(const void* out, const float* out_f32, const void* dout,
                                             const float* lse, const uint8_t* spd,
                                             const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                             void* context, size_t context_bytes, void* stream);
gt_status gt_biased_attn_bwd_step(const void* q, const void* k, const void* v, const void* dout, const float* bias,
                                  const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                  int32_t q_begin, int32_t q_end,
                                  int32_t kv_begin0, int32_t kv_end0, int32_t kv_begin1, int32_t kv_end1,
                                  float* dq_acc, float* dk_acc, float* dv_acc, double* dbias_acc,
                                  void* context, size_t context_bytes, void* stream);
gt_status gt_biased_attn_bwd_step_finish(const float* dq_acc, const float* dk_acc, const float* dv_acc,
                                         const double* dbias_acc,
                                         const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                         void* dq, void* dk, void* dv, float* dbias, void* stream);

/* ---------------------------------------------------------------------------------------
 * gt_biased_attn_fwd_chunked -- single-GPU analogue of graph-aware context parallelism
 * (Sec. GA-CP: ring steps over KV blocks; Eq. 2: the bias columns of each block are taken at
 * the block's global node indices; item 3: bias folded in before the softmax statistics).
 * The key/value rows are split into n_kv_chunks contiguous chunks of
 * w = round_up(ceil(N / n_kv_chunks), 128) rows (the last may be short or empty); each chunk
 * yields a partial (out_c, lse_c) using spd[i][j] at the GLOBAL column j; partials are then
 * merged:  lse = log sum_c exp(lse_c),  out = sum_c exp(lse_c - lse) out_c.
 * Results equal gt_biased_attn_fwd up to rounding.  Single graph only (n_graphs == 1).
 * lse_chunks: optional fp32 [n_kv_chunks, H, N] receiving lse_c (-inf for empty chunks), or NULL.
 * ------------------------------------------------------------------------------------- */
size_t gt_biased_attn_fwd_chunked_workspace(const gt_batch* batch, int32_t n_heads, int32_t head_dim,
                                            int32_t n_kv_chunks);
gt_status gt_biased_attn_fwd_chunked(const void* q, const void* k, const void* v,
                                     const uint8_t* spd, const int64_t* spd_offsets, const float* bias,
                                     const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                     void* out, float* lse,
                                     int32_t n_kv_chunks, float* lse_chunks,
                                     void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------
 * gt_feature_attn_fwd / gt_feature_attn_bwd -- Eq. 1 with a FEATURE bias in place of the distance-bucket
 * table.  The end-to-end model of the paper has an "attention bias dimension of 4" (Sec. "Experiments",
 * end-to-end configuration): every ordered node pair carries four bias features and each head weights
 * them.  The paper states the dimension only; the linear form is the reading taken here:
 *     S_ij = (q_i . k_j)/sqrt(head_dim) + sum_c weights[h][c] * features[i][j][c]     (c = 0..3)
 * features: uint8 [N, N, 4] (row i = query, column j = key, the four features of a pair in one 32-bit
 * word, base pointer 4-byte aligned); weights: fp32 [n_heads, 4].  Forward results as for
 * gt_biased_attn_fwd (out bf16 [N,H,d], lse fp32 [H,N]); the backward overwrites dq, dk, dv (bf16) and
 *     dweights[h][c] = sum_ij dS_ij * features[i][j][c]           (fp32 [n_heads, 4]),
 * a contraction instead of the bucket form's scatter.  The backward takes the forward's lse but not its output:
 * the per-query term dout_i . out_i is recomputed in fp32 as sum_j P_ij (dout_i . v_j), because the features have
 * a large common part and a term taken from the rounded bf16 output would leak it into dweights.  Single graph only (n_graphs == 1, else
 * GT_ERR_UNSUPPORTED); head_dim in {32, 64}.  This variant is a correctness-first fp32 path on the CUDA
 * cores (no tensor cores): it is meant for the model sizes the paper trains (1 024 - 8 192 nodes per
 * batch), not for the 65 536-node benchmark.  The forward needs no workspace and has no device status.
 * ------------------------------------------------------------------------------------- */
gt_status gt_feature_attn_fwd(const void* q, const void* k, const void* v, const uint8_t* features, const float* weights,
                              const gt_batch* batch, int32_t n_heads, int32_t head_dim,
                              void* out, float* lse, void* stream);
size_t gt_feature_attn_bwd_workspace(const gt_batch* batch, int32_t n_heads);
gt_status gt_feature_attn_bwd(const void* q, const void* k, const void* v, const void* dout, const float* lse,
                              const uint8_t* features, const float* weights,
                              const gt_batch* batch, int32_t n_heads, int32_t head_dim,
                              void* dq, void* dk, void* dv, float* dweights,
                              void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------
 * gt_feature_encode, gt_feature_code_table, gt_feature_code_dweights -- the feature bias above through the
 * tensor-core kernels of the bucket form, for CATEGORICAL features: when the node pairs of a graph carry at most 256
 * distinct feature vectors, numbering them c = 0..n_codes-1 gives, exactly (the same sums regrouped),
 *     sum_x weights[h][x] features[i][j][x] = table[h][code[i][j]],   table[h][c] = sum_x weights[h][x] vectors[c][x],
 *     dweights[h][x] = sum_c dtable[h][c] vectors[c][x],
 * so gt_biased_attn_fwd / gt_biased_attn_bwd (and their _ex, chunked and step forms) run on `codes` in place of the
 * SPD matrix, with max_dist = max(n_codes, 3) - 2 and `table` / `dtable` in place of bias / dbias.
 *
 * gt_feature_encode (once per batch, like gt_spd_build): features uint8 [N,N,4] (device, 4-byte aligned) -> codes
 * (device uint8, N rows of pitch N rounded up to 16, padding 255: the SPD layout of a single graph) and vectors
 * (device uint32 [256]: vectors[c] = features of code c as f0 + 256 f1 + 65536 f2 + 16777216 f3, zero beyond
 * n_codes).  Codes follow the ascending order of that word, so the result is deterministic.  Single graph only
 * (else GT_ERR_UNSUPPORTED).  With more than 256 distinct vectors the status word of `workspace` is set to
 * GT_ERR_UNSUPPORTED (reported by gt_check), `codes` is left unwritten and the caller falls back to
 * gt_feature_attn_fwd / _bwd.  Workspace: gt_feature_encode_workspace() bytes (about 41 KB), header zeroed by the
 * caller before first use.  gt_feature_encode_count synchronises the stream and returns the number of distinct
 * vectors found (it can exceed 256 when the encoding was given up).
 *
 * gt_feature_code_table: weights fp32 [n_heads,4] -> table fp32 [n_heads, n_codes] (1 <= n_codes <= 256; codes beyond
 * the ones found get 0).  gt_feature_code_dweights: dtable fp32 [n_heads, n_codes] -> dweights fp32 [n_heads,4]
 * (overwritten; fp64 sums).  Both take device pointers, launch one small kernel on `stream` and keep no state.
 * ------------------------------------------------------------------------------------- */
size_t gt_feature_encode_workspace(void);
gt_status gt_feature_encode(const uint8_t* features, const gt_batch* batch, uint8_t* codes, uint32_t* vectors,
                            void* workspace, size_t workspace_bytes, void* stream);
gt_status gt_feature_encode_count(void* workspace, void* stream, int32_t* n_codes_host);
gt_status gt_feature_code_table(const float* weights, const uint32_t* vectors, int32_t n_heads, int32_t n_codes,
                                float* table, void* stream);
gt_status gt_feature_code_dweights(const float* dtable, const uint32_t* vectors, int32_t n_heads, int32_t n_codes,
                                   float* dweights, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* GT_ATTN_H_ */

/*
 * la.h -- C boundary of the linear-attention layer library (libla_b200.so, sm_100a).
 *
 * One causal linear-attention layer with feature map phi and the causally masked
 * depthwise-convolution augmentation, in three modes:
 *
 *   prefill  (la_prefill)      grouped / chunkwise-parallel processing of T tokens,
 *   decode   (la_decode_step)  one token per sequence against the running state,
 *   verify   (la_verify_tree)  a draft-token tree against the committed state, which is
 *                              left untouched, followed by
 *   commit   (la_commit)       absorbing the accepted root-to-node path.
 *
 * Notation, per batch entry b and head h (d = head dimension):
 *   a_ij = phi(q_i) . phi(k_j)
 *   la_i = sum_{j<=i} a_ij v_j / (sum_{j<=i} a_ij + eps)
 *   o_i  = la_i + sum_{t<W} w[h,:,t] * v_{i-t}            (elementwise over channels)
 *   S[a][c] = sum_j phi(k_j)[a] v_j[c],  z[a] = sum_j phi(k_j)[a]
 * W counts the live causal taps of the convolution: the current token and W-1 past ones.
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers on the device that was current at la_create,
 *     16-byte aligned, densely packed, innermost dimension last.  Exceptions are marked
 *     "host".  q, k, v, o and the window use the io type of the context (fp32 or bf16);
 *     S, z and the convolution weights are always fp32.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is the
 *     default stream).  No entry point other than la_create / la_destroy allocates or frees
 *     memory, and none but la_last_device_status synchronises.
 *   - The caller owns all tensors and the state buffers.  The context owns one device
 *     status word.
 *   - Every entry point returns an la_status.  Problems the host can see (null or
 *     misaligned pointers, sizes out of range, unsupported head dimension) are rejected
 *     before anything is launched.  Problems only the device can see record a sticky code in
 *     the status word, which la_last_device_status returns; nothing ever traps.  A malformed
 *     tree or an accepted node outside the tree (LA_ERR_BAD_TREE) makes the kernel skip the
 *     affected sequence and leave its outputs and state unwritten.  A bounded wait that ran out
 *     (LA_ERR_TIMEOUT) ends the thread block where it stands: outputs of that call may be
 *     partly written and the state buffers it was updating are undefined afterwards -- restore
 *     them from a copy or restart the sequence.
 *   - LA_ERR_UNSUPPORTED from la_prefill / la_verify_tree means that the shape belongs to the
 *     tensor-core kernels but the driver cannot encode TMA tensor maps; the library does not
 *     fall back to a slower kernel behind the caller's back.
 */
#ifndef LA_B200_LA_H_
#define LA_B200_LA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LA_OK = 0,
  LA_ERR_INVALID_ARG = 1,   /* null / misaligned pointer, size out of range */
  LA_ERR_UNSUPPORTED = 2,   /* configuration the library has no kernel for */
  LA_ERR_CUDA = 3,          /* a CUDA runtime or driver call failed */
  LA_ERR_BAD_TREE = 4,      /* device: parent[n] not in [-1, n), path deeper than max_depth,
                               accepted node outside [-1, N) */
  LA_ERR_TIMEOUT = 5,       /* device: a bounded wait on an asynchronous copy or MMA ran out */
  LA_ERR_TOO_LARGE = 6      /* a size exceeds the fixed capacity of an entry point that cannot allocate */
} la_status;

typedef enum { LA_PHI_ELU1 = 0,   /* phi(x) = x + 1 for x > 0, exp(x) otherwise */
               LA_PHI_RELU = 1    /* phi(x) = max(x, 0) */
} la_phi;

typedef enum { LA_F32 = 0, LA_BF16 = 1 } la_dtype;

/* Limits of this build. */
#define LA_MAX_TAPS   32   /* W */
#define LA_MAX_NODES  64   /* N, one 64-bit ancestor mask per node */
#define LA_NOALLOC_MAX_SEQ 1024   /* largest B of la_verify_tree_noalloc */

typedef struct {
  int32_t  H;           /* heads */
  int32_t  d;           /* head dimension: 64 or 128 */
  int32_t  conv_taps;   /* W, 1..LA_MAX_TAPS */
  int32_t  chunk;       /* group size C of the grouped prefill; 0 = library default.  The
                           result does not depend on it; it only selects the tiling. */
  la_phi   phi;
  float    eps;         /* added to the denominator */
  la_dtype io_dtype;    /* type of q, k, v, o and the window */
  int32_t  max_nodes;   /* largest N passed to verify / commit, 1..LA_MAX_NODES */
  int32_t  max_depth;   /* longest accepted path; row length of path_out */
} la_config;

/* Running state of B sequences (caller-owned device buffers). */
typedef struct {
  float*   S;     /* [B, H, d, d]   S[a][c], c innermost */
  float*   z;     /* [B, H, d] */
  void*    win;   /* [B, H, W-1, d] io type, the last W-1 values of v, oldest first;
                     may be NULL when W == 1 */
  int64_t* pos;   /* [B] tokens absorbed so far */
} la_state;

typedef struct la_ctx la_ctx;

/* Library set-up.  la_create validates the configuration, allocates the device status word
 * on the current device and returns a context; la_destroy frees it.  Neither is
 * asynchronous. */
la_status la_create(const la_config* cfg /*host*/, la_ctx** out /*host*/);
la_status la_destroy(la_ctx* ctx);

/* Name of a status code (static string, never NULL). */
const char* la_status_str(la_status s);

/* Prefill: the grouped processing of Sec. 4.1 ("LA Augmentation for Autoregressive LLMs").
 * The sequence is cut into non-overlapping groups; inside a group the causally masked
 * product phi(Q) phi(K)^T V is formed in parallel, between groups only the group-level
 * cumulative sums S and z of the phi(K)^T V products are carried (Sec. 3 "Linear
 * Attentions" for the reordering phi(Q)(phi(K)^T V)); the masked depthwise convolution of
 * V (Sec. 4.1 "Revised LA Augmentation") is added to the output.
 *
 *   q, k, v     [B, H, T, d] io type, T >= 1
 *   conv_w      [H, d, W] fp32, tap 0 multiplies the current token
 *   init_state  0: start from an empty state (st is output only); 1: continue from st
 *   st          in-out; on return holds S, z, the window and pos after the T tokens
 *   o           [B, H, T, d] io type
 *
 * Kernels: bf16 io with d = 128 runs grouped on the tensor cores (128-token tiles); with more than
 * 5 taps its tap sum is formed in fp32, added to the attention term after that term has been
 * rounded to bf16, and the sum rounded to bf16 (with fewer taps both terms meet in fp32).  fp32 io, and
 * d = 64 in either type, take a CUDA-core kernel that walks the tokens in order -- the cumulative
 * sum taken literally, every product an fp32 multiply-add, which is what the fp32 tolerance
 * needs; it is correct for any T but far slower per token.
 */
la_status la_prefill(la_ctx* ctx, int32_t B, int32_t T, const void* q, const void* k, const void* v,
                     const float* conv_w, int32_t init_state, la_state* st /*host struct*/, void* o,
                     void* stream);

/* Prefill of the three-branch block: Sec. 4.1 "LA Augmentation for Autoregressive LLMs" as the paper describes it
 * (Fig. "la_aug"), where la_prefill computes the exact masked linear attention inside a group instead.  The
 * sequence is cut into non-overlapping groups of `group` tokens, counted from the first token of the sequence.
 * For token i of group g:
 *   middle branch   glob_i = phi(q_i)^T S_{<g} / (phi(q_i) . z_{<g} + eps): linear attention against the group-level
 *                   cumulative sums of the groups before g only (inside a group the local dependencies are bypassed);
 *                   0 where that denominator is 0 (no earlier group and eps = 0);
 *   left branch     loc_i = sum over j in g, j <= i of softmax_j(softmax_scale * q_i . k_j) v_j: causal softmax
 *                   attention inside the group, on the raw q and k;
 *   right branch    the masked depthwise convolution of v, as in la_prefill;
 *   o_i = alpha * glob_i + loc_i + conv_i     (alpha: the paper's hyper-parameter that balances global against local).
 *
 *   group          1 .. la_prefill_grouped_max_group(ctx) (what the kernel's shared memory holds: 128 for bf16 io
 *                  with d = 128, 256 for bf16 with d = 64, 128 / 64 for fp32 with d = 64 / 128); larger groups
 *                  return LA_ERR_UNSUPPORTED
 *   softmax_scale  multiplies q . k before the softmax (1 / sqrt(d) is the usual choice)
 *   init_state     1: continue from st, whose tokens must end at a group boundary (the library cannot see where
 *                  earlier groups ended and does not check)
 *   st             in-out as for la_prefill: on return S and z hold the sums over all tokens, the window the last
 *                  W-1 values of v, pos the token count
 *   other arguments as for la_prefill.
 *
 * Kernels: bf16 io with d = 128 and groups of 32 to 128 tokens run on the tensor cores, one 128-row tile per group
 * (a shorter group leaves the rest of its tile empty; the probabilities of the softmax are rounded to bf16 there
 * before they multiply v).  Everything else runs on the CUDA cores in fp32 (a register-tiled kernel, one thread
 * block per (batch, head)), several times slower per token. */
la_status la_prefill_grouped(la_ctx* ctx, int32_t B, int32_t T, const void* q, const void* k, const void* v,
                             const float* conv_w, int32_t group, float alpha, float softmax_scale, int32_t init_state,
                             la_state* st /*host struct*/, void* o, void* stream);
int32_t la_prefill_grouped_max_group(const la_ctx* ctx);

/* A prefill cut along the sequence, for several GPUs that each hold one stretch of a long sequence.  Sec. 4.1:
 * between groups only the cumulative sums of phi(k) v^T and of phi(k) are carried, so a stretch needs from all the
 * tokens before it just those sums and the last W-1 values of v.
 *
 * la_segment_state computes the sums of one stretch on their own: dS[a][c] = sum_j phi(k_j)[a] v_j[c],
 * dz[a] = sum_j phi(k_j)[a] over the T tokens given (K and V are read, Q is not needed).
 *   k, v   [B, H, T, d] io type;  dS [B, H, d, d] fp32 out;  dz [B, H, d] fp32 out
 *
 * la_state_prefix adds up parts: S_out = S_base + sum of the first `count` of the `nparts` parts in dS_parts
 * ([nparts, B, H, d, d], e.g. the all-gathered dS of all ranks, with count = this rank's index), likewise z.
 * S_base / z_base may both be NULL (an empty starting state).  la_prefill(init_state = 1) then continues from
 * (S_out, z_out, the last W-1 values of v before the stretch, the number of tokens before it).  S_out may not
 * overlap the parts. */
la_status la_segment_state(la_ctx* ctx, int32_t B, int32_t T, const void* k, const void* v, float* dS, float* dz,
                           void* stream);
la_status la_state_prefix(la_ctx* ctx, int32_t B, int32_t nparts, int32_t count, const float* dS_parts,
                          const float* dz_parts, const float* S_base, const float* z_base, float* S_out, float* z_out,
                          void* stream);

/* Decode: one token per sequence.  The cumulative sum of Sec. 4.1 (query t meets
 * sum_{i<=t} K_i V_i) as a recurrence: S += phi(k) v^T, z += phi(k), then
 * o = phi(q)^T S / (phi(q).z + eps) + conv, with the convolution reading the carried
 * window, which is then advanced by one token.
 *
 *   q, k, v  [B, H, d] io type;  st in-out;  o [B, H, d] io type
 */
la_status la_decode_step(la_ctx* ctx, int32_t B, const void* q, const void* k, const void* v,
                         const float* conv_w, la_state* st /*host struct*/, void* o, void* stream);

/* Verify: outputs for all N nodes of a per-sequence draft tree against the committed
 * state, which is read once and not modified (Sec. 4.2 "Proposed Solution"; the shared
 * cumulative-sum state of Sec. 5.3 "Comparison with Direct Integration").  Node n sees the
 * committed prefix, its ancestors and itself; tap t of the unfolded convolution reads the
 * t-th ancestor while one exists and the committed window behind the tree otherwise,
 * never a sibling.
 *
 *   q, k, v  [B, H, N, d] io type, 1 <= N <= max_nodes
 *   parent   [B, N] int32; -1 = child of the committed prefix; parent[n] < n
 *   st       read-only;  o [B, H, N, d] io type
 */
la_status la_verify_tree(la_ctx* ctx, int32_t B, int32_t N, const void* q, const void* k, const void* v,
                         const int32_t* parent, const float* conv_w, const la_state* st /*host struct*/,
                         void* o, void* stream);

/* Commit: absorb the accepted root-to-node path of each sequence exactly as if its tokens
 * had been decoded one by one (Sec. 4.2: later groups interact with the verified tokens of
 * earlier ones).  k, v and parent are the buffers given to la_verify_tree.
 *
 *   accept_node  [B] int32: deepest accepted node, -1 = nothing accepted (a no-op)
 *   st           in-out: S, z, window and pos advance by the path
 *   path_out     [B, max_depth] int32: the path root first, padded with -1
 *   commit_len   [B] int32: its length
 */
la_status la_commit(la_ctx* ctx, int32_t B, int32_t N, const void* k, const void* v, const int32_t* parent,
                    const int32_t* accept_node, la_state* st /*host struct*/, int32_t* path_out,
                    int32_t* commit_len, void* stream);

/* Greedy acceptance: which draft nodes does the verifier accept?  (Sec. 4.2: the original model acts as the
 * verifier and accepts or rejects the drafted tokens.  The rule implemented is the greedy one: a draft node is
 * accepted when its token is the verifier's most likely token at the node it hangs from -- at the committed prefix
 * for a child of the prefix -- and that node is accepted itself.)  Pure integer work; the result feeds la_commit.
 *
 *   parent       [B, N] int32 device, as for la_verify_tree
 *   draft_token  [B, N] int32 device: token id drafted at node n
 *   pred_root    [B]    int32 device: the verifier's arg-max token after the committed prefix
 *   pred         [B, N] int32 device: the verifier's arg-max token after node n (its guess for a child of n)
 *   accept_node  [B]    int32 device, out: the deepest accepted node, the smallest index among equally deep ones;
 *                       -1 when no child of the prefix matches
 *   accept_len   [B]    int32 device, out: the number of accepted draft tokens (the depth of accept_node; 0)
 *   next_token   [B]    int32 device, out, may be null: the verifier's token that follows the accepted chain
 *                       (pred[accept_node], or pred_root when nothing was accepted)
 *
 * A sequence whose parent array is invalid gets accept_node = -1, accept_len = 0, next_token = pred_root and the
 * device status LA_ERR_BAD_TREE.  Returns LA_ERR_INVALID_ARG for null pointers or N outside 1..max_nodes.
 */
la_status la_accept_greedy(la_ctx* ctx, int32_t B, int32_t N, const int32_t* parent, const int32_t* draft_token,
                           const int32_t* pred_root, const int32_t* pred, int32_t* accept_node, int32_t* accept_len,
                           int32_t* next_token, void* stream);

/* Acceptance by a per-node score and threshold: the sampling-based counterpart of la_accept_greedy.  (Sec. 4.2: the
 * original model accepts or rejects the drafted tokens, "resampling if needed"; the paper names no rule.  Both
 * published families reduce to one comparison per node, so the caller brings the two numbers: for rejection sampling
 * score = p(token) / q(token) under the verifier and the draft model and thresh = a uniform draw in [0, 1) -- the
 * random numbers are inputs, the library draws none; for typical acceptance score = p(token) and thresh = the
 * entropy-dependent bound.)  Node n passes when score[n] >= thresh[n] as float32 (a NaN on either side fails) and is
 * accepted when it passes and the node it hangs from is accepted; a child of the committed prefix when it passes.
 *
 *   parent       [B, N] int32 device, as for la_verify_tree
 *   score        [B, N] float32 device
 *   thresh       [B, N] float32 device
 *   accept_node  [B]    int32 device, out: the deepest accepted node, the smallest index among equally deep ones;
 *                       -1 when no child of the prefix passes.  The caller resamples after this node.
 *   accept_len   [B]    int32 device, out: the depth of accept_node (0 for none)
 *
 * Errors as for la_accept_greedy: an invalid parent array gives accept_node = -1, accept_len = 0 and the device
 * status LA_ERR_BAD_TREE; LA_ERR_INVALID_ARG for null pointers or N outside 1..max_nodes. */
la_status la_accept_threshold(la_ctx* ctx, int32_t B, int32_t N, const int32_t* parent, const float* score,
                              const float* thresh, int32_t* accept_node, int32_t* accept_len, void* stream);

/* Self-test of the bounded waits.  (No counterpart in the paper.)  Every wait of a kernel of this library on a
 * shared-memory barrier has a time limit, after which the kernel records LA_ERR_TIMEOUT in the status word and
 * returns instead of hanging the GPU.  This call launches a one-CTA kernel that waits, through the same helper, on a
 * barrier nobody arrives on, with a limit of limit_us microseconds (1 .. 1 000 000).  Afterwards
 * la_last_device_status returns LA_ERR_TIMEOUT, *waited_ns (device pointer to one int64, may be null) holds the time
 * the wait took, and the context is as usable as before (la_clear_device_status resets the status word).
 */
la_status la_selftest_wait_timeout(la_ctx* ctx, uint32_t limit_us, int64_t* waited_ns /*device*/, void* stream);

/* Tree verification for callers that cannot allocate device memory.  (The paper has no
 * counterpart to this entry point; it exists for the way the library is embedded.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a serving loop
 * whose memory was handed out up front by a pool that owns the whole device, in a plug-in
 * that is given a fixed workspace and a stream and nothing else, or at a point where an
 * allocation's implicit synchronisation would stall other streams.  Such a caller cannot
 * use la_create, because the context allocates its status word.
 *
 * It computes what la_verify_tree computes, from the same arguments, with the configuration
 * passed directly instead of a context, on the device that is current at the call.  It always
 * runs the fp32 CUDA-core kernel, so for bf16 io with d = 128 its results agree with
 * la_verify_tree (which rounds S and the scores to bf16 for the tensor cores) within the io
 * tolerance rather than bit for bit, and it is several times slower for that shape.  It calls
 * no allocating routine.  Its only scratch memory, one status word per
 * sequence, is a fixed array inside the library image; each GPU that loads the library
 * carries those LA_NOALLOC_MAX_SEQ * 4 bytes until the process ends.
 *
 *   B           1 .. LA_NOALLOC_MAX_SEQ; a larger batch is refused with LA_ERR_TOO_LARGE
 *               before anything is launched (split the batch instead)
 *   seq_status  [B] int32 device buffer or NULL.  If given, after the kernel it receives,
 *               per sequence, LA_OK or LA_ERR_BAD_TREE (that sequence's outputs were then
 *               left unwritten).
 *   other arguments as for la_verify_tree; cfg->max_nodes, max_depth and chunk are ignored
 *   (N is limited by LA_MAX_NODES).
 *
 * The first call on each device looks up the device address of the fixed array (and, as the
 * first use of the library on that device, makes the CUDA runtime load the kernel image); make
 * that first call outside any stream capture.  All calls share the array, which still holds the
 * previous call's codes on entry, so every call first clears the B words it uses, on
 * `stream`.  Two calls that overlap on the GPU (different streams, no ordering between
 * them) race on those words: keep calls to this entry point ordered on one device. */
la_status la_verify_tree_noalloc(const la_config* cfg /*host*/, int32_t B, int32_t N, const void* q,
                                 const void* k, const void* v, const int32_t* parent, const float* conv_w,
                                 const la_state* st /*host struct*/, void* o, int32_t* seq_status,
                                 void* stream);

/* Waits for `stream`, then returns the sticky device status (LA_OK if no kernel reported a
 * problem since the last la_clear_device_status). */
la_status la_last_device_status(la_ctx* ctx, void* stream);

/* Resets the device status word to LA_OK (asynchronous on `stream`). */
la_status la_clear_device_status(la_ctx* ctx, void* stream);

/* Selects the kernels of la_prefill and la_verify_tree: 0 = automatic (tensor-core kernels where
 * they apply: bf16 io, d = 128), 1 = always the fp32 CUDA-core kernels.  For testing one kernel against the other. */
la_status la_set_prefill_kernel(la_ctx* ctx, int32_t which);

/* Optional workspace for la_prefill.  With few (batch, head) chains and a long sequence -- fewer chains
 * than half the SMs, T >= 2048 -- the grouped processing of Sec. 4.1 is also cut along the sequence:
 * every segment first computes its own sum of phi(k) v^T, a prefix over the segments gives each its
 * starting state (the cumulative sum of Sec. 4.1 taken at segment level), and all segments then run
 * as independent thread blocks.  That needs la_prefill_workspace_bytes(ctx, B, T) bytes of device
 * memory, which the caller lends to the context here (16-byte aligned; it must stay valid until the
 * calls that use it have completed; NULL, 0 takes it back).  Without a large enough workspace
 * la_prefill runs every chain in one thread block; the results agree up to rounding order. */
la_status la_set_workspace(la_ctx* ctx, void* workspace, uint64_t bytes);
uint64_t  la_prefill_workspace_bytes(const la_ctx* ctx, int32_t B, int32_t T);

/* Number of kernels the library has launched through this context since creation. */
int64_t la_launch_count(const la_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif  /* LA_B200_LA_H_ */

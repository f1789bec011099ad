/*
 * tsd — blockwise verification for trajectory-level speculative decoding of
 * diffusion language models, as hand-written sm_100a CUDA kernels behind a
 * plain C ABI.
 *
 * One verification step scores every draft block of a trajectory tree in one
 * pass (paper Section 3.3): masked attention of each branch's rows over the
 * shared cached prefix/suffix K/V and over that branch's own rows, then a
 * per-row vocabulary softmax with confidence and top-k candidates (Eq. 2,
 * Section 3.2), then the per-branch acceptance test and the tree walk
 * (Section 3.3, "Verification procedure").
 *
 * Conventions for every entry point
 *   - Returns 0 (TSD_OK) or a negative tsd_error.  Nothing throws.
 *   - Pointers marked "device" are CUDA device addresses owned by the caller;
 *     the library never allocates, frees or synchronises, it only enqueues
 *     work on `stream` (a cudaStream_t; NULL = the default stream).
 *   - All argument checks run on the host before anything is launched; a
 *     rejected call launches nothing.  Device arrays cannot be checked on the
 *     host: a kernel that meets an inconsistent entry (for example a parent
 *     index out of range) ORs a TSD_STATUS_* bit into `*status` (device,
 *     nullable) and produces a defined, conservative result instead of
 *     trapping.  Copy the word back and pass it to tsd_check_status().
 *   - Results are deterministic: the same inputs give the same bits.
 *   - Non-finite inputs: -inf logits are ordered last with probability 0;
 *     NaN anywhere gives unspecified values but never a fault.  In the
 *     attention stage, rows that no query row of a 128-row query tile may read
 *     can hold anything, Inf and NaN included: cached rows at or past
 *     cache_lens[s] (whatever the unused capacity holds) and draft rows of
 *     branches that none of the tile's branches may read.  Draft K/V rows that
 *     SOME row of a query tile may read have to be finite: a masked key gets
 *     weight exactly 0, but 0 x NaN is NaN, so a non-finite value in one
 *     branch's V rows makes the outputs of the other branches of that tile
 *     (the 128 / R branches that share 128 consecutive draft rows) unspecified.
 */
#ifndef TSD_H_
#define TSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* tsd_stream_t; /* same type as cudaStream_t */

typedef enum {
  TSD_OK = 0,
  TSD_ERR_INVALID_ARG = -1, /* NULL, misaligned, out-of-range or inconsistent argument */
  TSD_ERR_UNSUPPORTED = -2, /* dtype / head_dim / rows_per_branch outside the supported set */
  TSD_ERR_WORKSPACE = -3,   /* caller-provided buffer smaller than the *_bytes() query */
  TSD_ERR_CUDA = -4,        /* a CUDA runtime call failed; see tsd_last_cuda_error() */
  TSD_ERR_TIMEOUT = -5,     /* a bounded device-side wait ran out (reported via status) */
  TSD_ERR_DEVICE_DATA = -6  /* a kernel met inconsistent device data (reported via status) */
} tsd_error;

typedef enum { TSD_F32 = 0, TSD_BF16 = 1 } tsd_dtype;

/* Which draft blocks count as verified (Section 3.3).  EXACT: the rows and
 * tokens a child adds equal the set that threshold decoding would unmask at
 * its parent; this is the test under which Theorem 1 holds.  TOP1: every token
 * the child adds equals its parent's arg-max at that row (the first clause of
 * the test in Section 3.3, "Verification procedure", taken literally; admits
 * trajectory drift). */
typedef enum {
  TSD_ACCEPT_EXACT = 0,
  TSD_ACCEPT_TOP1 = 1,
  /* The two relaxed alternatives the same passage mentions in passing (membership among the
   * top-k candidates; probability above the threshold), served by tsd_accept_relaxed only.  TOPK: every token the child adds is among its parent's first
   * topk_m candidates at that row.  PROB: every token the child adds has probability > tau
   * (strictly) under its parent's distribution at that row.  Both admit drift. */
  TSD_ACCEPT_TOPK = 2,
  TSD_ACCEPT_PROB = 3
} tsd_accept_rule;

/* Greedy search takes the first valid continuation per level; longest-path
 * search takes the deepest fully valid path (Section 3.3). */
typedef enum { TSD_SEARCH_GREEDY = 0, TSD_SEARCH_LONGEST = 1 } tsd_search;

/* Bits of the device status word. */
#define TSD_STATUS_TIMEOUT 0x1u     /* a bounded wait inside a kernel expired      */
#define TSD_STATUS_BAD_PARENT 0x2u  /* parent[b] outside [0, b) for some b > 0     */
#define TSD_STATUS_BAD_MASK 0x4u    /* mask blob header does not match the layout  */
#define TSD_STATUS_BAD_INDEX 0x8u   /* a position read from device memory is out of range */

/* tsd_verify_attention flags */
#define TSD_ATTN_FORCE_SIMT 0x1u /* use the CUDA-core kernel even where the tensor-core one applies */

/* Branch / position layout: the paper's prefix P, suffix S and draft blocks
 * B_i (Section 3.3).  Draft row index inside a sequence = branch * R + r. */
typedef struct {
  int32_t batch;           /* independent sequences                                        */
  int32_t n_branches;      /* tree nodes per sequence, node 0 = root; 1..256               */
  int32_t rows_per_branch; /* R: 32 (one block), 64 (current + next block) or 128          */
  int32_t n_cache;         /* cached prefix+suffix tokens per sequence (capacity), >= 0    */
  int32_t n_q_heads;
  int32_t n_kv_heads;      /* divides n_q_heads; query head h reads kv head h/(Hq/Hkv)     */
  int32_t head_dim;        /* 64 or 128                                                    */
  int32_t dtype;           /* tsd_dtype of Q, K, V and O                                   */
} tsd_layout;

const char* tsd_strerror(int err);
/* Text of the last CUDA runtime error seen by this thread's calls ("" if none). */
const char* tsd_last_cuda_error(void);
/* Decode a status word copied back from the device: TSD_OK, TSD_ERR_TIMEOUT or
 * TSD_ERR_DEVICE_DATA. */
int tsd_check_status(uint32_t status_word);

/* ---------------------------------------------------------------------------
 * Stage 1a — branch-isolation mask (Section 3.3, "Attention masking for
 * trajectory isolation"): every row of draft block B_i sees all cached tokens
 * and, bidirectionally, the rows of B_i itself; it sees no row of another
 * block B_j.  `vis` generalises the second rule (the inter-block variant of
 * Section 3.4 lets drafts read the other block's root).
 *
 *   vis        device, nullable: uint64 [batch, n_branches, ceil(n_branches/64)];
 *              bit j of vis[s][b] set = rows of branch b may read the draft keys
 *              of branch j.  Need not be symmetric.  The own-branch bit is
 *              always treated as set.  NULL = isolated branches.
 *   cache_lens device, nullable: int32 [batch], valid cached tokens per sequence
 *              (clamped to [0, n_cache]); NULL = n_cache everywhere.
 *   mask_out   device, 16-byte aligned, tsd_branch_mask_bytes() bytes: compact
 *              per-query-tile visibility lists read by tsd_verify_attention.
 *              Reusable across layers and steps while layout, vis and
 *              cache_lens stay the same.
 *   dense_out  device, nullable: uint8 [batch, B*R, n_cache + B*R], 1 = visible
 *              (for inspection; the attention kernels do not read it).
 * ------------------------------------------------------------------------- */
size_t tsd_branch_mask_bytes(const tsd_layout* layout);
int tsd_build_branch_mask(const tsd_layout* layout, const uint64_t* vis, const int32_t* cache_lens,
                          void* mask_out, size_t mask_bytes, uint8_t* dense_out,
                          tsd_stream_t stream);

/* ---------------------------------------------------------------------------
 * Stage 1b — verify attention (Section 3.3; App. A: cached prefix/suffix K/V
 * stay fixed, only block-level K/V change).  For every sequence s, query head
 * h and draft row i:
 *     O[i] = sum_j softmax_j(sm_scale * <q_i, k_j>) v_j
 * over the visible keys j = cached tokens below cache_lens[s] plus the draft
 * rows of the branches visible to i's branch.  bf16 (or fp32) in, fp32
 * accumulation, output in the input dtype.
 *
 *   mask       device: blob written by tsd_build_branch_mask for the same layout.
 *   q, out     device: [batch, B*R, n_q_heads, head_dim] addressed through the
 *              strides (in elements); head_dim contiguous; 16-byte aligned base
 *              and 16-byte multiples for every stride.
 *   k_cache, v_cache   device: [batch, n_cache, n_kv_heads, head_dim], shared strides c_*.
 *   k_draft, v_draft   device: [batch, B*R, n_kv_heads, head_dim], shared strides d_*.
 *   lse        device, nullable: fp32 [batch, n_q_heads, B*R], natural-log
 *              sum-exp of the scaled scores.
 *   sm_scale   usually 1/sqrt(head_dim).
 *   workspace  device, 16-byte aligned, tsd_verify_attention_workspace_bytes()
 *              bytes (may be 0, then NULL is accepted).
 *   flags      TSD_ATTN_* bits.
 * The tensor-core kernel (tcgen05 MMAs with TMEM accumulators, TMA-staged
 * tiles) serves bf16 with head_dim 128; other combinations run on CUDA cores.
 * ------------------------------------------------------------------------- */
size_t tsd_verify_attention_workspace_bytes(const tsd_layout* layout);
int tsd_verify_attention(const tsd_layout* layout, const void* mask,
                         const void* q, int64_t q_stride_b, int64_t q_stride_row, int64_t q_stride_head,
                         const void* k_cache, const void* v_cache,
                         int64_t c_stride_b, int64_t c_stride_row, int64_t c_stride_head,
                         const void* k_draft, const void* v_draft,
                         int64_t d_stride_b, int64_t d_stride_row, int64_t d_stride_head,
                         void* out, int64_t o_stride_b, int64_t o_stride_row, int64_t o_stride_head,
                         float* lse, float sm_scale, void* workspace, size_t workspace_bytes,
                         uint32_t flags, uint32_t* status, tsd_stream_t stream);

/* ---------------------------------------------------------------------------
 * Diagnostic for the time-out reporting path (no counterpart in the paper).
 * Every wait inside the attention kernel is bounded: a block whose wait runs out
 * ORs TSD_STATUS_TIMEOUT into the status word, stops issuing work and returns,
 * so the context stays usable and tsd_check_status() gives TSD_ERR_TIMEOUT.
 * This call launches one warp that runs that same bounded wait on a barrier
 * nothing will ever complete, with a limit of `poll_limit` polls (1..65536; a
 * few dozen microseconds at most), so that a caller, or a test, can see the
 * whole path work (kernel returns by itself, status word, decoding) without
 * making anything hang or fault.
 *   status   device uint32, required: receives TSD_STATUS_TIMEOUT.
 * ------------------------------------------------------------------------- */
int tsd_selftest_bounded_wait(uint32_t* status, uint32_t poll_limit, tsd_stream_t stream);

/* ---------------------------------------------------------------------------
 * Verify attention over an 8-bit K/V cache.  No counterpart in the paper, which
 * keeps the dual cache in the model's dtype: the cache is stored as e4m3 codes
 * (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities) with one
 * fp32 scale per (sequence, kv head), half the footprint of bf16.  A cached
 * value is bf16(decode(code) * scale) (product and rounding in fp32 -> bf16);
 * the call expands both caches into the workspace with a streaming kernel and
 * then runs tsd_verify_attention on the expanded copy, so results equal that
 * call on the dequantised cache bit for bit.  Arguments as for
 * tsd_verify_attention, except
 *   k_cache_e4m3, v_cache_e4m3   device uint8 [batch, n_cache, n_kv_heads, head_dim], strides
 *                c_* in elements (= bytes), multiples of 16, head_dim contiguous;
 *   k_scale, v_scale             device fp32 [batch, n_kv_heads], nullable (= 1);
 *   workspace    tsd_verify_attention_fp8_cache_workspace_bytes() bytes, 16-byte aligned; it is
 *                scratch (can be shared by all layers), the persistent cache stays 8-bit.
 * Only for layout dtype TSD_BF16, batch <= 65535 and fewer than 2^31 16-code
 * vectors per sequence and cache (else TSD_ERR_UNSUPPORTED).
 * ------------------------------------------------------------------------- */
size_t tsd_verify_attention_fp8_cache_workspace_bytes(const tsd_layout* layout);
int tsd_verify_attention_fp8_cache(const tsd_layout* layout, const void* mask, const void* q,
                                   int64_t q_stride_b, int64_t q_stride_row, int64_t q_stride_head,
                                   const uint8_t* k_cache_e4m3, const uint8_t* v_cache_e4m3,
                                   int64_t c_stride_b, int64_t c_stride_row, int64_t c_stride_head,
                                   const float* k_scale, const float* v_scale, const void* k_draft,
                                   const void* v_draft, int64_t d_stride_b, int64_t d_stride_row,
                                   int64_t d_stride_head, void* out, int64_t o_stride_b,
                                   int64_t o_stride_row, int64_t o_stride_head, float* lse,
                                   float sm_scale, void* workspace, size_t workspace_bytes,
                                   uint32_t flags, uint32_t* status, tsd_stream_t stream);

/* ---------------------------------------------------------------------------
 * Stage 2 — confidence and candidates (Eq. 2: c = max softmax(logits);
 * Section 3.2: top-k candidates per position).  One streaming pass over the
 * logits.  Per row: conf = largest softmax probability; topk_idx = the k first
 * vocabulary entries ordered by (logit descending, index ascending), decided on
 * the raw input values; topk_prob = their probabilities under the softmax over
 * the whole vocabulary (not renormalised); lse = log sum exp.
 *
 *   logits     device: [n_rows, vocab] of `dtype`, row r at logits + r*row_stride
 *              elements; base and row_stride*sizeof(elem) 16-byte aligned.
 *   k          1..8, k <= vocab.
 *   conf       device fp32 [n_rows];  topk_idx device int32 [n_rows, k];
 *   topk_prob  device fp32 [n_rows, k];  lse device fp32 [n_rows], nullable.
 *   workspace  device, 16-byte aligned, tsd_confidence_topk_workspace_bytes()
 *              bytes: per-segment partial results and per-row ticket words when
 *              a row is split across thread blocks (few rows); 0 bytes when it
 *              is not.  Zero it once before its first use (cudaMemsetAsync);
 *              after that it can be reused by later calls of any shape without
 *              clearing: a completed call leaves every ticket word it used at 0
 *              and the next call rewrites the partial slots it reads.  (A word
 *              counts as a live ticket only if it carries a 24-bit tag, so most
 *              leftover content is harmless, but only a zeroed buffer is
 *              guaranteed.)  Two calls that may overlap on the GPU need a
 *              workspace each.
 * ------------------------------------------------------------------------- */
size_t tsd_confidence_topk_workspace_bytes(int64_t n_rows, int32_t vocab, int32_t k);
int tsd_confidence_topk(const void* logits, int32_t dtype, int64_t n_rows, int32_t vocab,
                        int64_t row_stride, int32_t k, float* conf, int32_t* topk_idx,
                        float* topk_prob, float* lse, void* workspace, size_t workspace_bytes,
                        uint32_t* status, tsd_stream_t stream);

/* ---------------------------------------------------------------------------
 * Stage 2 without a caller workspace (no counterpart in the paper: an interface
 * convenience of this library).  Same computation and outputs as
 * tsd_confidence_topk, for callers that cannot obtain device memory at call
 * time: a server plug-in whose device pool is fixed at start-up, a decode loop
 * that may not call cudaMalloc because it would stall the device mid-step.
 * The per-segment partial results and per-row tickets go to a 1 MiB array that
 * is part of the library image (every GPU that loads the library holds it
 * until the process exits); tsd_confidence_topk_static_capacity() returns that
 * size.  The call itself allocates and frees nothing.
 *   - A shape whose scratch need exceeds the capacity is rejected with
 *     TSD_ERR_WORKSPACE and nothing is launched; compare
 *     tsd_confidence_topk_workspace_bytes() with the capacity beforehand, and
 *     fall back to tsd_confidence_topk with your own workspace.
 *   - Every call looks the array's device address up (cudaGetSymbolAddress,
 *     with the device current: a host-side query).  The first lookup on a
 *     device sets the library's module up there: make that first call before
 *     any stream capture begins.
 *   - All calls on a device share the one array, and it keeps whatever the
 *     previous call left: a completed call leaves every ticket word it used
 *     idle again and the next call overwrites the partial slots it reads.
 *     Two calls that overlap on the GPU (different streams, no ordering) would
 *     race on it: order them on one stream or with events.
 * Arguments as for tsd_confidence_topk, minus the workspace.
 * ------------------------------------------------------------------------- */
size_t tsd_confidence_topk_static_capacity(void);
int tsd_confidence_topk_static(const void* logits, int32_t dtype, int64_t n_rows, int32_t vocab,
                               int64_t row_stride, int32_t k, float* conf, int32_t* topk_idx,
                               float* topk_prob, float* lse, uint32_t* status, tsd_stream_t stream);

/* ---------------------------------------------------------------------------
 * Stage 3 — acceptance (Section 3.3 "Verification procedure"; Alg. 1 Phase 1
 * for the high/low confidence split; Eqs. 6-7 for the top-1 fallback).
 * Per node p the decode rule U(p) is what threshold decoding would unmask
 * next: the masked rows with conf > tau and their top-1 tokens, or, when there
 * are none, the single masked row of largest conf (lowest row on ties).
 * Edge parent->c is valid under `rule` (see tsd_accept_rule); a child that
 * adds nothing, alters a filled row or re-masks one is invalid.
 *
 *   parent     device int32 [batch, B]; parent[0] = -1, 0 <= parent[b] < b.
 *   state      device int32 [batch, B, R]: token id, or mask_id where masked.
 *   conf       device fp32 [batch, B, R] (stage 2 output).
 *   top1_idx   device int32, element (s,b,r) at top1_idx[((s*B+b)*R+r)*top1_stride]
 *              (pass topk_idx with top1_stride = k).
 *   edge_valid    device uint8 [batch, B]; root = 1.
 *   prefix_len    device int32 [batch, B]: leading valid edges on the path
 *                 root -> b (the branch's longest accepted trajectory prefix).
 *   accepted_node device int32 [batch];  accepted_len device int32 [batch] (its depth).
 *   n_new_tokens  device int32 [batch]: rows the accepted node holds beyond the root.
 *   unmask_flag   device uint8 [batch, R], unmask_tok device int32 [batch, R]:
 *                 U(accepted node), the caller's next root update; tok = -1
 *                 where flag = 0.
 * R is 1..128, B is 1..256.
 * ------------------------------------------------------------------------- */
int tsd_accept_trajectories(int32_t batch, int32_t n_branches, int32_t rows_per_branch,
                            const int32_t* parent, const int32_t* state, int32_t mask_id,
                            const float* conf, const int32_t* top1_idx, int32_t top1_stride,
                            float tau, int32_t rule, int32_t search,
                            uint8_t* edge_valid, int32_t* prefix_len, int32_t* accepted_node,
                            int32_t* accepted_len, int32_t* n_new_tokens, uint8_t* unmask_flag,
                            int32_t* unmask_tok, uint32_t* status, tsd_stream_t stream);

/* ---------------------------------------------------------------------------
 * Draft-tree construction for the next step (Alg. 1 "Confidence-Stratified
 * Trajectory Tree Construction", Phase 2; Section 3.2 hybrid expansion), fused
 * with the root update after acceptance so that a decode step stays on the
 * device.  Per sequence: next root = state of the accepted node + its unmask
 * set; candidate pool = top-k (token, probability) of the rows still masked in
 * that root, from the scores of the pass just verified (Section 3.1).
 * Level 1: the k most probable pool entries, one child each; deeper levels: one
 * child per frontier node (its most probable entry at a row it still masks);
 * after each level the `width` most probable children survive (siblings end up
 * in descending draft confidence); the tree holds at most `max_nodes` nodes
 * (the WxDy(n) naming: n + 1).  Ties: lower row, lower rank, earlier child.
 *
 *   prev_state    device int32 [batch, prev_branches, R]: block states of the verified tree.
 *   accepted_node device int32 [batch], nullable (= node 0).
 *   unmask_flag, unmask_tok   device [batch, R], both or neither: U(accepted node).
 *   topk_idx, topk_prob       device [batch, prev_branches, R, k]: stage 2 output of that pass.
 *   parent        device int32 [batch, max_nodes];  state device int32 [batch, max_nodes, R];
 *   node_prob     device fp32 [batch, max_nodes]: probability of the entry a node added (root 1);
 *   n_nodes       device int32 [batch].  Slots past n_nodes are copies of the root hanging off it.
 *   out_stride    branches per sequence in parent / state / node_prob (>= max_nodes): the tree
 *                 may be a slice of a larger forest (pass pointers to its first branch);
 *   node_base     added to every parent index written (the root still gets -1): the forest index
 *                 of this tree's root;  0 and out_stride = max_nodes for a tree of its own;
 *   enable        device uint8 [batch], nullable: 0 keeps that sequence's tree at its root
 *                 (the inter-block trigger of Eq. 3).
 * R 1..128, k 1..8, width 1..32, depth >= 0, max_nodes 1..256.
 * ------------------------------------------------------------------------- */
int tsd_build_draft_tree(int32_t batch, int32_t prev_branches, int32_t rows_per_branch, int32_t k,
                         const int32_t* prev_state, const int32_t* accepted_node,
                         const uint8_t* unmask_flag, const int32_t* unmask_tok, int32_t mask_id,
                         const int32_t* topk_idx, const float* topk_prob, int32_t width, int32_t depth,
                         int32_t max_nodes, int32_t out_stride, int32_t node_base, const uint8_t* enable,
                         int32_t* parent, int32_t* state, float* node_prob, int32_t* n_nodes,
                         uint32_t* status, tsd_stream_t stream);

/* ---------------------------------------------------------------------------
 * Inter-block speculation (Section 3.4, Eq. 3, Appendix D): one pass verifies
 * the tree of the current block B_t and a compact tree of the next block
 * B_{t+1}.  Joint layout: branches [0, n_cur) = tree of B_t with its root at 0,
 * branches [n_cur, n_branches) = tree of B_{t+1} with its root at n_cur; every
 * branch is one block of R rows; parent[] holds forest indices and
 * parent[n_cur] = -1.  None of the three calls below has a counterpart among the
 * stages of the single-block path; they are its inter-block variant.
 *
 * tsd_build_interblock_vis writes the `vis` bitsets for tsd_build_branch_mask:
 * the two roots read each other, a draft reads the other block's root, and
 * nobody but the draft itself reads a draft (so a root's scores never depend on
 * what was drafted).  n_cur = n_branches gives isolated branches.
 *   vis  device uint64 [batch, n_branches, ceil(n_branches/64)].
 *
 * tsd_interblock_trigger evaluates Eq. 3 per sequence from the pass just
 * verified: with c(b) = the largest confidence among the still-masked rows of
 * node b, trigger = c(node_next) > c(node_cur[s]) or c(node_next) > tau; a next
 * block without masked rows never triggers, a current block without masked
 * rows always does.
 *   state, conf  device [batch, n_branches, R] (int32 / fp32);
 *   node_cur     device int32 [batch], nullable (= 0): the accepted node of B_t's tree;
 *   node_next    index of B_{t+1}'s root;
 *   trigger      device uint8 [batch];  top_conf device fp32 [batch, 2], nullable: c(cur), c(next).
 *
 * tsd_accept_joint_trees runs the acceptance of tsd_accept_trajectories (rules
 * EXACT and TOP1) on both
 * trees in one launch.  Per-branch outputs (edge_valid, prefix_len) keep the
 * forest layout [batch, n_branches]; per-tree outputs are tree-major:
 * accepted_node, accepted_len, n_new_tokens [2, batch] and unmask_flag,
 * unmask_tok [2, batch, R]; accepted_node is a forest index.  With
 * n_cur = n_branches only tree 0 is written.  A parent outside its own tree sets
 * TSD_STATUS_BAD_PARENT and invalidates that edge.
 * ------------------------------------------------------------------------- */
int tsd_build_interblock_vis(int32_t batch, int32_t n_branches, int32_t n_cur, uint64_t* vis,
                             tsd_stream_t stream);

/* ---------------------------------------------------------------------------
 * The step after the path: commit what the pass accepted (Section 3.3: the
 * longest verified trajectory is kept; Section 3.1: its last node starts the
 * next pass; Theorem 1: each edge of the accepted path is one step of the
 * sequential decoder).  Per sequence: next root = state of the accepted node +
 * its unmask set, written to root_out and into the sequence's token buffer at
 * the block's position.  With the pass starting step_base sequential steps into
 * the block and accepting a node of depth n, a row filled by the path node at
 * depth j is logged at step step_base + j - 1, the rows of the unmask set at
 * step_base + n, and step_base moves on by n + 1 (by n if the accepted node had
 * no masked row left).
 *
 *   tree_root       forest index of the tree's root: 0 for a tree of its own; n_cur for the
 *                   next block's tree of a joint pass (Section 3.4), whose nodes, parents and
 *                   accepted_node are forest indices (as tsd_accept_joint_trees writes them);
 *   parent, state   device [batch, B] / [batch, B, R]: the verified tree (or forest);
 *   accepted_node   device int32 [batch], nullable (= the root);
 *   unmask_flag, unmask_tok   device [batch, R], both or neither;
 *   tokens          device int32, nullable: sequence s occupies tokens[s * seq_stride ...];
 *   block_start     device int32 [batch], nullable (= 0): first position of the block; a
 *                   block that does not fit in [0, seq_stride) sets TSD_STATUS_BAD_INDEX and
 *                   is not written;
 *   root_out        device int32 [batch, R], nullable;
 *   fill_step       device int32 [batch, R], nullable, in/out: only rows filled by this pass
 *                   are written (initialise with -1 at the start of a block);
 *   step_base       device int32 [batch], nullable (= 0), in/out;
 *   n_masked        device int32 [batch], nullable: rows still masked in the next root.
 * A parent chain that leaves the tree sets TSD_STATUS_BAD_PARENT and commits U(root) only.
 * R 1..128, B 1..256.
 * ------------------------------------------------------------------------- */
int tsd_commit_accepted(int32_t batch, int32_t n_branches, int32_t rows_per_branch, int32_t tree_root,
                        const int32_t* parent, const int32_t* state, const int32_t* accepted_node,
                        const uint8_t* unmask_flag, const int32_t* unmask_tok, int32_t mask_id,
                        int32_t* tokens, int64_t seq_stride, const int32_t* block_start,
                        int32_t* root_out, int32_t* fill_step, int32_t* step_base, int32_t* n_masked,
                        uint32_t* status, tsd_stream_t stream);

/* ---------------------------------------------------------------------------
 * Hand-over of the accepted node's K/V (Appendix A: the dual cache holds
 * prefix/suffix K/V for a whole block and is refreshed at block boundaries;
 * Section 3.1: a verification pass already holds what the next step needs).
 * The pass has computed draft K/V rows for every node of the tree; the rows of
 * the accepted node are the block's K/V under the tokens that were kept.  This
 * call copies them, per layer, to a destination of the caller's (typically the
 * block's position in that layer's cache) so that a block that has just been
 * completed need not be recomputed before it serves as cached context.  Whether
 * to use it or to recompute at the boundary, as the paper does, is the caller's
 * choice: the copied rows were computed while the block still held masked
 * positions elsewhere in the tree's other nodes, not in this one, so they are
 * exact for the accepted node's own content.
 * For sequence s and r < R:
 *     out[s, out_row0[s] + r, :, :] = draft[s, accepted_node[s] * R + r, :, :]
 *
 *   accepted_node   device int32 [batch], nullable (= node 0), a tree-local index as
 *                   tsd_accept_trajectories writes it;
 *   k_draft, v_draft  device [batch, B*R, n_kv_heads, head_dim], element strides d_*;
 *                   v_draft / v_out both NULL copies K only;
 *   k_out, v_out    device [batch, out_rows, n_kv_heads, head_dim], element strides o_*;
 *   out_row0        device int32 [batch], nullable (= 0): first destination row.
 * All bases 16-byte aligned, strides multiples of 16 bytes, head_dim contiguous and a
 * multiple of 16 bytes.  A node outside [0, B) or a destination outside
 * [0, out_rows) sets TSD_STATUS_BAD_INDEX and leaves that sequence unwritten.
 * ------------------------------------------------------------------------- */
int tsd_gather_accepted_kv(int32_t batch, int32_t n_branches, int32_t rows_per_branch, int32_t n_kv_heads,
                           int32_t head_dim, int32_t dtype, const int32_t* accepted_node,
                           const void* k_draft, const void* v_draft, int64_t d_stride_b,
                           int64_t d_stride_row, int64_t d_stride_head, void* k_out, void* v_out,
                           int64_t o_stride_b, int64_t o_stride_row, int64_t o_stride_head,
                           const int32_t* out_row0, int32_t out_rows, uint32_t* status,
                           tsd_stream_t stream);

/* ---------------------------------------------------------------------------
 * Acceptance under any of the four rules (Section 3.3, "Verification
 * procedure": the exact and top-1 tests, and the top-k-membership and
 * probability-above-tau alternatives), for one tree (n_cur = n_branches) or the two trees of a joint
 * pass; outputs laid out as for tsd_accept_joint_trees.  Combined with
 * TSD_SEARCH_LONGEST this is the longest-path search under trajectory drift.
 *
 *   topk_idx     device int32, candidates per (node, row) in descending probability,
 *                topk_stride apart (stage 2's topk_idx); entry 0 is the top prediction;
 *   topk_m       1..topk_stride: how many of them count for TSD_ACCEPT_TOPK;
 *   logits       device, nullable unless rule = TSD_ACCEPT_PROB: the logits of the pass,
 *                [batch * n_branches * R, vocab], rows row_stride elements apart, dtype as given;
 *   lse          device fp32 [batch * n_branches * R]: stage 2's log-sum-exp of each row
 *                (required with logits);
 *   draft_prob   device fp32 [batch, n_branches, R], nullable: probability, under the parent's
 *                distribution, of the token each node adds at each row, exp(logit - lse) in
 *                fp32 (0 where the node adds nothing); written whenever logits are given.  The
 *                PROB rule compares exactly these fp32 values with tau.
 * A drafted token outside [0, vocab) has probability 0.
 * ------------------------------------------------------------------------- */
int tsd_accept_relaxed(int32_t batch, int32_t n_branches, int32_t n_cur, int32_t rows_per_branch,
                       const int32_t* parent, const int32_t* state, int32_t mask_id, const float* conf,
                       const int32_t* topk_idx, int32_t topk_stride, int32_t topk_m, const void* logits,
                       int32_t dtype, int64_t vocab, int64_t row_stride, const float* lse, float tau,
                       int32_t rule, int32_t search, uint8_t* edge_valid, int32_t* prefix_len,
                       int32_t* accepted_node, int32_t* accepted_len, int32_t* n_new_tokens,
                       uint8_t* unmask_flag, int32_t* unmask_tok, float* draft_prob, uint32_t* status,
                       tsd_stream_t stream);
int tsd_interblock_trigger(int32_t batch, int32_t n_branches, int32_t rows_per_branch,
                           const int32_t* state, const float* conf, const int32_t* node_cur,
                           int32_t node_next, int32_t mask_id, float tau, uint8_t* trigger,
                           float* top_conf, uint32_t* status, tsd_stream_t stream);
int tsd_accept_joint_trees(int32_t batch, int32_t n_branches, int32_t n_cur, int32_t rows_per_branch,
                           const int32_t* parent, const int32_t* state, int32_t mask_id,
                           const float* conf, const int32_t* top1_idx, int32_t top1_stride, float tau,
                           int32_t rule, int32_t search, uint8_t* edge_valid, int32_t* prefix_len,
                           int32_t* accepted_node, int32_t* accepted_len, int32_t* n_new_tokens,
                           uint8_t* unmask_flag, int32_t* unmask_tok, uint32_t* status,
                           tsd_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* TSD_H_ */

/*
 * war.h -- C ABI of the batched SuffixDecoding speculate-and-verify step for one B200 (sm_100a).
 *
 * The paper (WAR: Workload-Aware Rollouts, Section 3 overview and Section 3.3 "SuffixDecoding") speeds up
 * low-load agentic RL rollouts with model-free speculative decoding: a cache of previously generated
 * trajectories is matched against each live request's current token pattern to produce draft tokens, the
 * target model verifies all drafts in one forward pass, and the request advances by every accepted token.
 * Sections 2.3 and 5.3 name the costs of that step: suffix lookup, draft construction, verification and
 * tree-mask handling.  This library is that step, entirely on the device:
 *
 *   war_index_build / war_index_append   the trajectory cache: suffix array + capped LCP over the corpus
 *   war_draft                            longest-suffix match + frequency-ranked draft token tree
 *   war_draft_scored                     the same from the best-scoring of several suffix lengths
 *   war_draft_local                      draft trees from each request's own context
 *   war_draft_pick                       choice between two draft trees by score
 *   war_verify_attn                      tree-masked GQA decode attention over a paged bf16 KV cache
 *   war_accept                           longest root path of the tree that equals the target's tokens
 *   war_commit                           the accepted tokens become context: KV rows, prefix length, tail window
 *
 * Conventions shared by every call
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  The caller owns every buffer it
 *     passes; the library neither frees nor keeps them beyond the stream order of the call.  The library
 *     owns only war_index_t objects (and build scratch it allocates and frees itself).
 *   - Every call enqueues its work on `stream` and returns without synchronising the host, except
 *     war_index_build / war_index_append (they size and free scratch) and war_device_status.
 *   - Errors are return codes.  Nothing throws, aborts or traps.  Problems visible on the host (null
 *     pointer, unsupported shape, capacity) are reported before anything is launched.  Problems only the
 *     device can see (a malformed parent array, a page index outside the pool, a bounded wait that ran
 *     out) set a sticky device status word, give the offending request an empty result (num_nodes = 0 /
 *     accept_len = 0 / untouched attention rows) and let the kernel finish normally; read the word with
 *     war_device_status.
 *   - Slot convention: a request's draft tree has at most N slots.  Slot 0 is the root = the request's
 *     last context token (parent -1).  Slots 1 .. num_nodes-1 are draft tokens with parent[j] < j.
 *     N therefore counts the root.  Limits: N <= 64, P <= 32, topk <= 8, D == 128.
 */
#ifndef WAR_H_
#define WAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    WAR_OK = 0,
    WAR_ERR_INVALID_ARG = 1,   /* null pointer, negative size, shape outside the stated limits      */
    WAR_ERR_OOM = 2,           /* a device allocation made by the library failed                      */
    WAR_ERR_CAPACITY = 3,      /* the index cannot hold the requested number of tokens                */
    WAR_ERR_CUDA = 4,          /* a CUDA runtime call or launch failed                                */
    WAR_ERR_TIMEOUT = 5,       /* device status only: a bounded in-kernel wait expired                */
    WAR_ERR_UNSUPPORTED = 6,   /* valid request this build has no kernel for (e.g. a strided pool)    */
    WAR_ERR_BAD_TREE = 7,      /* device status only: parent[j] outside [0, j) or num_nodes > N       */
    WAR_ERR_BAD_PAGE = 8       /* device status only: page table entry outside [0, num_pages)         */
} war_status_t;

typedef struct CUstream_st* war_stream_t;      /* same type as cudaStream_t */
typedef struct war_index war_index_t;          /* opaque; lives on the device that was current at build */

/* ------------------------------------------------------------------------------------------------
 * Trajectory cache (paper Section 3.3: SuffixDecoding keeps the token patterns of the trajectories generated so
 * far; an update interface outside the decode loop adds the new trajectories after each RL step).  Trajectory t is d_tokens[h_offsets[t] .. h_offsets[t+1]); token ids must lie in [0, vocab)
 * (checked on the device: WAR_ERR_INVALID_ARG, nothing added).
 * Inside the index the trajectories are joined with one unique negative separator each, so no match ever
 * straddles two trajectories.  The suffix array is ordered to depth max_depth (>= P + N of every later
 * war_draft call; <= 128) and LCP values are capped there.
 *   capacity_tokens  upper bound on (sum of trajectory lengths + number of trajectories) over the whole
 *                    life of the index, appends included.
 * war_index_append leaves the index answering every query exactly as a fresh build over the old
 * trajectories followed by the new ones would.  Exceeding the capacity returns WAR_ERR_CAPACITY and
 * leaves the index unchanged.  Both calls synchronise `stream` before returning (war_index_append_async, below,
 * does not).
 * Updating without blocking the drafts (the paper updates the cache asynchronously so that it does not block
 * the pipeline, Section 3.3): the index keeps two sets of (suffix array, LCP, buckets).  war_index_append builds
 * the new set beside the published one and publishes it just before it returns; the corpus is only written
 * behind what the published set refers to.  So ONE thread may run war_index_append (on its own stream) while other
 * threads keep calling war_draft on other streams: a draft kernel takes the set that is published at the moment
 * it STARTS on the device (it reads the published set's number from device memory), and that set stays intact
 * until the NEXT update starts.  The caller makes sure that update does not start before those drafts have
 * finished (an event, or one update per step).  Two updates must not overlap each other.  Cost: 5 more bytes per
 * token of capacity.
 * CUDA graphs: because the set is chosen on the device, a captured war_draft / war_draft_scored launch keeps
 * answering from the current index after any number of war_index_append / war_index_evict calls; nothing has to
 * be captured again.  (The graph holds the index handle's device addresses: destroy the index only when the graph
 * is no longer replayed.)
 * ------------------------------------------------------------------------------------------------ */
war_status_t war_index_build(const int32_t* d_tokens, const int64_t* h_offsets, int32_t T,
                             int32_t vocab, int32_t max_depth, int64_t capacity_tokens,
                             war_stream_t stream, war_index_t** out);
war_status_t war_index_append(war_index_t* ix, const int32_t* d_tokens, const int64_t* h_offsets, int32_t T,
                              war_stream_t stream);

/* war_index_append as a stream-ordered operation (paper Section 3.3: the cache is updated asynchronously, off the
 * critical path of training): the call only ENQUEUES the update on `stream` and returns; it never synchronises the
 * host, so one host thread can start the update on a side stream and go on launching steps on its main stream.
 * The new set of index arrays is built behind the work already in `stream` and published by the last kernel of the
 * update; a draft kernel that starts after that point answers from the grown index, one that starts earlier from
 * the old one (either way from a complete index), and the result is the one war_index_append gives.
 *   - Scratch comes from CUDA's stream-ordered allocator (cudaMallocAsync on `stream`), sized from the token and
 *     trajectory counts the host knows; the library lets the device's default memory pool keep what it frees.
 *   - The host-side state of the handle (war_index_info, the capacity check of the next update) advances at once;
 *     whatever uses the handle next -- another update, war_index_evict, war_index_export, destroying it -- must be
 *     ordered behind this one: enqueue it on the same stream, or wait for the stream first.  d_tokens must stay
 *     valid until the update has run; h_offsets may be reused when the call returns.
 *   - Nobody reads a flag back, so a token id outside [0, vocab) cannot make the call fail: it is stored as an
 *     end-of-trajectory mark (it matches nothing and nothing continues into it) and WAR_ERR_INVALID_ARG is
 *     recorded in the device status word.
 *   - At most 65 535 trajectories per call (WAR_ERR_UNSUPPORTED beyond); capacity as in war_index_append.  If the
 *     call returns an error, nothing has been published and the handle is as before.
 * The rule for updates beside running drafts is the one above: the set the drafts read stays intact until the NEXT
 * update starts. */
war_status_t war_index_append_async(war_index_t* ix, const int32_t* d_tokens, const int64_t* h_offsets, int32_t T,
                                    war_stream_t stream);

/* Windowed cache (the paper keeps the cache's memory overhead modest, Section 3.3, without naming a policy; this
 * is the simplest one): removes the n_oldest trajectories that were added first.  Afterwards every query answers
 * exactly as a fresh build on the remaining trajectories would.  The suffix array is filtered, not sorted again
 * (the remaining suffixes keep their order); LCP and buckets are recomputed.  Synchronises `stream`; allocates
 * and frees scratch of 4 bytes per stored token.  n_oldest must be in [0, T].  Unlike an append it moves the
 * corpus itself, so no war_draft call may be in flight on this index while it runs. */
war_status_t war_index_evict(war_index_t* ix, int32_t n_oldest, war_stream_t stream);

/* Export / import: the whole index as one host buffer (header, trajectory bounds, corpus, suffix array, LCP,
 * buckets), so that a replica that starts later, or restarts, takes the arrays instead of sorting again.  The paper
 * has no counterpart (its cache lives in the serving process).  war_index_export writes
 * war_index_export_bytes(ix) bytes to h_dst; war_index_import checks the header and the sizes (not the arrays'
 * contents: import only what an export wrote) and returns an index of the given capacity that answers exactly as the
 * exported one.  Both synchronise `stream`. */
size_t war_index_export_bytes(const war_index_t* ix);
war_status_t war_index_export(const war_index_t* ix, void* h_dst, size_t bytes, war_stream_t stream);
war_status_t war_index_import(const void* h_src, size_t bytes, int64_t capacity_tokens, war_stream_t stream,
                              war_index_t** out);

typedef struct {
    int64_t M;                  /* corpus entries in use: tokens + one separator per trajectory */
    int64_t capacity_tokens;
    int32_t T;                  /* trajectories */
    int32_t vocab;
    int32_t max_depth;
    int32_t reserved;
    const int32_t* d_corpus;    /* [M]  separator of trajectory t is -(t+1) */
    const int32_t* d_sa;        /* [M]  suffix array */
    const uint8_t* d_lcp;       /* [M]  min(lcp(sa[i-1], sa[i]), max_depth); lcp[0] = 0 */
    const int32_t* d_bucket;    /* [vocab+1] sa interval of every one-token string */
} war_index_info_t;
war_status_t war_index_info(const war_index_t* ix, war_index_info_t* out);
war_status_t war_index_destroy(war_index_t* ix);

/* ------------------------------------------------------------------------------------------------
 * Draft (paper Section 3: SuffixDecoding drafts by matching the request's current tokens against the stored
 * trajectories).  For each of B requests:
 *   match   the largest l <= min(P, tail_len) such that the last l tokens of the tail occur contiguously
 *           inside one stored trajectory (0 if none);
 *   tree    slot 0 = the last tail token, count[0] = occurrences of the matched string.  Every further slot
 *           is one continuation token; count = occurrences of matched string + root path (every occurrence
 *           counts, overlapping ones too).  Each slot offers its topk most frequent continuations (count
 *           descending, token id ascending); slots are created best-first from all offers (count
 *           descending, parent slot ascending, token id ascending) until N slots exist or no offer is left.
 *           If match_len < max(1, min_match) the tree is the root alone.
 * d_tail is int32 [B, P], right-aligned: the most recent token is d_tail[b, P-1]; only the last tail_len[b]
 * entries are read.  Tail tokens outside [0, vocab) never match.
 * Outputs: d_match_len [B], d_num_nodes [B], d_ids / d_parent / d_count [B, N] (d_count may be NULL).
 * Unused slots are written as ids = -1, parent = -1, count = 0.
 * Workload-aware switch (paper Section 3.3: speculation is enabled and disabled according to the
 * current batch size, and switching between the modes carries no state; Section 5.3: beyond a batch of about 16 speculation
 * costs more than it gains).  A request with tail_len[b] < 0 is not running: num_nodes = 0, match_len = 0.  The
 * effective batch size is the number of running requests, counted on the device in this call.  When
 * spec_batch_limit > 0 and the effective batch size exceeds it, nothing is looked up and every running request
 * gets the root alone (num_nodes = 1, match_len = 0, count = 0), so the step that follows is a plain decode step
 * through the same calls: no state is kept between calls and one captured CUDA graph serves both modes.
 * spec_batch_limit = 0 always speculates.
 * Two thresholds of the SuffixDecoding method the paper builds on (Section 3.3 takes that method's code base; the
 * paper itself names neither), both exact integer rules, both off when their numerator is 0:
 *   spec_factor_num / spec_factor_den   the tree has at most 1 + floor(match_len * num / den) slots, so a longer
 *                                       match earns a larger tree (den >= 1)
 *   min_prob_num / min_prob_den         a continuation is offered only if count(child) * den >= num * count(parent),
 *                                       i.e. its empirical probability after the parent's string is at least
 *                                       num / den (0 < num <= den)
 * ------------------------------------------------------------------------------------------------ */
typedef struct {
    int32_t B, P, N, topk, min_match;
    int32_t spec_batch_limit;
    int32_t spec_factor_num, spec_factor_den;
    int32_t min_prob_num, min_prob_den;
} war_draft_params_t;
war_status_t war_draft(const war_index_t* ix, const int32_t* d_tail, const int32_t* d_tail_len,
                       const war_draft_params_t* params,
                       int32_t* d_match_len, int32_t* d_num_nodes,
                       int32_t* d_ids, int32_t* d_parent, int32_t* d_count, war_stream_t stream);

/* Drafting from the best-scoring of several suffix lengths (a variant of the SuffixDecoding method that Section 3.3
 * adopts; the paper does not spell it out).  Candidates are the suffix lengths match_len, match_len - 1, ...,
 * n_lengths of them (1 <= n_lengths <= 32), never below max(1, min_match); every shorter suffix of an occurring
 * string occurs too, usually more often.  Each candidate gets its own tree by the rules of war_draft (its own root
 * interval, its own slot budget under spec_factor).  A tree's score is
 *     (sum of count[j], j = 1 .. num_nodes-1) / count[0]
 * = the sum over its slots of the empirical probability that the text continues with the slot's whole root path
 * = the number of draft tokens one expects to be accepted when the continuation is drawn from the occurrences of
 * the suffix.  The tree with the largest score is returned; scores are compared exactly (cross-multiplied 64-bit
 * integers); equal scores go to the longer suffix.  d_match_len [B] receives the longest match as in war_draft,
 * d_used_len [B] the length the returned tree was built from (0 where no tree was built).  With n_lengths = 1 the
 * outputs equal war_draft's.  The switch and the thresholds act as in war_draft.
 * Candidates run as separate thread blocks (B * n_lengths of them), so scoring costs no latency while the GPU
 * has idle SMs, which is when speculation is on.  d_workspace: device memory of
 * war_draft_scored_workspace_bytes(params, n_lengths) bytes (0 for invalid arguments), 4-byte aligned, owned by the
 * caller, overwritten by every call.  Nothing is allocated; the call can be captured in a CUDA graph. */
size_t war_draft_scored_workspace_bytes(const war_draft_params_t* params, int32_t n_lengths);
war_status_t war_draft_scored(const war_index_t* ix, const int32_t* d_tail, const int32_t* d_tail_len,
                              const war_draft_params_t* params, int32_t n_lengths, void* d_workspace,
                              int32_t* d_match_len, int32_t* d_used_len, int32_t* d_num_nodes,
                              int32_t* d_ids, int32_t* d_parent, int32_t* d_count, war_stream_t stream);

/* Drafting from each request's own context (a part of the SuffixDecoding method that Section 3.3 adopts; the paper
 * does not spell it out): text a rollout has produced or read once tends to come back inside the same trajectory.
 * d_ctx holds the contexts of all requests back to back (int32 token ids), d_ctx_off [B+1] (int64, DEVICE memory)
 * their bounds: request b owns c = d_ctx[d_ctx_off[b] .. d_ctx_off[b+1]), L tokens, the last one being the root of
 * its tree.  No index is kept (a context changes every step): the call scans the contexts.
 *   match   the largest l <= min(P, tail_len[b], L - 1) such that the last l tokens of c also occur ending at an
 *           earlier position e <= L - 2 (so that at least one token follows the occurrence inside the context);
 *           occurrences may overlap each other and the tail.  A token < 0 matches nothing and nothing continues
 *           into it.
 *   window  of all occurrences of that suffix only the 32 most recent ones (largest e) are used.
 *   tree    the rules of war_draft with the window as the occurrence list: count = number of window occurrences
 *           followed by the slot's root path inside the context (count[0] = size of the window, at most 32); topk,
 *           min_match, spec_factor, min_prob and the switch (tail_len < 0, spec_batch_limit) act as in war_draft.
 * Outputs as in war_draft (d_count may be NULL).  A request without tokens gets the root alone with id -1.
 * Contexts of 2^31 tokens or more set WAR_ERR_INVALID_ARG in the device status and give num_nodes = 0. */
war_status_t war_draft_local(const int32_t* d_ctx, const int64_t* d_ctx_off, const int32_t* d_tail_len,
                             const war_draft_params_t* params,
                             int32_t* d_match_len, int32_t* d_num_nodes,
                             int32_t* d_ids, int32_t* d_parent, int32_t* d_count, war_stream_t stream);

/* Choice between two draft trees per request, e.g. the one from the stored trajectories (war_draft) and the one
 * from the request's own context (war_draft_local).  A tree's score is (sum of count[j], j = 1 .. num_nodes-1) /
 * count[0], the number of draft tokens one expects to be accepted under the tree's own statistics (0 when count[0]
 * is 0); scores are compared exactly (128-bit products).  Tree b is taken only if its score is strictly larger.
 * All arrays are device memory, [B] or [B, N] as in war_draft; the count arrays of both inputs are required.
 * d_source [B] receives 0 or 1; the chosen tree is copied to d_match_len, d_num_nodes, d_ids, d_parent and, if not
 * NULL, d_count.  The outputs must not alias the inputs. */
war_status_t war_draft_pick(int32_t B, int32_t N,
                            const int32_t* a_match_len, const int32_t* a_num_nodes, const int32_t* a_ids,
                            const int32_t* a_parent, const int32_t* a_count,
                            const int32_t* b_match_len, const int32_t* b_num_nodes, const int32_t* b_ids,
                            const int32_t* b_parent, const int32_t* b_count,
                            int32_t* d_source, int32_t* d_match_len, int32_t* d_num_nodes,
                            int32_t* d_ids, int32_t* d_parent, int32_t* d_count, war_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * Verification attention (paper Section 3.3: the target model then verifies the predicted tokens
 * in one forward pass; Sections 2.3 / 5.3: this needs auxiliary attention-mask / tree-mask handling).
 * For request b, slot j < num_nodes[b], query head h (kv head h / (Hq/Hkv)):
 *     visible = { 0 .. prefix_len[b]-1 }  U  { prefix_len[b] + a : a == j or a is an ancestor of j }
 *     out[b,j,h,:] = sum_c softmax_c(scale * <q[b,j,h,:], K[c,:]>) * V[c,:]      (c over visible)
 *     lse[b,j,h]   = natural-log sum of exp of the same logits
 * bf16 inputs, fp32 accumulation, bf16 out, fp32 lse.  The tree mask is derived from d_parent on the device.
 * KV layout: logical position p of request b is row p % page_size of physical page
 * d_page_table[b, p / page_size]; slot a's K/V are at logical position prefix_len[b] + a (the caller writes
 * them before the call).  Pools are bf16 [num_pages, Hkv, page_size, D]; k_strides / v_strides give the
 * element strides of (page, head, token, d).  Two memory layouts are accepted, the same one for both pools:
 * head-major (strides = {Hkv*page_size*D, page_size*D, D, 1}; one copy per page and head, the faster one) and
 * token-major (a page stored as [token][head][d]: strides = {page_size*Hkv*D, D, Hkv*D, 1}).
 * Further: page_size 8, 16, 32, 64 or 128, D == 128, Hq % Hkv == 0,
 * (Hq/Hkv) * N <= 512, scale > 0; anything else returns WAR_ERR_UNSUPPORTED / WAR_ERR_INVALID_ARG.
 * Rows j >= num_nodes[b] of d_out / d_lse are left untouched.
 * d_workspace: war_verify_attn_workspace_bytes(params) bytes of device memory, 256-byte aligned, private to
 * the call while it runs (split-KV partial results, their arrival counters and the work list live there); its
 * contents before the call do not matter.
 *   kernel: 0 = default: the tensor-core kernel; with up to 64 requests (the low-load regime the step exists for)
 *               the whole call is ONE kernel launch: every thread block works out its own share of the work from
 *               prefix_len / num_nodes, and a request that was split between blocks is merged by one of them once
 *               its last piece is there (in a fixed order: results do not depend on timing).  With more requests a
 *               planning launch precedes the kernel and a combine launch follows it.
 *           1 = plain CUDA-core kernel, 2 = tensor-core kernel always with the separate planning and combine
 *               launches; both kept for A/B checks (0 and 2 give the same bits).
 * Contexts (max_pages_per_req * page_size) must stay below 2^30 tokens.
 * ------------------------------------------------------------------------------------------------ */
typedef struct {
    int32_t B, N, Hq, Hkv, D, page_size, max_pages_per_req, kernel;
    int64_t num_pages;
    float scale;
    int32_t reserved;
    int64_t k_strides[4], v_strides[4];
} war_attn_params_t;
size_t war_verify_attn_workspace_bytes(const war_attn_params_t* params);
war_status_t war_verify_attn(const void* d_q, const void* d_kpool, const void* d_vpool,
                             const int32_t* d_page_table, const int32_t* d_prefix_len,
                             const int32_t* d_num_nodes, const int32_t* d_parent,
                             const war_attn_params_t* params, void* d_workspace,
                             void* d_out, float* d_lse, war_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * war_verify_attn for callers that cannot allocate device memory.  The paper has no counterpart: this is a
 * packaging variant of the call above, for users such as an engine whose memory pool is already frozen when the
 * decode loop runs, a plugin that only ever receives its input and output buffers, or a thread that must not
 * enter the CUDA allocator.  Same arguments and results as war_verify_attn, without d_workspace: the scratch
 * (work list, split-KV partials) lives in one fixed array inside the library image, WAR_VERIFY_ATTN_NOALLOC_MAX_BYTES
 * long, which every GPU that loads the library holds until the process exits.
 *   - The call allocates nothing and frees nothing (no cudaMalloc/cudaFree, no allocating library routine).
 *   - If war_verify_attn_workspace_bytes(params) exceeds WAR_VERIFY_ATTN_NOALLOC_MAX_BYTES the call returns
 *     WAR_ERR_CAPACITY and launches nothing.
 *   - The first call on each device looks up the array's device address (with that device current); make that
 *     first call before starting any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's contents (the caller clears
 *     nothing: a call rewrites what it reads, or recognises it as left over from an earlier call).  Two calls that
 *     overlap on the GPU, e.g. on two streams, race on it; run them in stream order.
 * ------------------------------------------------------------------------------------------------ */
#define WAR_VERIFY_ATTN_NOALLOC_MAX_BYTES (64u * 1024u * 1024u)
war_status_t war_verify_attn_noalloc(const void* d_q, const void* d_kpool, const void* d_vpool,
                                     const int32_t* d_page_table, const int32_t* d_prefix_len,
                                     const int32_t* d_num_nodes, const int32_t* d_parent,
                                     const war_attn_params_t* params, void* d_out, float* d_lse,
                                     war_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * Accept (paper Section 2.3: verifying drafts leaves the target model's output distribution unchanged;
 * Section 3.3: with accepted drafts a request advances by several tokens at once).  The caller
 * supplies the target model's own token choices; a draft slot is accepted iff every slot on its root path
 * equals the target's choice there.
 *   target_mode 0: d_target_ids[b, p] is the token the target emits AFTER slot p; slot j matches iff
 *                  ids[j] == target[parent[j]].  bonus = target[result slot].
 *   target_mode 1: slot j matches iff ids[j] == target[j].  bonus = -1.
 * Result slot = deepest slot whose whole root path matches (ties: lowest slot).  d_accept_len [B] = its depth,
 * d_accept_path [B, N] = the slots from the root's child down to it, padded with -1, d_bonus [B].
 * ------------------------------------------------------------------------------------------------ */
war_status_t war_accept(const int32_t* d_ids, const int32_t* d_parent, const int32_t* d_num_nodes,
                        const int32_t* d_target_ids, int32_t B, int32_t N, int32_t target_mode,
                        int32_t* d_accept_len, int32_t* d_accept_path, int32_t* d_bonus, war_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * Commit (completes the step of paper Section 3.3: with accepted drafts a request advances by several tokens
 * in one forward pass; the paper does not spell the bookkeeping out).  After war_accept, makes the
 * accepted path the end of each request's context, so that the next war_draft / war_verify_attn can run on the
 * same buffers:
 *   KV cache    the K/V rows of the accepted slots (logical positions prefix_len + slot) move to positions
 *               prefix_len + 1 .. prefix_len + accept_len, in path order, inside the paged pool; no page is
 *               allocated or freed and rows of rejected slots are left as they are (dead)
 *   context     context' = context ++ ids[path[0]] .. ids[path[accept_len-1]] ++ bonus (when bonus >= 0)
 *   d_tail      [B, P] in/out, right-aligned: the last min(P, length) tokens of context'; entries left of the
 *               window are set to 0.  d_tail_len [B] in/out.
 *   d_prefix_len[B] in/out: the last token of context' is the next root.  bonus >= 0: += accept_len + 1 (the new
 *               root's K/V does not exist yet); bonus < 0 (per-node targets): += accept_len (the last accepted
 *               token, or the old root, stays the root).
 * d_accept_path [B, N] as written by war_accept (slots strictly increasing).  Pools: bf16, D = 128, strides in
 * elements as in war_attn_params_t with unit stride along d and the others multiples of 8 (rows are moved 16
 * bytes at a time); both pools are modified in place.
 * A request that is not running (tail_len[b] < 0, see war_draft) is left untouched and is no error.
 * A request whose path is malformed or whose rows lie beyond max_pages_per_req is left untouched and
 * WAR_ERR_BAD_TREE is recorded in the device status word; a page id outside [0, num_pages) records
 * WAR_ERR_BAD_PAGE and the move of that row is skipped (its destination keeps what it held).  Enqueues two kernels on `stream`; does not synchronise.
 * ------------------------------------------------------------------------------------------------ */
typedef struct {
    int32_t B, N, P;                 /* requests, slots per tree, tail window */
    int32_t Hkv, D, page_size, max_pages_per_req, reserved;
    int64_t num_pages;
    int64_t k_strides[4], v_strides[4];   /* [page, head, token, d] in elements */
} war_commit_params_t;
war_status_t war_commit(const int32_t* d_ids, const int32_t* d_accept_len, const int32_t* d_accept_path,
                        const int32_t* d_bonus, void* d_kpool, void* d_vpool, const int32_t* d_page_table,
                        const war_commit_params_t* params, int32_t* d_prefix_len, int32_t* d_tail,
                        int32_t* d_tail_len, war_stream_t stream);

/* Diagnostic, no counterpart in the paper: exercises the bounded waits of the attention kernel without the kernel.
 * Every wait inside the tensor-core kernel (on a tile that has not arrived, on a result that is not ready) gives up
 * after a time budget, records WAR_ERR_TIMEOUT in the device status word and tells the other waiters of its thread
 * block to stop, so that a lost signal ends the call with an error instead of hanging the GPU.  This call launches
 * one small thread block in which one warp waits, with a budget of budget_us microseconds (1 .. 1 000 000), on a
 * barrier that nobody will ever complete, and a second warp waits on the same barrier with the kernel's ordinary
 * budget (2 s).  Expected afterwards: d_result [4] (int64, device) = { 0, 0, t0, t1 } -- both waits gave up, the
 * first after about budget_us (t0, t1 in nanoseconds), the second released by the first, not by its own budget --
 * and war_device_status reads WAR_ERR_TIMEOUT.  The kernel returns normally; later calls work as before. */
war_status_t war_selftest_bounded_wait(int32_t budget_us, int64_t* d_result, war_stream_t stream);

/* Reads and clears the sticky device status word (synchronises `stream`).  *h_status receives a
 * war_status_t value: WAR_OK, or the first device-side problem seen since the last read. */
war_status_t war_device_status(war_stream_t stream, int32_t* h_status);
const char* war_status_string(war_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* WAR_H_ */

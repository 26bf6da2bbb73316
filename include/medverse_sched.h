/* Frontier scheduler: the host side that stands before and after one decode step.
 *
 * It keeps, per request, the Petri net of Sec. 3.2 in the transition-level form the attention planner takes (node v
 * owns place p_v and, unless v is a root, transition t_v with pre-set {p_u : u parent of v} and post-set {p_v}), the
 * marking M_k, and the page table behind the KV references k of every token tau = (h, k).  Each decode step it emits
 * the mv_dag_batch that mv_plan_dag takes; after the step it advances every running transition by one token.
 *
 *   - Roots (no parents) are the places M_0 marks: their tokens are already in the KV pool when the request is added.
 *   - The frontier F_k is Eq. 1: every input place marked, output place empty.  All of F_k decode concurrently, one
 *     token per step each; the marking advances only when all of them are complete (Sec. 3.3, execution loop).
 *   - Fork: siblings read the same pages; only a reference count changes.  Join: the step reads the union of its
 *     predecessors' page lists; nothing is copied (Sec. 4.3, Phase II).
 *   - Pages are handed out lowest free id first.  A page's count is one for the node that owns it plus one per running
 *     transition that reads it; a request's pages return to the pool when nothing of it is running or enabled.
 *
 * All pointers are HOST pointers.  The arrays behind an emitted batch, and behind mv_sched_rows, belong to the
 * scheduler and stay valid until the next mv_sched_step after a commit, or mv_sched_destroy.  Not thread safe.
 */
#ifndef MEDVERSE_SCHED_H_
#define MEDVERSE_SCHED_H_

#include "medverse_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mv_sched mv_sched;

typedef struct {
  int64_t requests_live;       /* requests with something running                                   */
  int64_t transitions_fired;   /* reasoning steps started so far (each exactly once)                 */
  int64_t forks;               /* started steps that share a predecessor with a sibling of their frontier */
  int64_t joins;               /* started steps with two or more predecessors                        */
  int64_t markings_advanced;   /* barriers passed (M_k -> M_{k+1}), summed over requests             */
  int64_t decode_steps;        /* batches emitted                                                    */
  int64_t rows_emitted;        /* rows (new tokens) in those batches                                 */
  int64_t pages_in_use;
  int64_t pages_peak;
} mv_sched_stats;

/* A scheduler over a pool of `num_pages` pages of `page_size` (16) tokens.
 * Errors: MV_ERR_INVALID_ARG (null, page_size != 16, num_pages < 0). */
mv_status mv_sched_create(int32_t page_size, int32_t num_pages, mv_sched** sched);
void mv_sched_destroy(mv_sched* sched);

/* Adds a request (Sec. 4.3, Phase I -> II hand-over: the parsed plan becomes the net and M_0) and starts its first
 * frontier.  parent_off/parent_idx: CSR parent lists, every parent index smaller than its child's.  node_tokens[v]:
 * for a root, its tokens already written to the pool (>= 0; its pages are allocated here, in node order); for any
 * other node, the tokens the step will emit (>= 1; mv_sched_commit can end it earlier).  The arrays are copied.
 * Not allowed between mv_sched_step and its mv_sched_commit (the rows of an emitted step are fixed).
 * Errors: MV_ERR_INVALID_ARG, MV_ERR_NOT_TOPOLOGICAL, MV_ERR_PAGE_CAPACITY (pool exhausted; nothing is added). */
mv_status mv_sched_add_request(mv_sched* sched, int32_t n_nodes, const int32_t* parent_off, const int32_t* parent_idx,
                               const int32_t* node_tokens, int32_t* request_id);

/* The batch of the next decode step: every request with running transitions, its nodes restricted to what those
 * transitions read (renumbered in their original order), node_len = tokens in the pool, node_new = 1 on running
 * transitions, and a fresh page for every transition whose next token opens one.  *n_rows = new tokens of the step;
 * 0 (and batch->n_req = 0) when nothing is running.  vis_mode = MV_VIS_ANCESTORS, pos_mode = MV_POS_MAX_PARENT_END,
 * the scheduling hints are zero: the caller sets them on its copy.  Calling it twice without mv_sched_commit in
 * between returns the same step.
 * Errors: MV_ERR_INVALID_ARG, MV_ERR_PAGE_CAPACITY (pool exhausted: the step is not emitted, state unchanged). */
mv_status mv_sched_step(mv_sched* sched, mv_dag_batch* batch, int32_t* n_rows);

/* Which transition every row of the last emitted batch belongs to: request id and node id (as given to
 * mv_sched_add_request), *n_rows entries each. */
mv_status mv_sched_rows(const mv_sched* sched, const int32_t** request_ids, const int32_t** node_ids, int32_t* n_rows);

/* After the decode step: every running transition has written one token.  finished (may be null): one byte per row
 * of the emitted batch, non-zero = the engine saw the end of the step, whatever its stated length.  Transitions that
 * are complete release what they read; a request whose frontier is complete advances its marking and starts the
 * next frontier, or, with nothing enabled, returns all its pages.
 * Errors: MV_ERR_INVALID_ARG (no batch emitted since the last commit). */
mv_status mv_sched_commit(mv_sched* sched, const uint8_t* finished);

/* Reference counts of the given pages (0 = free).  Errors: MV_ERR_INVALID_ARG (a page id out of range). */
mv_status mv_sched_page_refs(const mv_sched* sched, const int32_t* page_ids, int32_t n, int32_t* refs);

mv_status mv_sched_get_stats(const mv_sched* sched, mv_sched_stats* stats);

#ifdef __cplusplus
}
#endif
#endif  /* MEDVERSE_SCHED_H_ */

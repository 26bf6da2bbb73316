/*
 * medverse_attn.h -- C ABI of the B200-native topology-aware (DAG) attention library.
 *
 * The library implements the attention of DAG-structured parallel decoding: every active
 * branch of a request's reasoning DAG (a Petri-net transition, Sec. 3.2) decodes at the same time
 * against one shared paged KV cache; a query token attends to the shared prefix, the nodes on its
 * own path and itself, never to a concurrently running sibling (Eq. 3), and its rotary position
 * continues from its fork or join point instead of the flattened sequence offset (Sec. 4.2,
 * "Adaptive Position Indices").
 *
 * Conventions for every call
 *   - extern "C", plain pointers and sizes.  "host" / "device" is stated per argument.
 *   - Ownership: the caller owns every device buffer (Q/K/V/O, page pools, workspace, the plan's
 *     device table buffer).  The library never allocates or frees device memory.  An mv_plan owns
 *     only host memory (its tables, kept in page-locked memory so that uploads are asynchronous).
 *   - Streams: `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     The three kernel calls and mv_plan_upload are asynchronous; they return the launch status only.
 *   - Errors: an mv_status is returned; argument errors are found on the host before any launch.
 *     Kernels never trap: every device-side wait is bounded; when one runs out the CTA issues nothing further, waits
 *     (again bounded) for its copies and products in flight, frees its tensor memory and returns, and
 *     mv_plan_read_status() then gives MV_ERR_TIMEOUT.  mv_status_string() names a status.
 *   - Layouts: q, k, v, q_rot, out are [tokens][heads][head_dim], row-major, element type
 *     mv_attn_geom.dtype.  The K and V page pools are separate buffers of the same element type, each
 *     [num_pages][n_kv_heads][head_dim / 64][page_size][64]: the block of one (page, KV head) is contiguous
 *     (4 KB for bf16, head_dim 128) and holds the head vectors of its 16 tokens split into 64-element column
 *     blocks, so that one bulk tensor copy with the 128-byte shared-memory swizzle moves the whole block.
 *     Element c of token t of (page p, head h) is at ((p * n_kv_heads + h) * (head_dim / 64) + c / 64) * 1024
 *     + t * 64 + c % 64.  Only mv_rope_write_kv writes the pools and only mv_dag_decode_attn reads them.
 *   - Order: "new tokens" (rows) are ordered (request, node index, token index) ascending.
 *   - Supported geometry: head_dim 64 or 128; n_q_heads a multiple of n_kv_heads; page_size 16.
 *     Anything else returns MV_ERR_UNSUPPORTED.  There is no CPU fallback.
 */
#ifndef MEDVERSE_ATTN_H_
#define MEDVERSE_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MV_OK = 0,
  MV_ERR_INVALID_ARG = 1,      /* null pointer, negative size, inconsistent offsets, bad enum          */
  MV_ERR_NOT_TOPOLOGICAL = 2,  /* a parent index is not smaller than its child's index (or a cycle)     */
  MV_ERR_PAGE_CAPACITY = 3,    /* a node's page list is too short for node_len + node_new tokens        */
  MV_ERR_UNSUPPORTED = 4,      /* head_dim / dtype / group size / batch shape the kernel does not take  */
  MV_ERR_WORKSPACE = 5,        /* workspace or table buffer missing, too small or misaligned            */
  MV_ERR_CUDA = 6,             /* a CUDA runtime call failed (launch error, copy error)                 */
  MV_ERR_TIMEOUT = 7           /* a bounded device-side wait ran out (read with mv_plan_read_status)    */
} mv_status;

/* Which nodes a token may attend to.  The paper states the mask twice, differently (Eq. 3 masks only
 * same-frontier siblings; Sec. 3.2 / 4.3 let a branch inherit the history of its own path only). */
typedef enum {
  MV_VIS_ANCESTORS = 0,  /* prefix + transitive ancestors + the node itself (Sec. 3.2, Sec. 4.3 Join) */
  MV_VIS_LAYERWISE = 1   /* Eq. 3 literally: every node of an earlier frontier layer + the node itself */
} mv_vis_mode;

/* Where a node's position indices start (Sec. 4.2). */
typedef enum {
  MV_POS_MAX_PARENT_END = 0,  /* right after the largest index used by any parent (fork alignment and
                                 the join rule, applied node by node)                                   */
  MV_POS_FRONTIER_ALIGNED = 1 /* one start for a whole frontier layer: the largest end of the previous
                                 layer (the sentence on fork alignment read literally)                  */
} mv_pos_mode;

typedef enum { MV_F32 = 0, MV_BF16 = 1 } mv_dtype;

/* A batch of request DAGs.  HOST memory, caller-owned, read only during mv_plan_dag.
 * A node is one reasoning step (one Petri-net transition); node 0 of a request is normally the shared
 * prefix (prompt + linear plan, Sec. 4.3 Phase I).  Node indices inside a request are local. */
typedef struct {
  int32_t n_req;
  const int32_t* node_off;   /* [n_req+1]   CSR over nodes                                             */
  const int32_t* node_len;   /* [n_nodes]   tokens of the node already in the KV pool                  */
  const int32_t* node_new;   /* [n_nodes]   tokens appended by this step (decode: 1 on frontier nodes,
                                            0 elsewhere; prefill: the node's length)                   */
  const int32_t* parent_off; /* [n_nodes+1] CSR over parent lists                                      */
  const int32_t* parent_idx; /* local parent indices, each < its child's local index                   */
  const int32_t* page_off;   /* [n_nodes+1] CSR over page lists                                        */
  const int32_t* page_idx;   /* physical page ids; a node's pages hold only that node's tokens; the
                                last page may be partial; ceil((len+new)/page_size) pages are required */
  int32_t page_size;         /* 16 */
  int32_t vis_mode;          /* mv_vis_mode */
  int32_t pos_mode;          /* mv_pos_mode */
} mv_dag_batch;

typedef struct {
  int32_t n_q_heads, n_kv_heads, head_dim, page_size;
  int64_t num_pages;   /* pages in each of the K and V pools (see "Layouts" above for the block layout) */
  int32_t dtype;       /* mv_dtype of q/k/v/out and of the pools */
  float sm_scale;      /* softmax scale; 0 means 1/sqrt(head_dim) */
  double rope_base;    /* theta_i = rope_base^(-2i/head_dim) */
} mv_attn_geom;

/* Optional tuning of the decode work lists (all zero = the defaults). */
typedef struct {
  int32_t chunk_tokens;      /* longest KV slice of one work unit in tokens (multiple of page_size);
                                0 = no limit (slices are cut only where a CTA's equal share of the step ends)  */
  int32_t sched_ctas;        /* shares the step's KV stream is cut into = half-CTAs the decode kernel runs with
                                (0 = 296, two per SM of a 148-SM part)                                         */
} mv_plan_tuning;

typedef struct mv_plan mv_plan;

/* Canonical integer tables of a plan (host memory, owned by the plan, valid until the plan is
 * re-planned or destroyed).  "q-node" = a node that receives new tokens in this step. */
typedef enum {
  MV_TAB_LAYER = 0,         /* int32 [n_nodes]      frontier layer: 0 for roots, else 1 + max over parents (Eq. 1) */
  MV_TAB_POS_START = 1,     /* int32 [n_nodes]      first position index of the node (Sec. 4.2)                 */
  MV_TAB_POS_ID = 2,        /* int32 [n_new_tokens] position index of every new token                           */
  MV_TAB_SLOT = 3,          /* int64 [n_new_tokens] pool slot = page_id * page_size + offset in page            */
  MV_TAB_QNODE = 4,         /* int32 [n_qnodes]     global node index of every q-node, ascending                 */
  MV_TAB_QNODE_TOK_OFF = 5, /* int32 [n_qnodes+1]   offsets of each q-node's new tokens                          */
  MV_TAB_SEG_OFF = 6,       /* int32 [n_qnodes+1]   CSR over the q-node's visible segments                       */
  MV_TAB_SEG_NODE = 7,      /* int32 [n_segs]       global node index of the segment (ascending in a q-node)     */
  MV_TAB_SEG_LEN = 8,       /* int32 [n_segs]       node_len + node_new of that node                             */
  MV_TAB_KV_LEN = 9,        /* int64 [n_qnodes]     tokens visible to the last new token of the q-node           */
  /* The decode kernels' work lists, as int32 words, for tests that replay them on the host (the layout is the
   * kernels' own and may change): */
  MV_TAB_WORK_STAGES = 10,        /* 16 words per stage: page[4], valid tokens (a byte per page slot), page slots
                                     in use, row mask low word [4], row mask high word [4], 2 unused              */
  MV_TAB_WORK_UNITS = 11,         /* 8 words per unit: first stage, stages, first item row, rows, KV head, 3 unused */
  MV_TAB_WORK_ITEM_ROWS = 12,     /* 2 words per (unit, row): row, first partial slot or -1                       */
  MV_TAB_WORK_CTA_UNIT_OFF = 13,  /* [n_ctas + 1] CSR over the units of every share                               */
  MV_TAB_WORK_ROWKV_PART_OFF = 14 /* [n_rows * n_kv_heads + 1] CSR over the partial slots of a (row, KV head)     */
} mv_plan_table_id;

typedef struct {
  int64_t n_nodes, n_new_tokens, n_qnodes, n_segs;
  int64_t decode_ready;        /* 1 if mv_dag_decode_attn applies: every node receives at most one token, or at
                                  most 256 each with no receiving node visible to another of its request        */
  int64_t prefill_ready;       /* 1 if no node holds older tokens (mv_dag_prefill_attn applies)            */
  int64_t n_items;             /* decode: work units = (KV slice of a node, KV head, row set)                */
  int64_t n_partials;          /* decode: split-KV partial results, each holding group_size head vectors    */
  int64_t chunk_tokens;        /* decode: the slice limit in effect, or a CTA's share in tokens if none    */
  int64_t unique_kv_tokens;    /* tokens of every node at least one row sees, each once                    */
  int64_t per_row_kv_tokens;   /* sum over rows of visible tokens                                          */
  int64_t n_q_tiles;           /* prefill: query tiles                                                      */
  int64_t visible_pairs;       /* prefill: allowed (query, key) pairs                                      */
  int64_t tile_pairs;          /* prefill: (query, key) pairs inside the KV ranges the kernel walks,
                                  rounded up to whole 128x64 tiles                                         */
  int64_t max_page_id;         /* largest page id referenced                                                */
  int64_t max_item_rows;       /* decode: largest row set of a work item                                    */
  int64_t sched_kv_heads, sched_group; /* head counts the decode work lists were cut for (0: no geometry yet) */
  int64_t n_ctas;              /* decode: CTAs the step was cut for                                         */
  int64_t max_cta_cost;        /* decode: largest share handed to one CTA, in tokens of one KV head (a unit
                                  counts as its tokens + 48)                                                */
  int64_t append_tiles;        /* node append: 128-row query tiles over the paged cache (0 when no node of a
                                  decode_ready batch receives several tokens)                               */
  int64_t max_node_new;        /* most new tokens any node receives                                         */
} mv_plan_stats;

enum { MV_OP_ROPE_WRITE_KV = 0, MV_OP_DECODE_ATTN = 1, MV_OP_PREFILL_ATTN = 2, MV_OP_PREFILL_ATTN_BWD = 3 };

/* DAG -> segment planner (Eq. 1 layering; Eq. 3 / Sec. 4.3 visibility; Sec. 4.2 positions; Sec. 3.2 KV index
 * lists).  Host only, integers only, deterministic.
 *   batch  host, read during the call only: the paper-level description of the step, nothing else.
 *   geom   host, optional.  The canonical tables, mv_rope_write_kv and the prefill calls need no geometry.  The decode
 *          kernels' work lists are cut for a head count (units are per KV head; a node's rows are grouped so that
 *          rows * group size <= 64), so only n_q_heads and n_kv_heads are read.  With geom == NULL the plan keeps a copy
 *          of the batch instead and mv_plan_bind_geometry cuts the lists later, for any supported geometry; until then
 *          mv_dag_decode_attn returns MV_ERR_UNSUPPORTED.
 *   tuning host, optional (NULL = defaults).
 *   plan   in/out: if *plan is NULL a new plan is created; otherwise the existing plan is re-planned in
 *          place and its host buffers are reused (no allocation once they are large enough).  The caller
 *          must not re-plan while an mv_plan_upload of the same plan is still in flight on a stream.
 * Errors: MV_ERR_INVALID_ARG, MV_ERR_NOT_TOPOLOGICAL, MV_ERR_PAGE_CAPACITY, MV_ERR_UNSUPPORTED (head counts).  On
 * error *plan is unchanged if it was NULL and left in an unusable-but-destroyable state otherwise. */
mv_status mv_plan_dag(const mv_dag_batch* batch, const mv_attn_geom* geom, const mv_plan_tuning* tuning, mv_plan** plan);

/* Cuts (or re-cuts) the decode work lists of a plan that was made without a geometry, for `geom`'s head counts.  The
 * plan's canonical tables do not change; its device tables do: upload it again before the next kernel call.
 * Errors: MV_ERR_INVALID_ARG, MV_ERR_UNSUPPORTED (the plan was made with a geometry and kept no copy of its batch). */
mv_status mv_plan_bind_geometry(mv_plan* plan, const mv_attn_geom* geom, const mv_plan_tuning* tuning);

/* Canonical table access for parity checks.  *host_ptr points into the plan; *count is in elements. */
mv_status mv_plan_table(const mv_plan* plan, int which, const void** host_ptr, int64_t* count);

mv_status mv_plan_get_stats(const mv_plan* plan, mv_plan_stats* stats);

/* Bytes of device memory the plan's kernel tables need (positions, slots, page ids, work lists). */
size_t mv_plan_device_bytes(const mv_plan* plan);

/* Asynchronous host->device copy of the plan's kernel tables into `device_buf` (device, caller-owned,
 * 256-byte aligned, at least mv_plan_device_bytes(plan) bytes).  The plan remembers device_buf; the
 * kernel calls below read the tables from there, so device_buf must stay valid and unmodified while
 * calls that use this plan are in flight.  Errors: MV_ERR_WORKSPACE, MV_ERR_CUDA. */
mv_status mv_plan_upload(mv_plan* plan, void* device_buf, size_t device_buf_bytes, void* cuda_stream);

void mv_plan_destroy(mv_plan* plan);

/* Workspace bytes (device, caller-owned, 256-byte aligned) an op needs for this plan and geometry.
 * MV_OP_DECODE_ATTN: split-KV partial outputs and softmax statistics.  MV_OP_PREFILL_ATTN: the optional per-(token,
 * query head) log-sum-exp, n_new_tokens * n_q_heads floats (the call also runs without a workspace).
 * MV_OP_PREFILL_ATTN_BWD: as many floats again.  MV_OP_ROPE_WRITE_KV needs none (0). */
size_t mv_workspace_bytes(const mv_plan* plan, const mv_attn_geom* geom, int op);

/* RoPE with adaptive positions fused into the KV-cache write (P(i) of Eq. 2 at the indices of Sec. 4.2).
 * For new token t (n = n_new_tokens of the plan):
 *   q_rot[t] = RoPE(q[t], pos_id[t]);  k_pages[slot[t]] = k_rot[t] = RoPE(k[t], pos_id[t]);  v_pages[slot[t]] = v[t].
 * RoPE pairs element i with i + head_dim/2; the angle pos * rope_base^(-2i/head_dim) and its reduction modulo
 * pi/2 are evaluated in double precision, cos / sin of the reduced angle in float (within two float ulps of the
 * double-precision values at any position); the rotation is float; results are stored in `dtype`.
 *   q       device [n][n_q_heads][head_dim]   raw queries, or NULL (then q_rot is not written)
 *   k, v    device [n][n_kv_heads][head_dim]  raw keys / values
 *   q_rot   device [n][n_q_heads][head_dim]   out (may alias q); NULL exactly when q is NULL
 *   k_rot   device [n][n_kv_heads][head_dim]  out, optional (NULL to skip; may alias k): the rotated keys in
 *           token order, which is what mv_dag_prefill_attn reads
 *   k_pages, v_pages  device pools, updated in place at the new tokens' slots; both NULL skips the cache
 *           write (then k_rot must be given)
 * Requires mv_plan_upload first.  Errors: MV_ERR_INVALID_ARG, MV_ERR_UNSUPPORTED, MV_ERR_WORKSPACE, MV_ERR_CUDA. */
mv_status mv_rope_write_kv(const mv_plan* plan, const mv_attn_geom* geom, const void* q, const void* k,
                           const void* v, void* q_rot, void* k_rot, void* k_pages, void* v_pages,
                           void* cuda_stream);

/* Multi-branch decode attention (Eq. 2 with the DAG mask of Eq. 3 over a shared paged cache, Sec. 4.3
 * Fork / Join): for every row r (the single new token of a frontier node v) and query head h,
 *   out[r][h] = sum_j softmax_j(sm_scale * <q_rot[r][h], K_j>) V_j
 * over all tokens j of the nodes visible to v, the row's own just-written token included, so
 * mv_rope_write_kv must precede this call in stream order.  Pages shared by several rows of a request
 * (prefix, common ancestors) are read once per KV head and serve all those rows and the whole GQA group.
 * Node append (what follows a Join or the Phase I -> II hand-over of Sec. 4.3, where more than one token is
 * written to a node at once): a node may receive up to 256 new tokens, one row each in (node, token) order; new
 * token j of v then sees v's tokens 0 .. node_len(v) + j and every other visible node in full.  In a request
 * where some node receives several tokens, the nodes that receive tokens must not see one another, else the
 * plan is not decode_ready.  With head_dim 128, an even group size, 16-byte aligned q_rot and out, and some
 * node receiving at least 40 tokens, the step runs as 128-row query tiles over the paged cache (a node's
 * history is then read once per 128 new tokens); the workspace is still required but left untouched.
 *   q_rot   device [n_rows][n_q_heads][head_dim]  bf16
 *   k_pages, v_pages  device pools, bf16
 *   out     device [n_rows][n_q_heads][head_dim]  bf16
 *   workspace device, mv_workspace_bytes(plan, geom, MV_OP_DECODE_ATTN) bytes; contents are scratch
 * dtype must be MV_BF16 and the plan decode_ready, else MV_ERR_UNSUPPORTED. */
mv_status mv_dag_decode_attn(const mv_plan* plan, const mv_attn_geom* geom, const void* q_rot,
                             const void* k_pages, const void* v_pages, void* out, void* workspace,
                             size_t workspace_bytes, void* cuda_stream);

/* FP8 KV cache variant of the decode step (no counterpart in the paper: a storage format that halves the bytes a decode
 * step streams).  The pools hold 8-bit floats with 4 exponent and 3 mantissa bits (largest finite value 448, no
 * infinities), one scale per KV head: value = stored * scale[head].  kv_scale is a DEVICE array of 2 * n_kv_heads floats:
 * the K scales of all heads, then the V scales (positive; chosen by the caller, e.g. from calibration).
 * Pool layout: [num_pages][n_kv_heads][page_size][head_dim] bytes, K and V separate: the block of one (page, KV head) is
 * 2 KB, contiguous, one token per 128-byte row.
 *
 * mv_rope_write_kv_fp8 is mv_rope_write_kv writing such pools: k_pages8[slot[t]] = round(RoPE(k[t], pos_id[t]) / K scale),
 * v_pages8[slot[t]] = round(v[t] / V scale), rounding to nearest even and saturating at +-448; q_rot as before (bf16).
 * mv_dag_decode_attn_fp8 is mv_dag_decode_attn reading them: same plan, same work lists, same workspace, same result up
 * to the format's rounding.  Inside the kernel the queries and the softmax weights are 8-bit floats as well (one scale
 * per q-vector; each as a rounded value plus a rounded remainder, about seven bits of mantissa), so that both products
 * run on the tensor cores' 8-bit path straight on the pool bytes.
 * MV_BF16 queries and outputs, head_dim 128, single-token steps only (max one new token per node); anything else is
 * MV_ERR_UNSUPPORTED.  Other errors as for mv_rope_write_kv and mv_dag_decode_attn. */
mv_status mv_rope_write_kv_fp8(const mv_plan* plan, const mv_attn_geom* geom, const void* q, const void* k, const void* v,
                               void* q_rot, void* k_pages8, void* v_pages8, const float* kv_scale, void* cuda_stream);
mv_status mv_dag_decode_attn_fp8(const mv_plan* plan, const mv_attn_geom* geom, const void* q_rot, const void* k_pages8,
                                 const void* v_pages8, const float* kv_scale, void* out, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream);

/* Decode attention for callers that cannot allocate device memory.  (The paper has no counterpart: this is
 * a packaging variant of mv_dag_decode_attn, same arithmetic, same kernels.)
 *
 * Some hosts of this library may not call cudaMalloc or an allocating library routine on the decode path:
 * a serving loop whose memory pool is fixed at start-up and fully handed out, a plug-in that runs inside
 * another runtime's allocator-free region, or code that must not synchronise the device (cudaMalloc and
 * cudaFree do).  For them the split-KV scratch that mv_dag_decode_attn takes as `workspace` is replaced by
 * a fixed array of MV_STATIC_WORKSPACE_BYTES bytes that is part of the library image: every GPU on which
 * the library is loaded holds that much memory until the process exits.  The caller still passes q_rot,
 * the pools and out, exactly as for mv_dag_decode_attn; nothing is allocated or freed by this call.
 *
 *   - Limit: plans with mv_workspace_bytes(plan, geom, MV_OP_DECODE_ATTN) > MV_STATIC_WORKSPACE_BYTES are
 *     refused with MV_ERR_WORKSPACE before anything is launched (query it with mv_static_workspace_bytes()).
 *   - Set-up: the first call on each device looks up the array's device address (one cudaGetSymbolAddress,
 *     with the calling thread's current device).  That first call is a set-up call: with lazy module loading it is
 *     also the moment the driver brings the array into being on that device (and may synchronise).  Make it at
 *     start-up, outside any stream capture and outside the region in which nothing may be allocated; every later
 *     call on that device allocates and frees nothing.
 *   - Sharing: every call on a device uses the same array and finds the previous call's contents in it.
 *     The kernels write each partial result before they read it, so nothing needs clearing; but two calls
 *     whose kernels overlap on the GPU (different streams, no ordering between them) race on it.  Order such
 *     calls, or give all but one of them their own workspace through mv_dag_decode_attn.
 * Other errors are those of mv_dag_decode_attn. */
#define MV_STATIC_WORKSPACE_BYTES (16u << 20)
size_t mv_static_workspace_bytes(void);
mv_status mv_dag_decode_attn_static(const mv_plan* plan, const mv_attn_geom* geom, const void* q_rot,
                                    const void* k_pages, const void* v_pages, void* out, void* cuda_stream);

/* Topology-masked prefill attention over a flattened DAG sequence (Eq. 3; the training-time layout of
 * Sec. 4.2 and the engine's re-prefill): all tokens of the batch are new and contiguous in
 * (request, node, token) order;
 *   out[i][h] = sum_j softmax_j(sm_scale * <q_rot[i][h], k_rot[j]> + M_ij) v[j],
 * M_ij = 0 iff token j belongs to a node visible to node(i) and, inside node(i) itself, j <= i.
 * Key/value ranges no query of a tile may see are never visited (tile skipping).
 *   q_rot  device [T][n_q_heads][head_dim]   position-embedded queries
 *   k_rot  device [T][n_kv_heads][head_dim]  position-embedded keys
 *   v      device [T][n_kv_heads][head_dim]
 *   out    device [T][n_q_heads][head_dim]
 * dtype MV_F32 runs a float32 SIMT kernel, MV_BF16 the tensor-core kernel (float32 accumulation).
 * The plan must be prefill_ready, else MV_ERR_UNSUPPORTED.
 *   workspace  NULL, or device, 16-byte aligned, mv_workspace_bytes(plan, geom, MV_OP_PREFILL_ATTN) bytes: receives
 *              lse[i][h] = log2 sum_j 2^(sm_scale * log2(e) * <q_i, k_j> + M_ij) as float [T][n_q_heads], which
 *              mv_dag_prefill_attn_bwd takes.  Only the tcgen05 kernel (MV_BF16, head_dim 128, even group size,
 *              16-byte aligned tensors) writes it; with any other shape a non-NULL workspace is MV_ERR_UNSUPPORTED. */
mv_status mv_dag_prefill_attn(const mv_plan* plan, const mv_attn_geom* geom, const void* q_rot,
                              const void* k_rot, const void* v, void* out, void* workspace,
                              size_t workspace_bytes, void* cuda_stream);

/* Backward of mv_dag_prefill_attn: the attention the model is fine-tuned through (Sec. 5.1) is Eq. 2 with the mask of
 * Eq. 3 over the flattened training sequence at the position indices of Sec. 4.2.  Given dout = d loss / d out, with
 * P_ij = softmax_j(sm_scale * <q_i, k_j> + M_ij) per query head and delta_i = <dout_i, out_i>:
 *   dv[j]     = sum_i P_ij dout[i]                                    (summed over the query heads of j's KV head)
 *   dS_ij     = P_ij * (<dout[i], v[j]> - delta_i)
 *   dq_rot[i] = sm_scale * sum_j dS_ij k_rot[j],   dk_rot[j] = sm_scale * sum_i dS_ij q_rot[i]   (summed over the group)
 * The gradients are with respect to the position-embedded q_rot and k_rot (the rotation of mv_rope_write_kv is a fixed
 * orthogonal map per token).  Masked pairs contribute nothing; key tiles walk the transposed visibility (which query
 * runs see this key's node), so ranges no query can see are never visited.
 *   q_rot, k_rot, v, out   device, as given to / written by mv_dag_prefill_attn (bf16)
 *   dout      device [T][n_q_heads][head_dim] bf16
 *   lse       device [T][n_q_heads] float, as written by mv_dag_prefill_attn into its workspace
 *   dq_rot    device [T][n_q_heads][head_dim] bf16, out;  dk_rot, dv  device [T][n_kv_heads][head_dim] bf16, out
 *   workspace device, 256-byte aligned, mv_workspace_bytes(plan, geom, MV_OP_PREFILL_ATTN_BWD) bytes (scratch)
 * All tensors 16-byte aligned.  MV_BF16, head_dim 128 and an even group size only (MV_ERR_UNSUPPORTED otherwise); the plan
 * must be prefill_ready.  Deterministic (no atomics).  Errors: MV_ERR_INVALID_ARG, MV_ERR_UNSUPPORTED, MV_ERR_WORKSPACE,
 * MV_ERR_CUDA. */
mv_status mv_dag_prefill_attn_bwd(const mv_plan* plan, const mv_attn_geom* geom, const void* q_rot, const void* k_rot,
                                  const void* v, const void* out, const void* dout, const void* lse, void* dq_rot,
                                  void* dk_rot, void* dv, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* One decode step with HOST inputs and outputs (the end-to-end form of the path: Sec. 4.3 Phase II, one
 * frontier step).  Copies q, k, v (host, preferably page-locked, [n_rows][heads][head_dim]) to the device
 * staging buffer, uploads the plan, runs mv_rope_write_kv and mv_dag_decode_attn on `cuda_stream`, copies
 * `out` back to host memory and returns after enqueueing everything (asynchronous; synchronise the stream
 * before reading out_host).
 *   staging  device, caller-owned, mv_decode_step_staging_bytes(plan, geom) bytes, 256-byte aligned; holds
 *            the plan tables, q/k/v/out device copies and the decode workspace
 *   k_pages, v_pages  device pools (the resident KV cache) */
size_t mv_decode_step_staging_bytes(const mv_plan* plan, const mv_attn_geom* geom);
mv_status mv_decode_step_host(mv_plan* plan, const mv_attn_geom* geom, const void* q_host, const void* k_host,
                              const void* v_host, void* out_host, void* k_pages, void* v_pages, void* staging,
                              size_t staging_bytes, void* cuda_stream);

/* The same step starting from the batch description instead of a finished plan: the copies of q, k, v are
 * enqueued first and travel while the host plans the step (mv_plan_dag into *plan, which is created when NULL
 * and reused otherwise), then the step runs as in mv_decode_step_host.  The staging layout depends on the plan
 * only behind the q / k / v / out copies; size the buffer with mv_decode_step_staging_bytes on a plan of a batch
 * of the same shape (a too small buffer is refused with MV_ERR_WORKSPACE, possibly after the input copies were
 * enqueued).  *plan must not have an upload in flight (synchronise the stream between steps that share a plan).
 * Errors: those of mv_plan_dag and of mv_decode_step_host. */
mv_status mv_decode_step_host_batch(const mv_dag_batch* batch, mv_plan** plan, const mv_attn_geom* geom,
                                    const void* q_host, const void* k_host, const void* v_host, void* out_host,
                                    void* k_pages, void* v_pages, void* staging, size_t staging_bytes,
                                    void* cuda_stream);

/* The same step cut into slices that overlap (Sec. 4.3: the requests of a batch advance independently of one
 * another, so a batch may be cut between requests).  The batch is split into n_slices runs of consecutive requests with
 * about equal numbers of new tokens; every slice is planned on its own (plans[i], created when NULL, reused
 * otherwise) and runs as mv_decode_step_host_batch does, on one of two streams that the library keeps per device
 * (created by the first call on that device, with two event pairs, and kept until the process exits): slice i + 1's
 * inputs travel while slice i computes, and slice i's output travels while slice i + 1 computes.  The work starts
 * behind everything already enqueued on `cuda_stream`, and `cuda_stream` continues behind all of it: synchronise
 * `cuda_stream` before reading out_host, as with the other forms.  Rows of q, k, v, out are those of the whole batch
 * (a slice's rows are consecutive).  Results are those of the unsliced call up to the rounding order of the split-KV
 * merge (a slice's key ranges are cut for its own share of the step).
 *   plans    host array of n_slices plan pointers (in/out); none may have an upload in flight
 *   n_slices 1 .. min(8, batch->n_req)
 *   staging  device, 256-byte aligned; mv_decode_step_pipelined_staging_bytes(plans, n_slices, geom) bytes after
 *            mv_decode_step_pipelined_plan on a batch of the same shape (0 if a plan is missing or invalid)
 * The library's two streams and their events are shared by every call on a device: host threads must not run this
 * call on the same device at the same time.
 * mv_decode_step_pipelined_plan plans the slices only (host work; for sizing the staging buffer).
 * Errors: MV_ERR_INVALID_ARG (n_slices out of range, a slice without a request, null pointers), MV_ERR_WORKSPACE,
 * MV_ERR_CUDA, and those of mv_plan_dag; after an error, work of earlier slices may already be enqueued. */
mv_status mv_decode_step_pipelined_plan(const mv_dag_batch* batch, mv_plan** plans, int32_t n_slices,
                                        const mv_attn_geom* geom);
size_t mv_decode_step_pipelined_staging_bytes(mv_plan* const* plans, int32_t n_slices, const mv_attn_geom* geom);
mv_status mv_decode_step_host_pipelined(const mv_dag_batch* batch, mv_plan** plans, int32_t n_slices,
                                        const mv_attn_geom* geom, const void* q_host, const void* k_host,
                                        const void* v_host, void* out_host, void* k_pages, void* v_pages,
                                        void* staging, size_t staging_bytes, void* cuda_stream);

/* Reads the device-side status word of the kernels that last ran with this plan's uploaded tables: MV_OK, or
 * MV_ERR_TIMEOUT if a bounded wait inside a kernel ran out (the kernel then still terminated, with an
 * undefined result).  Copies 4 bytes device->host on `cuda_stream` and synchronises that stream.
 *   status  host, out */
mv_status mv_plan_read_status(const mv_plan* plan, void* cuda_stream, int32_t* status);

const char* mv_status_string(mv_status s);

/* Number of kernel launches the library has issued in this process since load (diagnostic counter). */
int64_t mv_launch_count(void);

/* Self-tests (diagnostics; no counterpart in the paper, nothing of the attention path runs).
 *
 * mv_selftest_bounded_wait: every wait inside the kernels is bounded and reports through the plan's status word
 * (mv_plan_read_status).  This call exercises that mechanism alone: one thread of a one-CTA kernel waits, with the
 * same bounded wait and a limit of `limit_ns` nanoseconds (1 .. 100 000 000), on a barrier that nothing ever
 * completes; when the limit has passed it records MV_ERR_TIMEOUT in the status word of `plan` (which must have been
 * uploaded) and returns.  No copy or product is in flight, the context stays usable; upload the plan again to clear
 * the word.  Asynchronous on `cuda_stream`.  Errors: MV_ERR_INVALID_ARG, MV_ERR_WORKSPACE, MV_ERR_CUDA.
 *
 * mv_selftest_tmap_cache: the launchers keep the tensor maps of recent calls in a small cache keyed by (device index,
 * up to three base pointers, row count, one more word).  This call runs the same lookup on a private instance with
 * four entries: returns 1 if the key is cached, else 0 after caching it (the oldest entry is replaced); reset != 0
 * empties the instance first.  Host only. */
mv_status mv_selftest_bounded_wait(const mv_plan* plan, uint64_t limit_ns, void* cuda_stream);
int32_t mv_selftest_tmap_cache(int32_t device, const void* a, const void* b, const void* c, int64_t rows, int64_t aux,
                               int32_t reset);

#ifdef __cplusplus
}
#endif
#endif /* MEDVERSE_ATTN_H_ */

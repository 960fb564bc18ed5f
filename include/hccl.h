/*
 * hccl.h - C ABI of the B200 collective executor.
 *
 * The library follows the paper's "compiled communication" model (Sec. I,
 * Sec. III-B.2): the host compiles a collective into a complete description
 * (a work packet made of subgraphs of work-queue elements, WQEs, with their
 * dependencies) and a small, fixed set of execution units runs it on their
 * own. Here the execution units are the thread blocks of one persistent
 * sm_100a kernel launched on a caller-chosen number of SMs (the analogue of the
 * message engines, Sec. II-A.2), and the per-WQE work is what the near-memory
 * compute unit does: copies and FP32-internal sums on FP32/BF16/FP16 buffers.
 *
 * All ranks are virtual: R send buffers and R receive buffers live in the
 * memory of ONE GPU. There is no network, no second GPU.
 *
 * Conventions
 *  - Every call returns hccl_status_t; out-parameters are written only on
 *    HCCL_OK. No exceptions cross this boundary.
 *  - Pointers named host_* / plain arrays of counts are HOST memory. Pointers
 *    named dev_*, the entries of sendbufs/recvbufs and the workspace are DEVICE
 *    memory owned by the caller. The library allocates no device memory and
 *    creates no streams.
 *  - A plan owns its host tables. hccl_plan_destroy frees them; it never
 *    touches device memory.
 *  - hccl_execute is asynchronous on the given stream. A plan must not be in
 *    flight twice at once. Device-side failures (timeout, malformed table) never
 *    trap: they are recorded in the workspace and read back with
 *    hccl_plan_status after the stream has been synchronised. After a
 *    device-side failure the plan must be bound again before reuse.
 *  - Only sum reductions exist (Sec. II-A.2). Element types: FP32, BF16, FP16.
 *  - A plan or graph handle is not thread-safe: use one handle from one host thread at a time. Different
 *    handles may be used from different threads.
 */
#ifndef HCCL_B200_H
#define HCCL_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HCCL_MAX_RANKS 256 /* the paper's largest job is 256 ranks (Sec. V-A) */

typedef enum {
    HCCL_OK = 0,
    HCCL_ERR_INVALID_ARG = 1,
    HCCL_ERR_DTYPE = 2,
    HCCL_ERR_COUNT_MISMATCH = 3, /* recvcounts[d][s] != sendcounts[s][d], or shard sizes do not add up */
    HCCL_ERR_OVERLAP = 4,        /* receive ranges of one rank overlap, or a send buffer aliases a receive buffer */
    HCCL_ERR_ALIGNMENT = 5,      /* a buffer is not aligned to its element size / workspace not 256-B aligned */
    HCCL_ERR_WORKSPACE = 6,      /* workspace too small */
    HCCL_ERR_BUSY = 7,
    HCCL_ERR_CUDA = 8,           /* a CUDA runtime call failed; see hccl_last_cuda_error() */
    HCCL_ERR_TIMEOUT = 9,        /* device side: a dependency or WAIT did not come true within timeout_ns */
    HCCL_ERR_BAD_DESCRIPTOR = 10,/* device side: a table entry failed its checks */
    HCCL_ERR_NOT_BOUND = 11,     /* execute before bind */
    HCCL_ERR_HAZARD = 12         /* compile-time check: two conflicting WQEs are not ordered by a dependency */
} hccl_status_t;

typedef enum { HCCL_FP32 = 0, HCCL_BF16 = 1, HCCL_FP16 = 2 } hccl_dtype_t; /* the NMC's three types, Sec. II-A.2 */

typedef enum {
    HCCL_ALGO_RING = 0,      /* unidirectional ring, reduce-scatter then all-gather (Sec. III-B.2, Fig. 5) */
    HCCL_ALGO_ONESHOT = 1,   /* "all-to-all style": every rank reads every peer once (Sec. V-F, PE kernels) */
    HCCL_ALGO_RING_FUSED = 2,/* the ring's sums in the ring's order, but each chunk's chain collapsed into
                                one multi-input reduction (cf. NOOP-joined tree reductions, Sec. III-B.2).
                                Reported as its own algorithm, never as "ring". */
    HCCL_ALGO_RING_2LEVEL = 3,/* topology-aware two-level ring (Sec. V-D): ranks form racks of opts.rack_size; sums
                                run round each rack's ring first, then round the ring of racks, and results
                                are gathered across racks first, then inside each rack, so that only 1/rack_size
                                of the data ever crosses between racks. AllReduce and AllGather. */
    HCCL_ALGO_FANOUT = 4,    /* one-shot with the destinations fused: each piece of the result is produced once
                                (AllReduce: one sum over all ranks in rank order 0..R-1, the one-shot's order;
                                AllGather: one read of the chunk) and written into all R receive buffers by the
                                same work item. Possible only because the virtual ranks share one memory; not in
                                the paper. Reported as its own algorithm, never as "one-shot". */
    HCCL_ALGO_TREE = 5,      /* AllReduce by a binary tree of two-input sums (tree-based NMC reduction, Sec.
                                III-B.2): per granule of opts.chunk_bytes, neighbours in rank order are added in
                                pairs level by level (an odd one out moves up unchanged), FP32 partials in scratch,
                                one rounding at the root into rank 0's buffer, then a binomial tree of copies to
                                every rank. Dependency depth 2*ceil(log2 R). */
    HCCL_ALGO_AUTO = 6       /* AllReduce only: the planner picks between the paper's two forms by size (the
                                algorithm, and with it the cost of generating the packet, changes with the size,
                                Sec. V-B): ONESHOT while R times the bytes per rank is at most 32 MiB (every rank
                                reads R buffers: the work grows with R squared), RING beyond. */
} hccl_algo_t;

/* Which data mover the executor uses for aligned bulk work. AUTO: the planner decides: the bulk engine for
 * copies that do not wait on one another (AllToAllv, one-shot and fan-out AllGather) and for reductions with
 * 256 MiB of input or more; the register engine for hop-by-hop copies, smaller reductions and all
 * multi-input sums. Graphs compiled directly (hccl_graph_compile) default to the register engine. */
typedef enum {
    HCCL_ENGINE_AUTO = 0,
    HCCL_ENGINE_LSU = 1,  /* 128-bit vector loads/stores through registers */
    HCCL_ENGINE_BULK = 2  /* cp.async.bulk (TMA) global->shared->global with mbarrier pipelining; with static chains
                             (ring reductions) the forwarding kernel, see HCCL_FLAG_STATIC_CHAINS */
} hccl_engine_t;

/* Ticket order of a reduction plan. */
#define HCCL_FLAG_LEVEL_MAJOR 1u /* all chains' step t before any chain's step t+1 (max parallelism);
                                    default is chain-group-major so partials stay in L2 */
#define HCCL_FLAG_CHECK_HAZARDS 2u /* run the host hazard checker at compile time, fail with HCCL_ERR_HAZARD */
#define HCCL_FLAG_STAGED_RING 4u /* keep the paper's separate transfer and compute WQEs: COPY the peer's
                                    partial into this rank's staging slot, then REDUCE (A=A+B). Default fuses
                                    the pair into one REDUCE that reads the peer's buffer directly. */

#define HCCL_FLAG_BIDIRECTIONAL 8u /* flat ring AllReduce / ReduceScatter: granules of a chunk alternate direction, even
                                     ones travel r -> r+1, odd ones r -> r-1 (a bidirectional ring, Sec. III-B.2) */

#define HCCL_FLAG_STATIC_CHAINS 16u /* if every dependency of the packet is a tile-by-tile link (HCCL_DEP_ELEMENTWISE
                                      between WQEs cut into the same number of tiles) and the groups of WQEs linked
                                      that way are equally long (the chains of a small ring; the copies of one
                                      chunk in a hop-by-hop AllGather; a granule's tree of sums), run tile k of a
                                      whole group inside ONE block, in issue order: a barrier of that block then
                                      stands where a device counter and a poll across SMs would. Ignored when the
                                      packet has another shape. On the bulk engine only packets of simple chains
                                      (one predecessor, one successor) of REDUCE items, optionally followed by
                                      plain copies, or of copies of one send-buffer range, run this way, in the forwarding kernel: a block walks a piece of
                                      14336 elements through all steps of its chain with the running FP32 sums in
                                      registers; every step's result is stored where its descriptor says, none is
                                      read back. The planners ask for it themselves where it pays (rings with about
                                      a chain of tiles per SM or more, each chain with a scratch slot of its own). */
#define HCCL_FLAG_DYNAMIC_TICKETS 32u /* keep the planners from asking for HCCL_FLAG_STATIC_CHAINS */
#define HCCL_FLAG_DEVICE_TABLES 64u /* hccl_plan_alltoallv_dynamic: build descriptors and tiles on the device and run
                                      them on the ordinary executor (always so beyond 64 ranks) */

/* Options. A zero field means "default". */
typedef struct {
    int32_t sm_budget;      /* thread blocks of the persistent executor = "message engines" (default 148). An upper
                               bound: a plan never launches more blocks than it has work items or static chains,
                               and a ring planner left to the default may launch exactly one block per tile of a
                               ring step. hccl_plan_info reports the number used. */
    int32_t engine;         /* hccl_engine_t */
    uint64_t chunk_bytes;   /* ring pipelining granule inside a shard/chunk, in bytes of the data type (default 2 MiB) */
    uint64_t tile_bytes;    /* work-item size, bytes of the widest operand (default: chosen from size and sm_budget) */
    uint64_t timeout_ns;    /* bound on every device-side wait (default 2e9) */
    uint32_t flags;         /* HCCL_FLAG_* */
    int32_t chain_group;    /* chains scheduled together in chain-group-major order; FP32 scratch slots are recycled
                               every two groups. Default: all chains together (a slot per chain, no recycling) while
                               the FP32 partials take at most 32 MiB (AllReduce rings: 48 MiB), else as many as keep one
                               group-step's partials at 64 MiB, half the L2 (16 for 2 MiB granules of 16-bit data) */
    int32_t threads;        /* threads per block, multiple of 32. Register engine: one control warp + workers (default 512,
                               at least 64). Bulk engine: DMA, control and publishing warps + compute warps (default 352, at least 128);
                               its forwarding kernel (static chains) always runs 256 threads and its own stages */
    int32_t stages;         /* bulk engine: shared-memory stages per block, 2..8 (default: 4 of 48 KiB; copy-only plans on 100 blocks
                               or more: 3, since the memory is then the limit and fewer bytes in flight per block serve it better) */
    int32_t cluster;        /* register engine: launch blocks in clusters of this size (2, 4, 8) so that they sit on
                               neighbouring SMs; 0/1 = no clusters. Ignored unless it divides the block count. */
    int32_t light;          /* register engine: nonzero = the 64-register build (several blocks per SM). With 64-128 threads such a
                               block is small enough to be placed on an SM that a large compute kernel's block already occupies:
                               12 of them moved 230-240 GB/s beside a saturating bf16 GEMM for 1.9-4.6 % of its rate (16: 300 GB/s for 2.8-5.6 %), where two
                               full-size blocks (two SMs held) cost it 6 % */
    int32_t copy_by_warps;  /* bulk engine: who stores COPY stages. 1 = the compute warps (a stage is free as soon as it is read;
                               best per-block rate), 2 = the bulk unit, 0 = compute warps below 100 blocks, bulk unit otherwise */
    int32_t rack_size;      /* ranks per rack for HCCL_ALGO_RING_2LEVEL and for cross-rack byte accounting (default 16,
                               the paper's rack, Sec. V-D) */
    int32_t stage_kib;      /* bulk engine: KiB per shared-memory stage, 12 to 96 (default 48; multiples of 12 split evenly for every operand mix); with
                               opts.stages left at 0 the number of stages keeps 192 KiB in flight (at most 8 stages) */
    int32_t quantum;        /* 0: persistent blocks (sm_budget of them run until the packet is done). > 0: short-lived blocks,
                               each leaves after this many work items and as many blocks are launched as that takes; how many
                               run at once is then the block scheduler's choice. On a stream of lower priority than a
                               concurrent compute kernel's they fill the SMs that kernel leaves idle (the tail of its last
                               wave, the gap between launches) and hold none against it. Ticket dispatch only: ignored by
                               plans that run as static chains and by device-resident plans; refused by hccl_server_start */
} hccl_opts_t;

/* Fills *o with the options measured to let a collective run beside a saturating compute kernel for less than 5 % of
 * that kernel's rate (the overlap experiment of Sec. V-E; 8192^3 bf16 GEMM, AllToAllv of config 4: 1.9-4.6 % at
 * 230-240 GB/s over a dozen runs): 12 persistent blocks of the register engine's 64-register build with 128 threads each, which are small
 * enough to share an SM with a block of the compute kernel and so hold no SM against it. Every other field is zeroed
 * (defaults). The library's general defaults aim at a GPU of its own instead: one full-size block per SM. */
void hccl_opts_for_overlap(hccl_opts_t* o);

typedef struct hccl_plan hccl_plan_t;   /* opaque, host-owned: a compiled, cacheable work packet (Sec. V-B) */
typedef struct hccl_graph hccl_graph_t; /* opaque, host-owned: a work packet under construction */

/* ------------------------------------------------------------------------
 * Collective planners (Sec. III-B.2 "Data Path"; collectives named in Sec. V-A, V-D).
 * Each validates its arguments, builds the WQE graph of the chosen schedule and
 * compiles it. Counts are int64. Nothing here touches the GPU.
 * ------------------------------------------------------------------------ */

/* AllReduce(sum): every rank r ends with Y_r[i] = round(sum_q X_q[i]), i < count.
 * RING: chunk c = elements [floor(c*count/R), floor((c+1)*count/R)); reduce-scatter step t has rank
 * (c+t+2) mod R add its own chunk c to its predecessor's partial, so chunk c is summed as
 * ((X_{c+1}+X_{c+2})+...)+X_c in FP32 and ends on rank c; all-gather step u copies it to rank c+u+1.
 * FP32 data keeps partials in the receive buffers; 16-bit data keeps FP32 partials in workspace
 * scratch and is rounded once, on the last reduce step. ONESHOT: R independent R-input sums in rank
 * order 0..R-1. FANOUT: that sum formed once per element and stored into all R receive buffers (same
 * bits as ONESHOT). RING_FUSED, RING_2LEVEL, TREE: see hccl_algo_t. Send and receive buffers: count elements each. */
hccl_status_t hccl_plan_allreduce(int R, int64_t count, hccl_dtype_t dt, hccl_algo_t algo,
                                  const hccl_opts_t* opts, hccl_plan_t** out);

/* ReduceScatter(sum): rank r ends with Y_r[j] = round(sum_q X_q[o_r + j]), j < recvcounts[r],
 * o_r = sum of recvcounts below r. count = elements in every send buffer; recvcounts == NULL means
 * the floor split of count over R ranks; otherwise sum(recvcounts) must equal count
 * (HCCL_ERR_COUNT_MISMATCH). RING: each shard is cut into granules of opts->chunk_bytes and each
 * granule is an independent chain of R-1 reductions with FP32 partials in scratch. RING_FUSED: the same sums
 * in the same order as one multi-input sum per granule. ONESHOT: every rank sums its shard over all ranks
 * itself, in rank order 0..R-1. */
hccl_status_t hccl_plan_reducescatter(int R, const int64_t* recvcounts, int64_t count, hccl_dtype_t dt,
                                      hccl_algo_t algo, const hccl_opts_t* opts, hccl_plan_t** out);

/* AllGather(v): Y_r[o_q + j] = X_q[j] for all r, q; sendcounts[q] elements from rank q (NULL: count each).
 * algo RING copies hop by hop (rank r receives chunk (r-u-1) mod R from rank r-1 at step u);
 * ONESHOT has every rank read every peer directly (issued chunk by chunk, so a chunk's R reads follow one
 * another); FANOUT reads each chunk once and writes it into all R receive buffers from the same work item;
 * RING_2LEVEL gathers across racks first, then inside each rack. */
hccl_status_t hccl_plan_allgather(int R, const int64_t* sendcounts, int64_t count, hccl_dtype_t dt,
                                  hccl_algo_t algo, const hccl_opts_t* opts, hccl_plan_t** out);

/* AllToAllv (the collective that dominates recommendation training, Sec. I; its per-peer sizes and
 * offsets are the metadata of Sec. IV-B.2). All matrices are R x R row-major, in units of rows of
 * row_elems elements: sendcounts[s*R+d], sdispls[s*R+d] describe X_s; recvcounts[d*R+s], rdispls[d*R+s]
 * describe Y_d. For every (s,d), k < sendcounts[s][d]:
 *     row rdispls[d][s]+k of Y_d  =  row sdispls[s][d]+k of X_s      (byte for byte)
 * and no other byte of any Y is written. sdispls == NULL / rdispls == NULL mean packed (exclusive
 * prefix sums of the counts). recvcounts == NULL means the transpose of sendcounts; otherwise it must
 * equal it (HCCL_ERR_COUNT_MISMATCH). Send ranges may overlap or leave gaps; receive ranges of one
 * rank must not overlap (HCCL_ERR_OVERLAP). Zero counts are legal and cost nothing. */
hccl_status_t hccl_plan_alltoallv(int R, const int64_t* sendcounts, const int64_t* sdispls,
                                  const int64_t* recvcounts, const int64_t* rdispls, hccl_dtype_t dt,
                                  int64_t row_elems, const hccl_opts_t* opts, hccl_plan_t** out);

/* Device-resident AllToAllv ("AllToAllvDynamic", Sec. IV-B.2): for exchanges whose per-peer sizes are
 * produced on the device (a routing kernel) and must not travel through the host. The plan fixes only
 * R, the row size and the CAPACITY of every buffer in rows (max_send_rows[s] for X_s, max_recv_rows[d] for
 * Y_d); R <= HCCL_MAX_RANKS. Up to 64 ranks one kernel holds the whole count matrix in shared memory and
 * moves the rows itself. Beyond 64 ranks, from 1 GiB of send capacity on, or with HCCL_FLAG_DEVICE_TABLES, an execution is two launches: a small
 * kernel (one block per source rank) writes the R*R descriptors and their tiles into the bound workspace
 * -- the work requests are patched on the device, as the paper puts it -- and the ordinary executor
 * (opts.engine, default the bulk engine) runs them; the workspace is sized for the capacities. Before hccl_execute, hccl_plan_set_dynamic_metadata names the DEVICE array of R*R int64
 * counts (counts[s*R+d] rows from s to d) that the kernel reads when it runs, and optionally two DEVICE
 * arrays [d*R+s] that receive each destination's counts and displacements for the consumer of the result.
 * Layout is packed on both sides (exclusive prefix sums, computed in the kernel with warp scans). The
 * counts may change between executions of the same bound plan; combined with hccl_plan_set_trigger the
 * collective can be enqueued before the counts exist and is released by the producer's signal
 * (Sec. IV-B.3). If a count is negative, a source's rows exceed max_send_rows or a destination's rows
 * exceed max_recv_rows, no byte of a receive buffer is written and hccl_plan_status reports
 * HCCL_ERR_BAD_DESCRIPTOR (the two optional output arrays are then unspecified). */
hccl_status_t hccl_plan_alltoallv_dynamic(int R, const int64_t* max_send_rows, const int64_t* max_recv_rows,
                                          hccl_dtype_t dt, int64_t row_elems, const hccl_opts_t* opts,
                                          hccl_plan_t** out);
hccl_status_t hccl_plan_set_dynamic_metadata(hccl_plan_t*, const int64_t* dev_sendcounts,
                                             int64_t* dev_recvcounts_out, int64_t* dev_rdispls_out);

/* ------------------------------------------------------------------------
 * Work-packet builder: the paper's own vocabulary (Sec. III-B.2). A work packet is a set of
 * subgraphs that run in parallel; a subgraph is a list of WQEs issued in order; a WQE is a copy or
 * sum (the NMC forms S=A+B, A=A+B, B=A+B, A=B), a WAIT/SET on a memory location, or a NOOP that only
 * carries dependencies. The planners above are built on this; it is public so that schedules and
 * dependency kinds can be tested directly.
 * ------------------------------------------------------------------------ */
typedef enum {
    HCCL_OP_COPY = 0,     /* dst[0:count) = a[0:count)   count in BYTES, any alignment            (A=B) */
    HCCL_OP_REDUCE = 1,   /* dst[i] = round(f32(a[i]) + f32(b[i])), count in ELEMENTS; dst may alias a or b
                             exactly (A=A+B, B=A+B) or be separate (S=A+B) */
    HCCL_OP_REDUCE_N = 2, /* dst[i] = round(((f32(a_0[i]) + f32(a_1[i])) + ...) + f32(a_{nsrc-1}[i])) where a_k is
                             buffer a.kind of rank (a.rank + k) mod R at byte offset a.offset.
                             COPY and REDUCE_N may name several destinations (ndst > 1): the same bytes are then
                             written at dst.offset into the receive buffer of every rank (dst.rank + k) mod R,
                             k < ndst, from one read of the sources. The NMC of the paper has no such form (its ranks do
                             not share a memory); here it plays the part of a one-to-many send replicated inside the switch. */
    HCCL_OP_WAIT = 3,     /* block until signal slot a.offset compares true against value (+ epoch*value_per_epoch) */
    HCCL_OP_SET = 4,      /* store value (+ epoch*value_per_epoch) to signal slot dst.offset */
    HCCL_OP_NOOP = 5      /* nothing; exists to carry dependencies */
} hccl_op_t;

typedef enum {
    HCCL_BUF_SEND = 0,    /* X_rank: read-only for the library */
    HCCL_BUF_RECV = 1,    /* Y_rank */
    HCCL_BUF_SCRATCH = 2, /* library scratch inside the bound workspace (rank ignored) */
    HCCL_BUF_SIGNAL = 3,  /* 64-bit signal slots inside the workspace; offset = slot index. They persist across
                             executions, hence the paper's "monotonic increasing values" */
    HCCL_BUF_USER_SIGNAL = 4 /* a caller-supplied device uint64 array (hccl_plan_set_user_signals); offset = index */
} hccl_buf_t;

typedef struct {
    int32_t kind;   /* hccl_buf_t */
    int32_t rank;
    int64_t offset; /* bytes (data buffers) or slot index (signals) */
} hccl_ref_t;

/* Dependency kinds of Sec. III-B.2, as bit flags on a WQE. */
#define HCCL_DEP_FENCE 1u     /* the NEXT WQE of this subgraph does not start until this one has completed */
#define HCCL_DEP_SYNC 2u      /* wait for ALL previous WQEs of this subgraph */
#define HCCL_DEP_WQE_SYNC 4u  /* wait for the WQE whose id is dep_wqe (any subgraph, must be older) */
#define HCCL_DEP_RECV_SYNC 8u /* wait for all earlier WQEs of this subgraph that bring data INTO the subgraph's rank */
#define HCCL_DEP_SEND_SYNC 16u/* wait for all earlier WQEs of this subgraph that read data OUT OF the subgraph's rank
                                 into another rank (its buffers are released) */
/* Refinement of WQE_SYNC for pipelining (not a sixth kind): element k of this WQE needs only element k of
 * dep_wqe, so tile k may start as soon as tile k of dep_wqe is done. Honoured only when both WQEs are cut
 * into the same number of tiles; otherwise the whole of dep_wqe is waited for. The schedule's author is
 * responsible for the claim; hccl_plan_check_hazards verifies it tile by tile. */
#define HCCL_DEP_ELEMENTWISE 32u
#define HCCL_DEP_ELEMENTWISE2 64u /* the same claim for dep_wqe2 */

/* Cache hints on data WQEs. READ_ONCE: no source byte of this WQE is read by any other WQE of the packet
 * (it is streamed through the L2 with an evict-first policy). */
#define HCCL_HINT_READ_ONCE 1
/* LAST_READ_A (REDUCE whose operand A is in scratch): after this WQE nothing reads A's bytes again before they are
 * rewritten, so the executor may tell the L2 to drop those lines instead of writing them back to memory (the
 * cache-partition idea of Sec. II-A.3: temporary communication buffers should not cost the application).
 * Honoured by the bulk engine; a hint only. */
#define HCCL_HINT_LAST_READ_A 2

typedef enum { HCCL_CMP_EQ = 0, HCCL_CMP_NE = 1, HCCL_CMP_GE = 2, HCCL_CMP_GT = 3, HCCL_CMP_LE = 4, HCCL_CMP_LT = 5 } hccl_cmp_t;

typedef struct {
    int32_t op;                       /* hccl_op_t */
    int32_t dtype_dst, dtype_a, dtype_b; /* hccl_dtype_t; ignored by COPY/WAIT/SET/NOOP */
    hccl_ref_t dst, a, b;
    int64_t count;                    /* bytes (COPY) or elements (REDUCE, REDUCE_N) */
    int32_t nsrc;                     /* REDUCE_N only: 1..R */
    uint32_t dep_flags;               /* HCCL_DEP_* */
    int64_t dep_wqe;                  /* with HCCL_DEP_WQE_SYNC */
    int64_t dep_wqe2;                 /* optional second WQE_SYNC target, -1 if unused */
    int32_t cmp;                      /* WAIT: hccl_cmp_t */
    int32_t hints;                    /* data WQEs: HCCL_HINT_* */
    int32_t ndst;                     /* COPY, REDUCE_N: number of destinations, 0 or 1 = one; > 1 needs dst.kind RECV */
    int32_t reserved;                 /* 0 */
    int64_t tile_count;               /* tile size in units of count; 0 = derived from opts.tile_bytes */
    uint64_t value, value_per_epoch;  /* WAIT/SET: effective value = value + epoch*value_per_epoch, epoch = 1,2,.. per execute */
} hccl_wqe_t;

/* R ranks; send_bytes[r] / recv_bytes[r] = declared extent of X_r / Y_r (every WQE is bounds-checked
 * against them at add time), scratch_bytes = library scratch wanted, n_signals = signal slots. */
hccl_status_t hccl_graph_create(int R, const int64_t* send_bytes, const int64_t* recv_bytes,
                                int64_t scratch_bytes, int32_t n_signals, hccl_graph_t** out);
/* A new subgraph acting for virtual rank `rank` (used by RECV_SYNC/SEND_SYNC). Returns its index. */
hccl_status_t hccl_graph_add_subgraph(hccl_graph_t*, int rank, int32_t* subgraph);
/* Append a WQE to a subgraph. Issue order across the packet = order of these calls. *wqe_id gets its id. */
hccl_status_t hccl_graph_add_wqe(hccl_graph_t*, int32_t subgraph, const hccl_wqe_t* wqe, int64_t* wqe_id);
/* Lower to descriptors, tiles and synchronisation objects. The graph can be destroyed afterwards. */
hccl_status_t hccl_graph_compile(const hccl_graph_t*, const hccl_opts_t* opts, hccl_plan_t** out);
void hccl_graph_destroy(hccl_graph_t*);

/* ------------------------------------------------------------------------
 * Binding, execution, status (work-packet upload and cached re-enqueue, Sec. V-B, V-C).
 * ------------------------------------------------------------------------ */

/* Bytes of device workspace the plan needs: tables + counters + signals + FP32 scratch. */
hccl_status_t hccl_plan_workspace_bytes(const hccl_plan_t*, size_t* bytes);

/* Upload the tables into dev_workspace (256-B aligned, >= workspace bytes) with one host-to-device copy
 * on `stream` (a cudaStream_t passed as void*), zero the counters, reset the epoch. The workspace must
 * stay valid and untouched by others while the plan is used. Synchronises the stream before returning. */
hccl_status_t hccl_plan_bind(hccl_plan_t*, void* dev_workspace, size_t bytes, void* stream);

/* Enqueue one execution: a single kernel launch on `stream`. sendbufs/recvbufs are HOST arrays of R
 * DEVICE pointers (element-size aligned; 16-B alignment enables the fast paths; misaligned buffers are
 * handled correctly on a slow path). Send buffers are only read. Receive buffers are written only in
 * the declared ranges. Returns HCCL_ERR_OVERLAP if any send extent intersects any receive extent
 * (in-place operation is not supported). */
hccl_status_t hccl_execute(hccl_plan_t*, const void* const* sendbufs, void* const* recvbufs, void* stream);

/* Execution for callers that cannot allocate device memory. (The paper has no counterpart to this call;
 * it exists for the library's users.) Some callers must not call cudaMalloc at the point where they need a
 * collective: code that runs under a framework allocator's lock or inside its out-of-memory and
 * garbage-collection hooks, where asking for memory again would deadlock; processes that have already
 * handed every free byte of the GPU to another pool, so that cudaMalloc simply fails; and latency-critical
 * sections that cannot take the device-wide synchronisation cudaMalloc may imply. For them the library
 * carries its own workspace: a fixed array of HCCL_NOALLOC_WORKSPACE_BYTES = 8 MiB in the library's device
 * image, which every GPU that loads the library holds until the process exits.
 *
 * Runs `plan` once with that array in place of a bound workspace (the plan need not be bound; a bound
 * plan's own workspace and epoch are not touched). The register-path executor is used whatever
 * opts.engine says. sendbufs/recvbufs as in hccl_execute. Plans whose hccl_plan_workspace_bytes exceed
 * 8 MiB are refused with HCCL_ERR_WORKSPACE (for reductions on 16-bit data choose a small opts.chunk_bytes:
 * the FP32 scratch is 2 * chain_group granules); plans with a trigger and device-resident plans
 * (hccl_plan_alltoallv_dynamic) are refused with HCCL_ERR_INVALID_ARG. The call allocates nothing on the device: it calls no cudaMalloc/cudaFree and no
 * allocating library routine.
 *
 * All calls share the one array, and it keeps the previous call's contents: each call rewrites the
 * tables, control words, dependency counters and signal slots before launching, and leaves the FP32
 * scratch as it is (every execution writes a scratch slot before reading it). Two calls that overlap on
 * the GPU would race on the array; within one process the library serialises them, and the call therefore
 * BLOCKS: it waits for `stream` and returns the device-side verdict (HCCL_OK, HCCL_ERR_TIMEOUT,
 * HCCL_ERR_BAD_DESCRIPTOR) directly. Calls from different processes use different copies of the array.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that
 * device current); make that first call outside any stream capture. */
#define HCCL_NOALLOC_WORKSPACE_BYTES (8u << 20)
hccl_status_t hccl_execute_noalloc(hccl_plan_t*, const void* const* sendbufs, void* const* recvbufs, void* stream);

/* The same through HOST data: copies each host_send[r] (send extent of rank r) into dev_send[r], executes,
 * and copies each receive extent back into host_recv[r]; all asynchronous on `stream` (use pinned host
 * memory for true asynchrony). Device staging buffers are the caller's. */
hccl_status_t hccl_execute_host(hccl_plan_t*, const void* const* host_send, void* const* host_recv,
                                void* const* dev_send, void* const* dev_recv, void* stream);

/* ------------------------------------------------------------------------
 * AllToAllv through HOST buffers, pipelined by destination (the paper spreads an AllToAllv over several
 * subgraphs to keep the links busy, Sec. IV-A; here the link is the host interface and the pieces are
 * windows of destination ranks). The destinations are cut into n_windows contiguous groups by received
 * bytes; the first and last few groups are smaller, since only their copy-in and copy-out overlap nothing. For window g: the rows bound for its destinations are copied host->device (with packed
 * send displacements they are one contiguous slice of every send buffer), exchanged by a sub-plan that
 * holds only those segments, and the window's receive buffers are copied device->host. The three steps
 * run on three caller-supplied streams, ordered by events, so that copy-in of window g+1, exchange of g
 * and copy-out of g-1 overlap and both directions of the host link are busy at once.
 *   create    host only; sendcounts as in hccl_plan_alltoallv, packed displacements; n_windows is clamped
 *             to [1, R]; windows that would receive nothing are merged into their neighbours.
 *   bind      uploads every sub-plan's tables into the caller's workspace (workspace_bytes, 256-aligned)
 *             and creates the ordering events (no device memory is allocated).
 *   execute   asynchronous; everything has completed when stream_out has. host buffers should be pinned.
 *             dev_send / dev_recv are the caller's staging buffers (full extents, as for hccl_execute).
 *             A second execute may be enqueued at once, on the same three streams: its copies-in start when
 *             the first call's last exchange has run, and its exchange of a window when the first call's
 *             copy-out of that window has finished. The host buffers of a call must stay untouched until
 *             stream_out has passed that call.
 *   status    after synchronising stream_out: the first device-side failure of any window, else HCCL_OK.
 *   windows   first_dest[g] .. first_dest[g+1]-1 are window g's destinations (n_windows+1 entries).
 * ------------------------------------------------------------------------ */
typedef struct hccl_hostpipe hccl_hostpipe_t;
hccl_status_t hccl_hostpipe_alltoallv_create(int R, const int64_t* sendcounts, hccl_dtype_t dt, int64_t row_elems,
                                             int n_windows, const hccl_opts_t* opts, hccl_hostpipe_t** out);
hccl_status_t hccl_hostpipe_windows(const hccl_hostpipe_t*, int32_t* n_windows, int32_t* first_dest /* [R+1] room */);
hccl_status_t hccl_hostpipe_workspace_bytes(const hccl_hostpipe_t*, size_t* bytes);
hccl_status_t hccl_hostpipe_bind(hccl_hostpipe_t*, void* dev_workspace, size_t bytes, void* stream);
hccl_status_t hccl_hostpipe_execute(hccl_hostpipe_t*, const void* const* host_send, void* const* host_recv,
                                    void* const* dev_send, void* const* dev_recv, void* stream_in, void* stream_exec,
                                    void* stream_out);
hccl_status_t hccl_hostpipe_status(hccl_hostpipe_t*, hccl_status_t* device_status, int64_t* detail);
void hccl_hostpipe_destroy(hccl_hostpipe_t*);

/* Resident, doorbell-fed execution (the express-doorbell idea of Sec. II-A.3 and the cached re-enqueue of
 * Sec. V-B, without any launch per collective). hccl_server_start launches the register engine ONCE as a
 * long-lived kernel bound to this plan and these buffers; afterwards hccl_server_ring is a single store
 * into the doorbell record and costs no CUDA call, the resident blocks execute the plan once per ring, and
 * hccl_server_wait spins (on the host) until the record says so. host_doorbell points to 64 bytes of
 * pinned, MAPPED host memory owned by the caller (cudaHostAlloc with cudaHostAllocMapped, or torch pinned
 * memory), 64-byte aligned; it must stay valid until the kernel has left. All blocks must be resident at
 * once (sm_budget blocks of opts.threads threads; HCCL_ERR_INVALID_ARG otherwise). The kernel leaves by
 * itself when no ring arrives for idle_timeout_ns (default 100 ms; then hccl_server_ring returns
 * HCCL_ERR_TIMEOUT and the server can be started again), after hccl_server_stop, or after a failed
 * execution (whose verdict hccl_server_ring / hccl_server_wait then return). While the server runs, use
 * only these calls on the plan, and do not synchronise the whole device: the kernel occupies `stream` until
 * it leaves. Rings are served in order; ring again only after the previous ring was waited for.
 * hccl_server_stop only asks the kernel to leave and returns at once: synchronise the server's `stream` after
 * it, before the plan is executed, bound or served again (until the kernel has left, its blocks still use the
 * workspace's ticket, exit count and counters). */
typedef struct {
    uint64_t request, completed, stop, exited, status, detail;
    uint64_t t_seen_ns, t_done_ns; /* device clock (%globaltimer) when the kernel saw the last ring and when that execution's last
                                      block had left: the part of a ring-to-wait round trip that is spent on the device */
} hccl_doorbell_t;
hccl_status_t hccl_server_start(hccl_plan_t*, const void* const* sendbufs, void* const* recvbufs, void* host_doorbell,
                                uint64_t idle_timeout_ns, void* stream);
hccl_status_t hccl_server_ring(hccl_plan_t*);
hccl_status_t hccl_server_wait(hccl_plan_t*, uint64_t timeout_ns);
hccl_status_t hccl_server_stop(hccl_plan_t*);

/* Device-triggered execution (Sec. IV-B.3): give the plan a caller-owned device array of uint64 that
 * HCCL_BUF_USER_SIGNAL refs index; hccl_plan_set_trigger makes every execution (a) hold all work until
 * user signal slot wait_slot satisfies cmp against wait_value + epoch*wait_per_epoch, and (b) store
 * set_value + epoch*set_per_epoch into slot set_slot once everything has completed. Pass a negative
 * slot to disable either half. Must be called before hccl_plan_bind. */
hccl_status_t hccl_plan_set_user_signals(hccl_plan_t*, void* dev_signals, int64_t n_slots);
hccl_status_t hccl_plan_set_trigger(hccl_plan_t*, int64_t wait_slot, int32_t cmp, uint64_t wait_value,
                                    uint64_t wait_per_epoch, int64_t set_slot, uint64_t set_value,
                                    uint64_t set_per_epoch);

/* After the stream has been synchronised: the device-side verdict of the LAST execution. The device numbers
 * its own executions (epoch = completed executions of the bound workspace + 1), so hccl_execute is a plain
 * kernel launch that can be captured in a CUDA graph and replayed; replays count as executions.
 * *device_status is HCCL_OK, HCCL_ERR_TIMEOUT or HCCL_ERR_BAD_DESCRIPTOR; *detail is the tile index
 * involved or, on HCCL_OK, the number of executions completed since the plan was bound. */
hccl_status_t hccl_plan_status(hccl_plan_t*, hccl_status_t* device_status, int64_t* detail);

typedef struct {
    int64_t n_wqe;            /* WQEs in the packet */
    int64_t n_tiles;          /* work items the executor dispatches */
    int64_t n_syncs;          /* device-side dependency counters */
    int64_t chain_depth;      /* longest dependency chain, in WQEs */
    int64_t schedule_bytes;   /* sum over WQEs of bytes read + bytes written (what the schedule moves) */
    int64_t compulsory_bytes; /* every input byte read once + every output byte written once */
    int64_t scratch_bytes;
    int64_t send_bytes_total, recv_bytes_total; /* declared extents */
    int32_t R, sm_budget, threads, engine;
    int64_t tile_bytes;       /* the largest work item cut, in bytes of its widest operand */
    int64_t epoch;            /* executions enqueued since the last bind */
    int64_t crossrack_bytes;  /* bytes that data WQEs move between ranks of different racks (racks of opts.rack_size):
                                 what would cross the scale-out network with real ranks (Sec. II-A.3, V-D) */
    int64_t static_chains;    /* 0: tiles are handed out by ticket; otherwise the number of chains of tiles that run
                                 inside one block each (HCCL_FLAG_STATIC_CHAINS), chain_depth tiles per chain */
} hccl_plan_info_t;
hccl_status_t hccl_plan_info(const hccl_plan_t*, hccl_plan_info_t* out);

/* Tracing (the per-work-packet and per-subgraph counters of Sec. V-C, per work item here): give the plan a
 * caller-owned DEVICE array of capacity_items x 4 uint64 and every later execution records, for work item i,
 * [4i] = i | block << 32, [4i+1] = time it was claimed, [4i+2] = time its data movement was released (all
 * dependencies met), [4i+3] = time its last byte was stored (bulk COPY: its last store issued); %globaltimer
 * nanoseconds. Items beyond the capacity are not recorded. Pass capacity 0 to switch tracing off. The
 * resident executor and hccl_execute_noalloc do not trace. */
hccl_status_t hccl_plan_set_trace(hccl_plan_t*, void* dev_trace, int64_t capacity_items);

/* Byte offsets of the regions inside a bound workspace, in this order: control block, dependency counters,
 * signal slots, descriptors (64 B each), tiles (32 B each), wait lists (8 B per entry), FP32 scratch, total.
 * For tools that inspect a workspace, and for tests that damage a table on purpose. */
hccl_status_t hccl_plan_layout(const hccl_plan_t*, int64_t offsets[8]);

/* Declared extent, in bytes, of rank r's send / receive buffer. */
hccl_status_t hccl_plan_extents(const hccl_plan_t*, int rank, int64_t* send_bytes, int64_t* recv_bytes);

void hccl_plan_destroy(hccl_plan_t*);
const char* hccl_status_string(hccl_status_t);
const char* hccl_last_cuda_error(void); /* text of the last CUDA failure seen by this thread, "" if none */
int hccl_version(void);

/* ------------------------------------------------------------------------
 * Plan verification on the host (debugging aids for schedules; never part of hccl_execute).
 * ------------------------------------------------------------------------ */

/* Hazard check: every pair of work items whose byte ranges intersect with at least one writer must be
 * ordered by a dependency path. *n_violations = pairs found unordered (0 = clean). Cost grows with the
 * number of conflicting pairs; meant for small and medium plans. */
hccl_status_t hccl_plan_check_hazards(const hccl_plan_t*, int64_t* n_violations);

/* Run the compiled tables on HOST buffers in a random dependency-respecting order drawn from `seed`
 * (seed 0 = ticket order). A schedule debugging aid only: it validates what the planner emitted
 * without a GPU. host_scratch must hold scratch_bytes (see hccl_plan_info); may be NULL if zero. */
hccl_status_t hccl_plan_interpret_host(const hccl_plan_t*, const void* const* host_send, void* const* host_recv,
                                       void* host_scratch, uint64_t* host_signals, uint64_t seed);

#ifdef __cplusplus
}
#endif
#endif /* HCCL_B200_H */

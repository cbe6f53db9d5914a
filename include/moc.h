/*
 * moc -- batched evaluation of rematerialization sequences on one NVIDIA B200 (sm_100a).
 *
 * C ABI of the shared library libmoc_b200.so.  The operations are those of the rematerialization
 * problem of "Moccasin: Efficient Tensor Rematerialization for Neural Networks" (arXiv 2304.14463):
 * given a compute DAG G=(V,E) with per-node duration w_v and output size m_v, and a candidate
 * execution sequence in which every node runs between 1 and C times, report the total duration,
 * the peak memory footprint and whether the sequence meets the data dependencies and a memory
 * budget M (Section 1, problem statement; Section 2, Eqs. 1-8).
 *
 * Conventions
 *   - nodes are 0..n-1; an edge (u,v) means "v consumes the output of u" (Section 1);
 *   - a sequence seq[0..T) lists node ids in execution order; position t is the t-th *filled*
 *     compute event of Section 2 (empty events contribute to neither duration nor peak);
 *   - each occurrence ("copy") of a node is one active retention interval [s,e] of Section 2 with
 *     s = its position; its end e ("free step") is the last step that consumes this copy before
 *     the node is computed again (Eq. 3: intervals of one node do not overlap; Eq. 5: a consumer
 *     at step t needs a copy with s+1 <= t <= e, and the most recent earlier copy is the one
 *     charged, which makes every interval as short as the sequence permits); a copy nobody
 *     consumes has e = s (Eq. 2); the last copy of a node without successors is the result of the
 *     computation and stays resident to step T-1;
 *   - memory in use at step t is the sum of m over the copies with s <= t <= e, both ends
 *     inclusive (Eq. 4); the peak is the maximum over the steps (Section 2).
 *
 * Per-sequence status codes (never an error return; bad sequences cannot fault the GPU):
 *     1  dependencies met and peak <= M                      peak, duration valid
 *     0  dependencies met, peak > M                           peak, duration valid
 *    -1  some consumer has no earlier copy of a predecessor  peak = -1, duration valid (Eq. 5)
 *    -2  malformed: length outside [n, C*n], id outside [0,n), a node absent (Eq. 7) or computed
 *        more than C times (Section 2, C_v)                  peak = duration = -1
 *
 * Every function returns MOC_OK or a negative error code and never throws or aborts;
 * moc_last_error() gives the text for the calling thread.  "HOST" / "DEVICE" below says where a
 * pointer must live.  The caller owns every array; the library owns the handle, its device copy
 * of the graph and grow-only scratch attached to the handle.  Because of that scratch, calls on
 * one handle must be ordered (issue them from one thread, on one stream, or synchronise between
 * streams); different handles are independent.  There is no CPU fallback: without a CUDA device
 * every call that needs one fails with MOC_ERR_CUDA.
 */
#ifndef MOC_H_
#define MOC_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MOC_OK 0
#define MOC_ERR_ARG (-1)      /* null pointer, negative size, value outside its documented range   */
#define MOC_ERR_RANGE (-2)    /* edge endpoint outside [0,n)                                       */
#define MOC_ERR_CYCLE (-3)    /* self-loop or directed cycle                                       */
#define MOC_ERR_OVERFLOW (-4) /* negative weight, or 8*sum(w) or 8*sum(m) would not fit in 62 bits  */
#define MOC_ERR_CUDA (-5)     /* a CUDA runtime call failed (text in moc_last_error)               */
#define MOC_ERR_NOMEM (-6)    /* host or device allocation failed                                  */

#define MOC_MAX_COPIES 8      /* largest admissible C                                              */

typedef struct moc_graph moc_graph; /* opaque */

/*
 * Problem data of Section 1: DAG, durations, output sizes.
 *   n        number of nodes, >= 1
 *   n_edges  number of (u,v) pairs in `edges`, >= 0
 *   edges    HOST, 2*n_edges ints, pair k = (edges[2k], edges[2k+1]) = (u,v): v consumes u.
 *            Duplicates are accepted and merged.  May be NULL when n_edges == 0.
 *   w, m     HOST, n values each, all >= 0 (opaque integer units).
 *   out      receives the handle; device copies live on the CUDA device current at the call.
 * Errors: MOC_ERR_ARG, MOC_ERR_RANGE, MOC_ERR_CYCLE, MOC_ERR_OVERFLOW, MOC_ERR_CUDA,
 * MOC_ERR_NOMEM; *out is NULL on error.  Synchronous (copies the graph before returning).
 * The maximum number of copies per node starts at C = 2 (Section 4.3 uses C_v = 2 throughout).
 */
int moc_graph_create(int32_t n, int64_t n_edges, const int32_t* edges, const int64_t* w,
                     const int64_t* m, moc_graph** out);

/* Sets the cap C on copies per node (the paper's C_v, uniform over nodes; Section 2).
 * 1 <= C <= MOC_MAX_COPIES, else MOC_ERR_ARG.  Per-node caps set earlier are dropped. */
int moc_graph_set_max_copies(moc_graph* g, int32_t C);

/*
 * Per-node caps C_v (Section 2: node v has at most C_v retention intervals).
 *   caps   HOST, n ints, each in [1, C] for the handle's current C; NULL restores the uniform cap.
 * A sequence with more than C_v copies of node v gets status -2.  The length bound stays
 * n <= T <= C*n.  moc_graph_set_max_copies resets the caps to uniform.  Synchronises the device
 * (work in flight may still read the old caps), then copies.  Errors: MOC_ERR_ARG, MOC_ERR_CUDA,
 * MOC_ERR_NOMEM.
 */
int moc_graph_set_node_caps(moc_graph* g, const int32_t* caps);

/* Frees the handle with its device memory.  NULL is accepted.  The caller must have
 * synchronised every stream that still runs work of this handle. */
void moc_graph_destroy(moc_graph* g);

/* Facts about a handle (any pointer may be NULL): node count, number of distinct edges, current
 * C, and whether memory sums are accumulated in 64 bits (1) or provably fit 32 bits (0) at that C. */
int moc_graph_info(const moc_graph* g, int32_t* n, int64_t* n_edges, int32_t* C, int32_t* wide);

/*
 * Evaluates B sequences (objective Eq. 1, memory constraint Eq. 4, precedence Eq. 5, peak as
 * defined in Section 2).
 *   seqs          DEVICE, int32, packed back to back: sequence b occupies
 *                 seqs[offs[b] .. offs[b]+len_b) with len_b = max(lens[b], 0) and offs the
 *                 exclusive prefix sum of len_b.  Must hold sum(len_b) ints, 4-byte aligned.
 *   lens          DEVICE, B ints.
 *   B             number of sequences, >= 0 (0: nothing is launched, MOC_OK).
 *   M             memory budget.
 *   out_peak      DEVICE, B int64: peak memory footprint (or -1, see status codes).
 *   out_dur       DEVICE, B int64: total duration with recomputations (or -1).
 *   out_feasible  DEVICE, B int32: status code 1 / 0 / -1 / -2.
 *   stream        a cudaStream_t (NULL = default stream).  The call only enqueues work; outputs
 *                 are valid once the stream has been synchronised.
 * Errors: MOC_ERR_ARG (null pointer with B > 0, B < 0), MOC_ERR_CUDA, MOC_ERR_NOMEM (scratch
 * growth; happens only when B exceeds every earlier B on this handle).
 * The library cannot see how large a device buffer is: outputs shorter than B entries, or a seqs
 * buffer shorter than the lengths add up to, make the kernels read or write outside them.  The
 * caller (the Python binding does it for the outputs) checks the sizes.
 */
int moc_eval_batch(const moc_graph* g, const int32_t* seqs, const int32_t* lens, int32_t B,
                   int64_t M, int64_t* out_peak, int64_t* out_dur, int32_t* out_feasible,
                   void* stream);

/*
 * Same evaluation with every array in HOST memory (pinned memory makes the copies asynchronous
 * with respect to the host, pageable memory works too): copies seqs (n_steps ints, which must be
 * at least sum(max(lens[b],0))) and lens to device staging owned by the handle, evaluates, copies
 * the three outputs back and synchronises `stream` before returning.  Large batches travel in
 * four chunks of whole sequences (a half, a quarter and two eighths of the steps): a copy stream
 * owned by the handle brings one chunk while `stream` evaluates the one before, so that only the
 * evaluation of the small last chunk is not hidden, and the results return in a single copy
 * through a pinned block of the handle.  One call at a time per handle.
 */
int moc_eval_batch_host(const moc_graph* g, const int32_t* seqs, int64_t n_steps,
                        const int32_t* lens, int32_t B, int64_t M, int64_t* out_peak,
                        int64_t* out_dur, int32_t* out_feasible, void* stream);

/*
 * moc_eval_batch_host with the node ids as HOST uint16 (graphs with n <= 65535, else MOC_ERR_ARG):
 * half the bytes cross the host link, which is what bounds the host entry point; the ids are widened
 * on the device in front of the evaluation.  An id >= n is out of range as before (status -2).
 * Everything else as moc_eval_batch_host.
 */
int moc_eval_batch_host16(const moc_graph* g, const uint16_t* seqs, int64_t n_steps,
                          const int32_t* lens, int32_t B, int64_t M, int64_t* out_peak,
                          int64_t* out_dur, int32_t* out_feasible, void* stream);

/*
 * moc_eval_batch for callers that must not allocate device memory.  (The paper has no counterpart:
 * this is a deployment variant of moc_eval_batch, with identical results.)
 *
 * Who needs it: a caller that has handed the whole device to its own memory pool, a latency-bound
 * loop that cannot afford the driver's allocator lock or the device-wide synchronisation that
 * cudaFree implies, or a process running under a fixed memory partition.  moc_eval_batch keeps its
 * packing offsets (B+1 int64) in scratch that it allocates on the handle and regrows when B grows;
 * this entry point keeps them in a fixed array inside the library image instead, and calls no
 * cudaMalloc, cudaFree or other allocating routine.
 *
 *   - The array holds MOC_NOALLOC_MAX_B + 1 offsets (512 KB).  It is part of the library's device
 *     image: every GPU on which the library is used holds it until the process exits.
 *   - B > MOC_NOALLOC_MAX_B is rejected with MOC_ERR_ARG.  So is a graph whose per-sequence state
 *     does not fit in shared memory (more than 65534 steps per sequence, or n*C too large): that
 *     case needs a global workspace, which only moc_eval_batch provides.
 *   - The first call on each device looks up the array's device address (once per device, with
 *     that device current) and prepares the launch plan of the handle.  Make that first call
 *     outside of any stream capture.
 *   - All calls on a device, from every handle and stream, share the one array.  Each call
 *     rewrites the B+1 entries it uses before reading them, so stale contents of an earlier call
 *     never matter and nothing needs clearing; but two calls that overlap on the GPU (different
 *     streams without an ordering between them) race on it and give wrong results.  Order them.
 *
 * Arguments, outputs, asynchrony and status codes are exactly those of moc_eval_batch.
 */
#define MOC_NOALLOC_MAX_B 65536
int moc_eval_batch_noalloc(const moc_graph* g, const int32_t* seqs, const int32_t* lens, int32_t B,
                           int64_t M, int64_t* out_peak, int64_t* out_dur, int32_t* out_feasible,
                           void* stream);

/*
 * Memory profile of one sequence (the per-event sums of Eq. 4 and the interval ends of Section 2).
 *   seq          DEVICE, len int32 node ids.
 *   out_profile  DEVICE, len int64: memory in use at every step.
 *   out_free     DEVICE, len int32: free step of the copy executed at each step; may be NULL.
 *   out_status   DEVICE, 1 int32: -2 / -1 as above, otherwise 1.  When the status is negative
 *                both arrays are filled with -1.
 * Asynchronous on `stream` like moc_eval_batch.  len < 0 is MOC_ERR_ARG.
 */
int moc_mem_profile(const moc_graph* g, const int32_t* seq, int32_t len, int64_t* out_profile,
                    int32_t* out_free, int32_t* out_status, void* stream);

/*
 * ---- Solutions in the paper's own variables ------------------------------------------------------
 *
 * Checks B solutions given as retention intervals against Eqs. 2-8 as printed (Section 2), with the
 * duration of Eq. 1 and the peak of the usage of Eq. 4, e.g. to validate what a constraint solver
 * returned.  Node v has C slots (the handle's C); slot i has a start s, an end e (events, 1-based)
 * and a flag a (1 active, 0 inactive).
 *   s, e, a      DEVICE, B*n*C int32 each, index [b][v][i].
 *   D            size of the event domain {1..D}: normally C*n (Section 2) or n(n+1)/2 (staged).
 *   topo_index   DEVICE, n int32: 1-based index of every node in the input topological order; selects
 *                the staged model of the subsection "Complexity Reduction by Enforcing an Initial
 *                Topological Ordering" (stage j = events j(j-1)/2+1 .. j(j+1)/2; an active interval of
 *                the node with index k starts at event k of a stage j >= k; its first interval at the
 *                last event of stage k).  Requires D = n(n+1)/2.  NULL: the plain model.
 *   M            memory budget of Eq. 4.
 *   out_mask     DEVICE, B int32: bit 0 set when Eq. 2 (s <= e, every slot) is violated, bit 1 Eq. 3
 *                (e_v^i <= s_v^{i+1}, every slot), bit 2 Eq. 4 (peak > M), bit 3 Eq. 5 (an active
 *                interval of a consumer v starts at t without an active interval of a predecessor u
 *                with s_u + 1 <= t <= e_u), bit 4 Eq. 6 (two slots of different nodes share a start;
 *                plain model only), bit 5 Eq. 7 (first slot inactive), bit 6 Eq. 8 (s or e outside
 *                {1..D}, a outside {0,1}), bit 7 the staged rule.  When bit 6 is set nothing else is
 *                evaluated: mask = 64, peak = duration = -1, length = -1.
 *   out_peak     DEVICE, B int64: max over the events of the sum of m over active intervals with
 *                s <= t <= e.
 *   out_dur      DEVICE, B int64: sum of w over active intervals.
 *   out_seqs     DEVICE, B rows of n*C int32, or NULL: the execution sequence the solution stands for
 *                (its active intervals in the order of their starts), usable with moc_eval_batch after
 *                packing; only the first out_lens[b] entries of a row are written.
 *   out_lens     DEVICE, B int32, or NULL: number of active intervals, or -1 when two of them start at
 *                the same event (no sequential execution; the row is then left untouched).
 * Asynchronous on `stream`; allocates nothing.  MOC_ERR_ARG when the domain and the intervals of one
 * solution do not fit in the shared memory of one block ((D/32)*12 + n*C*8 bytes, roughly).
 * Per-node caps of the handle are not applied here: every node has the handle's C slots.
 */
int moc_check_intervals(const moc_graph* g, const int32_t* s, const int32_t* e, const int32_t* a,
                        int32_t B, int64_t D, const int32_t* topo_index, int64_t M, int64_t* out_peak,
                        int64_t* out_dur, int32_t* out_mask, int32_t* out_seqs, int32_t* out_lens,
                        void* stream);

/*
 * ---- Incremental evaluation of edited sequences ------------------------------------------------
 *
 * A search looks at many sequences that differ from an evaluated one ("parent") by a single edit.
 * Retention intervals are local to the copies of a node (Section 2: Eq. 3 orders the intervals of one
 * node, Eq. 5 ties the end of an interval to the consumers of that node), so an edit of a copy of node
 * x changes only the intervals of x and of the predecessors of x; the memory profile of Eq. 4 changes
 * inside a window around them and is shifted elsewhere.  moc_cache_build evaluates the parents once and
 * keeps their profile, its prefix and suffix maxima, the free steps and the positions of every node's
 * copies on the device; moc_eval_edits then scores any number of edits of those parents from the
 * cache.  The results are exactly those moc_eval_batch gives for the edited sequences.
 *
 * Limits: handles with C <= 2 (the setting of Section 4.3) and C*n <= 65534; per-node caps are honoured.
 * The cache refers to the graph handle, which must outlive it.  A call of moc_graph_set_max_copies or
 * moc_graph_set_node_caps makes the cached parents stale: moc_eval_edits (and a moc_search_run that scores
 * its proposals from a cache) then fails with MOC_ERR_ARG until moc_cache_build has run again; a changed
 * C needs a new cache.  The cache owns, per parent, 4 + 3 * (4 or 8) bytes for each of its C*n possible steps
 * (sequence and free steps in 16 bits, usage and its prefix and suffix maxima in 32 or 64 bits as the graph's
 * sums need) and 4 bytes per node, all allocated by moc_cache_create.
 */
typedef struct moc_cache moc_cache; /* opaque */

/* Room for up to max_parents parents.  Errors: MOC_ERR_ARG (C > 2, sequences too long for the
 * on-chip state), MOC_ERR_CUDA, MOC_ERR_NOMEM. */
int moc_cache_create(const moc_graph* g, int32_t max_parents, moc_cache** out);

/*
 * Evaluates P parents (seqs, lens: DEVICE, packed as for moc_eval_batch) against budget M and fills
 * the cache; parent k of later moc_eval_edits calls is sequence k of this call.  out_peak, out_dur,
 * out_status (DEVICE, P each, any may be NULL) receive the same values as moc_eval_batch.
 * Asynchronous on `stream`; two kernels; no allocation.  1 <= P <= max_parents.
 */
int moc_cache_build(moc_cache* c, const int32_t* seqs, const int32_t* lens, int32_t P, int64_t M,
                    int64_t* out_peak, int64_t* out_dur, int32_t* out_status, void* stream);

/*
 * Scores B edits.  Edit b takes parent parent[b] (sequence of T steps) and
 *     op[b] = 0  inserts a further copy of node seq[q[b]] in front of index j[b], 0 <= j <= T;
 *     op[b] = 1  removes step q[b]  (j[b] is ignored);
 *     op[b] = 2  removes step q[b] and puts its node back in front of index j[b] of the shortened
 *                sequence, 0 <= j <= T-1;
 * with 0 <= q[b] < T: the edits of the search entry points.  All arrays DEVICE, B entries.
 *   out_peak, out_dur, out_status: what moc_eval_batch reports for the edited sequence (status
 *   1 / 0 / -1 / -2 with the same sentinels).  Two more cases: an edit whose parent index, op, q or
 *   j is out of range gets status -2 (peak = dur = -1); an edit of a parent whose own status is
 *   negative gets status MOC_STATUS_PARENT_INVALID (-3, peak = dur = -1): such a parent has no
 *   profile to start from, evaluate the edited sequence with moc_eval_batch.
 *   out_window (DEVICE, B int32, may be NULL): number of steps of the edited sequence whose usage had
 *   to be recomputed (0 when the edit was refused before that point): the cost of the edit.
 * Asynchronous on `stream` (ordered after moc_cache_build on the same stream); one kernel; no
 * allocation.
 */
#define MOC_STATUS_PARENT_INVALID (-3)
int moc_eval_edits(const moc_cache* c, const int32_t* parent, const int32_t* op, const int32_t* q,
                   const int32_t* j, int32_t B, int64_t M, int64_t* out_peak, int64_t* out_dur,
                   int32_t* out_status, int32_t* out_window, void* stream);

/* Frees the cache; NULL is accepted.  Synchronise its streams first. */
void moc_cache_destroy(moc_cache* c);

/*
 * ---- Local search over sequences (Section 3, "Optimization in Two Phases") -------------------------
 *
 * P independent chains each hold one sequence and its evaluation.  One generation proposes, for
 * every chain, one edited copy of its sequence, evaluates all proposals as one batch with the
 * evaluator above, and replaces a chain's sequence by its proposal when the proposal's status is
 * >= 0 and its key
 *         ( max(peak, M), duration )                 (sequences with status < 0 rank last)
 * is not larger than the chain's.  This folds the paper's two phases into one order: while a chain
 * is over the budget the first component, the Phase 1 objective max(M_var, M), goes down; once
 * peak <= M it equals M for everything that can still be accepted, so the duration (Eq. 1) alone
 * decides under the memory constraint of Eq. 4, which is Phase 2.  Equal keys are accepted, so a
 * chain can drift across plateaus.
 *
 * Proposal of chain c in generation k for a sequence of T steps (T = 0 proposes nothing): with
 * (r0, r1, r2, r3) = Philox4x32-10(counter = (k, first_chain + c, 0, 0), key = (seed mod 2^32,
 * seed div 2^32)) (Salmon, Moraes, Dror, Shaw, SC 2011),
 *     op = r0 mod 3 (all kinds enabled, see moc_search_set_kinds), q = r1 mod T;
 *     op 0  insert: a further copy of node seq[q] is put in front of index j = r2 mod (T+1);
 *     op 1  delete: element q is removed;
 *     op 2  move:   element q is removed and put back in front of index j = r2 mod T of the
 *                   shortened sequence.
 * Whether a proposal is admissible is left to the evaluator (length outside [n, C*n], a node without
 * a copy or with more than C copies give status -2; a consumer moved in front of its producer gives
 * status -1), and such proposals are refused.
 *
 * The handle owns all device memory of the search (2 rows of C*n ints per chain plus 60 bytes per
 * chain) and refers to the graph handle, which must outlive it and keep its C.  Calls on one search
 * handle, and calls on its graph handle, must be ordered like calls on a graph handle.
 */
typedef struct moc_search moc_search; /* opaque */

/*
 * Starts a search from P sequences.
 *   seqs, lens   DEVICE, packed as for moc_eval_batch; every length must lie in [0, C*n]
 *                (MOC_ERR_ARG otherwise).  Sequences may be invalid (status < 0): such a chain
 *                accepts the first proposal with status >= 0.
 *   M            memory budget;  seed: key of the random draws.
 *   first_chain  global number of chain 0.  A population split over several handles (one per
 *                GPU) evolves exactly like the unsplit one when every part is given the global
 *                number of its first chain; 0 for a single handle.  first_chain + P <= 2^32.
 * Copies the sequences, evaluates them and synchronises `stream` before returning.
 * Errors: MOC_ERR_ARG, MOC_ERR_CUDA, MOC_ERR_NOMEM; *out is NULL on error.
 */
int moc_search_create(const moc_graph* g, const int32_t* seqs, const int32_t* lens, int32_t P,
                      int64_t M, uint64_t seed, uint32_t first_chain, void* stream,
                      moc_search** out);

/* Enqueues n_generations further generations on `stream` (asynchronous; two kernels per generation
 * plus one at the end, no allocation, no synchronisation).  Generations are numbered from 0 over
 * the life of the handle; the result does not depend on how they are split over calls. */
int moc_search_run(moc_search* s, int32_t n_generations, void* stream);

/*
 * Chooses the kinds of edit the following generations may propose: bit 0 insert (MOC_EDIT_INSERT),
 * bit 1 delete (MOC_EDIT_DELETE), bit 2 move (MOC_EDIT_MOVE); default all three.  With k kinds
 * enabled a proposal takes the (r0 mod k)-th enabled kind in this order.  MOC_EDIT_MOVE alone
 * searches over the orders of the sequences without adding or removing a copy: started from
 * topological orders it is a search for a no-rematerialization order of low peak (Section 1: the
 * peak depends on the topological order).  kinds outside 1..7 is MOC_ERR_ARG.
 */
#define MOC_EDIT_INSERT 1u
#define MOC_EDIT_DELETE 2u
#define MOC_EDIT_MOVE 4u
int moc_search_set_kinds(moc_search* s, uint32_t kinds);

/*
 * Proposals per chain and generation, and how they are scored.
 *   samples      E >= 1.  Proposal e = 0..E-1 of chain c in generation k draws
 *                Philox4x32-10(counter = (k, first_chain + c, e, 0)); the chain's candidate is the
 *                proposal with the smallest key among those with status >= 0, the lowest e among
 *                equals, and it replaces the chain's sequence when its key is not larger.  E = 1 is
 *                the single proposal described above.
 *   incremental  0 (MOC_SEARCH_WRITTEN_OUT): every proposal is written out and evaluated from scratch
 *                (E must be 1);
 *                1 (MOC_SEARCH_SCORE_AUTO): proposals are scored from the cached evaluation of the chain's
 *                sequence and only accepted ones are written out; the library picks the scoring kernel
 *                (a warp per chain from E = 24 on when the graph fits it, else the kernel of moc_eval_edits);
 *                2 (MOC_SEARCH_SCORE_EDIT): the same through moc_eval_edits: a generation is four
 *                kernels (draw, moc_eval_edits, pick, rebuild of the changed cache entries);
 *                3 (MOC_SEARCH_SCORE_CHAIN): the same with a warp per chain: the chain's cache entry is
 *                staged in shared memory once and its E proposals are drawn, scored and settled there;
 *                a generation is two kernels (that one and the rebuild).  MOC_ERR_ARG when the entry
 *                and the correction lists (4 + 2 * largest in-degree entries) of four chains do not
 *                fit the shared memory of an SM.
 *                1 to 3 need C <= 2 and a valid sequence (status >= 0) in every chain at the time of
 *                the call (MOC_ERR_ARG otherwise).  All four give identical chains.
 * Synchronises the device, allocates (the cache of the chains, 28 bytes per proposal); after it
 * moc_search_run allocates nothing.
 */
#define MOC_SEARCH_WRITTEN_OUT 0
#define MOC_SEARCH_SCORE_AUTO 1
#define MOC_SEARCH_SCORE_EDIT 2
#define MOC_SEARCH_SCORE_CHAIN 3
int moc_search_set_samples(moc_search* s, int32_t samples, int32_t incremental);

/*
 * Copies the chains' current state to DEVICE arrays of the caller (any pointer may be NULL):
 *   out_rows      P rows of `stride` ints (moc_search_info); row c holds chain c's sequence in its
 *                 first out_lens[c] entries, the rest of the row is left untouched;
 *   out_lens, out_status, out_accepted   P int32 (accepted = proposals accepted so far);
 *   out_peak, out_dur                    P int64.
 * Asynchronous on `stream`.
 */
int moc_search_state(const moc_search* s, int32_t* out_rows, int32_t* out_lens, int64_t* out_peak,
                     int64_t* out_dur, int32_t* out_status, int32_t* out_accepted, void* stream);

/*
 * Best chain: smallest key among the chains with status >= 0, lowest index among equals.
 *   out_seq    DEVICE, C*n ints, receives its sequence; may be NULL.
 *   out_best   DEVICE, 6 int64: chain index (-1 when no chain is valid; the next four are then
 *              0, -1, -1, -2), length, peak, duration, status, and the number of proposals
 *              accepted so far over all chains.
 * Asynchronous on `stream`.
 */
int moc_search_best(const moc_search* s, int32_t* out_seq, int64_t* out_best, void* stream);

/* Facts about a search handle (any pointer may be NULL): number of chains, ints per exported row,
 * generations enqueued so far. */
int moc_search_info(const moc_search* s, int32_t* P, int32_t* stride, uint32_t* generation);

/* Frees the handle and its device memory; NULL is accepted.  Synchronise its streams first. */
void moc_search_destroy(moc_search* s);

/*
 * Launch shape override for moc_eval_batch, for tuning.  threads_per_sequence is the number of
 * threads that cooperate on one sequence (32, 64, 128, 256, 512 or 1024; 0 = choose from the
 * graph size), sequences_per_block how many sequences one thread block works on at a time
 * (0 = choose).  Results never depend on it.  MOC_ERR_ARG for unsupported values.
 */
int moc_graph_set_launch(moc_graph* g, int32_t threads_per_sequence, int32_t sequences_per_block);

/*
 * Which evaluation kernel moc_eval_batch uses, and in what shape.  The library has three families
 * for the operation of Section 2 (Eqs. 1-8) -- four with the packed variant for up to four copies --;
 * all give the same results, and MOC_KERNEL_AUTO (the
 * default) picks the fastest one that can serve the graph.  The call exists so that tests can
 * compare every family with the oracle and so that launch shapes can be measured.
 *   MOC_KERNEL_AUTO   a = b = 0.
 *   MOC_KERNEL_GROUP  a group of a threads (0, 32 .. 1024) per sequence, b sequences per block
 *                     (0 = choose); any C <= MOC_MAX_COPIES.  Same as moc_graph_set_launch(a, b).
 *   MOC_KERNEL_WARP   one warp per sequence, b warps per block (0 or 4..16), a = 0; C <= 2.
 *   MOC_KERNEL_LANE   one sequence per lane: a block keeps a group of a sequences (0, 8, 16, 32)
 *                     on chip and its b warps (0, 8, 16, 24 or 32; a multiple of a) share the work on them;
 *                     C <= 2 and a graph whose state for a group fits in shared memory.
 *   MOC_KERNEL_BLOCK  one block of a threads (0, or a multiple of 32 in 64..1024) per sequence with
 *                     the copies of a node packed into one 64-bit word, b = 0; C <= 4 and sequences
 *                     of at most 32766 steps whose state fits in shared memory.
 * MOC_ERR_ARG for an unknown kind or shape; a kind that cannot serve the graph with its current C
 * is reported by the next moc_eval_batch (MOC_ERR_ARG), which evaluates nothing.
 */
#define MOC_KERNEL_AUTO 0
#define MOC_KERNEL_GROUP 1
#define MOC_KERNEL_WARP 2
#define MOC_KERNEL_LANE 3
#define MOC_KERNEL_BLOCK 4
int moc_graph_set_kernel(moc_graph* g, int32_t kind, int32_t a, int32_t b);

/*
 * Measurement hook: while set, every moc_eval_batch on this handle records `before` right before
 * and `after` right after its evaluation kernel (the dominant kernel; the offsets kernel lies
 * outside the pair), on the stream of the call.  Both are cudaEvent_t created by the caller with
 * timing enabled; pass NULL, NULL to switch the hook off.  The caller reads the elapsed time after
 * synchronising.  Costs two event records per call, so leave it off outside of measurements.
 */
int moc_graph_set_timing_events(moc_graph* g, void* before, void* after);

/* Number of kernels the most recent moc_eval_batch / moc_mem_profile / moc_search_run on this
 * thread launched. */
int moc_last_launch_count(void);

/* Text of the most recent error on the calling thread ("" if none). Owned by the library. */
const char* moc_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* MOC_H_ */

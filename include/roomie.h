/*
 * roomie.h - C ABI of the B200 (sm_100a) implementation of Roomie's occupancy-based
 * kernel-interference model and placement rule.
 *
 * The library evaluates, in batch and on the GPU, the analytical model of
 * "Roomie: Interference-Aware Colocation for Efficient Model Serving":
 *   - per-kernel theoretical occupancy (Section 3.1, Eq. 1),
 *   - the pairwise interference walk over two models' kernel sequences with its
 *     alignment set, median and overlap factor (Section 3.2, Eq. 2, Eq. 4; Algorithm 1),
 *   - the greedy pairwise-sum multi-model estimate (Algorithm 1, outer loops),
 *   - argmin placement under a degradation budget (Section 3.4, Algorithm 2).
 *
 * General conventions
 *   - Every data pointer is a DEVICE pointer owned by the caller unless its comment says
 *     "host".  The library never allocates or frees device memory and keeps no pointer after a
 *     call returns; scratch space is passed in as `workspace`.  Two documented exceptions:
 *     roomie_pair_interference_static works in a fixed array inside the library image instead
 *     of a workspace, and roomie_profile_enable creates CUDA events (host-side objects).  On the
 *     host, the size arithmetic of the pair calls keeps two small per-thread vectors.
 *   - Calls only enqueue work on `stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) and return without synchronising, except where a comment says otherwise.
 *   - Return value: ROOMIE_OK or a negative roomie_status.  Data-dependent conditions
 *     (a timeline too long for 31-bit ticks, a negative duration) cannot be seen by the host
 *     at enqueue time: kernels record them as sticky bits in the library's `status` word,
 *     which the caller reads after synchronising (see ROOMIE_FLAG_*).
 *   - No call is re-entrant on the same workspace: two calls that share a workspace must be
 *     ordered on the GPU (same stream or an event dependency).
 */
#ifndef ROOMIE_H
#define ROOMIE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ROOMIE_OK = 0,
    ROOMIE_ERR_INVALID_ARG = -1, /* NULL pointer, size 0 where not allowed, index out of range   */
    ROOMIE_ERR_RANGE = -2,       /* a GPU-spec field does not fit the packed demand record       */
    ROOMIE_ERR_CUDA = -3,        /* a CUDA runtime call failed; see roomie_last_cuda_error()     */
    ROOMIE_ERR_CAPACITY = -4     /* workspace too small, or more alignments than supported       */
} roomie_status;

/* sticky bits of roomie_library.status (device word) */
#define ROOMIE_FLAG_TICK_OVERFLOW 1u /* a profile's timeline reached 2^31 ticks (1 tick = 1 ns) */
#define ROOMIE_FLAG_BAD_TIME 2u      /* a duration or gap was negative, NaN or >= 2^31 ns       */
#define ROOMIE_FLAG_WORKSPACE 4u     /* internal: a kernel ran out of planned workspace        */
#define ROOMIE_FLAG_WAIT_TIMEOUT 8u  /* internal: a bounded wait on an asynchronous copy expired */

/* Per-SM limits of the MODELLED GPU (Section 3.1: warp capacity W, registers, shared memory;
 * the block-slot limit and the SM count complete the launch model).
 * Limits of the packed record: threads_per_sm/32 <= 255, blocks_per_sm <= 255,
 * regs_per_sm < 2^18, smem_per_sm < 2^20; num_sms >= 1.  Otherwise ROOMIE_ERR_RANGE. */
typedef struct roomie_gpu_spec {
    uint32_t num_sms;
    uint32_t regs_per_sm;
    uint32_t smem_per_sm;    /* bytes */
    uint32_t threads_per_sm;
    uint32_t blocks_per_sm;
} roomie_gpu_spec;

/* Struct-of-arrays kernel table: the launch configuration of n kernels (all profiles
 * concatenated).  dim3 grids/blocks are flattened to element counts by the caller. */
typedef struct roomie_kernel_table {
    uint32_t n;
    const uint32_t *grid_blocks;     /* [n] blocks in the grid          */
    const uint32_t *block_threads;   /* [n] threads per block           */
    const uint32_t *regs_per_thread; /* [n] 0 = no register limit       */
    const uint32_t *smem_per_block;  /* [n] bytes, 0 = no smem limit    */
} roomie_kernel_table;

/* Outputs of roomie_occupancy; any pointer may be NULL to skip that output. */
typedef struct roomie_occ_out {
    uint32_t *packed4;        /* [n] bytes {b_lim, b_res, limiter, warps} = bits 0-7, 8-15, 16-23, 24-31 */
    float *occ;               /* [n] Eq. 1 at the resident block count: warps / W                  */
    float *occ_theo;          /* [n] Eq. 1 with the grid ignored: W_b * b_lim / W                  */
    uint32_t *phi;            /* [4][n] per-SM demand: warps, registers, smem bytes, block slots   */
    uint32_t *n_unlaunchable; /* [1] kernels whose single block exceeds the SM (b_lim = 0); the
                                 call ADDS to this word, zero it first                            */
} roomie_occ_out;

/* Section 3.1, Eq. 1.  For every kernel: warps per block W_b = ceil(threads/32); block limits
 * floor(W/W_b) (warps), blocks_per_sm (slots), floor(R/(regs*32*W_b)) (registers),
 * floor(S/smem) (shared memory); b_lim = their minimum, limiter = 0 warps / 1 slots /
 * 2 registers / 3 shared memory (first minimum in that order); resident blocks
 * b_res = min(b_lim, ceil(grid/num_sms)), limiter 4 when the grid is the stricter bound;
 * o = W_b * b_res / W as one float32 division.  A kernel with b_lim = 0 gets o = 0. */
int roomie_occupancy(const roomie_kernel_table *table /* host struct of device arrays */,
                     const roomie_gpu_spec *spec /* host */, const roomie_occ_out *out /* host struct */,
                     void *stream);

/* Which kernel roomie_occupancy launches for these arguments (host arithmetic on the pointer values and
 * n only; nothing is dereferenced, no CUDA call is made; the paper has no counterpart).  Arrays need only
 * their elements' own 4-byte alignment: bit 0 of the result is set when the 128-bit kernel is used, which
 * takes n >= 4 and every input column and every packed4 / occ / occ_theo output (NULL counts as aligned) on
 * a 16-byte boundary; bits 4-7 tell which of the four rows of phi (row c starts at phi + c*n) take 128-bit
 * stores there.  0 = the scalar kernel.  Negative: ROOMIE_ERR_INVALID_ARG (NULL struct). */
int roomie_occupancy_variant(const roomie_kernel_table *table /* host */, const roomie_occ_out *out /* host */);

/* A kernel library prepared for the interference walk.  The caller allocates every array and
 * fills the struct (host memory); roomie_library_build writes the device arrays.
 * Record layout (16 bytes per kernel, the unit the walk streams):
 *   u32 start tick, u32 end tick (start + duration), u64 packed per-SM demand phi
 *   (bits 0-19 registers, 20-29 warps, 32-53 shared-memory bytes, 54-63 block slots; the top
 *   bit of every field is a zero guard bit). */
typedef struct roomie_library {
    uint32_t num_profiles;        /* P                                                           */
    uint32_t num_kernels;         /* K = offsets_host[P]                                         */
    const uint32_t *offsets_host; /* host [P+1] first kernel of each profile; must stay valid
                                     while the struct is in use                                   */
    uint32_t *offsets;            /* device [P+1]                                                */
    void *records;                /* device [K] x 16 bytes, 16-byte aligned                      */
    uint64_t *T;                  /* device [P] isolated inference time = sum of kernel ticks     */
    uint32_t *status;             /* device [1] sticky ROOMIE_FLAG_* bits; zero it before build   */
    roomie_gpu_spec spec;
} roomie_library;

/* The occupancy share o_i/(o_i+o_j) of Algorithm 1 line 13 is evaluated from the resident warps of
 * the two kernels (W cancels): a charged delay is (ticks * (1/(warps_i + warps_j))) * warps_i in
 * float32, the reciprocal to one unit in the last place. */

/* Builds the library from a kernel table plus isolated durations and inter-kernel gaps
 * (microseconds, float32, device arrays [K]).  Times become integer ticks of 1 ns:
 * max(1, rint(d*1000)) and rint(g*1000), float32 product, round-half-even.  Kernel k of a
 * profile starts at the sum of the durations and gaps before it (Section 3.2: a model is a
 * sequence of kernels).  Copies offsets_host to the device (synchronous for pageable memory).
 * Errors: INVALID_ARG, RANGE (spec), CUDA.  Overflow of 31-bit ticks and bad time values set
 * status bits. */
int roomie_library_build(const roomie_library *lib /* host */, const roomie_kernel_table *table /* host */,
                         const float *dur_us, const float *gap_us, void *stream);

/* Options of the pairwise walk and of placement. */
#define ROOMIE_WALK_TIMELINE 0 /* event-driven: the kernel that ends first is replaced (Section 3.2);
                                  only the time both kernels overlap is charged                  */
#define ROOMIE_WALK_LOCKSTEP 1 /* Algorithm 1 as printed: both indices advance together, the whole
                                  duration d_k is charged                                        */
/* Section 3.2 in full instead of Algorithm 1's closed-form delay: adjusted occupancy (a kernel that
 * shares the SM runs with the blocks b~ the partition policy leaves it, at the rate o~/o = b~/b),
 * two-phase execution (interference ends when the first of the two kernels completes), stretched
 * timelines.  One value per partition policy the paper names:
 *   EQUAL    each of the two kernels may use half of every SM resource;
 *   PRIORITY the kernel of the pair's first model keeps its blocks, the other gets the remainder;
 *   FCFS     the same with priority to the kernel that started earlier (first model on a tie).
 * Time is in whole ticks here too: the work of a kernel is d_k * b block-ticks, a kernel running with
 * b~ blocks does b~ of them per tick and completes after ceil(work left / b~) ticks, and a tick spent
 * with b~ of b blocks delays it by (b - b~)/b; so which kernel completes first, and which started
 * earlier, never depends on rounding.
 * The alignment set, median, gamma and /T are applied as for the other modes; V is 0 and `evals`
 * counts simulation events (a gap ends or a kernel completes).  With PRIORITY, P[a][b] and P[b][a] of
 * an unordered pair both come from the walk in which the lower-numbered profile has priority. */
#define ROOMIE_WALK_DETAILED_EQUAL 2
#define ROOMIE_WALK_DETAILED_PRIORITY 3
#define ROOMIE_WALK_DETAILED_FCFS 4
typedef struct roomie_opts {
    int32_t walk_mode;      /* ROOMIE_WALK_*                                                      */
    uint32_t n_align;       /* A: alignment set = A x A evenly spaced start indices floor(t*q/A);
                               0 = the full Cartesian product q_i x q_j.  With ROOMIE_WALK_LOCKSTEP
                               that is Algorithm 1 exactly as printed and is served for any profile
                               length (all alignments of a pair are suffix sums along the diagonals
                               of one q_i x q_j table, exact median by radix select); with
                               ROOMIE_WALK_TIMELINE, or when per-alignment detail is requested,
                               at most 4096 alignments per pair                                  */
    int32_t start_filter;   /* 1: keep only alignments whose two start kernels interfere (Eq. 2) */
    float lambda;           /* degradation budget of Algorithm 2 (the paper uses 0.5)            */
    uint32_t max_residents; /* placement calls: 0, or the slot count of the cluster state they are
                               given (anything else is ROOMIE_ERR_INVALID_ARG); the state's own
                               max_residents is what counts                                       */
    int32_t admit_rule;     /* ROOMIE_ADMIT_*: which quantity must stay below lambda             */
    int32_t objective;      /* ROOMIE_OBJECTIVE_*: which quantity the chosen GPU minimises       */
} roomie_opts;
/* Algorithm 2 as printed admits a GPU when the MEAN drop of its would-be model set is below lambda
 * and picks the lowest mean.  Its comment asks that "no variant has a performance drop beyond
 * lambda" (ADMIT_MAX: the largest member drop), and Section 3.4 notes that the objective can be
 * substituted: OBJECTIVE_MAX picks the GPU whose worst-hit member suffers least, OBJECTIVE_ARRIVAL
 * the GPU on which the arriving model itself suffers least.  Ties go to the lowest GPU index. */
#define ROOMIE_ADMIT_MEAN 0
#define ROOMIE_ADMIT_MAX 1
#define ROOMIE_OBJECTIVE_MEAN 0
#define ROOMIE_OBJECTIVE_MAX 1
#define ROOMIE_OBJECTIVE_ARRIVAL 2

/* Unordered profile pairs (a <= b, diagonal included) are numbered row-major over the upper
 * triangle: (0,0), (0,1), ..., (0,P-1), (1,1), ...; there are P(P+1)/2 of them. */

/* Bytes of workspace that let roomie_pair_matrix process pairs [pair_begin, pair_end) in one
 * batch (a smaller workspace makes it split the range).  0 on invalid arguments.
 * For ROOMIE_WALK_LOCKSTEP with n_align = 0 the workspace is optional help, not a need: it holds
 * the counter a persistent grid takes its pairs from and per-CTA lists of candidate values that
 * save the exact median one of its three passes over a pair's table; the figure returned is what
 * lets the library's largest tables use the lists (at most about 1.2 GB), any size >= 256 bytes
 * is accepted and gives the same bits. */
size_t roomie_pair_workspace_bytes(const roomie_library *lib /* host */, const roomie_opts *opts /* host */,
                                   uint64_t pair_begin, uint64_t pair_end);

/* Algorithm 1 lines 6-20 for every unordered pair in [pair_begin, pair_end): for each
 * alignment (s_i, s_j) of the alignment set the walk accumulates the delay
 *   delta_i += overlap * o_i/(o_i+o_j)   whenever phi_i + phi_j > Phi in any resource (Eq. 2),
 * then  P[i][j] = max(q_i/q_j, 1) * median(delta_i) / T_i  (relative slowdown of i caused by j,
 * Eq. 4 for M = {i, j}), and P[j][i] from the same walks.  Median of an even count is the
 * mean of the two middle values; an empty alignment set gives 0.
 *   P_out      [P*P] row-major float32; only entries of the requested pairs are written.
 *   evals_out  optional [1]: set to the number of kernel pairings scored by this call.
 *   workspace  device scratch, 256-byte aligned, any size >= the need of the largest single
 *              pair; contents are undefined afterwards.
 * Errors: INVALID_ARG, CAPACITY (workspace cannot hold one pair; more than 4096 alignments
 * per pair), CUDA. */
int roomie_pair_matrix(const roomie_library *lib /* host */, const roomie_opts *opts /* host */,
                       uint64_t pair_begin, uint64_t pair_end, float *P_out, uint64_t *evals_out,
                       void *workspace, size_t workspace_bytes, void *stream);

/* Per-alignment detail of one pair (all device arrays of `capacity` entries, any may be NULL).
 * Kept alignments are listed in alignment-set order (s_i major, s_j minor). */
typedef struct roomie_pair_detail {
    uint32_t capacity;
    uint32_t *n_kept;  /* [1] number of alignments kept (may exceed capacity)       */
    uint32_t *s_i;     /* start index in profile a                                   */
    uint32_t *s_j;     /* start index in profile b                                   */
    float *delta_i;    /* accumulated delay of a, ticks                              */
    float *delta_j;    /* accumulated delay of b, ticks                              */
    uint64_t *V;       /* TIMELINE: ticks of interfering overlap (= delta_i+delta_j);
                          LOCKSTEP: summed durations of both kernels of interfering pairings */
    uint32_t *evals;   /* pairings scored by the walk                                */
} roomie_pair_detail;

/* Bytes of workspace roomie_pair_interference needs for the pair (a, b) under `opts` (with or
 * without detail).  0 on invalid arguments or when the pair has more than 4096 alignments. */
size_t roomie_pair_interference_workspace_bytes(const roomie_library *lib /* host */, uint32_t a, uint32_t b,
                                                const roomie_opts *opts /* host */);

/* The same computation for ONE ordered pair (a, b), any order, a == b allowed:
 * out2[0] = P[a][b], out2[1] = P[b][a].  `detail` (host struct) may be NULL.  `workspace`: device,
 * 256-byte aligned, at least roomie_pair_interference_workspace_bytes(lib, a, b, opts) bytes
 * (ROOMIE_ERR_CAPACITY otherwise). */
int roomie_pair_interference(const roomie_library *lib /* host */, uint32_t a, uint32_t b,
                             const roomie_opts *opts /* host */, float *out2, uint64_t *evals_out,
                             const roomie_pair_detail *detail, void *workspace, size_t workspace_bytes,
                             void *stream);

/* roomie_pair_interference without a workspace argument (the paper has no counterpart: this is
 * a deployment aid).  It is meant for callers that cannot obtain device memory of their own:
 * a placement controller living beside an inference runtime whose allocator already owns the
 * whole device, a plug-in that is handed raw device pointers but no allocator, or a service
 * loop in which a cudaMalloc would stall every stream of the device.  The scratch the walk
 * needs lives in a fixed array of ROOMIE_STATIC_SCRATCH_BYTES inside the library image; every
 * GPU that loads the library holds that array until the process exits.  Inputs and outputs are
 * still the caller's.  The call allocates nothing: no cudaMalloc, no cudaFree, no allocating
 * library routine.
 *   - Same arguments, results and errors as roomie_pair_interference; a pair whose scratch need
 *     exceeds the array (very long profiles combined with many alignments) is refused with
 *     ROOMIE_ERR_CAPACITY and nothing is enqueued.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress,
 *     with that device current) and remembers it; make that first call during start-up, before
 *     any stream capture begins.
 *   - All calls on a device share the one array.  Each call clears what it needs cleared, so
 *     calls issued one after the other on a stream are independent, but two calls whose GPU
 *     work overlaps (different streams without an ordering between them, or different host
 *     threads) race on the array and give wrong results: serialise them. */
#define ROOMIE_STATIC_SCRATCH_BYTES (1u << 20)
int roomie_pair_interference_static(const roomie_library *lib /* host */, uint32_t a, uint32_t b,
                                    const roomie_opts *opts /* host */, float *out2, uint64_t *evals_out,
                                    const roomie_pair_detail *detail, void *stream);

/* Algorithm 1, outer loops, given the pairwise terms (performance_drop(M)), batched over
 * n_sets independent model sets.  Set s is M = resident_ids[s*max_residents + 0..count[s])
 * followed by incoming[s] (profile ids, duplicates allowed = replicas).
 *   mu_out   [n_sets * (max_residents+1)]: mu_i = sum over the OTHER members j, in slot order with
 *            the incoming model last, of Pmat[id_i][id_j]; float32 additions in exactly that order.
 *            Slot count[s] holds the incoming model's mu; later slots are left untouched.
 *   mean_out [n_sets]: (sum of mu_i in slot order) / |M|.
 * Either output may be NULL.  Errors: INVALID_ARG (max_residents > 64), CUDA. */
int roomie_multi_estimate(const float *Pmat, uint32_t P, const int32_t *resident_ids,
                          const uint32_t *count, const int32_t *incoming, uint32_t n_sets,
                          uint32_t max_residents, float *mu_out, float *mean_out, void *stream);

/* Cluster state, updated in place by roomie_place (host struct of device arrays). */
typedef struct roomie_cluster_state {
    uint32_t num_gpus;      /* G <= 1024                                                     */
    uint32_t max_residents; /* R <= 64 slots per GPU, and G * R <= 8192 (the state of one
                               stream lives in one SM's shared memory)                       */
    int32_t *ids;           /* [G*R] profile id per slot, residents packed first, -1 = free  */
    uint32_t *expiry;       /* [G*R] arrival tick at which the resident leaves, 0 = never    */
    uint32_t *count;        /* [G] residents per GPU                                         */
    uint32_t *tick;         /* [1] arrivals processed so far                                 */
} roomie_cluster_state;

/* Algorithm 2 applied to a stream of n arrivals, in order.  For arrival k (tick = *tick + k):
 * residents whose expiry tick is <= tick leave (order kept); every GPU with a free slot is
 * scored what-if by the multi-model estimate with the arrival added; a GPU is admissible
 * when its mean drop is < lambda; the admissible GPU with the lowest mean is chosen, the
 * lowest index on ties; with no admissible GPU the arrival is deferred (-1) and not added.
 * A placed model gets expiry tick + lifetime (lifetime 0 = never leaves).
 *   arr_id [n] profile ids, arr_life [n] lifetimes in arrival ticks;
 *   gpu_out [n]; mean_out [n] (optional) mean drop of the chosen GPU; mu_arr_out [n]
 *   (optional) predicted drop of the arriving model there.
 * Decisions are taken in float32 with the fixed summation order of roomie_multi_estimate;
 * opts->admit_rule and opts->objective select the variants described at roomie_opts.
 * Profile ids are checked on the device, where they live: an arrival whose id is outside [0, P) is
 * not placed and gets gpu_out = ROOMIE_PLACE_BAD_ID (the state is left as it was); a cluster state
 * that holds such an id among its residents makes every arrival of the call come back that way.
 * Errors: INVALID_ARG (shape limits above, unknown rule or objective, opts->max_residents that
 * contradicts the state), CUDA. */
#define ROOMIE_PLACE_BAD_ID (-2)
int roomie_place(const float *Pmat, uint32_t P, const roomie_cluster_state *state /* host struct */,
                 const int32_t *arr_id, const uint32_t *arr_life, uint32_t n, const roomie_opts *opts /* host */,
                 int32_t *gpu_out, float *mean_out, float *mu_arr_out, void *stream);

/* roomie_place for num_streams INDEPENDENT arrival streams at once (what-if scenarios, one
 * cluster per tenant, placement-quality studies): one CTA per stream, so streams run side by
 * side where a single stream is a dependent chain.  Every per-stream array is the single-stream
 * array repeated num_streams times, stream-major: states->ids and ->expiry [S][G*R], ->count
 * [S][G], ->tick [S]; arr_id, arr_life and the outputs [S][n].  All streams share Pmat, the
 * cluster shape, n and the options.  Same decisions as num_streams calls of roomie_place. */
int roomie_place_batch(const float *Pmat, uint32_t P, const roomie_cluster_state *states /* host struct */,
                       const int32_t *arr_id, const uint32_t *arr_life, uint32_t n, uint32_t num_streams,
                       const roomie_opts *opts /* host */, int32_t *gpu_out, float *mean_out, float *mu_arr_out,
                       void *stream);

/* Placement quality (Section 5, "Deployment accuracy evaluation against optimal strategies"): for each of
 * num_scenarios model lists, the deployment of its n models on num_gpus identical GPUs, at most
 * max_residents per GPU, with the lowest average predicted drop - found by trying every assignment
 * (model 0 fixed on GPU 0).  With the pairwise-sum estimate of Algorithm 1 the average drop is
 *     cost = ( sum over i < j on the same GPU of (Pmat[m_i][m_j] + Pmat[m_j][m_i]) ) / n,
 * evaluated in float32: one add per pair term, terms accumulated model by model (j ascending, its
 * partners i < j ascending), one division.
 *   models      [S][n] profile ids (duplicates = replicas)
 *   best_cost   [S] lowest cost, -1 when n > num_gpus * max_residents
 *   best_assign [S][n] optional: GPU of every model in the optimal deployment that comes first in
 *               lexicographic order of (GPU of model 1, GPU of model 2, ...)
 *   workspace   roomie_optimal_workspace_bytes(S) bytes of device scratch
 * Limits: n <= 16, num_gpus <= 15, max_residents <= 15, num_gpus^(n-1) <= 2^32, S <= 65535
 * (INVALID_ARG / CAPACITY otherwise). */
size_t roomie_optimal_workspace_bytes(uint32_t num_scenarios);
int roomie_optimal_assignment(const float *Pmat, uint32_t P, const int32_t *models, uint32_t n,
                              uint32_t num_scenarios, uint32_t num_gpus, uint32_t max_residents,
                              float *best_cost, int32_t *best_assign, void *workspace, size_t workspace_bytes,
                              void *stream);

/* The same cost for GIVEN deployments (e.g. the one Algorithm 2 arrived at): gpu_of [S][n], a negative
 * entry = model not deployed (it takes part in no term but still counts in n). */
int roomie_assignment_cost(const float *Pmat, uint32_t P, const int32_t *models, const int32_t *gpu_of,
                           uint32_t n, uint32_t num_scenarios, float *cost_out, void *stream);

/* Text of a roomie_status; the last CUDA error code/text seen by this thread's calls. */
const char *roomie_strerror(int status);
const char *roomie_last_cuda_error(void);

/* Launch statistics of the calling thread since the last reset: kernels launched by this
 * library (used by benchmarks to report launches per step). */
uint64_t roomie_launch_count(void);
void roomie_reset_launch_count(void);

/* Self-test of the library's bounded waits (the paper has no counterpart).  The pairwise walk stages its
 * tiles with asynchronous copies and waits for them on a barrier, with a time limit; a wait that runs out
 * sets ROOMIE_FLAG_WAIT_TIMEOUT in the library's status word and ends the CTA instead of hanging the GPU.
 * This call launches one CTA that waits, with `limit_ns` (1 .. 1e9) as the limit, for a copy that is never
 * issued: afterwards *status (device word, e.g. roomie_library.status or a word of the caller's) has
 * ROOMIE_FLAG_WAIT_TIMEOUT set and the context is still usable.  Errors: INVALID_ARG, CUDA. */
int roomie_selftest_bounded_wait(uint32_t *status /* device */, uint64_t limit_ns, void *stream);

/* Measurement aid (the paper has no counterpart).  While enabled, the calling thread's pair
 * calls bracket every launch of the pairwise walk kernel with a pair of CUDA events recorded on
 * the call's stream (at most 256 pairs are kept; later launches are not recorded).
 * roomie_profile_walk_ms synchronises on the recorded events, returns their summed elapsed time in
 * milliseconds and the number of launches through the pointers (host), and forgets them.
 * Enabling allocates the events (host-side objects only); disabling destroys them. */
int roomie_profile_enable(int on);
int roomie_profile_walk_ms(float *total_ms /* host */, uint32_t *launches /* host */);

#ifdef __cplusplus
}
#endif
#endif /* ROOMIE_H */

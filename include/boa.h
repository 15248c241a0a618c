/*
 * boa.h -- C interface of the B200 (sm_100a) library for batched, beamwidth-adaptive,
 * range-filtered graph beam search (BOA / BOA+).
 *
 * All functions are extern "C", take plain pointers and sizes, return an int
 * status (BOA_OK == 0, negative == error), never throw, abort or print.  Unless a
 * parameter says "host", a pointer is a DEVICE pointer on the current CUDA
 * device and must be 16-byte aligned.  The caller owns every buffer it passes.
 * `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 */
#ifndef BOA_H
#define BOA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct boa_index boa_index; /* opaque */

enum { BOA_F32 = 0, BOA_U8 = 1 };            /* element type of the stored vectors      */
enum { BOA_ATTR_I32 = 0, BOA_ATTR_F32 = 1,   /* cell type of one attribute column       */
       BOA_ATTR_SET32 = 2 };                 /* 32-bit membership mask (see boa_search)  */
enum { BOA_METRIC_L2 = 0, BOA_METRIC_COSINE = 1 }; /* distance of the search             */

enum {
    BOA_OK = 0,
    BOA_EINVAL = -1, /* bad argument (null, range, alignment, unsupported shape) */
    BOA_ENOMEM = -2, /* device or host allocation failed                         */
    BOA_ECUDA = -3,  /* a CUDA call failed; boa_last_cuda_error() has its code   */
    BOA_EGRAPH = -4, /* the graph names a node id >= N                           */
    BOA_ETOOBIG = -5 /* boa_search_noalloc: Q or Lmax beyond its fixed scratch   */
};

#define BOA_NO_ID 0xFFFFFFFFu /* "no edge" in graph rows, "no result" in out_ids */
#define BOA_MAX_ATTRS 8
#define BOA_MAX_DEGREE 64
#define BOA_MAX_WIDTH 1024 /* largest beamwidth / pool capacity */
#define BOA_MAX_PHASES 8
#define BOA_MAX_POINTS ((int64_t)1 << 28)
#define BOA_PQ_MAX_SUBSPACES 64 /* largest M of a product-quantisation codebook */
#define BOA_PQ_MAX_K 32         /* largest k of a search that traverses on PQ distances */

/* Keys of boa_set_param. */
enum {
    BOA_PARAM_EPS = 0,      /* confidence threshold eps of Eq. 3; default 0.05               */
    BOA_PARAM_GROWTH = 1,   /* alpha of Algorithm 1: width of phase p+1 = min(Lmax, alpha*w_p); default 4 */
    BOA_PARAM_TAU = 2,      /* residual fraction tau of Algorithm 1; default 0                */
    BOA_PARAM_MODE = 3,     /* 0 = restart every phase from the entry point (Algorithm 1 as
                               printed), 1 = resume: later phases continue from the pool the
                               earlier ones built (the "redundancy avoidance" paragraph)      */
    BOA_PARAM_PLUS_K = 4,   /* 0 or 1 = BOA; K >= 2 = BOA+: the first phase is issued as K
                               sub-batches and wider phases overlap them ("Pipelining
                               Multiple Batches").  The sub-batches run one after another,
                               so K is capped by BOA_PARAM_PLUS_MIN_SUB                      */
    BOA_PARAM_CAP_MULT = 5, /* a phase at width L gives up after CAP_MULT*L + CAP_ADD        */
    BOA_PARAM_CAP_ADD = 6,  /*   expansions; defaults 8 and 64                               */
    BOA_PARAM_TABLE_KB = 7, /* 0 = default (6 or 4, whichever keeps 20 query warps per SM
                               within 196 KB of shared memory; 1 with PQ traversal, where the
                               distance table decides how many warps fit and a node scored
                               twice costs little); else KB of shared memory
                               per query for the table of recently scored ids: 1, 2, 3, 4,
                               6, 8, 12, 16 or 24 (doubled automatically while an index of
                               more than 2^25 points needs tags wider than 16 bits).  Never
                               changes results.                                              */
    BOA_PARAM_MAX_WARPS_PER_SM = 8, /* 0 = as many query warps per SM as fit; else a cap.
                               Never changes results.                                        */
    BOA_PARAM_TABLE_TAGS = 10, /* 0 (default) = the table keeps 10-bit tags, three to a 4-byte
                               bucket, when the index is small enough for that (up to 2^20
                               points with the default 4 KB), else 16-bit tags, four to an
                               8-byte bucket; 16 = always the latter.  Never changes
                               results.                                                      */
    BOA_PARAM_LAMBDA = 11,  /* weight lambda of the filter penalty in the score the search
                               orders by, dist + lambda*phi ("Graph construction" paragraph;
                               phi = number of violated predicates).  Default +infinity: any
                               violated predicate outweighs any distance, keys order by
                               (phi, d^2, id).  A finite value >= 0 orders by the score
                               d^2 + lambda*phi (squared distance, one fp32 fused
                               multiply-add), ties by id.  Answers are filter-valid either
                               way; a finite lambda lets invalid nodes push valid ones out
                               of the pool.                                                  */
    BOA_PARAM_PQ = 12,      /* 1 = traverse on product-quantised distances (needs
                               boa_index_attach_pq) and rank the filter-valid beam entries by
                               exact distance when a phase has converged: Algorithm 2's PQDist
                               line and the "Re-rank exact" step of Section "BOA Implementation
                               on a GPU System".  0 (default) = exact distances throughout.
                               With 1, k <= BOA_PQ_MAX_K and BOA_PARAM_EXPAND_W must be 1.     */
    BOA_PARAM_CHAINS = 15,  /* 2: the two halves of the batch go through all their phases
                               independently, one on the caller's stream and one on a stream of
                               the index, joined before `stream` goes on: the launches of one
                               half fill the GPU while the last, partly empty wave of the other
                               half's phase drains (the observation of "Pipelining Multiple
                               Batches": phases of different queries do not depend on each
                               other).  1: the batch goes through its phases as one, the
                               schedule of Algorithm 1 as printed.  0 (default): 2 while the
                               widest phase is at most 128, else 1.  Same results in every
                               case.  Two chains need BOA+ off, tau = 0 and more than one
                               phase.                                                        */
    BOA_PARAM_PLUS_MIN_SUB = 14, /* BOA+: the fewest queries a sub-batch may hold; K is lowered
                               (down to plain BOA) until Q / K reaches it.  0 (default) = twice
                               the queries the GPU searches at once (2 x 20 x SM count); 1 =
                               always K sub-batches.                                         */
    BOA_PARAM_HOST_IN_PLACE = 13, /* boa_search_host only.  1 (default): buffers in page-locked host
                               memory that the device can address are read and written in
                               place by the search kernels; 0: always staged through device
                               copies.  Results are the same either way.                     */
    BOA_PARAM_EXPAND_W = 9  /* nodes expanded per iteration of Algorithm 2.  1 (default) is
                               the algorithm as printed (one node per iteration, Section
                               "How Filtered Search Works").  2 is an extension: the first
                               two unexpanded beam
                               entries are marked and their rows scored together (first
                               node's row first), at most as many as the expansion cap
                               leaves.  Changes which nodes get expanded, hence results.  */
};

/*
 * Build a search index (problem statement of the paper's Background section: points
 * p = (x_p, a_p) with m numeric attributes, and a proximity graph of out-degree <= R).
 *
 *   vectors     [N][D] row-major, float (BOA_F32) or uint8_t (BOA_U8); D % 4 == 0 for
 *               floats, D % 16 == 0 for bytes; values must be finite
 *   attrs       [N][m] row-major 4-byte cells; column j is int32 or float per attr_types[j]
 *   attr_types  HOST array [m]
 *   graph       [N][R] node ids, BOA_NO_ID pads short rows; self references and
 *               repeated ids inside a row are tolerated (ignored by the search)
 *   entry       start node s of every search (the entry medoid of Algorithm 2); -1 = the
 *               point nearest to the coordinate-wise mean, lower id on ties
 *
 * The index copies and re-lays-out everything into device memory it owns, so the
 * inputs may be freed when the call returns.  The call synchronises `stream`.
 * Errors: BOA_EINVAL (nulls, N < 1, N > BOA_MAX_POINTS, m outside 1..8, R outside 1..64,
 * bad D, misaligned pointers, entry >= N), BOA_EGRAPH, BOA_ENOMEM, BOA_ECUDA.
 */
int boa_index_create(boa_index** out, const void* vectors, int vec_dtype, int64_t N, int D,
                     const void* attrs, const int* attr_types, int m, const uint32_t* graph, int R,
                     int64_t entry, void* stream);

/*
 * Build a proximity graph on the GPU (Background section, "Graph construction": Vamana
 * insertion -- a beam search over the graph built so far collects candidates for each new
 * point, a pruning step keeps at most R diverse out-neighbours by the alpha-dominance rule --
 * with the threshold pruning the paper adopts: the pruning runs once per attribute threshold,
 * each run with a degree budget of R/T and only over candidates whose attribute distance to
 * the point is within the threshold, so part of every row links attribute-near points.
 * Candidates come from one filter-aware search per threshold, filtered to that window).
 * Not part of the search hot path; its output is the `graph` argument of boa_index_create.
 *
 *   vectors     [N][D] as for boa_index_create
 *   attr_pos    [N][m_pos] float: where the point sits in each attribute (for instance its
 *               rank divided by N); the distance of two points in attribute j is the
 *               absolute difference of their positions
 *   R, Lb       out-degree and the beamwidth of the build's searches (Lb <= 128, T*Lb + R <= 256)
 *   alpha       dominance factor >= 1 on distances (applied squared to squared distances)
 *   thresholds  HOST array [T][m_pos], T <= 8: pass i admits the candidates whose distance in
 *               every attribute j is <= thresholds[i][j] (+infinity leaves the attribute
 *               free; a row of +infinity is the plain Vamana pass) and may add
 *               R*(i+1)/T - R*i/T neighbours
 *   B           largest batch; batches are [start, start+size) in index order with size =
 *               min(B, points inserted so far) (1, 1, 2, 4, ...); every point of a batch
 *               searches the graph as it stood before the batch
 *   passes      sweeps over all points (the second and later ones in batches of B)
 *   cap_in      reverse edges: at most this many requesters (lowest ids first) are
 *               considered per target and batch (<= 64)
 *   entry       start node of the build's searches, -1 = the medoid as in boa_index_create
 *   out_graph   [N][R] device; BOA_NO_ID pads
 *   n_batches   HOST, may be NULL
 *
 * Deterministic: the same inputs give the same graph.  Synchronises `stream`; allocates and
 * frees its own scratch (a search index over the vectors among it).
 * Errors: BOA_EINVAL (nulls, sizes out of range), BOA_ENOMEM, BOA_ECUDA.
 */
int boa_graph_build(const void* vectors, int vec_dtype, int64_t N, int D, const float* attr_pos, int m_pos,
                    int R, int Lb, float alpha, const float* thresholds, int T, int B, int passes,
                    int cap_in, int64_t entry, uint32_t* out_graph, int64_t* n_batches, void* stream);

/*
 * Give the index a product-quantisation codebook (Section "BOA Implementation on a GPU
 * System": PQ codes and quantisation pivots live in GPU memory; a query's distance table
 * holds the distance from each of its subvectors to every centroid of that subspace, and a
 * candidate's PQ distance is the sum of the table entries its code selects).
 *
 *   pivots  [M][K][D/M] float: centroid c of subspace m; subspace m covers dimensions
 *           [m*D/M, (m+1)*D/M) of the vectors
 *   codes   [N][M] uint8_t: index of the centroid that stands for point p in subspace m
 *
 * M a multiple of 16 in 16..BOA_PQ_MAX_SUBSPACES that divides D, 1 <= K <= 256.  The
 * codebook is trained by the caller; both arrays are copied into index-owned memory (the
 * call synchronises `stream`).  Attaching does not switch PQ traversal on: set BOA_PARAM_PQ.
 * The distance table costs M*K*4 bytes of shared memory per resident query.
 * Errors: BOA_EINVAL (nulls, bad M or K, misaligned pointers), BOA_ENOMEM, BOA_ECUDA.
 */
int boa_index_attach_pq(boa_index* index, const float* pivots, const uint8_t* codes, int M, int K,
                        void* stream);

/*
 * Choose the distance (Definition 1 allows the Euclidean norm or cosine distance; the paper
 * itself uses the Euclidean norm, which is the default here).  BOA_METRIC_COSINE: float
 * vectors only; the index rescales its copy of the vectors to unit length (in place, once:
 * going back is BOA_EINVAL), every search rescales a copy of its queries, and out_dists
 * holds cosine distances 1 - cos(x, q) (a zero vector has distance 0.5 to everything),
 * computed as half the squared Euclidean distance of the unit vectors.  The confidence test
 * of Eq. 3 then compares cosine distances.  The entry point stays the one chosen at
 * creation.  A PQ codebook attached to a cosine index must have been trained on unit-length
 * vectors.  boa_search_noalloc supports the Euclidean metric only.  Synchronises `stream`.
 */
int boa_index_set_metric(boa_index* index, int metric, void* stream);

/*
 * A second handle on the same index data, for searches that run at the same time as the
 * first handle's (the paper's "Pipelining Multiple Batches" carried to whole batches: while
 * the last, partly empty wave of one batch's wide phase drains, the narrow phase of the next
 * batch fills the GPU from another stream).  boa_search keeps its survivor lists, counters,
 * statistics and carried pools in its handle, so two searches in flight need two handles.
 * The new handle shares the vectors, attribute cells, graph and PQ codebook of `src` (no
 * copy), copies src's parameters, schedule and range-penalty scales as they stand, and owns
 * its own scratch (allocated on its first search), so it costs a few MB.
 *
 * Rules: `src` must be fully set up before (boa_index_attach_pq and boa_index_set_metric are
 * BOA_EINVAL on a shared handle, and calling them on `src` afterwards is not seen by, or
 * breaks, its shares) and must outlive every handle shared from it; each handle is used by
 * one search at a time, and `src` is not being searched by another thread while it is shared;
 * parameters set on one handle do not reach the other.
 * Errors: BOA_EINVAL, BOA_ENOMEM, BOA_ECUDA; *out is NULL then.
 */
int boa_index_share(boa_index** out, boa_index* src);

/* Free the index and everything it owns (a shared handle: its scratch only).  NULL is accepted. */
int boa_index_destroy(boa_index* index);

/* The start node the index uses (host value). */
int64_t boa_index_entry(const boa_index* index);

/*
 * Algorithm 1 (BOA) over one batch: every query is searched with Algorithm 2
 * (filter-aware beam search) at beamwidth L0; queries that fail the confidence test of
 * Eq. 3 are compacted and searched again at wider beamwidths up to Lmax.  L0 == Lmax is
 * the fixed-beamwidth baseline.
 *
 *   queries   [Q][D] float
 *   lo, hi    [Q][m] closed bounds, cell types as the index's columns; lo > hi is legal
 *             (empty valid set); an unconstrained attribute gets the type's full range; an
 *             equality predicate is lo == hi.  For a BOA_ATTR_SET32 column (the equality /
 *             subset filters the paper's Conclusion mentions: the cell is the set of tags
 *             the point carries) lo is the set of wanted tags and hi the mode: 0 = the
 *             point must carry at least one of them, non-zero = all of them
 *   out_ids   [Q][k]  ids of the filter-valid nearest points found, ascending by
 *             (squared distance, id), duplicate-free; BOA_NO_ID fills unused slots
 *   out_dists [Q][k]  squared L2 distances in fp32; +inf in unused slots
 *
 * Asynchronous on `stream`: no host synchronisation; outputs are valid once the stream
 * has run the enqueued work.  Scratch memory is owned by the index and grows (a device
 * allocation) only when Q or Lmax exceed every earlier call's; two searches on one
 * index must not overlap in time.  With BOA+ a second stream owned by the index is
 * used and joined back into `stream` before the call's work ends.
 * Errors (before any launch): BOA_EINVAL for nulls, Q < 0, k < 1, k > L0, L0 > Lmax,
 * Lmax > BOA_MAX_WIDTH, misaligned pointers.  Q == 0 is a no-op.
 */
int boa_search(boa_index* index, const float* queries, int64_t Q, const void* lo, const void* hi,
               int k, int L0, int Lmax, uint32_t* out_ids, float* out_dists, void* stream);

/*
 * boa_search with HOST buffers: the end-to-end call of a caller whose queries arrive in host
 * memory and whose results are read on the host (the problem statement's (q_i, f_i) -> K_f
 * with the transfers included).  Copies queries, lo and hi to index-owned device staging
 * buffers on `stream`, runs boa_search there, copies out_ids and out_dists back and
 * SYNCHRONISES `stream` before it returns, so the outputs are ready to read.  When all five
 * buffers are page-locked host memory mapped into the device's address space (cudaHostAlloc,
 * cudaHostRegister) and start on 16 bytes, nothing is staged: the kernels read each query over
 * the host link when they start on it and write its results straight back
 * (BOA_PARAM_HOST_IN_PLACE = 0 turns that off).
 *
 *   queries, lo, hi, out_ids, out_dists   HOST pointers, shapes and meaning as in boa_search;
 *       page-locked memory lets the copies run at full speed and asynchronously, pageable
 *       memory works too.  No alignment requirement.
 *   everything else as in boa_search (same results, statistics, parameter handling).
 *
 * The staging buffers grow (cudaMalloc) the first time a batch is larger than any before.
 * Errors: as boa_search, plus BOA_ENOMEM for the staging buffers.
 */
int boa_search_host(boa_index* index, const float* queries, int64_t Q, const void* lo, const void* hi, int k,
                    int L0, int Lmax, uint32_t* out_ids, float* out_dists, void* stream);

/*
 * boa_search for callers that must not allocate device memory.  (The paper has no
 * counterpart: this is a service of the library, not a step of the method.)
 *
 * Who needs it: a serving loop that has handed all device memory to its own pools and
 * runs with allocation forbidden; a latency-critical caller that cannot afford the
 * device-wide synchronisation a cudaMalloc or cudaFree may imply; code running inside a
 * region where the CUDA runtime refuses allocation.  boa_search grows index-owned
 * scratch with cudaMalloc the first time a batch is larger than any before; this
 * variant never does.  Its scratch (survivor lists, counters, per-query statistics and
 * the pools carried between phases) is a fixed array of about 4.1 MiB inside the
 * library image, so every GPU that loads the library holds that much until the process
 * exits.
 *
 * Same arguments, outputs and asynchronous behaviour as boa_search, same results, with
 * these differences:
 *   - Q <= BOA_NOALLOC_MAX_Q and Lmax <= BOA_NOALLOC_MAX_WIDTH, else BOA_ETOOBIG and
 *     nothing is enqueued;
 *   - it calls no cudaMalloc, cudaFree or other allocating routine; the first call on a
 *     device looks up the device address of the fixed array (one cudaGetSymbolAddress),
 *     so make that first call outside any stream capture;
 *   - all calls on one device share the one array, whatever the index: it keeps the
 *     previous call's contents (what must start at zero is cleared on `stream` at the
 *     start of each call), and two calls whose GPU work overlaps in time race on it --
 *     run them one after the other, on one stream or ordered by events;
 *   - boa_get_stats and boa_get_phase_counts do not cover this call: they keep
 *     describing the last boa_search on the index.
 */
#define BOA_NOALLOC_MAX_Q 1024
#define BOA_NOALLOC_MAX_WIDTH 512
int boa_search_noalloc(boa_index* index, const float* queries, int64_t Q, const void* lo,
                       const void* hi, int k, int L0, int Lmax, uint32_t* out_ids, float* out_dists,
                       void* stream);

/*
 * Replace the violation count in the finite-lambda score by the numeric distance to the
 * range (the range filter distance the paper's graph-construction paragraph names; the
 * paper's own system counts violated predicates, which stays the default): score =
 * d^2 + lambda * sum_j scales[j] * dist_j, where dist_j is how far attribute j lies outside
 * its range (0 inside; integer cells exact, float cells one subtraction, NaN infinitely
 * far, a violated membership predicate 1), added over j in ascending order in fp32.
 * Validity of an answer is still decided by the predicates alone.
 *   scales  HOST array [m], every entry finite and > 0; NULL goes back to the count
 * Needs a finite BOA_PARAM_LAMBDA at search time (else boa_search returns BOA_EINVAL);
 * not combined with PQ traversal or expansion width 2.  Synchronises `stream`.
 */
int boa_set_range_penalty(boa_index* index, const float* scales, void* stream);

/* Set one parameter (keys above).  BOA_EINVAL for an unknown key or a value out of range. */
int boa_set_param(boa_index* index, int key, double value);

/* Explicit phase widths (HOST array, strictly increasing, 1..BOA_MAX_PHASES entries)
   replacing the geometric schedule of Algorithm 1; n == 0 restores it.  With an
   explicit schedule boa_search requires L0 == widths[0] and Lmax == widths[n-1]. */
int boa_set_schedule(boa_index* index, const int* widths, int n);

/*
 * Per-query statistics of the last boa_search on this index, copied on `stream` into
 * caller DEVICE buffers of Q int32 each (any may be NULL):
 *   final_L   width of the last phase the query ran (its mean is the paper's L_avg)
 *   n_expand  nodes expanded, summed over the phases the query ran
 *   n_scored  neighbour distances computed (a node forgotten by the bounded table of
 *             scored ids and met again is counted again)
 *   flags     bit 0: a phase stopped at its expansion cap
 */
int boa_get_stats(boa_index* index, int32_t* final_L, int32_t* n_expand, int32_t* n_scored,
                  int32_t* flags, void* stream);

/* With PQ traversal: rows fetched per query for the final exact ranking, summed over the
   phases it ran (DEVICE buffer of Q int32, copied on `stream`); zeros otherwise. */
int boa_get_rerank_counts(boa_index* index, int32_t* n_rerank, void* stream);

/* Number of queries that entered each phase of the last search: writes up to n values
   into the HOST array `active` and returns the number of phases in *n_phases.
   Synchronises `stream`. */
int boa_get_phase_counts(boa_index* index, int64_t* active, int n, int* n_phases, void* stream);

/* Bytes of index-owned scratch a search of Q queries up to width Lmax needs. */
int boa_workspace_bytes(const boa_index* index, int64_t Q, int Lmax, size_t* bytes);

/* Number of kernel launches the last boa_search enqueued. */
int boa_last_launch_count(const boa_index* index);

/* Device-side status word of the last search on this index (HOST int, synchronises
   `stream`): 0 = fine.  The search kernel has no wait on a flag, barrier or peer and
   every loop in it is bounded by the expansion cap, so no bit is raised today; the word
   is where a kernel that has to give up would say so (bit 0 is reserved for "a wait
   timed out, outputs of the affected launches are incomplete"). */
int boa_device_status(boa_index* index, int* status, void* stream);

/* cudaError_t of the most recent failing CUDA call made by this library (0 if none). */
int boa_last_cuda_error(void);

/* Static text for a status code. */
const char* boa_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* BOA_H */

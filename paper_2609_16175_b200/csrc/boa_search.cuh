// Warp-per-query filter-aware beam search (Algorithm 2) with the confidence test
// (Eq. 3) and survivor compaction (the gather step of Algorithm 1) fused
// into its epilogue.  sm_100a only.
//
// One warp (one CTA of 32 threads) owns one query from start to convergence.  Its
// candidate pool, the table of recently scored ids and the query vector live in
// shared memory.  A pool entry is one 64-bit key
//     [63:60] phi (violated predicates)  [59:29] fp32 bits of d^2  [28:1] id  [0] expanded
// so that integer order of keys is the lexicographic order (phi, d^2, id): the
// lambda -> infinity reading of the paper's score dist + lambda*phi.  With a finite
// lambda the key carries the score itself (layout at pack_key).
//
// Neighbour records (the vector, one 32-byte-aligned row each; the attribute cells sit in a
// compact array of their own that stays in L2) are read with 16-byte read-only loads straight into registers: eight
// rows per pass, 8 lanes per row, every lane issues all its loads of the pass (two
// rows, up to four chunks each) before the first use, so a warp keeps 4 KB in flight
// and an SM with 20 resident warps about 80 KB.  Two staged variants were measured
// first and dropped: one cp.async.bulk (TMA) copy per row into shared memory needs a
// uniform-datapath instruction sequence per row, and 16-byte cp.async copies spend
// as long issuing as waiting; both were 40 % slower than register loads on the 1M x
// 128-d workload because the kernel is bound by instruction issue and dependent
// latency, not by the number of bytes in flight.
//
// The table of recently scored ids stores 16-bit tags in 4-way buckets of 8 bytes or, when
// the index is small enough for 10-bit tags, 10-bit tags in 3-way buckets of 4 bytes (half
// again as many ids in the same shared memory); the least recently met way is replaced.  An id is first mapped by an odd multiplier modulo 2^id_bits (a
// bijection); the high bits pick the bucket (with 3*2^kb buckets: the bucket group, and
// the low part modulo 3 the bucket inside it) and the rest is the tag, so bucket + tag
// identify the id exactly: the table can forget an id, it can never report an unseen id
// as seen.
// A forgotten id that is met again is scored again and then recognised by its key
// in the pool (or rejected again by the pool's worst key), so results never change.
//
// Distances are accumulated in a fixed order: a row is cut into 16-byte chunks,
// chunk c belongs to lane (c mod 8) of an 8-lane group, each lane runs
// acc = fmaf(x-q, x-q, acc) over its chunks in ascending order, and the eight
// partial sums meet in a butterfly (xor 4, 2, 1).  Eight neighbours are scored per
// warp pass, two per 8-lane group sharing one butterfly.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace boa {

// Query warps per SM the register allocation is tuned for: five per scheduler (at most 96
// registers a thread).  The kernel is bound by dependent latency, so the fifth warp per
// scheduler pays (9 % on the 1M x 128-d workload against four at 104 registers) although a
// few values spill.
#ifndef BOA_MIN_CTAS
#define BOA_MIN_CTAS 20
#endif
// Rows per 8-lane group and scoring pass for rows of one / two 16-byte chunks per lane.
#ifndef BOA_SHORT_RPG1
#define BOA_SHORT_RPG1 4
#endif
#ifndef BOA_SHORT_RPG2
#define BOA_SHORT_RPG2 4
#endif

// L2 prefetch of the rows about to be scored: all of an expansion's rows are requested as
// soon as they are known, so only the first scoring pass waits for DRAM.  Measured on B200:
// +2 to +5 % for rows of 384 and 512 bytes (three scoring passes of eight rows); nothing
// or a loss for 128-byte rows (16 to a pass already) and for rows of several KB (the
// requests cost more issue slots than the latency they hide), so only rows of 129..512
// bytes use it.  Requesting the adjacency row of the probable next node the same way
// measured as no gain and is not done.
#ifndef BOA_PREFETCH_ROWS
#define BOA_PREFETCH_ROWS 1
#endif

constexpr uint32_t kNoId = 0xFFFFFFFFu;
constexpr int kThreads = 32;           // one warp per CTA
constexpr uint64_t kKeyMax = ~0ull;

enum : uint32_t { kStatusCopyTimeout = 1u };   // reserved: no wait in the kernel can time out

// Keeps the compiler from moving code across this point.
#define BOA_SCHED_FENCE() asm volatile("" ::: "memory")

// Optional per-section cycle counters (build with -DBOA_SECTION_TIMERS; off in the product).

#ifdef BOA_SECTION_TIMERS
#define BOA_T_DECL long long t_prev_ = clock64(); long long t_acc_[12] = {0}
#define BOA_T_MARK(i) do { long long t_now_ = clock64(); t_acc_[i] += t_now_ - t_prev_; t_prev_ = t_now_; } while (0)
#define BOA_T_FLUSH(ptr) do { if (lane == 0 && (ptr)) for (int i_ = 0; i_ < 12; ++i_) atomicAdd((unsigned long long*)(ptr) + i_, (unsigned long long)t_acc_[i_]); } while (0)
#else
#define BOA_T_DECL
#define BOA_T_MARK(i)
#define BOA_T_FLUSH(ptr)
#endif

struct SearchParams {
    // index
    const uint8_t* rec;       // [N] records: the vector, padded to rec_stride
    const uint32_t* attrs;    // [N][m] attribute cells
    const uint32_t* graph;    // [N][R]
    int64_t N;
    int D, m, R;
    int rec_stride;           // bytes, multiple of 32
    int nchunks;              // 16-byte chunks of one vector
    uint32_t attr_float_mask; // bit j set: column j is float
    uint32_t attr_set_mask;   // bit j set: column j holds membership masks (EXT kernels)
    const float* pen_scales;  // [8] per-attribute scale of the distance-to-range penalty, or null:
                              // the score's filter term is then the violation count (EXT kernels)
    uint32_t entry;
    // product quantisation (PQ kernels only): D = pq_M * pq_dsub
    const uint8_t* pq_codes;  // [N][pq_M] centroid index per subspace, rows of pq_M bytes (multiple of 16)
    const float* pq_pivots;   // [pq_M][pq_K][pq_dsub]
    int pq_M, pq_K, pq_dsub;
    // batch
    const float* queries;     // [Q][D]
    const int32_t* lo;        // [Q][m]
    const int32_t* hi;
    uint32_t* out_ids;        // [Q][k]
    float* out_d2;
    int64_t Q;
    int k;
    // phase
    int L;                    // beamwidth: expandable prefix of the pool
    int C;                    // pool capacity (L in restart mode, Lmax in resume mode)
    int table_bytes;          // shared memory of the table of recently scored ids (multiple of 16)
    int table_narrow;         // 0: 8-byte buckets of four 16-bit tags; 1: 4-byte buckets of three 10-bit tags
    int table_mul3;           // 1 when the bucket count is 3*2^kb, 0 when it is 2^kb
    int id_bits;              // bits of a node id (ids < 2^id_bits)
    int low_bits;             // id_bits - kb: bits of a mapped id below its bucket group
    int max_expand;           // expansions after which a phase gives up
    int first_phase;          // statistics start from zero
    int resume_in;            // load the pool a narrower phase spilled
    int spill_out;            // uncertain queries spill their pool for the next phase
    int last_phase;           // nobody is appended to a survivor list
    float c_eps;              // (1-eps)^2 rounded once to fp32
    int eps_mode;             // 0: use c_eps; -1: never confident; 1: confident iff > k valid
    double tau_q;             // tau * Q: a phase runs only while |A| > tau*Q
    int fin;                  // 1: keys order by the score d^2 + lambda*phi (finite lambda)
    float lambda;
    // work list of this launch: positions [begin, end) of in_list (identity when null)
    const uint32_t* in_list;
    const uint32_t* in_begin_ptr;  // device values read at kernel start (null: use constants)
    const uint32_t* in_end_ptr;
    uint32_t in_begin, in_end;
    const uint32_t* active_count;  // |A| of this phase for the tau test (null: Q)
    uint32_t* ticket;              // work counter of this launch, zero at start
    uint32_t* out_list;            // survivors of this phase
    uint32_t* out_count;
    uint32_t* status;              // device status word (kStatus* bits)
#ifdef BOA_SECTION_TIMERS
    unsigned long long* timers;    // section cycle counters of debug builds
#endif
    // per-query state
    int32_t* final_L;
    int32_t* n_expand;
    int32_t* n_scored;
    int32_t* flags;
    int32_t* n_rerank;        // PQ kernels: rows fetched for the final exact ranking
    uint64_t* spill;          // [Q][spill_stride] pools carried between phases (resume)
    int32_t* spill_size;      // [Q]
    int spill_stride;
};

// ---------------------------------------------------------------- helpers
// Two key layouts.  Lexicographic (lambda -> infinity): phi on top, then the distance bits.
// Finite lambda: the score bits on top, then the id; phi rides below the id, where it
// cannot change the order of two different nodes.
//     fin == false: [63:60] phi  [59:29] fp32 bits of d^2    [28:1] id            [0] expanded
//     fin == true : [63:33] fp32 bits of d^2 + lambda*phi    [32:5] id  [4:1] phi [0] expanded
__device__ __forceinline__ uint64_t pack_key(bool fin, uint32_t phi, float key, uint32_t id)
{
    const uint64_t bits = __float_as_uint(key) & 0x7FFFFFFFu;
    return fin ? ((bits << 33) | ((uint64_t)id << 5) | ((uint64_t)phi << 1))
               : (((uint64_t)phi << 60) | (bits << 29) | ((uint64_t)id << 1));
}
__device__ __forceinline__ uint32_t key_id(bool fin, uint64_t k)
{
    return (uint32_t)(k >> (fin ? 5 : 1)) & 0x0FFFFFFFu;
}
// d^2 in the lexicographic layout; the score in the other (equal to d^2 where phi == 0)
__device__ __forceinline__ float key_d2(bool fin, uint64_t k)
{
    return __uint_as_float((uint32_t)(k >> (fin ? 33 : 29)) & 0x7FFFFFFFu);
}
__device__ __forceinline__ uint32_t key_phi(bool fin, uint64_t k)
{
    return fin ? ((uint32_t)(k >> 1) & 0xFu) : (uint32_t)(k >> 60);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
// Predicated read-only loads.  When the predicate is false nothing is loaded and the
// outputs keep whatever the registers held: callers never use them in that case.
template <int N>
__device__ __forceinline__ void ldg_chunks(uint4 (&v)[N], const uint8_t* ptr, bool pred)
{
    static_assert(N >= 1 && N <= 4, "one to four 16-byte chunks, 128 bytes apart");
    if (N == 1) {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %5, 0;\n\t"
            "@p ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];\n\t}"
            : "=r"(v[0].x), "=r"(v[0].y), "=r"(v[0].z), "=r"(v[0].w)
            : "l"(ptr), "r"((uint32_t)pred));
    } else if (N == 2) {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %9, 0;\n\t"
            "@p ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%8];\n\t"
            "@p ld.global.nc.v4.u32 {%4,%5,%6,%7}, [%8+128];\n\t}"
            : "=r"(v[0].x), "=r"(v[0].y), "=r"(v[0].z), "=r"(v[0].w), "=r"(v[N > 1 ? 1 : 0].x),
              "=r"(v[N > 1 ? 1 : 0].y), "=r"(v[N > 1 ? 1 : 0].z), "=r"(v[N > 1 ? 1 : 0].w)
            : "l"(ptr), "r"((uint32_t)pred));
    } else if (N == 3) {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %13, 0;\n\t"
            "@p ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%12];\n\t"
            "@p ld.global.nc.v4.u32 {%4,%5,%6,%7}, [%12+128];\n\t"
            "@p ld.global.nc.v4.u32 {%8,%9,%10,%11}, [%12+256];\n\t}"
            : "=r"(v[0].x), "=r"(v[0].y), "=r"(v[0].z), "=r"(v[0].w), "=r"(v[N > 1 ? 1 : 0].x),
              "=r"(v[N > 1 ? 1 : 0].y), "=r"(v[N > 1 ? 1 : 0].z), "=r"(v[N > 1 ? 1 : 0].w),
              "=r"(v[N > 2 ? 2 : 0].x), "=r"(v[N > 2 ? 2 : 0].y), "=r"(v[N > 2 ? 2 : 0].z),
              "=r"(v[N > 2 ? 2 : 0].w)
            : "l"(ptr), "r"((uint32_t)pred));
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %17, 0;\n\t"
            "@p ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%16];\n\t"
            "@p ld.global.nc.v4.u32 {%4,%5,%6,%7}, [%16+128];\n\t"
            "@p ld.global.nc.v4.u32 {%8,%9,%10,%11}, [%16+256];\n\t"
            "@p ld.global.nc.v4.u32 {%12,%13,%14,%15}, [%16+384];\n\t}"
            : "=r"(v[0].x), "=r"(v[0].y), "=r"(v[0].z), "=r"(v[0].w), "=r"(v[N > 1 ? 1 : 0].x),
              "=r"(v[N > 1 ? 1 : 0].y), "=r"(v[N > 1 ? 1 : 0].z), "=r"(v[N > 1 ? 1 : 0].w),
              "=r"(v[N > 2 ? 2 : 0].x), "=r"(v[N > 2 ? 2 : 0].y), "=r"(v[N > 2 ? 2 : 0].z),
              "=r"(v[N > 2 ? 2 : 0].w), "=r"(v[N > 3 ? 3 : 0].x), "=r"(v[N > 3 ? 3 : 0].y),
              "=r"(v[N > 3 ? 3 : 0].z), "=r"(v[N > 3 ? 3 : 0].w)
            : "l"(ptr), "r"((uint32_t)pred));
    }
}
__device__ __forceinline__ uint4 ldg_stream128(const void* ptr, bool pred)
{
    uint4 v;
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %5, 0;\n\t"
        "@p ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];\n\t}"
        : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
        : "l"(ptr), "r"((uint32_t)pred));
    return v;
}
__device__ __forceinline__ uint32_t ldg_stream32(const void* ptr, bool pred)
{
    uint32_t v;
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t"
        "@p ld.global.nc.u32 %0, [%1];\n\t}"
        : "=r"(v)
        : "l"(ptr), "r"((uint32_t)pred));
    return v;
}
// Ask for the 128-byte line holding `ptr` to be brought into L2; nothing waits for it.
__device__ __forceinline__ void prefetch_l2(const void* ptr)
{
    asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
}
__device__ __forceinline__ float sq_acc4u(float acc, uint4 x, float4 q);

__device__ __forceinline__ float sq_acc4(float acc, float4 x, float4 q)
{
    float d;
    d = x.x - q.x; acc = fmaf(d, d, acc);
    d = x.y - q.y; acc = fmaf(d, d, acc);
    d = x.z - q.z; acc = fmaf(d, d, acc);
    d = x.w - q.w; acc = fmaf(d, d, acc);
    return acc;
}
__device__ __forceinline__ float sq_acc4u(float acc, uint4 x, float4 q)
{
    return sq_acc4(acc, make_float4(__uint_as_float(x.x), __uint_as_float(x.y), __uint_as_float(x.z),
                                    __uint_as_float(x.w)), q);
}
// Four bytes of a uint8 row against four query values.  A byte b becomes the float b exactly
// by a byte permute into the mantissa of 2^23 and one subtraction: full-rate instructions
// instead of an integer-to-float conversion per element.
__device__ __forceinline__ float sq_acc_bytes(float acc, uint32_t w, float4 q)
{
    const float magic = 8388608.0f;                     // 2^23 = 0x4B000000
    float d;
    d = (__uint_as_float(__byte_perm(w, 0x4B000000u, 0x7440)) - magic) - q.x; acc = fmaf(d, d, acc);
    d = (__uint_as_float(__byte_perm(w, 0x4B000000u, 0x7441)) - magic) - q.y; acc = fmaf(d, d, acc);
    d = (__uint_as_float(__byte_perm(w, 0x4B000000u, 0x7442)) - magic) - q.z; acc = fmaf(d, d, acc);
    d = (__uint_as_float(__byte_perm(w, 0x4B000000u, 0x7443)) - magic) - q.w; acc = fmaf(d, d, acc);
    return acc;
}

// acc + sum over the 16 byte pairs of two 16-byte chunks of a[i]*b[i]
__device__ __forceinline__ uint32_t dot4_bytes(uint4 a, uint4 b, uint32_t acc)
{
    acc = __dp4a(a.x, b.x, acc);
    acc = __dp4a(a.y, b.y, acc);
    acc = __dp4a(a.z, b.z, acc);
    acc = __dp4a(a.w, b.w, acc);
    return acc;
}

// Bitonic sort of 32*RS keys held one per (lane, slot); element index = lane + 32*slot.
template <int RS>
__device__ __forceinline__ void sort_keys(uint64_t (&x)[RS], int lane)
{
#pragma unroll
    for (int k = 2; k <= 32 * RS; k <<= 1) {
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
            if (j >= 32) {
                // partners sit in the same lane, t slots apart
                const int t = j >> 5;
#pragma unroll
                for (int s = 0; s < RS; ++s) {
                    if ((s & t) == 0 && (s | t) < RS) {
                        const uint64_t a = x[s], b = x[s | t];
                        const bool up = ((32 * s) & k) == 0;
                        const uint64_t mn = a < b ? a : b, mx = a < b ? b : a;
                        x[s] = up ? mn : mx;
                        x[s | t] = up ? mx : mn;
                    }
                }
            } else {
#pragma unroll
                for (int s = 0; s < RS; ++s) {
                    const int e = lane + 32 * s;
                    uint64_t y = __shfl_xor_sync(0xffffffffu, x[s], j);
                    const bool up = (e & k) == 0;
                    const bool lower = (lane & j) == 0;
                    const uint64_t mn = x[s] < y ? x[s] : y;
                    const uint64_t mx = x[s] < y ? y : x[s];
                    x[s] = (lower == up) ? mn : mx;
                }
            }
        }
    }
}

// Per-warp shared memory carve-up (bytes), shared by host and device.
struct WarpSmem {
    int pool_off, nk_off, cand_off, hash_off, q_off, pq_off, top_off, total;
};
constexpr int kPqMaxK = 32;            // largest k of a PQ search: its final ranking keeps k keys per warp
// q_in_smem: the query vector is kept in shared memory (only when lanes do not hold their
// slices of it in registers).
__host__ __device__ inline WarpSmem warp_smem_layout(int C, int table_bytes, int D, int RS, bool q_in_smem,
                                                      int pq_entries = 0)
{
    WarpSmem s;
    int off = 0;
    s.pool_off = off;  off += ((C + 1) & ~1) * 8;
    s.nk_off = off;    off += 32 * RS * 8;
    s.q_off = off;     off += q_in_smem ? ((D * 4 + 15) & ~15) : 0;
    s.hash_off = off;  off += table_bytes;
    s.cand_off = off;  off += 32 * RS * 4;
    s.pq_off = off;    off += pq_entries * 4;                     // distance table of the query
    s.top_off = off;   off += pq_entries ? kPqMaxK * 8 : 0;       // best exact keys of the final ranking
    s.total = (off + 127) & ~127;
    return s;
}

// ---------------------------------------------------------------- the kernel
// VT: 0 = float vectors, 1 = uint8 vectors.  RN: adjacency slots per lane and node (1:
// R <= 32, 2: R <= 64).  W: nodes expanded per iteration (1 = Algorithm 2 as printed; 2 =
// the first two unexpanded beam entries together, an extension).  CPL: 16-byte chunks of a row per lane of an 8-lane group when that is
// at most 4 (the lane then keeps its slices of the query in registers and the chunk
// loop is unrolled); 0 = any length, query slices read from shared memory.  EXACT: the
// row has exactly 8*CPL chunks, so no lane ever has a chunk missing.
// PQ: the traversal orders by product-quantised distances (a per-query table of
// subvector-to-centroid distances in shared memory, one look-up per subspace and candidate,
// a lane per candidate); when a phase has converged the filter-valid beam entries are ranked
// by exact distance with the same row-scoring code the exact search uses.
// EXT: membership-mask columns and the distance-to-range penalty (kept out of the default
// kernels, whose register allocation has no room to spare).
template <int VT, int RN, int W, int CPL, bool EXACT, bool PQ = false, bool EXT = false>
__global__ void __launch_bounds__(kThreads, (PQ ? 8 : BOA_MIN_CTAS)) boa_search_kernel(const SearchParams p)
{
    static_assert(W == 1 || W == 2, "expansion width 1 or 2");
    static_assert(!PQ || W == 1, "PQ traversal expands one node per iteration");
    static_assert(!EXT || (W == 1 && !PQ), "extended predicates: one node per iteration, exact distances");
    constexpr int RS = RN * W;                      // adjacency slots per lane and iteration
    extern __shared__ __align__(128) uint8_t smem_raw[];
    const int lane = threadIdx.x;
    const int g = lane & 7;        // lane inside its 8-lane group
    const int gi = lane >> 3;      // group index 0..3
    const unsigned lt_mask = (1u << lane) - 1u;
    constexpr int QF4 = (VT == 0) ? 1 : 4;          // float4 slices of the query per chunk
    constexpr int NQ = (CPL > 0) ? CPL * QF4 : 1;

    const WarpSmem lay = warp_smem_layout(p.C, p.table_bytes, p.D, RS, CPL == 0 && !PQ, PQ ? p.pq_M * p.pq_K : 0);
    float* pq_table = reinterpret_cast<float*>(smem_raw + lay.pq_off);
    uint64_t* topk = reinterpret_cast<uint64_t*>(smem_raw + lay.top_off);
    uint64_t* pool = reinterpret_cast<uint64_t*>(smem_raw + lay.pool_off);
    uint64_t* nk = reinterpret_cast<uint64_t*>(smem_raw + lay.nk_off);
    uint32_t* cand = reinterpret_cast<uint32_t*>(smem_raw + lay.cand_off);
    uint16_t* hash = reinterpret_cast<uint16_t*>(smem_raw + lay.hash_off);
    float4* qs = reinterpret_cast<float4*>(smem_raw + lay.q_off);

    const bool fin = p.fin != 0;
    const uint32_t id_mask = (p.id_bits >= 32) ? 0xFFFFFFFFu : ((1u << p.id_bits) - 1u);
    const uint32_t low_mask = (1u << p.low_bits) - 1u;

    // work range of this launch
    const uint32_t w_begin = p.in_begin_ptr ? *p.in_begin_ptr : p.in_begin;
    const uint32_t w_end = p.in_end_ptr ? *p.in_end_ptr : p.in_end;
    if (p.active_count) {
        // loop condition of Algorithm 1: a phase runs only while |A| exceeds tau * rho
        if (!((double)(*p.active_count) > p.tau_q)) return;
    }
    const uint32_t n_work = w_end > w_begin ? w_end - w_begin : 0u;

    BOA_T_DECL;

    for (;;) {
        uint32_t t = 0;
        if (lane == 0) t = atomicAdd(p.ticket, 1u);
        t = __shfl_sync(0xffffffffu, t, 0);
        if (t >= n_work) break;
        const uint32_t qi = p.in_list ? p.in_list[w_begin + t] : (w_begin + t);

        // ---- load the query, its bounds; clear the table of scored ids
        {
            // PQ traversal needs the whole query only for the final exact ranking: it is read
            // from global memory there and its shared-memory copy is left out (the per-query
            // distance table decides how many warps fit)
            if (CPL == 0 && !PQ) {
                const float4* qsrc = reinterpret_cast<const float4*>(p.queries + (size_t)qi * p.D);
                for (int i = lane; i < p.D / 4; i += 32) qs[i] = qsrc[i];
            }
            const uint4 ff = make_uint4(~0u, ~0u, ~0u, ~0u);
            uint4* h4 = reinterpret_cast<uint4*>(hash);
            for (int i = lane; i < p.table_bytes / 16; i += 32) h4[i] = ff;
        }
        int32_t my_lo = 0, my_hi = 0;
        if (g < p.m) {
            my_lo = p.lo[(size_t)qi * p.m + g];
            my_hi = p.hi[(size_t)qi * p.m + g];
        }
        const bool my_float = (p.attr_float_mask >> g) & 1u;
        const bool my_set = EXT && ((p.attr_set_mask >> g) & 1u);
        const bool pen_on = EXT && p.pen_scales != nullptr;
        const float my_scale = (pen_on && g < p.m) ? __ldg(p.pen_scales + g) : 0.0f;
        __syncwarp();
        const float4* qglob = reinterpret_cast<const float4*>(p.queries + (size_t)qi * p.D);   // PQ, long rows
        float4 qreg[NQ];           // this lane's slices of the query (CPL > 0)
        if (CPL > 0) {
            const float4* qsrc = reinterpret_cast<const float4*>(p.queries + (size_t)qi * p.D);
#pragma unroll
            for (int i = 0; i < (CPL > 0 ? CPL : 1); ++i) {
                const int c = g + 8 * i;
#pragma unroll
                for (int f = 0; f < QF4; ++f)
                    qreg[i * QF4 + f] = (c < p.nchunks) ? __ldg(qsrc + c * QF4 + f) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        // Byte rows against a query whose elements are themselves whole numbers 0..255 (the
        // usual case when data and queries come from one byte-valued source): every term
        // (x-q)^2 and every partial sum of at most 256 of them is an integer below 2^24, so
        // fp32 accumulation in any order is exact and equals the integer sum.  The distance
        // is then computed with 4-way byte dot products, sum x*x - 2 sum x*q + sum q*q, two
        // instructions per four elements instead of sixteen.  The query bytes take the place
        // of the first float slices in qreg; qq_lane is this lane's sum q*q.
        bool q_bytes = false;
        int qq_lane = 0;
        if (VT == 1 && (CPL == 1 || CPL == 2)) {
            bool ok = true;
#pragma unroll
            for (int j = 0; j < NQ; ++j) {
                const float4 v = qreg[j];
                ok = ok && v.x >= 0.f && v.x <= 255.f && v.x == truncf(v.x) && v.y >= 0.f && v.y <= 255.f &&
                     v.y == truncf(v.y) && v.z >= 0.f && v.z <= 255.f && v.z == truncf(v.z) && v.w >= 0.f &&
                     v.w <= 255.f && v.w == truncf(v.w);
            }
            q_bytes = __all_sync(0xffffffffu, ok);
            if (q_bytes) {
                uint32_t wq[NQ];
#pragma unroll
                for (int j = 0; j < NQ; ++j) {
                    const float4 v = qreg[j];
                    wq[j] = (uint32_t)v.x | ((uint32_t)v.y << 8) | ((uint32_t)v.z << 16) | ((uint32_t)v.w << 24);
                    qq_lane = (int)__dp4a(wq[j], wq[j], (uint32_t)qq_lane);
                }
#pragma unroll
                for (int i = 0; i < (CPL > 0 ? CPL : 1); ++i)
                    qreg[i] = make_float4(__uint_as_float(wq[4 * i + 0]), __uint_as_float(wq[4 * i + 1]),
                                          __uint_as_float(wq[4 * i + 2]), __uint_as_float(wq[4 * i + 3]));
            }
        }

        if (PQ) {
            // distance table of this query: entry (m, c) = squared distance between the m-th
            // subvector of q and centroid c of subspace m, one fused multiply-add per dimension
            // in ascending order; a lane per entry
            const int entries = p.pq_M * p.pq_K;
            const float* qv = p.queries + (size_t)qi * p.D;
            for (int e = lane; e < entries; e += 32) {
                const int m = e / p.pq_K;
                const float* piv = p.pq_pivots + (size_t)e * p.pq_dsub;
                const float* qm = qv + m * p.pq_dsub;
                float acc = 0.0f;
                if ((p.pq_dsub & 3) == 0) {
                    for (int i = 0; i < p.pq_dsub; i += 4) {
                        const float4 pv = __ldg(reinterpret_cast<const float4*>(piv + i));
                        const float4 qq = __ldg(reinterpret_cast<const float4*>(qm + i));
                        acc = sq_acc4(acc, qq, pv);
                    }
                } else {
                    for (int i = 0; i < p.pq_dsub; ++i) {
                        const float d = __ldg(qm + i) - __ldg(piv + i);
                        acc = fmaf(d, d, acc);
                    }
                }
                pq_table[e] = acc;
            }
            __syncwarp();
        }

        // Scores cand[0..cnt) straight from global memory: eight rows per pass, every lane
        // loads its own 16-byte chunks of two rows into registers (all loads of a pass are
        // issued before the first use), distance + violated predicates -> nk[0..cnt).
        // reduce the two partial-sum sets of a pass, count violated predicates, write the keys
        auto finish_pass = [&](int cnt, float a0, float a1, uint32_t av0, uint32_t av1, uint32_t id0,
                               uint32_t id1, int j0, int j1, bool act0, bool act1) {
            const bool hi4 = (lane & 4) != 0;
            float v = hi4 ? a1 : a0;
            const float w = hi4 ? a0 : a1;
            v += __shfl_xor_sync(0xffffffffu, w, 4);
            v += __shfl_xor_sync(0xffffffffu, v, 2);
            v += __shfl_xor_sync(0xffffffffu, v, 1);
            bool v0, v1;
            float e0 = 0.0f, e1 = 0.0f;      // EXT: this lane's attribute's distance to its range
            if (my_float) {
                const float l = __int_as_float(my_lo), h = __int_as_float(my_hi);
                const float c0 = __uint_as_float(av0), c1 = __uint_as_float(av1);
                v0 = !(c0 >= l && c0 <= h);
                v1 = !(c1 >= l && c1 <= h);
                if (EXT) {
                    e0 = c0 < l ? l - c0 : (c0 > h ? c0 - h : (v0 ? __int_as_float(0x7f800000) : 0.0f));
                    e1 = c1 < l ? l - c1 : (c1 > h ? c1 - h : (v1 ? __int_as_float(0x7f800000) : 0.0f));
                }
            } else if (my_set) {
                // membership: lo = the wanted tags; hi == 0: at least one of them, else all of them
                const uint32_t h0 = av0 & (uint32_t)my_lo, h1 = av1 & (uint32_t)my_lo;
                v0 = my_hi == 0 ? h0 == 0u : h0 != (uint32_t)my_lo;
                v1 = my_hi == 0 ? h1 == 0u : h1 != (uint32_t)my_lo;
                e0 = v0 ? 1.0f : 0.0f;
                e1 = v1 ? 1.0f : 0.0f;
            } else {
                v0 = (int32_t)av0 < my_lo || (int32_t)av0 > my_hi;
                v1 = (int32_t)av1 < my_lo || (int32_t)av1 > my_hi;
                if (EXT) {
                    // exact in double, rounded once
                    const int32_t c0 = (int32_t)av0, c1 = (int32_t)av1;
                    e0 = c0 < my_lo ? (float)((double)my_lo - (double)c0) : (c0 > my_hi ? (float)((double)c0 - (double)my_hi) : 0.0f);
                    e1 = c1 < my_lo ? (float)((double)my_lo - (double)c1) : (c1 > my_hi ? (float)((double)c1 - (double)my_hi) : 0.0f);
                }
            }
            const unsigned bal0 = __ballot_sync(0xffffffffu, v0 && act0 && g < p.m);
            const unsigned bal1 = __ballot_sync(0xffffffffu, v1 && act1 && g < p.m);
            const unsigned bal = hi4 ? bal1 : bal0;
            const int jj = hi4 ? j1 : j0;
            float pen = 0.0f;
            if (pen_on) {
                // the attributes' scaled distances, added in ascending attribute order
                const float s0 = __fmul_rn(e0, my_scale), s1 = __fmul_rn(e1, my_scale);
                float p0 = 0.0f, p1 = 0.0f;
                for (int a = 0; a < p.m; ++a) {
                    p0 = __fadd_rn(p0, __shfl_sync(0xffffffffu, s0, (lane & ~7) + a));
                    p1 = __fadd_rn(p1, __shfl_sync(0xffffffffu, s1, (lane & ~7) + a));
                }
                pen = hi4 ? p1 : p0;
            }
            if ((g & 3) == 0 && jj < cnt)
            {
                const uint32_t phi = __popc((bal >> (8 * gi)) & 0xFFu);
                // finite lambda: one fused multiply-add gives the score the pool orders by
                if (fin) nk[jj] = pack_key(true, phi, __fmaf_rn(p.lambda, pen_on ? pen : (float)phi, v), hi4 ? id1 : id0);
                else nk[jj] = pack_key(false, phi, v, hi4 ? id1 : id0);
            }
        };

        // Scores cand[0..cnt) straight from global memory: eight rows per pass, every lane
        // loads its own 16-byte chunks of two rows into registers (all loads of a pass are
        // issued before the first use), distance + violated predicates -> nk[0..cnt).  For
        // short rows the loads of the next pass are issued as soon as the multiply-adds of
        // this pass have freed the registers, before its reduction.
        auto score = [&](int cnt) {
            BOA_T_MARK(3);
            const int ga = (g < p.m) ? g : 0;
            if (CPL == 1 || CPL == 2) {
                // short rows: RPG rows per 8-lane group and pass (16 or 32 rows a pass), so that
                // a row list of 40 costs two or three dependent round trips instead of six
                constexpr int NC = (CPL > 0 ? CPL : 1);
                constexpr int RPG = (CPL == 1) ? BOA_SHORT_RPG1 : BOA_SHORT_RPG2;
                constexpr int RPP = 4 * RPG;
                uint4 x[RPG][NC];
                uint32_t av[RPG], id[RPG];
                auto issue_pass = [&](int r0) {
#pragma unroll
                    for (int t = 0; t < RPG; ++t) {
                        const int j = r0 + gi + 4 * t;
                        const bool act = j < cnt;
                        id[t] = cand[act ? j : 0];
                        const uint8_t* row = p.rec + (size_t)id[t] * p.rec_stride;
                        if (EXACT) {
                            ldg_chunks<NC>(x[t], row + 16 * g, act);
                        } else {
#pragma unroll
                            for (int i = 0; i < NC; ++i) {
                                const int c = g + 8 * i;
                                x[t][i] = ldg_stream128(row + 16 * c, act && c < p.nchunks);
                            }
                        }
                        av[t] = ldg_stream32(p.attrs + (size_t)id[t] * p.m + ga, act && g < p.m);
                    }
                };
                issue_pass(0);
#pragma unroll 1
                for (int r0 = 0; r0 < cnt; r0 += RPP) {
                    BOA_T_MARK(4);
                    BOA_SCHED_FENCE();        // every load of the pass is issued before its first use
                    float a[RPG];
                    uint32_t c_av[RPG], c_id[RPG];
#pragma unroll
                    for (int t = 0; t < RPG; ++t) {
                        a[t] = 0.0f;
                        if (VT == 1 && q_bytes) {
                            uint32_t xx = 0u, xq = 0u;
#pragma unroll
                            for (int i = 0; i < NC; ++i) {
                                if (!EXACT && g + 8 * i >= p.nchunks) continue;
                                xx = dot4_bytes(x[t][i], x[t][i], xx);
                                xq = dot4_bytes(x[t][i], make_uint4(__float_as_uint(qreg[i].x), __float_as_uint(qreg[i].y),
                                                                    __float_as_uint(qreg[i].z), __float_as_uint(qreg[i].w)), xq);
                            }
                            // this lane's sum of (x-q)^2: a whole number in [0, 2^24)
                            a[t] = (float)((int)xx - 2 * (int)xq + qq_lane);
                        } else {
#pragma unroll
                            for (int i = 0; i < NC; ++i) {
                                if (!EXACT && g + 8 * i >= p.nchunks) continue;
                                if (VT == 0) {
                                    a[t] = sq_acc4u(a[t], x[t][i], qreg[i]);
                                } else {
                                    a[t] = sq_acc_bytes(a[t], x[t][i].x, qreg[4 * i + 0]);
                                    a[t] = sq_acc_bytes(a[t], x[t][i].y, qreg[4 * i + 1]);
                                    a[t] = sq_acc_bytes(a[t], x[t][i].z, qreg[4 * i + 2]);
                                    a[t] = sq_acc_bytes(a[t], x[t][i].w, qreg[4 * i + 3]);
                                }
                            }
                        }
                        c_av[t] = av[t];
                        c_id[t] = id[t];
                    }
                    BOA_SCHED_FENCE();
                    if (r0 + RPP < cnt) issue_pass(r0 + RPP);
                    BOA_SCHED_FENCE();
#pragma unroll
                    for (int u = 0; u < RPG; u += 2) {
                        const int ja = r0 + gi + 4 * u, jb = r0 + gi + 4 * (u + 1);
                        finish_pass(cnt, a[u], a[u + 1], c_av[u], c_av[u + 1], c_id[u], c_id[u + 1], ja, jb,
                                    ja < cnt, jb < cnt);
                    }
                    BOA_T_MARK(6);
                }
            } else if (CPL > 0) {
                uint4 x0[CPL > 0 ? CPL : 1], x1[CPL > 0 ? CPL : 1];
                uint32_t av0, av1, id0, id1;
                bool act0, act1;
                int j0, j1;
                auto issue_pass = [&](int r0) {
                    j0 = r0 + gi; j1 = r0 + 4 + gi;
                    act0 = j0 < cnt; act1 = j1 < cnt;
                    id0 = cand[act0 ? j0 : 0]; id1 = cand[act1 ? j1 : 0];
                    const uint8_t* row0 = p.rec + (size_t)id0 * p.rec_stride;
                    const uint8_t* row1 = p.rec + (size_t)id1 * p.rec_stride;
                    if (EXACT) {
                        // one predicate per row; chunk i sits 128 bytes after chunk i-1
                        ldg_chunks<(CPL > 0 ? CPL : 1)>(x0, row0 + 16 * g, act0);
                        ldg_chunks<(CPL > 0 ? CPL : 1)>(x1, row1 + 16 * g, act1);
                    } else {
#pragma unroll
                        for (int i = 0; i < (CPL > 0 ? CPL : 1); ++i) {
                            const int c = g + 8 * i;
                            x0[i] = ldg_stream128(row0 + 16 * c, act0 && c < p.nchunks);
                            x1[i] = ldg_stream128(row1 + 16 * c, act1 && c < p.nchunks);
                        }
                    }
                    av0 = ldg_stream32(p.attrs + (size_t)id0 * p.m + ga, act0 && g < p.m);
                    av1 = ldg_stream32(p.attrs + (size_t)id1 * p.m + ga, act1 && g < p.m);
                };
                issue_pass(0);
#pragma unroll 1
                for (int r0 = 0; r0 < cnt; r0 += 8) {
                    BOA_T_MARK(4);
                    BOA_SCHED_FENCE();        // every load of the pass is issued before its first use
                    float a0 = 0.0f, a1 = 0.0f;
#pragma unroll
                    for (int i = 0; i < (CPL > 0 ? CPL : 1); ++i) {
                        if (!EXACT && g + 8 * i >= p.nchunks) continue;
                        if (VT == 0) {
                            a0 = sq_acc4u(a0, x0[i], qreg[i]);
                            a1 = sq_acc4u(a1, x1[i], qreg[i]);
                        } else {
                            a0 = sq_acc_bytes(a0, x0[i].x, qreg[4 * i + 0]);
                            a1 = sq_acc_bytes(a1, x1[i].x, qreg[4 * i + 0]);
                            a0 = sq_acc_bytes(a0, x0[i].y, qreg[4 * i + 1]);
                            a1 = sq_acc_bytes(a1, x1[i].y, qreg[4 * i + 1]);
                            a0 = sq_acc_bytes(a0, x0[i].z, qreg[4 * i + 2]);
                            a1 = sq_acc_bytes(a1, x1[i].z, qreg[4 * i + 2]);
                            a0 = sq_acc_bytes(a0, x0[i].w, qreg[4 * i + 3]);
                            a1 = sq_acc_bytes(a1, x1[i].w, qreg[4 * i + 3]);
                        }
                    }
                    const uint32_t c_av0 = av0, c_av1 = av1, c_id0 = id0, c_id1 = id1;
                    const int c_j0 = j0, c_j1 = j1;
                    const bool c_act0 = act0, c_act1 = act1;
                    BOA_SCHED_FENCE();
                    if (r0 + 8 < cnt) issue_pass(r0 + 8);
                    BOA_SCHED_FENCE();
                    finish_pass(cnt, a0, a1, c_av0, c_av1, c_id0, c_id1, c_j0, c_j1, c_act0, c_act1);
                    BOA_T_MARK(6);
                }
            } else {
#pragma unroll 1
                for (int r0 = 0; r0 < cnt; r0 += 8) {
                    const int j0 = r0 + gi, j1 = r0 + 4 + gi;
                    const bool act0 = j0 < cnt, act1 = j1 < cnt;
                    const uint32_t id0 = cand[act0 ? j0 : 0], id1 = cand[act1 ? j1 : 0];
                    const uint8_t* row0 = p.rec + (size_t)id0 * p.rec_stride;
                    const uint8_t* row1 = p.rec + (size_t)id1 * p.rec_stride;
                    float a0 = 0.0f, a1 = 0.0f;
                    const uint32_t av0 = ldg_stream32(p.attrs + (size_t)id0 * p.m + ga, act0 && g < p.m);
                    const uint32_t av1 = ldg_stream32(p.attrs + (size_t)id1 * p.m + ga, act1 && g < p.m);
                    // long rows: four chunks of each row in flight per lane at a time
                    for (int c0 = g; c0 < p.nchunks; c0 += 32) {
                        uint4 x0[4], x1[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int c = c0 + 8 * i;
                            x0[i] = ldg_stream128(row0 + 16 * c, act0 && c < p.nchunks);
                            x1[i] = ldg_stream128(row1 + 16 * c, act1 && c < p.nchunks);
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int c = c0 + 8 * i;
                            if (c < p.nchunks) {
                                if (VT == 0) {
                                    const float4 qq = PQ ? __ldg(qglob + c) : qs[c];
                                    a0 = sq_acc4u(a0, x0[i], qq);
                                    a1 = sq_acc4u(a1, x1[i], qq);
                                } else {
                                    const float4 q0 = PQ ? __ldg(qglob + 4 * c + 0) : qs[4 * c + 0];
                                    const float4 q1 = PQ ? __ldg(qglob + 4 * c + 1) : qs[4 * c + 1];
                                    const float4 q2 = PQ ? __ldg(qglob + 4 * c + 2) : qs[4 * c + 2];
                                    const float4 q3 = PQ ? __ldg(qglob + 4 * c + 3) : qs[4 * c + 3];
                                    a0 = sq_acc_bytes(a0, x0[i].x, q0);
                                    a1 = sq_acc_bytes(a1, x1[i].x, q0);
                                    a0 = sq_acc_bytes(a0, x0[i].y, q1);
                                    a1 = sq_acc_bytes(a1, x1[i].y, q1);
                                    a0 = sq_acc_bytes(a0, x0[i].z, q2);
                                    a1 = sq_acc_bytes(a1, x1[i].z, q2);
                                    a0 = sq_acc_bytes(a0, x0[i].w, q3);
                                    a1 = sq_acc_bytes(a1, x1[i].w, q3);
                                }
                            }
                        }
                    }
                    BOA_T_MARK(4);
                    finish_pass(cnt, a0, a1, av0, av1, id0, id1, j0, j1, act0, act1);
                    BOA_T_MARK(6);
                }
            }
            __syncwarp();
        };

        // PQ scoring of cand[0..cnt): a lane per candidate.  The lane reads the candidate's
        // code (pq_M bytes) and attribute cells, counts the violated predicates (the bounds sit
        // in lanes 0..m-1 and are handed round by shuffles) and adds the pq_M table entries the
        // code selects, in ascending subspace order -> nk[0..cnt).
        auto score_pq = [&](int cnt) {
#pragma unroll
            for (int s = 0; s < RS; ++s) {
                const int j = lane + 32 * s;
                const bool act = j < cnt;
                const uint32_t id = act ? cand[j] : 0u;
                uint32_t phi = 0;
                for (int a = 0; a < p.m; ++a) {
                    const int32_t l = __shfl_sync(0xffffffffu, my_lo, a);
                    const int32_t h = __shfl_sync(0xffffffffu, my_hi, a);
                    const uint32_t cell = ldg_stream32(p.attrs + (size_t)id * p.m + a, act);
                    bool v;
                    if ((p.attr_float_mask >> a) & 1u)
                        v = !(__uint_as_float(cell) >= __int_as_float(l) && __uint_as_float(cell) <= __int_as_float(h));
                    else
                        v = (int32_t)cell < l || (int32_t)cell > h;
                    phi += (act && v) ? 1u : 0u;
                }
                float d = 0.0f;
                const uint8_t* code = p.pq_codes + (size_t)id * p.pq_M;
                for (int c0 = 0; c0 < p.pq_M; c0 += 16) {
                    const uint4 cw = ldg_stream128(code + c0, act);
                    if (act) {
                        const uint32_t w4[4] = {cw.x, cw.y, cw.z, cw.w};
#pragma unroll
                        for (int t = 0; t < 16; ++t) {
                            const uint32_t c = (w4[t >> 2] >> (8 * (t & 3))) & 0xFFu;
                            d = d + pq_table[(c0 + t) * p.pq_K + c];
                        }
                    }
                }
                if (act) nk[j] = fin ? pack_key(true, phi, __fmaf_rn(p.lambda, (float)phi, d), id)
                                     : pack_key(false, phi, d, id);
            }
            __syncwarp();
        };
        // the distance the traversal orders by
        auto score_search = [&](int cnt) {
            if (PQ) score_pq(cnt);
            else score(cnt);
        };

        // Returns true when id was not in the table; records it either way.
        auto hash_test_and_set = [&](uint32_t id) -> bool {
            const uint32_t h = (id * 0x9E3779B1u) & id_mask;
            // (high part, low part) -> (bucket, tag), one to one: with 3*2^kb buckets the low
            // part picks one of three buckets of its group and its third is the tag
            const uint32_t top = h >> p.low_bits, low = h & low_mask;
            const uint32_t third = __umulhi(low, 0xAAAAAAABu) >> 1;        // low / 3
            const uint32_t tag = p.table_mul3 ? third : low;
            const uint32_t bucket = p.table_mul3 ? top * 3u + (low - 3u * third) : top;
            // least recently met first out: the tag moves (or enters) to way 0, the ways
            // before its old place move up by one, a new tag pushes the last way out.  The
            // all-ones tag marks an empty way: an id with that tag is never recorded.
            if (p.table_narrow) {
                uint32_t* slot = reinterpret_cast<uint32_t*>(hash) + bucket;
                const uint32_t b = *slot;
                const uint32_t w0 = b & 0x3FFu, w1 = (b >> 10) & 0x3FFu, w2 = (b >> 20) & 0x3FFu;
                const bool found = (w0 == tag) | (w1 == tag) | (w2 == tag);
                const bool fresh = !found | (tag == 0x3FFu);
                if (tag != 0x3FFu && w0 != tag)
                    *slot = tag | (w0 << 10) | (((w1 == tag) ? w2 : w1) << 20) | 0xC0000000u;
                return fresh;
            }
            uint2* slot = reinterpret_cast<uint2*>(hash + 4 * bucket);
            const uint2 b = *slot;
            const uint32_t w0 = b.x & 0xFFFFu, w1 = b.x >> 16, w2 = b.y & 0xFFFFu, w3 = b.y >> 16;
            const bool found = (w0 == tag) | (w1 == tag) | (w2 == tag) | (w3 == tag);
            const bool fresh = !found | (tag == 0xFFFFu);
            if (tag != 0xFFFFu && w0 != tag) {
                const uint32_t hi = (w1 == tag) ? b.y : (w1 | (((w2 == tag) ? w3 : w2) << 16));
                *slot = make_uint2(tag | (w0 << 16), hi);
            }
            return fresh;
        };
        // first unexpanded entry at or after `from` among the first `lim`, or -1
        auto first_unexpanded = [&](int from, int lim) -> int {
            for (int b0 = from & ~31; b0 < lim; b0 += 32) {
                const int i = b0 + lane;
                const bool un = (i >= from) && (i < lim) && ((pool[i] & 1ull) == 0ull);
                const unsigned bal = __ballot_sync(0xffffffffu, un);
                if (bal) return b0 + __ffs(bal) - 1;
            }
            return -1;
        };
        // adjacency row of node `id` into slots [base, base + RN); id == kNoId: an empty row
        auto load_row_ids = [&](uint32_t id, uint32_t (&out)[RS], int base) {
            const uint32_t* grow = p.graph + (size_t)(id == kNoId ? 0u : id) * p.R;
#pragma unroll
            for (int s = 0; s < RN; ++s) {
                const int j = lane + 32 * s;
                out[base + s] = (id != kNoId && j < p.R) ? __ldg(grow + j) : kNoId;
            }
        };

        // ---- pool: fresh from the entry point, or what a narrower phase left
        int n;                 // entries in the pool
        int cur = 0;           // every entry before cur is expanded
        int n_exp = 0, n_sc = 0;
        bool capped = false;
        if (p.resume_in) {
            n = p.spill_size[qi];
            const uint64_t* src = p.spill + (size_t)qi * p.spill_stride;
            for (int i = lane; i < n; i += 32) {
                const uint64_t e = src[i];
                pool[i] = e;
                hash_test_and_set(key_id(fin, e));
            }
            __syncwarp();
        } else {
            if (lane == 0) cand[0] = p.entry;
            __syncwarp();
            score_search(1);
            if (lane == 0) {
                pool[0] = nk[0];
                hash_test_and_set(p.entry);
            }
            n = 1;
            __syncwarp();
        }

        // ---- Algorithm 2 main loop
        BOA_T_MARK(0);
        int pos = first_unexpanded(0, n < p.L ? n : p.L);
        int pos2 = -1;                 // W == 2: the second node of this iteration, or -1
        uint32_t nb[RS];
        bool have_row = false;         // nb[] already holds the adjacency rows of this iteration
        for (;;) {
            if (pos < 0) break;                                   // converged
            if (n_exp >= p.max_expand) { capped = true; break; }
            if (!have_row) {
                load_row_ids(key_id(fin, pool[pos]), nb, 0);
                if (W > 1) {
                    pos2 = (n_exp + 1 < p.max_expand) ? first_unexpanded(pos + 1, n < p.L ? n : p.L) : -1;
                    load_row_ids(pos2 >= 0 ? key_id(fin, pool[pos2]) : kNoId, nb, RN);
                }
            }
            __syncwarp();
            if (lane == 0) {
                pool[pos] |= 1ull;
                if (W > 1 && pos2 >= 0) pool[pos2] |= 1ull;
            }
            cur = ((W > 1 && pos2 >= 0) ? pos2 : pos) + 1;
            n_exp += (W > 1 && pos2 >= 0) ? 2 : 1;
            have_row = false;
            // The probable next node is the next unexpanded entry of the pool as it is now (it
            // is, unless a key scored in this iteration ranks before it): its adjacency row is
            // requested here, a whole scoring pass ahead of its use.  Only for one node per
            // iteration and R <= 32: with longer rows the requests wasted on wrong guesses
            // cost more than the hidden latency saves.
            constexpr bool PRED = (W == 1 && RN == 1);
            int pred_pos = -1;
            uint32_t nbp[RS];
            if (PRED) {
                pred_pos = first_unexpanded(cur, n < p.L ? n : p.L);
                load_row_ids(pred_pos >= 0 ? key_id(fin, pool[pred_pos]) : kNoId, nbp, 0);
            }
            BOA_T_MARK(1);

            // drop ids scored before, compact the rest
            int cnt = 0;
#pragma unroll
            for (int s = 0; s < RS; ++s) {
                if (W > 1 && s == RN) __syncwarp();   // the second row sees what the first recorded
                const bool fresh = (nb[s] != kNoId) && hash_test_and_set(nb[s]);
                const unsigned bal = __ballot_sync(0xffffffffu, fresh);
                if (fresh) {
                    cand[cnt + __popc(bal & lt_mask)] = nb[s];
                    if (BOA_PREFETCH_ROWS && p.rec_stride > 128 && p.rec_stride <= 512) {
                        const uint8_t* row = p.rec + (size_t)nb[s] * p.rec_stride;
                        for (int off = 0; off < p.rec_stride; off += 128) prefetch_l2(row + off);
                        prefetch_l2(p.attrs + (size_t)nb[s] * p.m);
                    }
                }
                cnt += __popc(bal);
            }
            __syncwarp();
            BOA_T_MARK(2);
            int kept = 0, live = 0;
            uint64_t x[RS];
            bool keep[RS];
            int pos_new[RS];
            int rank_s[RS];
            if (cnt > 0) {
                n_sc += cnt;
                // gather + distance + range check (fused)
                score_search(cnt);

                // new keys that cannot enter a full pool are dropped right away
                const uint64_t worst = (n == p.C) ? (pool[n - 1] >> 1) : (kKeyMax >> 1);
#pragma unroll
                for (int s = 0; s < RS; ++s) {
                    const int j = lane + 32 * s;
                    x[s] = (j < cnt) ? nk[j] : kKeyMax;
                    if (x[s] != kKeyMax && (x[s] >> 1) >= worst) x[s] = kKeyMax;
                    live += __popc(__ballot_sync(0xffffffffu, x[s] != kKeyMax));
                }
            }
            if (live > 0) {
                // sort the survivors: by counting for a handful, bitonic otherwise
                if (live <= 8) {
                    // every live key counts the live keys before it (equal keys, which two rows
                    // of one iteration can produce, order by where they sit), then moves there
                    int r[RS];
#pragma unroll
                    for (int s = 0; s < RS; ++s) r[s] = 0;
#pragma unroll
                    for (int s2 = 0; s2 < RS; ++s2) {
                        const unsigned m2 = __ballot_sync(0xffffffffu, x[s2] != kKeyMax);
                        for (unsigned mm = m2; mm; mm &= mm - 1) {
                            const int src = __ffs(mm) - 1;
                            const uint64_t y = __shfl_sync(0xffffffffu, x[s2], src);
#pragma unroll
                            for (int s = 0; s < RS; ++s) {
                                const bool before = (RS == 1) ? (y < x[s])
                                    : (y < x[s] || (y == x[s] && src + 32 * s2 < lane + 32 * s));
                                r[s] += before ? 1 : 0;
                            }
                        }
                    }
                    __syncwarp();
#pragma unroll
                    for (int s = 0; s < RS; ++s)
                        if (x[s] != kKeyMax) nk[r[s]] = x[s];
                    __syncwarp();
#pragma unroll
                    for (int s = 0; s < RS; ++s) x[s] = (s == 0 && lane < live) ? nk[lane] : kKeyMax;
                } else {
                    sort_keys<RS>(x, lane);
                }
                BOA_T_MARK(7);

                // rank of every new key in the pool, found by the whole warp for one key at
                // a time: lane l holds the last key of the l-th block of `stride` pool entries;
                // one ballot finds the block, a second one the place inside it.  Keys the
                // pool already holds (same key, expanded or not) are dropped.
                bool dup_s[RS];
#pragma unroll
                for (int s = 0; s < RS; ++s) { rank_s[s] = 0; dup_s[s] = false; }
                if (W > 1) {
                    // two rows of one iteration can hold the same id, and the table may have
                    // forgotten it in between: equal keys are neighbours after the sort, the
                    // later one is dropped
#pragma unroll
                    for (int s = 0; s < RS; ++s) {
                        uint64_t pv = __shfl_up_sync(0xffffffffu, x[s], 1);
                        if (s > 0) {
                            const uint64_t last = __shfl_sync(0xffffffffu, x[s - 1], 31);
                            if (lane == 0) pv = last;
                        }
                        dup_s[s] = (s > 0 || lane > 0) && x[s] != kKeyMax && pv == x[s];
                    }
                }
                if (live <= 10) {
                    const int stride = (n + 31) >> 5;
                    const int pend = ((lane + 1) * stride < n) ? (lane + 1) * stride : n;
                    const uint64_t piv = (lane * stride < n) ? (pool[pend - 1] | 1ull) : kKeyMax;
#pragma unroll 2
                    for (int j = 0; j < live; ++j) {
                        const uint64_t xj = __shfl_sync(0xffffffffu, x[0], j) | 1ull;
                        const int base = __popc(__ballot_sync(0xffffffffu, piv < xj)) * stride;
                        const int idx = base + lane;
                        const uint64_t e = (lane < stride && idx < n) ? (pool[idx] | 1ull) : kKeyMax;
                        int r = base + __popc(__ballot_sync(0xffffffffu, e < xj));
                        r = r < n ? r : n;
                        const bool dj = __ballot_sync(0xffffffffu, e == xj) != 0u;
                        if (j == lane) { rank_s[0] = r; dup_s[0] = dup_s[0] || dj; }
                    }
                } else {
                    // many keys: every lane searches for its own (4-ary, same trip count for
                    // all lanes, selects instead of branches)
                    int trips = 0;
                    for (int span = n; span > 0; span >>= 2) ++trips;
#pragma unroll
                    for (int s = 0; s < RS; ++s) {
                        const uint64_t xo = x[s] | 1ull;
                        int lo_i = 0, hi_i = (x[s] != kKeyMax) ? n : 0;
                        for (int it = 0; it < trips; ++it) {
                            const int len = hi_i - lo_i;
                            const bool on = len > 0;
                            const int q1 = lo_i + (len >> 2), q2 = lo_i + (len >> 1);
                            const int q3 = lo_i + ((3 * len) >> 2);
                            const uint64_t k1 = pool[on ? q1 : 0] | 1ull;
                            const uint64_t k2 = pool[on ? q2 : 0] | 1ull;
                            const uint64_t k3 = pool[on ? q3 : 0] | 1ull;
                            const bool c1 = k1 < xo, c2 = k2 < xo, c3 = k3 < xo;
                            const int nlo = c3 ? q3 + 1 : (c2 ? q2 + 1 : (c1 ? q1 + 1 : lo_i));
                            const int nhi = c3 ? hi_i : (c2 ? q3 : (c1 ? q2 : q1));
                            lo_i = on ? nlo : lo_i;
                            hi_i = on ? nhi : hi_i;
                        }
                        rank_s[s] = lo_i;
                        dup_s[s] = dup_s[s] || ((lo_i < n) && ((pool[lo_i] | 1ull) == xo));
                    }
                }
#pragma unroll
                for (int s = 0; s < RS; ++s) {
                    const bool valid = x[s] != kKeyMax;
                    const int lo_i = rank_s[s];
                    const bool dup = valid && dup_s[s];
#ifdef BOA_SECTION_TIMERS
                    t_acc_[11] += __popc(__ballot_sync(0xffffffffu, dup));   // keys found again in the pool
#endif
                    const bool nd = valid && !dup;
                    const unsigned bal = __ballot_sync(0xffffffffu, nd);
                    const int pidx = kept + __popc(bal & lt_mask);
                    pos_new[s] = lo_i + pidx;
                    keep[s] = nd && (pos_new[s] < p.C);
                    kept += __popc(__ballot_sync(0xffffffffu, keep[s]));
                }
                BOA_T_MARK(8);
            }
            if (kept == 0) {
                // pool unchanged: the next node is simply the next unexpanded entry
                if (PRED) {
                    pos = pred_pos;
#pragma unroll
                    for (int s = 0; s < RS; ++s) nb[s] = nbp[s];
                    have_row = pos >= 0;
                } else {
                    pos = first_unexpanded(cur, n < p.L ? n : p.L);
                }
                continue;
            }
            // smallest rank among the kept keys = rank of the first kept key; and that key
            int rmin = 0;
            uint64_t first_new = 0;
#pragma unroll
            for (int s = RS - 1; s >= 0; --s) {
                const unsigned kb = __ballot_sync(0xffffffffu, keep[s]);
                if (kb) {
                    rmin = __shfl_sync(0xffffffffu, rank_s[s], __ffs(kb) - 1);
                    first_new = __shfl_sync(0xffffffffu, x[s], __ffs(kb) - 1);
                }
            }

            // ---- which node is expanded next?  Decide on the pool as it is, translate the
            // position, and start loading that node's adjacency row before the merge.
            {
                const int lim_old = n < p.L ? n : p.L;
                const int pos_old = PRED ? pred_pos : first_unexpanded(cur, lim_old);
                int pos_old_new = -1;
                if (pos_old >= 0) {
                    int sh = 0;                       // kept keys ranked at or before it
#pragma unroll
                    for (int s = 0; s < RS; ++s)
                        sh += __popc(__ballot_sync(0xffffffffu, keep[s] && rank_s[s] <= pos_old));
                    pos_old_new = pos_old + sh;
                }
                const int n_new = (n + kept < p.C) ? n + kept : p.C;
                const int lim_new = n_new < p.L ? n_new : p.L;
                if (W == 1) {
                    int next_pos;
                    const bool new_first = pos_old_new < 0 || rmin < pos_old_new;
                    if (new_first) next_pos = rmin;              // the smallest new key comes first
                    else next_pos = pos_old_new;
                    if (next_pos >= lim_new) next_pos = -1;
                    pos = next_pos;
                    if (pos >= 0 && n_exp < p.max_expand) {
                        if (new_first || !PRED) {
                            load_row_ids(key_id(fin, new_first ? first_new : pool[pos_old]), nb, 0);
                        } else {
#pragma unroll
                            for (int s = 0; s < RS; ++s) nb[s] = nbp[s];     // requested a pass ago
                        }
                        have_row = true;
                    }
                } else {
                    // the next two nodes are the two smallest merged places among: the first
                    // two unexpanded old entries and the first two kept new keys
                    constexpr int kNone = 0x7fffffff;
                    const int a0 = pos_old_new >= 0 ? pos_old_new : kNone;
                    const uint32_t a0id = pos_old >= 0 ? key_id(fin, pool[pos_old]) : kNoId;
                    int a1 = kNone;
                    uint32_t a1id = kNoId;
                    if (pos_old >= 0) {
                        const int o2 = first_unexpanded(pos_old + 1, lim_old);
                        if (o2 >= 0) {
                            int sh = 0;
#pragma unroll
                            for (int s = 0; s < RS; ++s)
                                sh += __popc(__ballot_sync(0xffffffffu, keep[s] && rank_s[s] <= o2));
                            a1 = o2 + sh;
                            a1id = key_id(fin, pool[o2]);
                        }
                    }
                    const int b0 = rmin;
                    const uint32_t b0id = key_id(fin, first_new);
                    int b1 = kNone;
                    uint32_t b1id = kNoId;
                    {
                        bool skipped = false;
#pragma unroll
                        for (int s = 0; s < RS; ++s) {
                            unsigned mk = __ballot_sync(0xffffffffu, keep[s]);
                            if (!skipped && mk) { mk &= mk - 1; skipped = true; }
                            if (b1 == kNone && mk) {
                                const int src = __ffs(mk) - 1;
                                b1 = __shfl_sync(0xffffffffu, pos_new[s], src);
                                b1id = key_id(fin, __shfl_sync(0xffffffffu, x[s], src));
                            }
                        }
                    }
                    int p1, p2;
                    uint32_t id1, id2;
                    if (a0 < b0) {
                        p1 = a0; id1 = a0id;
                        if (a1 < b0) { p2 = a1; id2 = a1id; } else { p2 = b0; id2 = b0id; }
                    } else {
                        p1 = b0; id1 = b0id;
                        if (a0 < b1) { p2 = a0; id2 = a0id; } else { p2 = b1; id2 = b1id; }
                    }
                    if (p1 >= lim_new) p1 = -1;
                    if (p1 < 0 || p2 >= lim_new || !(n_exp + 1 < p.max_expand)) p2 = -1;
                    pos = p1;
                    pos2 = p2;
                    if (pos >= 0 && n_exp < p.max_expand) {
                        load_row_ids(id1, nb, 0);
                        load_row_ids(pos2 >= 0 ? id2 : kNoId, nb, RN);
                        have_row = true;
                    }
                }
            }

            // ---- merge.  A bitmap marks the places the new keys take in the merged pool;
            // every other place d receives the old entry d - (new places before d).  Places
            // are filled four 32-entry chunks at a time, top chunks first, all reads of a
            // group before its writes (a source never lies above its destination).
            {
                uint32_t* occ = cand;                    // 32 words: places < 1024
                uint32_t* pre = reinterpret_cast<uint32_t*>(nk);   // new places before each word (nk is free here)
                occ[lane] = 0u;
                __syncwarp();
#pragma unroll
                for (int s = 0; s < RS; ++s)
                    if (keep[s]) atomicOr(&occ[pos_new[s] >> 5], 1u << (pos_new[s] & 31));
                __syncwarp();
                {
                    const int c_l = __popc(occ[lane]);
                    int inc = c_l;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const int t = __shfl_up_sync(0xffffffffu, inc, o);
                        if (lane >= o) inc += t;
                    }
                    pre[lane] = (uint32_t)(inc - c_l);
                }
                __syncwarp();
                const int n_new = (n + kept < p.C) ? n + kept : p.C;
                const int top = (n_new - 1) >> 5, bot = rmin >> 5;
                for (int ct = top; ct >= bot; ct -= 4) {
                    uint64_t e[4];
                    bool wr[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int c = ct - u;
                        const int cc = c >= bot ? c : bot;
                        const int d = cc * 32 + lane;
                        const uint32_t w = occ[cc];
                        const int src = d - (int)pre[cc] - __popc(w & lt_mask);
                        wr[u] = (c >= bot) && !((w >> lane) & 1u) && (d >= rmin) && (d < n_new) && (src != d);
                        e[u] = wr[u] ? pool[src] : 0ull;
                    }
                    __syncwarp();
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (wr[u]) pool[(ct - u) * 32 + lane] = e[u];
                    __syncwarp();
                }
#pragma unroll
                for (int s = 0; s < RS; ++s)
                    if (keep[s]) pool[pos_new[s]] = x[s];
                n = n_new;
                if (rmin < cur) cur = rmin;
                __syncwarp();
            }
            BOA_T_MARK(9);
        }
        // ---- result: the k nearest filter-valid entries; V = the valid ones among the first L
        const int lim = n < p.L ? n : p.L;
        int nv_beam = 0;            // |V|
        float d2k = 0.0f, d2max = 0.0f;     // k-th and last distance of V
        int n_rr = 0;               // PQ: rows fetched for the final ranking
        if (PQ) {
            // Final ranking by exact distance: the filter-valid beam entries, 32 pool places at a
            // time, are scored exactly (same code as the exact search) and merged into the 32
            // best keys found so far, kept sorted in shared memory as (d^2 bits, id).
            topk[lane] = kKeyMax;
            uint32_t mx = 0u;                         // largest exact d^2 (its bits) over V
            __syncwarp();
            for (int b0 = 0; b0 < lim; b0 += 32) {
                const int i = b0 + lane;
                const uint64_t e = (i < lim) ? pool[i] : 0ull;
                const bool ok = (i < lim) && (key_phi(fin, e) == 0u);
                const unsigned bal = __ballot_sync(0xffffffffu, ok);
                const int cntc = __popc(bal);
                if (cntc == 0) continue;
                if (ok) cand[__popc(bal & lt_mask)] = key_id(fin, e);
                __syncwarp();
                score(cntc);
                uint64_t x2[2];
                x2[0] = kKeyMax;
                if (lane < cntc) {
                    const uint64_t kx = nk[lane];
                    const uint32_t bits = __float_as_uint(key_d2(fin, kx));
                    x2[0] = ((uint64_t)bits << 32) | key_id(fin, kx);
                    mx = bits > mx ? bits : mx;
                }
                x2[1] = topk[lane];
                __syncwarp();
                sort_keys<2>(x2, lane);
                topk[lane] = x2[0];
                n_rr += cntc;
                __syncwarp();
            }
            mx = __reduce_max_sync(0xffffffffu, mx);
            nv_beam = n_rr;
            for (int i = lane; i < p.k; i += 32) {
                uint32_t id = kNoId;
                float d2 = __int_as_float(0x7f800000);
                if (i < n_rr && i < kPqMaxK) {
                    const uint64_t kx = topk[i];
                    id = (uint32_t)kx;
                    d2 = __uint_as_float((uint32_t)(kx >> 32));
                }
                p.out_ids[(size_t)qi * p.k + i] = id;
                p.out_d2[(size_t)qi * p.k + i] = d2;
            }
            if (nv_beam > p.k) {
                d2k = __uint_as_float((uint32_t)(topk[p.k - 1] >> 32));
                d2max = __uint_as_float(mx);
            }
        } else if (!fin) {
            // valid entries sort first
            for (int b0 = 0; b0 < lim; b0 += 32) {
                const int i = b0 + lane;
                const bool ok = (i < lim) && (key_phi(false, pool[i]) == 0u);
                nv_beam += __popc(__ballot_sync(0xffffffffu, ok));
            }
            for (int i = lane; i < p.k; i += 32) {
                uint32_t id = kNoId;
                float d2 = __int_as_float(0x7f800000);
                if (i < n) {
                    const uint64_t e = pool[i];
                    if (key_phi(false, e) == 0u) { id = key_id(false, e); d2 = key_d2(false, e); }
                }
                p.out_ids[(size_t)qi * p.k + i] = id;
                p.out_d2[(size_t)qi * p.k + i] = d2;
            }
            if (nv_beam > p.k) {
                d2k = key_d2(false, pool[p.k - 1]);
                d2max = key_d2(false, pool[nv_beam - 1]);
            }
        } else {
            // valid entries lie among invalid ones: one pass over the pool
            int have = 0;           // valid entries met so far
            for (int b0 = 0; b0 < n; b0 += 32) {
                const int i = b0 + lane;
                const uint64_t e = (i < n) ? pool[i] : 0ull;
                const bool ok = (i < n) && (key_phi(true, e) == 0u);
                const float d2 = key_d2(true, e);           // phi == 0: the score is d^2
                const unsigned bal = __ballot_sync(0xffffffffu, ok);
                const int r = have + __popc(bal & lt_mask);
                if (ok && r < p.k) {
                    p.out_ids[(size_t)qi * p.k + r] = key_id(true, e);
                    p.out_d2[(size_t)qi * p.k + r] = d2;
                }
                const unsigned balb = __ballot_sync(0xffffffffu, ok && i < lim);
                const int rb = nv_beam + __popc(balb & lt_mask);
                const unsigned kth = __ballot_sync(0xffffffffu, ok && i < lim && rb == p.k - 1);
                if (kth) d2k = __shfl_sync(0xffffffffu, d2, __ffs(kth) - 1);
                if (balb) d2max = __shfl_sync(0xffffffffu, d2, 31 - __clz(balb));
                nv_beam += __popc(balb);
                have += __popc(bal);
            }
            for (int i = lane; i < p.k; i += 32)
                if (i >= have) {
                    p.out_ids[(size_t)qi * p.k + i] = kNoId;
                    p.out_d2[(size_t)qi * p.k + i] = __int_as_float(0x7f800000);
                }
        }

        // ---- confidence test (Eq. 3) and compaction of the uncertain
        bool uncertain = true;
        if (nv_beam > p.k) {
            if (p.eps_mode < 0) uncertain = true;
            else if (p.eps_mode > 0) uncertain = false;
            else uncertain = !(d2k >= p.c_eps * d2max);
        }
        if (lane == 0) {
            p.final_L[qi] = p.L;
            if (p.first_phase) {
                p.n_expand[qi] = n_exp;
                p.n_scored[qi] = n_sc;
                p.flags[qi] = capped ? 1 : 0;
                p.n_rerank[qi] = n_rr;
            } else {
                p.n_expand[qi] += n_exp;
                p.n_scored[qi] += n_sc;
                if (capped) p.flags[qi] |= 1;
                if (PQ) p.n_rerank[qi] += n_rr;
            }
        }
        if (uncertain && !p.last_phase) {
            if (p.spill_out) {
                uint64_t* dst = p.spill + (size_t)qi * p.spill_stride;
                for (int i = lane; i < n; i += 32) dst[i] = pool[i];
                if (lane == 0) p.spill_size[qi] = n;
            }
            if (lane == 0) {
                const uint32_t slot = atomicAdd(p.out_count, 1u);
                p.out_list[slot] = qi;
            }
        }
        __syncwarp();
        BOA_T_MARK(10);
    }
    BOA_T_FLUSH(p.timers);
}

}  // namespace boa

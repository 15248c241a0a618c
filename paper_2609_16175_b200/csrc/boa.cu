// C interface of the library: index construction, the phase driver of Algorithm 1
// (BOA) and the overlapped schedule of BOA+, statistics.  sm_100a only.
#include "../../include/boa.h"

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <new>

#include "boa_search.cuh"

namespace {

thread_local int g_last_cuda = 0;

#define BOA_CUDA(expr)                                   \
    do {                                                 \
        cudaError_t e__ = (expr);                        \
        if (e__ != cudaSuccess) {                        \
            g_last_cuda = (int)e__;                      \
            return e__ == cudaErrorMemoryAllocation ? BOA_ENOMEM : BOA_ECUDA; \
        }                                                \
    } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The index's buffers live on the device that was current when it was built: a search
// launched with another device current would hand its kernels foreign pointers.
inline bool on_device(int device)
{
    int cur = -1;
    return cudaGetDevice(&cur) == cudaSuccess && cur == device;
}

// ------------------------------------------------------------------ index build kernels
// Record i = [vector bytes | zero padding], rec_stride bytes.  The attribute cells live in
// an array of their own ([N][m], a few MB that stay in L2), so a scored row costs whole
// 64-byte DRAM bursts of vector data only.
__global__ void build_records_kernel(const uint8_t* __restrict__ vec, const int32_t* __restrict__ attrs,
                                     uint8_t* __restrict__ rec, int64_t N, int vec_bytes, int m,
                                     int stride)
{
    const int cps = stride / 16;
    const int64_t total = N * cps;
    for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = idx / cps;
        const int off = (int)(idx % cps) * 16;
        uint4 v;
        if (off + 16 <= vec_bytes) {
            v = *reinterpret_cast<const uint4*>(vec + row * vec_bytes + off);
        } else {
            uint32_t w[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int a = (off + 4 * t - vec_bytes) / 4;
                w[t] = (a >= 0 && a < m) ? (uint32_t)attrs[row * m + a] : 0u;
            }
            v = make_uint4(w[0], w[1], w[2], w[3]);
        }
        *reinterpret_cast<uint4*>(rec + row * stride + off) = v;
    }
}

// Copy the graph; self references and repeats inside a row become BOA_NO_ID, so the
// search never meets one id twice in a row.  Flags ids >= N.
__global__ void clean_graph_kernel(const uint32_t* __restrict__ in, uint32_t* __restrict__ out,
                                   int64_t N, int R, int* __restrict__ bad)
{
    for (int64_t row = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; row < N;
         row += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t* src = in + row * R;
        uint32_t* dst = out + row * R;
        for (int j = 0; j < R; ++j) {
            uint32_t id = src[j];
            if (id != BOA_NO_ID) {
                if ((int64_t)id >= N) { atomicOr(bad, 1); id = BOA_NO_ID; }
                else if ((int64_t)id == row) id = BOA_NO_ID;
                else {
                    for (int t = 0; t < j; ++t)
                        if (src[t] == id) { id = BOA_NO_ID; break; }
                }
            }
            dst[j] = id;
        }
    }
}

__device__ __forceinline__ double elem_at(const void* vec, int dtype, int64_t i)
{
    return dtype == BOA_U8 ? (double)reinterpret_cast<const uint8_t*>(vec)[i]
                           : (double)reinterpret_cast<const float*>(vec)[i];
}

// partial[b][d] = sum over rows b, b+nb, b+2nb, ... of x[row][d]   (fixed order)
__global__ void column_partial_kernel(const void* vec, int dtype, int64_t N, int D, double* partial)
{
    const int nb = gridDim.x;
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
        double s = 0.0;
        for (int64_t r = blockIdx.x; r < N; r += nb) s += elem_at(vec, dtype, r * D + d);
        partial[(size_t)blockIdx.x * D + d] = s;
    }
}
__global__ void column_mean_kernel(const double* partial, int nb, int64_t N, int D, double* mean)
{
    const int d = blockIdx.x * blockDim.x + threadIdx.x;
    if (d >= D) return;
    double s = 0.0;
    for (int b = 0; b < nb; ++b) s += partial[(size_t)b * D + d];
    mean[d] = s / (double)N;
}
// One warp per point: squared distance to the mean in double; per-block argmin.
__global__ void medoid_block_kernel(const void* vec, int dtype, int64_t N, int D, const double* mean,
                                    double* best_d, int64_t* best_i)
{
    __shared__ double sd[8];
    __shared__ int64_t si[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double bd = INFINITY;
    int64_t bi = INT64_MAX;
    for (int64_t r = blockIdx.x * 8 + warp; r < N; r += (int64_t)gridDim.x * 8) {
        double s = 0.0;
        for (int d = lane; d < D; d += 32) {
            const double x = elem_at(vec, dtype, r * D + d) - mean[d];
            s += x * x;
        }
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (s < bd || (s == bd && r < bi)) { bd = s; bi = r; }
    }
    if (lane == 0) { sd[warp] = bd; si[warp] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w)
            if (sd[w] < bd || (sd[w] == bd && si[w] < bi)) { bd = sd[w]; bi = si[w]; }
        best_d[blockIdx.x] = bd;
        best_i[blockIdx.x] = bi;
    }
}

__global__ void fill_outputs_kernel(uint32_t* ids, float* d2, int64_t n, int32_t* final_L,
                                    int32_t* n_expand, int32_t* n_scored, int32_t* flags, int32_t* n_rerank,
                                    int64_t Q)
{
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n;
         i += (int64_t)gridDim.x * blockDim.x) {
        ids[i] = BOA_NO_ID;
        d2[i] = __int_as_float(0x7f800000);
        if (i < Q) { final_L[i] = 0; n_expand[i] = 0; n_scored[i] = 0; flags[i] = 0; n_rerank[i] = 0; }
    }
}

// Cosine metric: scale rows to unit length.  One thread per row: the sum of squares runs in
// double over the elements in ascending order, the row is multiplied by 1/sqrt(sum) in double
// and rounded to float (a zero row stays zero).  dst may be src.
__global__ void unit_rows_kernel(const float* src, int64_t src_stride, float* dst, int64_t dst_stride,
                                 int64_t n, int D)
{
    for (int64_t r = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; r < n; r += (int64_t)gridDim.x * blockDim.x) {
        const float* x = src + r * src_stride;
        float* y = dst + r * dst_stride;
        double s = 0.0;
        for (int i = 0; i < D; ++i) s += (double)x[i] * (double)x[i];
        const double inv = s > 0.0 ? 1.0 / sqrt(s) : 0.0;
        for (int i = 0; i < D; ++i) y[i] = (float)((double)x[i] * inv);
    }
}

// out[i] *= 0.5 (cosine distance = half the squared distance of the unit vectors); +inf stays
__global__ void halve_kernel(float* out, int64_t n)
{
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        out[i] *= 0.5f;
}

// dst[0] = src[0]: freezes a survivor count at a point of a stream's order.
__global__ void copy_word_kernel(uint32_t* dst, const uint32_t* src) { *dst = *src; }

}  // namespace

// ------------------------------------------------------------------ the index
struct boa_index {
    int64_t N = 0;
    int D = 0, m = 0, R = 0, vec_dtype = 0;
    int rec_stride = 0, nchunks = 0;
    uint32_t* attr_cells = nullptr;    // [N][m] attribute cells
    uint32_t attr_float_mask = 0;
    uint32_t attr_set_mask = 0;        // columns holding membership masks
    float* pen_scales = nullptr;       // [8] device copy of the range-penalty scales, or null (count)
    int64_t entry = 0;
    uint8_t* rec = nullptr;
    uint32_t* graph = nullptr;
    int device = 0, num_sms = 0;
    int shared = 0;                    // made by boa_index_share: rec, attr_cells, graph, pq_* belong to another handle
    int metric = BOA_METRIC_L2;
    // device staging of boa_search_host: queries [ws_host_Q][D], lo and hi [ws_host_Q][m], outputs [ws_host_Q][ws_host_k]
    float* hq = nullptr; int32_t* hlo = nullptr; int32_t* hhi = nullptr; uint32_t* hids = nullptr; float* hd2 = nullptr;
    int64_t ws_host_Q = 0;
    int ws_host_k = 0;
    int chains = 0;                    // 2: the batch is searched as two halves, each on a stream of its own; 1: as one; 0: chosen per call
    int last_split = 0;
    int64_t plus_min_sub = 0;          // smallest BOA+ sub-batch; 0 = twice the resident query warps
    int host_in_place = 1;             // boa_search_host reads mapped page-locked buffers in place
    float* qunit = nullptr;            // [ws_qunit][D] unit-length copies of a batch's queries (cosine)
    int64_t ws_qunit = 0;
    // product quantisation (optional)
    uint8_t* pq_codes = nullptr;       // [N][pq_M]
    float* pq_pivots = nullptr;        // [pq_M][pq_K][D / pq_M]
    int pq_M = 0, pq_K = 0, use_pq = 0;
    // parameters
    double eps = 0.05, growth = 4.0, tau = 0.0;
    int mode = 0, plus_k = 0, cap_mult = 8, cap_add = 64, table_kb = 0, max_ctas = 0, expand_w = 1, table_tags = 0;
    double lambda = INFINITY;          // weight of the filter penalty; infinity = lexicographic keys
    int n_sched = 0;
    int sched[BOA_MAX_PHASES] = {0};
    // scratch
    int64_t ws_Q = 0;
    int ws_spill = 0;
    uint32_t* lists = nullptr;     // [2][BOA_MAX_PHASES][ws_Q]: survivor lists (second set: BOA+ pool 2)
    uint32_t* counters = nullptr;  // see enum below
    int32_t* stats = nullptr;      // [5][ws_Q]
    uint64_t* spill = nullptr;     // [ws_Q][ws_spill]
    int32_t* spill_size = nullptr; // [ws_Q]
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    // last search
    int64_t last_Q = 0;
    int last_phases = 0;
    int last_launches = 0;
    int last_widths[BOA_MAX_PHASES] = {0};
};

namespace {
// layout of boa_index::counters (uint32 words)
constexpr int kCntCount = 0;                          // [P+1] survivors entering phase p (p>=1)
constexpr int kCntCount2 = 16;                        // [P+1] the same for the second pool of BOA+ (p>=2)
constexpr int kCntSnap = 32;                          // [pool] frozen end of phase 1's list
constexpr int kCntStatus = 47;                        // device status bits
constexpr int kCntTicket = 48;                        // one per launch
constexpr int kMaxLaunches = 128;
constexpr int kCntWords = kCntTicket + kMaxLaunches;   // 176: the 64-bit words after it stay aligned
#ifdef BOA_SECTION_TIMERS
constexpr size_t kTimerBytes = 12 * sizeof(unsigned long long);   // debug builds: cycle counters
#else
constexpr size_t kTimerBytes = 0;
#endif

// ---- scratch of boa_search_noalloc: lives in the library image, never allocated
constexpr int64_t kNoAllocMaxQ = BOA_NOALLOC_MAX_Q;
constexpr int kNoAllocMaxWidth = BOA_NOALLOC_MAX_WIDTH;
constexpr size_t kNaCounters = 0;                                             // 1 KiB
constexpr size_t kNaLists = 1024;                                             // [phases][Q] u32
constexpr size_t kNaStats = kNaLists + (size_t)2 * BOA_MAX_PHASES * kNoAllocMaxQ * 4;
constexpr size_t kNaSpillSize = kNaStats + (size_t)5 * kNoAllocMaxQ * 4;
constexpr size_t kNaSpill = kNaSpillSize + (size_t)kNoAllocMaxQ * 4;
constexpr size_t kNaBytes = kNaSpill + (size_t)kNoAllocMaxQ * kNoAllocMaxWidth * 8;
static_assert(kCntWords * 4 + kTimerBytes <= 1024, "counter block must fit its slot");
static_assert(kNaSpill % 256 == 0 && kNaStats % 256 == 0, "sub-buffers stay aligned");

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNaBytes];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an address a
// kernel can use: the device address is asked for once per device and kept here.
constexpr int kMaxDevices = 64;
std::atomic<unsigned char*> g_noalloc_ptr[kMaxDevices];

int noalloc_scratch(unsigned char** out)
{
    int dev = 0;
    BOA_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return BOA_EINVAL;
    unsigned char* cached = g_noalloc_ptr[dev].load(std::memory_order_acquire);
    if (!cached) {
        // two threads may both ask; they get the same address
        void* ptr = nullptr;
        BOA_CUDA(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
        cached = static_cast<unsigned char*>(ptr);
        g_noalloc_ptr[dev].store(cached, std::memory_order_release);
    }
    *out = cached;
    return BOA_OK;
}

static_assert(BOA_PQ_MAX_K == boa::kPqMaxK, "header and kernel agree on the largest k of a PQ search");

typedef void (*SearchKernel)(const boa::SearchParams);

struct KernelChoice {
    SearchKernel fn;
    int rs;
    bool q_in_smem;     // the generic-length kernels keep the query in shared memory
};

template <int VT, int CPL, int W, bool PQ, bool EXT>
KernelChoice pick_rn(int R, bool exact)
{
    if (R <= 32) {
        if (exact) return {boa::boa_search_kernel<VT, 1, W, CPL, (CPL > 0), PQ, EXT>, W, CPL == 0 && !PQ};
        return {boa::boa_search_kernel<VT, 1, W, CPL, false, PQ, EXT>, W, CPL == 0 && !PQ};
    }
    if (exact) return {boa::boa_search_kernel<VT, 2, W, CPL, (CPL > 0), PQ, EXT>, 2 * W, CPL == 0 && !PQ};
    return {boa::boa_search_kernel<VT, 2, W, CPL, false, PQ, EXT>, 2 * W, CPL == 0 && !PQ};
}
template <int VT, int CPL>
KernelChoice pick_rs(int R, bool exact, int expand_w, bool pq, bool ext)
{
    if (pq) return pick_rn<VT, CPL, 1, true, false>(R, exact);
    if (ext) return pick_rn<VT, CPL, 1, false, true>(R, exact);
    return expand_w == 2 ? pick_rn<VT, CPL, 2, false, false>(R, exact) : pick_rn<VT, CPL, 1, false, false>(R, exact);
}

KernelChoice pick_kernel(const boa_index* ix)
{
    const int cpl = (ix->nchunks + 7) / 8;      // 16-byte chunks per lane of an 8-lane group
    const bool exact = ix->nchunks == 8 * cpl;
    const bool pq = ix->use_pq != 0;
    const bool ext = ix->attr_set_mask != 0 || ix->pen_scales != nullptr;
    if (ix->vec_dtype == BOA_F32) {
        switch (cpl) {
            case 1: return pick_rs<0, 1>(ix->R, exact, ix->expand_w, pq, ext);
            case 2: return pick_rs<0, 2>(ix->R, exact, ix->expand_w, pq, ext);
            case 3: return pick_rs<0, 3>(ix->R, exact, ix->expand_w, pq, ext);
            case 4: return pick_rs<0, 4>(ix->R, exact, ix->expand_w, pq, ext);
            default: return pick_rs<0, 0>(ix->R, false, ix->expand_w, pq, ext);
        }
    }
    switch (cpl) {
        case 1: return pick_rs<1, 1>(ix->R, exact, ix->expand_w, pq, ext);
        case 2: return pick_rs<1, 2>(ix->R, exact, ix->expand_w, pq, ext);
        default: return pick_rs<1, 0>(ix->R, false, ix->expand_w, pq, ext);
    }
}

// Table of recently scored ids: size in KB (a power of two, or three times one) -> bucket
// count, bucket-group bits and the bits left for group-local addressing.  Buckets are 4
// bytes (three 10-bit tags) when the tags of this index fit 10 bits at that bucket count,
// else 8 bytes (four 16-bit tags).  `tags` forces the wide form when it is 16.
struct TableShape { int bytes, narrow, mul3, id_bits, low_bits; };
TableShape choose_table(const boa_index* ix, int default_kb)
{
    int kb_size = ix->table_kb ? ix->table_kb : default_kb;
    TableShape t;
    t.id_bits = 1;
    while (((int64_t)1 << t.id_bits) < ix->N) ++t.id_bits;
    for (;;) {
        t.mul3 = (kb_size % 3 == 0) ? 1 : 0;
        t.bytes = kb_size * 1024;
        for (t.narrow = (ix->table_tags == 16 ? 0 : 1); t.narrow >= 0; --t.narrow) {
            const int groups = (t.mul3 ? kb_size / 3 : kb_size) * (t.narrow ? 256 : 128);   // 2^kb
            int kb = 0;
            while ((1 << kb) < groups) ++kb;
            if (kb > t.id_bits) kb = t.id_bits;
            t.low_bits = t.id_bits - kb;
            // tags must fit; an id whose tag is all ones (the empty mark) is simply never
            // recorded, which the narrow form accepts for one id in 1024
            const uint32_t max_tag = ((1u << t.low_bits) - 1u) / (t.mul3 ? 3u : 1u);
            if (t.narrow ? max_tag <= 0x3FFu : max_tag < 0xFFFFu) return t;
        }
        t.narrow = 0;
        if (kb_size >= 1024) return t;
        kb_size *= 2;
    }
}

// Default table size of a launch.  The register allocation lets 20 query warps live on an
// SM; their shared memory (plus the 1 KB the system reserves per CTA) has to stay within
// 196 KB, the largest carve-out that still leaves the L1 cache about 60 KB for the rows in
// flight: with the next carve-out step (28 KB of L1) the same kernel ran 35 % slower on the
// 1M x 128-d workload.  So: the largest of 6, 4, 3, 2 KB that fits.  Rows shorter than 256
// bytes need little L1 and take 6 KB; so does a launch that no size fits (query vector in
// shared memory): fewer warps are resident then anyway.
// PQ traversal: a node scored a second time costs one more sum of table look-ups, not a row,
// while the distance table already limits how many warps fit; the smallest table wins there
// (c5, M = 48, K = 64: 1 KB is 10 % faster than 6 KB at every width measured).
int default_table_kb(const boa_index* ix, const KernelChoice& kc, int C)
{
    if (ix->use_pq) return 1;
    if (ix->rec_stride < 256) return 6;
    const int sizes[4] = {6, 4, 3, 2};
    for (int i = 0; i < 4; ++i) {
        const boa::WarpSmem lay = boa::warp_smem_layout(C, sizes[i] * 1024, ix->D, kc.rs, kc.q_in_smem,
                                                        ix->use_pq ? ix->pq_M * ix->pq_K : 0);
        if ((int64_t)BOA_MIN_CTAS * (lay.total + 1024) <= 196 * 1024) return sizes[i];
    }
    return 6;
}

int phase_widths(const boa_index* ix, int L0, int Lmax, int* w)
{
    if (ix->n_sched > 0) {
        for (int i = 0; i < ix->n_sched; ++i) w[i] = ix->sched[i];
        return ix->n_sched;
    }
    int n = 0;
    double cur = L0;
    w[n++] = L0;
    while (w[n - 1] < Lmax && n < BOA_MAX_PHASES) {
        cur = cur * ix->growth;
        int next = cur >= (double)Lmax ? Lmax : (int)cur;
        if (next <= w[n - 1]) next = w[n - 1] + 1;
        if (next > Lmax || n == BOA_MAX_PHASES - 1) next = Lmax;
        w[n++] = next;
    }
    return n;
}

int ensure_workspace(boa_index* ix, int64_t Q, int Lmax)
{
    const int need_spill = ix->mode == 1 ? ((Lmax + 1) & ~1) : 0;
    if (ix->counters == nullptr) {
        BOA_CUDA(cudaMalloc(&ix->counters, kCntWords * sizeof(uint32_t) + kTimerBytes));
        BOA_CUDA(cudaMemset(ix->counters, 0, kCntWords * sizeof(uint32_t) + kTimerBytes));
    }
    if (Q > ix->ws_Q || need_spill > ix->ws_spill) {
        const int64_t nq = Q > ix->ws_Q ? Q : ix->ws_Q;
        const int ns = need_spill > ix->ws_spill ? need_spill : ix->ws_spill;
        cudaFree(ix->lists); cudaFree(ix->stats); cudaFree(ix->spill); cudaFree(ix->spill_size);
        ix->lists = nullptr; ix->stats = nullptr; ix->spill = nullptr; ix->spill_size = nullptr;
        ix->ws_Q = 0; ix->ws_spill = 0;
        BOA_CUDA(cudaMalloc(&ix->lists, (size_t)2 * BOA_MAX_PHASES * nq * sizeof(uint32_t)));
        BOA_CUDA(cudaMalloc(&ix->stats, (size_t)5 * nq * sizeof(int32_t)));
        BOA_CUDA(cudaMalloc(&ix->spill_size, (size_t)nq * sizeof(int32_t)));
        if (ns > 0) BOA_CUDA(cudaMalloc(&ix->spill, (size_t)nq * ns * sizeof(uint64_t)));
        ix->ws_Q = nq;
        ix->ws_spill = ns;
    }
    return BOA_OK;
}

struct LaunchPlan {
    boa_index* ix;
    KernelChoice kc;
    boa::SearchParams base;
    int n_phases;
    int widths[BOA_MAX_PHASES];
    int launches;
};

// One launch of Algorithm 2 over positions [begin, end) of phase p's work list.
// `chain` picks the set of survivor lists and counters (0 everywhere except the second
// pooled escalation of BOA+); phase 1 always reads the one list the first phase wrote.
int launch_phase(LaunchPlan& lp, int p, cudaStream_t st, const uint32_t* begin_ptr,
                 const uint32_t* end_ptr, uint32_t begin, uint32_t end, uint32_t expected_items,
                 int chain = 0, bool use_active_count = true, bool own_first = false)
{
    boa_index* ix = lp.ix;
    if (lp.launches >= kMaxLaunches) return BOA_EINVAL;
    boa::SearchParams sp = lp.base;
    const int L = lp.widths[p];
    const int Lmax = lp.widths[lp.n_phases - 1];
    sp.L = L;
    sp.C = ix->mode == 1 ? Lmax : L;
    {
        const TableShape t = choose_table(ix, default_table_kb(ix, lp.kc, sp.C));
        sp.table_bytes = t.bytes; sp.table_narrow = t.narrow; sp.table_mul3 = t.mul3;
        sp.id_bits = t.id_bits; sp.low_bits = t.low_bits;
    }
    sp.max_expand = ix->cap_mult * L + ix->cap_add;
    sp.first_phase = p == 0;
    sp.resume_in = (ix->mode == 1 && p > 0);
    sp.last_phase = p == lp.n_phases - 1;
    sp.spill_out = (ix->mode == 1 && !sp.last_phase);
    uint32_t* lists_c = ix->lists + (size_t)chain * BOA_MAX_PHASES * ix->ws_Q;
    uint32_t* cnt_c = ix->counters + (chain == 0 ? kCntCount : kCntCount2);
    // own_first: the chain's first phase wrote the chain's own phase-1 list (two-chain schedule)
    sp.in_list = p == 0 ? nullptr : ((p == 1 && !own_first) ? ix->lists : lists_c) + (size_t)p * ix->ws_Q;
    sp.in_begin_ptr = begin_ptr;
    sp.in_end_ptr = end_ptr;
    sp.in_begin = begin;
    sp.in_end = end;
    sp.active_count = (p == 0 || !use_active_count) ? nullptr : ix->counters + kCntCount + p;
    sp.ticket = ix->counters + kCntTicket + lp.launches;
    sp.out_list = lists_c + (size_t)(p + 1 < BOA_MAX_PHASES ? p + 1 : p) * ix->ws_Q;
    sp.out_count = cnt_c + p + 1;

    const boa::WarpSmem lay = boa::warp_smem_layout(sp.C, sp.table_bytes, ix->D, lp.kc.rs, lp.kc.q_in_smem,
                                                    ix->use_pq ? ix->pq_M * ix->pq_K : 0);
    const size_t smem = (size_t)lay.total;
    if (smem > 48 * 1024) {
        BOA_CUDA(cudaFuncSetAttribute((const void*)lp.kc.fn, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)smem));
    }
    int per_sm = 0;
    BOA_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, (const void*)lp.kc.fn,
                                                           boa::kThreads, smem));
    if (per_sm < 1) return BOA_EINVAL;
    if (ix->max_ctas > 0 && per_sm > ix->max_ctas) per_sm = ix->max_ctas;
    int64_t grid = (int64_t)per_sm * ix->num_sms;
    const int64_t need = (int64_t)expected_items;
    if (need < grid) grid = need < 1 ? 1 : need;
    lp.kc.fn<<<(unsigned)grid, boa::kThreads, smem, st>>>(sp);
    BOA_CUDA(cudaGetLastError());
    lp.launches++;
    return BOA_OK;
}

}  // namespace

// ------------------------------------------------------------------ C interface
extern "C" {

int boa_last_cuda_error(void) { return g_last_cuda; }

const char* boa_strerror(int status)
{
    switch (status) {
        case BOA_OK: return "ok";
        case BOA_EINVAL: return "invalid argument";
        case BOA_ENOMEM: return "out of memory";
        case BOA_ECUDA: return "CUDA call failed";
        case BOA_EGRAPH: return "graph names a node id outside the index";
        case BOA_ETOOBIG: return "batch or beamwidth beyond the fixed scratch of boa_search_noalloc";
        default: return "unknown status";
    }
}

int boa_index_create(boa_index** out, const void* vectors, int vec_dtype, int64_t N, int D,
                     const void* attrs, const int* attr_types, int m, const uint32_t* graph, int R,
                     int64_t entry, void* stream)
{
    if (!out) return BOA_EINVAL;
    *out = nullptr;
    if (!vectors || !attrs || !attr_types || !graph) return BOA_EINVAL;
    if (N < 1 || N > BOA_MAX_POINTS) return BOA_EINVAL;
    if (m < 1 || m > BOA_MAX_ATTRS || R < 1 || R > BOA_MAX_DEGREE) return BOA_EINVAL;
    if (vec_dtype != BOA_F32 && vec_dtype != BOA_U8) return BOA_EINVAL;
    if (D < 1 || (vec_dtype == BOA_F32 && D % 4 != 0) || (vec_dtype == BOA_U8 && D % 16 != 0))
        return BOA_EINVAL;
    if (D > 16384) return BOA_EINVAL;
    if (!aligned16(vectors) || !aligned16(attrs) || !aligned16(graph)) return BOA_EINVAL;
    if (entry >= N || entry < -1) return BOA_EINVAL;
    for (int j = 0; j < m; ++j)
        if (attr_types[j] != BOA_ATTR_I32 && attr_types[j] != BOA_ATTR_F32 && attr_types[j] != BOA_ATTR_SET32)
            return BOA_EINVAL;

    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    boa_index* ix = new (std::nothrow) boa_index();
    if (!ix) return BOA_ENOMEM;
    auto fail = [&](int code) { boa_index_destroy(ix); return code; };
#define BOA_TRY(expr)                                                      \
    do {                                                                   \
        cudaError_t e__ = (expr);                                          \
        if (e__ != cudaSuccess) {                                          \
            g_last_cuda = (int)e__;                                        \
            return fail(e__ == cudaErrorMemoryAllocation ? BOA_ENOMEM : BOA_ECUDA); \
        }                                                                  \
    } while (0)

    ix->N = N; ix->D = D; ix->m = m; ix->R = R; ix->vec_dtype = vec_dtype;
    const int vec_bytes = vec_dtype == BOA_U8 ? D : 4 * D;
    ix->nchunks = vec_bytes / 16;
    ix->rec_stride = (vec_bytes + 31) & ~31;
    for (int j = 0; j < m; ++j)
        if (attr_types[j] == BOA_ATTR_F32) ix->attr_float_mask |= 1u << j;
        else if (attr_types[j] == BOA_ATTR_SET32) ix->attr_set_mask |= 1u << j;
    BOA_TRY(cudaGetDevice(&ix->device));
    BOA_TRY(cudaDeviceGetAttribute(&ix->num_sms, cudaDevAttrMultiProcessorCount, ix->device));
    BOA_TRY(cudaMalloc(&ix->rec, (size_t)N * ix->rec_stride));
    BOA_TRY(cudaMalloc(&ix->graph, (size_t)N * R * sizeof(uint32_t)));
    BOA_TRY(cudaMalloc(&ix->attr_cells, (size_t)N * m * sizeof(uint32_t)));
    BOA_TRY(cudaMemcpyAsync(ix->attr_cells, attrs, (size_t)N * m * sizeof(uint32_t),
                            cudaMemcpyDeviceToDevice, st));
    BOA_TRY(cudaStreamCreateWithFlags(&ix->side, cudaStreamNonBlocking));
    BOA_TRY(cudaEventCreateWithFlags(&ix->ev_fork, cudaEventDisableTiming));
    BOA_TRY(cudaEventCreateWithFlags(&ix->ev_join, cudaEventDisableTiming));

    const int blocks = ix->num_sms * 8;
    build_records_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const uint8_t*>(vectors),
                                                 reinterpret_cast<const int32_t*>(attrs), ix->rec, N,
                                                 vec_bytes, 0, ix->rec_stride);
    BOA_TRY(cudaGetLastError());
    int* d_bad = nullptr;
    BOA_TRY(cudaMalloc(&d_bad, sizeof(int)));
    cudaError_t e = cudaMemsetAsync(d_bad, 0, sizeof(int), st);
    if (e == cudaSuccess) {
        clean_graph_kernel<<<blocks, 128, 0, st>>>(graph, ix->graph, N, R, d_bad);
        e = cudaGetLastError();
    }
    int h_bad = 0;
    if (e == cudaSuccess) e = cudaMemcpyAsync(&h_bad, d_bad, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    cudaFree(d_bad);
    BOA_TRY(e);
    if (h_bad) return fail(BOA_EGRAPH);

    if (entry >= 0) {
        ix->entry = entry;
    } else {
        // medoid: the point nearest to the coordinate-wise mean, lower id on ties
        const int nb = (int)(N < 1024 ? N : 1024);
        const int mb = (int)((N + 7) / 8 < 2048 ? (N + 7) / 8 : 2048);
        double *partial = nullptr, *mean = nullptr, *bd = nullptr;
        int64_t* bi = nullptr;
        e = cudaMalloc(&partial, (size_t)nb * D * sizeof(double));
        if (e == cudaSuccess) e = cudaMalloc(&mean, (size_t)D * sizeof(double));
        if (e == cudaSuccess) e = cudaMalloc(&bd, (size_t)mb * sizeof(double));
        if (e == cudaSuccess) e = cudaMalloc(&bi, (size_t)mb * sizeof(int64_t));
        double* h_bd = (double*)malloc((size_t)mb * sizeof(double));
        int64_t* h_bi = (int64_t*)malloc((size_t)mb * sizeof(int64_t));
        if (e == cudaSuccess && h_bd && h_bi) {
            column_partial_kernel<<<nb, 128, 0, st>>>(vectors, vec_dtype, N, D, partial);
            column_mean_kernel<<<(D + 127) / 128, 128, 0, st>>>(partial, nb, N, D, mean);
            medoid_block_kernel<<<mb, 256, 0, st>>>(vectors, vec_dtype, N, D, mean, bd, bi);
            e = cudaGetLastError();
            if (e == cudaSuccess)
                e = cudaMemcpyAsync(h_bd, bd, (size_t)mb * sizeof(double), cudaMemcpyDeviceToHost, st);
            if (e == cudaSuccess)
                e = cudaMemcpyAsync(h_bi, bi, (size_t)mb * sizeof(int64_t), cudaMemcpyDeviceToHost, st);
            if (e == cudaSuccess) e = cudaStreamSynchronize(st);
            if (e == cudaSuccess) {
                double best = INFINITY;
                int64_t besti = INT64_MAX;
                for (int b = 0; b < mb; ++b)
                    if (h_bd[b] < best || (h_bd[b] == best && h_bi[b] < besti)) {
                        best = h_bd[b]; besti = h_bi[b];
                    }
                ix->entry = besti;
            }
        }
        const bool host_oom = !h_bd || !h_bi;
        free(h_bd); free(h_bi);
        cudaFree(partial); cudaFree(mean); cudaFree(bd); cudaFree(bi);
        if (host_oom) return fail(BOA_ENOMEM);
        BOA_TRY(e);
    }
#undef BOA_TRY
    *out = ix;
    return BOA_OK;
}

int boa_index_share(boa_index** out, boa_index* src)
{
    if (!out || !src) return BOA_EINVAL;
    if (!on_device(src->device)) return BOA_EINVAL;
    *out = nullptr;
    boa_index* ix = new (std::nothrow) boa_index(*src);      // data pointers and parameters as they stand
    if (!ix) return BOA_ENOMEM;
    ix->shared = 1;
    // everything a search writes is this handle's own, allocated on first use
    ix->hq = nullptr; ix->hlo = nullptr; ix->hhi = nullptr; ix->hids = nullptr; ix->hd2 = nullptr;
    ix->ws_host_Q = 0; ix->ws_host_k = 0;
    ix->qunit = nullptr; ix->ws_qunit = 0;
    ix->ws_Q = 0; ix->ws_spill = 0;
    ix->lists = nullptr; ix->counters = nullptr; ix->stats = nullptr; ix->spill = nullptr; ix->spill_size = nullptr;
    ix->side = nullptr; ix->ev_fork = nullptr; ix->ev_join = nullptr;
    ix->pen_scales = nullptr;
    ix->last_Q = 0; ix->last_phases = 0; ix->last_launches = 0;
    cudaError_t e = cudaStreamCreateWithFlags(&ix->side, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ix->ev_fork, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ix->ev_join, cudaEventDisableTiming);
    if (e == cudaSuccess && src->pen_scales) {
        e = cudaMalloc(&ix->pen_scales, BOA_MAX_ATTRS * sizeof(float));
        if (e == cudaSuccess)
            e = cudaMemcpy(ix->pen_scales, src->pen_scales, BOA_MAX_ATTRS * sizeof(float), cudaMemcpyDeviceToDevice);
    }
    if (e != cudaSuccess) {
        g_last_cuda = (int)e;
        boa_index_destroy(ix);
        return e == cudaErrorMemoryAllocation ? BOA_ENOMEM : BOA_ECUDA;
    }
    *out = ix;
    return BOA_OK;
}

int boa_index_destroy(boa_index* ix)
{
    if (!ix) return BOA_OK;
    if (!ix->shared) {
        cudaFree(ix->rec); cudaFree(ix->attr_cells); cudaFree(ix->graph);
        cudaFree(ix->pq_codes); cudaFree(ix->pq_pivots);
    }
    cudaFree(ix->lists); cudaFree(ix->counters);
    cudaFree(ix->stats); cudaFree(ix->spill); cudaFree(ix->spill_size);
    cudaFree(ix->qunit); cudaFree(ix->pen_scales);
    cudaFree(ix->hq); cudaFree(ix->hlo); cudaFree(ix->hhi); cudaFree(ix->hids); cudaFree(ix->hd2);
    if (ix->side) cudaStreamDestroy(ix->side);
    if (ix->ev_fork) cudaEventDestroy(ix->ev_fork);
    if (ix->ev_join) cudaEventDestroy(ix->ev_join);
    delete ix;
    return BOA_OK;
}

int64_t boa_index_entry(const boa_index* ix) { return ix ? ix->entry : -1; }

// For the graph builder in this library (not declared in the public header): the index's own
// copy of the graph, which the builder fills in while it searches it.
uint32_t* boa_internal_graph(boa_index* ix) { return ix ? ix->graph : nullptr; }

int boa_set_param(boa_index* ix, int key, double v)
{
    if (!ix || v != v) return BOA_EINVAL;
    switch (key) {
        case BOA_PARAM_EPS: ix->eps = v; return BOA_OK;
        case BOA_PARAM_GROWTH: if (!(v > 1.0)) return BOA_EINVAL; ix->growth = v; return BOA_OK;
        case BOA_PARAM_TAU: if (v < 0.0) return BOA_EINVAL; ix->tau = v; return BOA_OK;
        case BOA_PARAM_MODE: if (v != 0.0 && v != 1.0) return BOA_EINVAL; ix->mode = (int)v; return BOA_OK;
        case BOA_PARAM_PLUS_K:
            if (v < 0.0 || v > 64.0 || v != floor(v)) return BOA_EINVAL;
            ix->plus_k = (int)v; return BOA_OK;
        case BOA_PARAM_CAP_MULT:
            if (v < 0.0 || v > 1024.0 || v != floor(v)) return BOA_EINVAL;
            ix->cap_mult = (int)v; return BOA_OK;
        case BOA_PARAM_CAP_ADD:
            if (v < 0.0 || v > 1e6 || v != floor(v)) return BOA_EINVAL;
            ix->cap_add = (int)v; return BOA_OK;
        case BOA_PARAM_TABLE_KB: {
            const int kb = (int)v;
            bool ok = v == floor(v) && kb >= 0 && kb <= 24;
            if (ok && kb > 0) {
                int t = (kb % 3 == 0) ? kb / 3 : kb;
                ok = (t & (t - 1)) == 0;               // a power of two, or three times one
            }
            if (!ok) return BOA_EINVAL;
            ix->table_kb = kb; return BOA_OK;
        }
        case BOA_PARAM_MAX_WARPS_PER_SM:
            if (v < 0.0 || v > 64.0 || v != floor(v)) return BOA_EINVAL;
            ix->max_ctas = (int)v; return BOA_OK;
        case BOA_PARAM_TABLE_TAGS:
            if (v != 0.0 && v != 16.0) return BOA_EINVAL;
            ix->table_tags = (int)v; return BOA_OK;
        case BOA_PARAM_LAMBDA:
            // finite values must stay finite as fp32: an overflow to +inf would turn the
            // score of every filter-valid node into inf * 0
            if (!(v >= 0.0) || (!isinf(v) && v > 3.4028234663852886e38)) return BOA_EINVAL;
            ix->lambda = v; return BOA_OK;
        case BOA_PARAM_EXPAND_W:
            if (v != 1.0 && v != 2.0) return BOA_EINVAL;
            ix->expand_w = (int)v; return BOA_OK;
        case BOA_PARAM_PQ:
            if ((v != 0.0 && v != 1.0) || (v == 1.0 && !ix->pq_codes)) return BOA_EINVAL;
            ix->use_pq = (int)v; return BOA_OK;
        case BOA_PARAM_CHAINS:
            if (v != 0.0 && v != 1.0 && v != 2.0) return BOA_EINVAL;
            ix->chains = (int)v; return BOA_OK;
        case BOA_PARAM_PLUS_MIN_SUB:
            if (v < 0.0 || v > 2147483647.0 || v != floor(v)) return BOA_EINVAL;
            ix->plus_min_sub = (int64_t)v; return BOA_OK;
        case BOA_PARAM_HOST_IN_PLACE:
            if (v != 0.0 && v != 1.0) return BOA_EINVAL;
            ix->host_in_place = (int)v; return BOA_OK;
        default: return BOA_EINVAL;
    }
}

int boa_set_schedule(boa_index* ix, const int* widths, int n)
{
    if (!ix || n < 0 || n > BOA_MAX_PHASES || (n > 0 && !widths)) return BOA_EINVAL;
    for (int i = 0; i < n; ++i) {
        if (widths[i] < 1 || widths[i] > BOA_MAX_WIDTH) return BOA_EINVAL;
        if (i > 0 && widths[i] <= widths[i - 1]) return BOA_EINVAL;
    }
    ix->n_sched = n;
    for (int i = 0; i < n; ++i) ix->sched[i] = widths[i];
    return BOA_OK;
}

int boa_workspace_bytes(const boa_index* ix, int64_t Q, int Lmax, size_t* bytes)
{
    if (!ix || !bytes || Q < 0 || Lmax < 1 || Lmax > BOA_MAX_WIDTH) return BOA_EINVAL;
    size_t b = kCntWords * sizeof(uint32_t);
    b += (size_t)2 * BOA_MAX_PHASES * Q * sizeof(uint32_t) + (size_t)6 * Q * sizeof(int32_t);
    if (ix->mode == 1) b += (size_t)Q * ((Lmax + 1) & ~1) * sizeof(uint64_t);
    *bytes = b;
    return BOA_OK;
}

int boa_search(boa_index* ix, const float* queries, int64_t Q, const void* lo, const void* hi, int k,
               int L0, int Lmax, uint32_t* out_ids, float* out_dists, void* stream)
{
    if (!ix) return BOA_EINVAL;
    if (Q < 0 || Q > (int64_t)0x7FFFFFFF) return BOA_EINVAL;
    if (k < 1 || k > L0 || L0 > Lmax || Lmax > BOA_MAX_WIDTH) return BOA_EINVAL;
    if (ix->n_sched > 0 && (L0 != ix->sched[0] || Lmax != ix->sched[ix->n_sched - 1])) return BOA_EINVAL;
    if (ix->use_pq && (k > boa::kPqMaxK || ix->expand_w != 1)) return BOA_EINVAL;
    // membership columns and the range penalty have kernels for one node per iteration and
    // exact distances; the penalty is a term of the finite-lambda score
    const bool ext = ix->attr_set_mask != 0 || ix->pen_scales != nullptr;
    if (ext && (ix->use_pq || ix->expand_w != 1)) return BOA_EINVAL;
    if (ix->pen_scales && isinf(ix->lambda)) return BOA_EINVAL;
    if (Q == 0) { ix->last_Q = 0; ix->last_phases = 0; ix->last_launches = 0; return BOA_OK; }
    if (!queries || !lo || !hi || !out_ids || !out_dists) return BOA_EINVAL;
    if (!on_device(ix->device)) return BOA_EINVAL;
    if (!aligned16(queries) || !aligned16(lo) || !aligned16(hi) || !aligned16(out_ids) ||
        !aligned16(out_dists))
        return BOA_EINVAL;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

    int rc = ensure_workspace(ix, Q, Lmax);
    if (rc != BOA_OK) return rc;
    if (ix->metric == BOA_METRIC_COSINE) {
        // the kernels work on unit-length vectors: the index's rows already are, the queries
        // of this batch are copied
        if (Q > ix->ws_qunit) {
            cudaFree(ix->qunit);
            ix->qunit = nullptr; ix->ws_qunit = 0;
            BOA_CUDA(cudaMalloc(&ix->qunit, (size_t)Q * ix->D * sizeof(float)));
            ix->ws_qunit = Q;
        }
        unit_rows_kernel<<<(unsigned)((Q + 127) / 128), 128, 0, st>>>(queries, ix->D, ix->qunit, ix->D, Q, ix->D);
        BOA_CUDA(cudaGetLastError());
        queries = ix->qunit;
    }

    LaunchPlan lp;
    lp.ix = ix;
    lp.kc = pick_kernel(ix);
    lp.n_phases = phase_widths(ix, L0, Lmax, lp.widths);
    lp.launches = 0;
    boa::SearchParams& b = lp.base;
    memset(&b, 0, sizeof(b));
    b.rec = ix->rec; b.graph = ix->graph; b.N = ix->N; b.D = ix->D; b.m = ix->m; b.R = ix->R;
    b.rec_stride = ix->rec_stride; b.nchunks = ix->nchunks;
    b.attrs = ix->attr_cells; b.status = ix->counters + kCntStatus;
#ifdef BOA_SECTION_TIMERS
    b.timers = reinterpret_cast<unsigned long long*>(ix->counters + kCntWords);
#endif
    b.attr_float_mask = ix->attr_float_mask; b.entry = (uint32_t)ix->entry;
    b.attr_set_mask = ix->attr_set_mask; b.pen_scales = ix->pen_scales;
    b.queries = queries;
    b.lo = reinterpret_cast<const int32_t*>(lo);
    b.hi = reinterpret_cast<const int32_t*>(hi);
    b.out_ids = out_ids; b.out_d2 = out_dists; b.Q = Q; b.k = k;
    b.tau_q = ix->tau * (double)Q;
    b.fin = isinf(ix->lambda) ? 0 : 1;
    b.lambda = b.fin ? (float)ix->lambda : 0.0f;
    if (ix->eps < 0.0) b.eps_mode = -1;
    else if (ix->eps >= 1.0) b.eps_mode = 1;
    else {
        // Eq. 3 on norms with squared distances as keys: (1-eps)^2; on cosine distances: 1-eps
        b.eps_mode = 0;
        b.c_eps = ix->metric == BOA_METRIC_COSINE ? (float)(1.0 - ix->eps)
                                                  : (float)((1.0 - ix->eps) * (1.0 - ix->eps));
    }
    b.final_L = ix->stats; b.n_expand = ix->stats + ix->ws_Q; b.n_scored = ix->stats + 2 * ix->ws_Q;
    b.flags = ix->stats + 3 * ix->ws_Q;
    b.n_rerank = ix->stats + 4 * ix->ws_Q;
    b.pq_codes = ix->pq_codes; b.pq_pivots = ix->pq_pivots; b.pq_M = ix->pq_M; b.pq_K = ix->pq_K;
    b.pq_dsub = ix->pq_M ? ix->D / ix->pq_M : 0;
    b.spill = ix->spill; b.spill_size = ix->spill_size; b.spill_stride = ix->ws_spill;

    ix->last_Q = Q;
    ix->last_phases = lp.n_phases;
    for (int p = 0; p < lp.n_phases; ++p) ix->last_widths[p] = lp.widths[p];

    BOA_CUDA(cudaMemsetAsync(ix->counters, 0, kCntWords * sizeof(uint32_t), st));
    lp.launches = 0;
    int extra_launches = 0;

    if (!((double)Q > b.tau_q)) {
        // Algorithm 1's loop body never runs: every query returns "nothing found"
        const int64_t n = Q * k > Q ? Q * k : Q;
        fill_outputs_kernel<<<ix->num_sms * 4, 256, 0, st>>>(out_ids, out_dists, Q * k, b.final_L,
                                                            b.n_expand, b.n_scored, b.flags, b.n_rerank, Q);
        (void)n;
        BOA_CUDA(cudaGetLastError());
        ix->last_launches = 1;
        ix->last_phases = 0;
        return BOA_OK;
    }

    // BOA+ splits the first phase into sub-batches that run one after another: a sub-batch
    // smaller than about twice the queries the GPU searches at once (one per resident warp)
    // would leave it partly empty, so K is lowered until the sub-batches are that large
    int K = (ix->plus_k >= 2 && lp.n_phases > 1 && ix->tau == 0.0) ? ix->plus_k : 1;
    {
        const int64_t min_sub = ix->plus_min_sub > 0 ? ix->plus_min_sub : (int64_t)2 * 20 * ix->num_sms;
        if (K > 1 && Q / min_sub < K) K = (int)(Q / min_sub);
        if (K < 2) K = 1;
    }
    uint32_t* cnt = ix->counters + kCntCount;
    uint32_t* snap = ix->counters + kCntSnap;
    ix->last_split = 0;
    // chosen per call: two chains while the widest phase is at most 128 (measured: with wider last
    // phases one query per warp slot lasts so long that splitting the batch only delays the second half)
    const int chains = ix->chains != 0 ? ix->chains : (lp.widths[lp.n_phases - 1] <= 128 ? 2 : 1);
    if (K == 1 && chains == 2 && lp.n_phases > 1 && ix->tau == 0.0 && Q >= 2) {
        // Two chains: the halves of the batch go through all their phases independently, one on
        // the caller's stream, one on the side stream, each with its own survivor lists and
        // counters.  A query's phases depend on each other, different queries' do not: while
        // the partly empty last wave of one half's phase drains, the other half's launches fill
        // the GPU.  Every query is searched exactly as in the one-chain schedule.
        ix->last_split = 1;
        BOA_CUDA(cudaEventRecord(ix->ev_fork, st));
        BOA_CUDA(cudaStreamWaitEvent(ix->side, ix->ev_fork, 0));
        const uint32_t half = (uint32_t)(Q / 2);
        for (int c = 0; c < 2; ++c) {
            cudaStream_t cs = c == 0 ? st : ix->side;
            const uint32_t b0 = c == 0 ? 0u : half, b1 = c == 0 ? half : (uint32_t)Q;
            uint32_t* cnt_c = ix->counters + (c == 0 ? kCntCount : kCntCount2);
            rc = launch_phase(lp, 0, cs, nullptr, nullptr, b0, b1, b1 - b0, c, false, true);
            if (rc != BOA_OK) return rc;
            for (int p = 1; p < lp.n_phases; ++p) {
                rc = launch_phase(lp, p, cs, nullptr, cnt_c + p, 0u, 0u, b1 - b0, c, false, true);
                if (rc != BOA_OK) return rc;
            }
        }
        BOA_CUDA(cudaEventRecord(ix->ev_join, ix->side));
        BOA_CUDA(cudaStreamWaitEvent(st, ix->ev_join, 0));
    } else if (K == 1) {
        // BOA: one launch per phase, each over the survivors of the one before
        rc = launch_phase(lp, 0, st, nullptr, nullptr, 0u, (uint32_t)Q, (uint32_t)Q);
        if (rc != BOA_OK) return rc;
        for (int p = 1; p < lp.n_phases; ++p) {
            rc = launch_phase(lp, p, st, nullptr, cnt + p, 0u, 0u, (uint32_t)Q);
            if (rc != BOA_OK) return rc;
        }
    } else {
        // BOA+: the first phase goes out as K sub-batches on the caller's stream.  The
        // survivors gathered up to the middle sub-batch are escalated together through all
        // wider phases on the side stream while the remaining narrow sub-batches run; the
        // survivors of the second half follow as a second pool on the caller's stream,
        // concurrently with the first pool.  Each pool has its own lists from phase 2 on.
        const int mid = (K + 1) / 2;
        for (int j = 0; j < K; ++j) {
            const uint32_t b0 = (uint32_t)((Q * j) / K), b1 = (uint32_t)((Q * (j + 1)) / K);
            if (b1 > b0) {
                rc = launch_phase(lp, 0, st, nullptr, nullptr, b0, b1, b1 - b0);
                if (rc != BOA_OK) return rc;
            }
            if (j + 1 == mid || j + 1 == K) {
                const int chain = (j + 1 == K && mid != K) ? 1 : 0;
                // freeze the end of the phase-1 list at this point of the caller's stream
                copy_word_kernel<<<1, 1, 0, st>>>(snap + chain, cnt + 1);
                extra_launches++;
                BOA_CUDA(cudaGetLastError());
                cudaStream_t cs = st;
                if (chain == 0 && mid != K) {
                    BOA_CUDA(cudaEventRecord(ix->ev_fork, st));
                    BOA_CUDA(cudaStreamWaitEvent(ix->side, ix->ev_fork, 0));
                    cs = ix->side;
                }
                uint32_t* cnt_c = ix->counters + (chain == 0 ? kCntCount : kCntCount2);
                for (int p = 1; p < lp.n_phases; ++p) {
                    const uint32_t* beginp = (p == 1 && chain == 1) ? snap + 0 : nullptr;
                    const uint32_t* endp = (p == 1) ? snap + chain : cnt_c + p;
                    rc = launch_phase(lp, p, cs, beginp, endp, 0u, 0u, (uint32_t)Q, chain, false);
                    if (rc != BOA_OK) return rc;
                }
            }
        }
        if (mid != K) {
            BOA_CUDA(cudaEventRecord(ix->ev_join, ix->side));
            BOA_CUDA(cudaStreamWaitEvent(st, ix->ev_join, 0));
        }
    }
    if (ix->metric == BOA_METRIC_COSINE) {
        halve_kernel<<<ix->num_sms * 2, 256, 0, st>>>(out_dists, Q * k);
        BOA_CUDA(cudaGetLastError());
        extra_launches += 2;
    }
    ix->last_launches = lp.launches + extra_launches;
    return BOA_OK;
}

int boa_get_stats(boa_index* ix, int32_t* final_L, int32_t* n_expand, int32_t* n_scored, int32_t* flags,
                  void* stream)
{
    if (!ix) return BOA_EINVAL;
    if (ix->last_Q == 0) return BOA_OK;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int32_t* dst[4] = {final_L, n_expand, n_scored, flags};
    for (int i = 0; i < 4; ++i) {
        if (!dst[i]) continue;
        BOA_CUDA(cudaMemcpyAsync(dst[i], ix->stats + (size_t)i * ix->ws_Q,
                                 (size_t)ix->last_Q * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
    }
    return BOA_OK;
}

int boa_index_attach_pq(boa_index* ix, const float* pivots, const uint8_t* codes, int M, int K, void* stream)
{
    if (!ix || !pivots || !codes) return BOA_EINVAL;
    if (M < 16 || M > BOA_PQ_MAX_SUBSPACES || M % 16 != 0 || ix->D % M != 0) return BOA_EINVAL;
    if (K < 1 || K > 256) return BOA_EINVAL;
    if (!aligned16(pivots) || !aligned16(codes) || !on_device(ix->device) || ix->shared) return BOA_EINVAL;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    cudaFree(ix->pq_codes); cudaFree(ix->pq_pivots);
    ix->pq_codes = nullptr; ix->pq_pivots = nullptr; ix->pq_M = 0; ix->pq_K = 0; ix->use_pq = 0;
    const size_t cb = (size_t)ix->N * M, pb = (size_t)M * K * (ix->D / M) * sizeof(float);
    BOA_CUDA(cudaMalloc(&ix->pq_codes, cb));
    BOA_CUDA(cudaMalloc(&ix->pq_pivots, pb));
    BOA_CUDA(cudaMemcpyAsync(ix->pq_codes, codes, cb, cudaMemcpyDeviceToDevice, st));
    BOA_CUDA(cudaMemcpyAsync(ix->pq_pivots, pivots, pb, cudaMemcpyDeviceToDevice, st));
    BOA_CUDA(cudaStreamSynchronize(st));
    ix->pq_M = M; ix->pq_K = K;
    return BOA_OK;
}

int boa_set_range_penalty(boa_index* ix, const float* scales, void* stream)
{
    if (!ix || !on_device(ix->device)) return BOA_EINVAL;
    if (!scales) {
        cudaFree(ix->pen_scales);
        ix->pen_scales = nullptr;
        return BOA_OK;
    }
    float h[BOA_MAX_ATTRS] = {0};
    for (int j = 0; j < ix->m; ++j) {
        if (!(scales[j] > 0.0f) || isinf(scales[j])) return BOA_EINVAL;
        h[j] = scales[j];
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (!ix->pen_scales) BOA_CUDA(cudaMalloc(&ix->pen_scales, sizeof(h)));
    BOA_CUDA(cudaMemcpyAsync(ix->pen_scales, h, sizeof(h), cudaMemcpyHostToDevice, st));
    BOA_CUDA(cudaStreamSynchronize(st));
    return BOA_OK;
}

int boa_index_set_metric(boa_index* ix, int metric, void* stream)
{
    if (!ix || (metric != BOA_METRIC_L2 && metric != BOA_METRIC_COSINE)) return BOA_EINVAL;
    if (metric == ix->metric) return BOA_OK;
    // the rows are rescaled in place, once: there is no way back to the Euclidean metric
    if (ix->metric != BOA_METRIC_L2 || ix->vec_dtype != BOA_F32 || !on_device(ix->device) || ix->shared) return BOA_EINVAL;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    float* rows = reinterpret_cast<float*>(ix->rec);
    unit_rows_kernel<<<ix->num_sms * 8, 128, 0, st>>>(rows, ix->rec_stride / 4, rows, ix->rec_stride / 4, ix->N, ix->D);
    BOA_CUDA(cudaGetLastError());
    BOA_CUDA(cudaStreamSynchronize(st));
    ix->metric = BOA_METRIC_COSINE;
    return BOA_OK;
}

int boa_get_rerank_counts(boa_index* ix, int32_t* n_rerank, void* stream)
{
    if (!ix || !n_rerank) return BOA_EINVAL;
    if (ix->last_Q == 0) return BOA_OK;
    BOA_CUDA(cudaMemcpyAsync(n_rerank, ix->stats + (size_t)4 * ix->ws_Q, (size_t)ix->last_Q * sizeof(int32_t),
                             cudaMemcpyDeviceToDevice, reinterpret_cast<cudaStream_t>(stream)));
    return BOA_OK;
}

int boa_get_phase_counts(boa_index* ix, int64_t* active, int n, int* n_phases, void* stream)
{
    if (!ix || !active || n < 0) return BOA_EINVAL;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (n_phases) *n_phases = ix->last_phases;
    if (ix->last_Q == 0 || ix->last_phases == 0) return BOA_OK;
    uint32_t h[BOA_MAX_PHASES + 1] = {0};
    uint32_t h2[BOA_MAX_PHASES + 1] = {0};
    BOA_CUDA(cudaMemcpyAsync(h, ix->counters + kCntCount, sizeof(h), cudaMemcpyDeviceToHost, st));
    BOA_CUDA(cudaMemcpyAsync(h2, ix->counters + kCntCount2, sizeof(h2), cudaMemcpyDeviceToHost, st));
    BOA_CUDA(cudaStreamSynchronize(st));
    const double tau_q = ix->tau * (double)ix->last_Q;
    bool stopped = false;
    for (int p = 0; p < n && p < ix->last_phases; ++p) {
        const int64_t a = p == 0 ? ix->last_Q : (int64_t)h[p] + ((p >= 2 || ix->last_split) ? (int64_t)h2[p] : 0);
        if (!((double)a > tau_q)) stopped = true;
        active[p] = stopped ? 0 : a;
    }
    return BOA_OK;
}

int boa_last_launch_count(const boa_index* ix) { return ix ? ix->last_launches : 0; }

int boa_search_host(boa_index* ix, const float* queries, int64_t Q, const void* lo, const void* hi, int k,
                    int L0, int Lmax, uint32_t* out_ids, float* out_dists, void* stream)
{
    if (!ix) return BOA_EINVAL;
    if (Q < 0 || Q > (int64_t)0x7FFFFFFF || k < 1 || k > BOA_MAX_WIDTH) return BOA_EINVAL;
    if (Q == 0) return boa_search(ix, nullptr, 0, nullptr, nullptr, k, L0, Lmax, nullptr, nullptr, stream);
    if (!queries || !lo || !hi || !out_ids || !out_dists) return BOA_EINVAL;
    if (!on_device(ix->device)) return BOA_EINVAL;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    {
        // Page-locked host memory that is mapped into the device's address space is read and
        // written in place: the kernels fetch each query over the host link when they start on
        // it and write its results straight back, so no transfer is serialised before or after
        // the search.
        auto mapped = [](const void* p, const void** dp) {
            cudaPointerAttributes a;
            if (cudaPointerGetAttributes(&a, p) != cudaSuccess) { cudaGetLastError(); return false; }
            if (a.type != cudaMemoryTypeHost || !a.devicePointer) return false;
            *dp = a.devicePointer;
            return aligned16(*dp);
        };
        const void *dq, *dlo, *dhi, *dids, *dd2;
        if (ix->host_in_place && mapped(queries, &dq) && mapped(lo, &dlo) && mapped(hi, &dhi) && mapped(out_ids, &dids) &&
            mapped(out_dists, &dd2)) {
            const int rc = boa_search(ix, static_cast<const float*>(dq), Q, dlo, dhi, k, L0, Lmax,
                                      static_cast<uint32_t*>(const_cast<void*>(dids)),
                                      static_cast<float*>(const_cast<void*>(dd2)), stream);
            const cudaError_t e = cudaStreamSynchronize(st);
            if (rc != BOA_OK) return rc;
            BOA_CUDA(e);
            return BOA_OK;
        }
    }
    if (Q > ix->ws_host_Q || k > ix->ws_host_k) {
        const int64_t nq = Q > ix->ws_host_Q ? Q : ix->ws_host_Q;
        const int nk = k > ix->ws_host_k ? k : ix->ws_host_k;
        BOA_CUDA(cudaStreamSynchronize(st));        // an earlier call's copies may still read the old buffers
        cudaFree(ix->hq); cudaFree(ix->hlo); cudaFree(ix->hhi); cudaFree(ix->hids); cudaFree(ix->hd2);
        ix->hq = nullptr; ix->hlo = nullptr; ix->hhi = nullptr; ix->hids = nullptr; ix->hd2 = nullptr;
        ix->ws_host_Q = 0; ix->ws_host_k = 0;
        BOA_CUDA(cudaMalloc(&ix->hq, (size_t)nq * ix->D * sizeof(float)));
        BOA_CUDA(cudaMalloc(&ix->hlo, (size_t)nq * ix->m * sizeof(int32_t)));
        BOA_CUDA(cudaMalloc(&ix->hhi, (size_t)nq * ix->m * sizeof(int32_t)));
        BOA_CUDA(cudaMalloc(&ix->hids, (size_t)nq * nk * sizeof(uint32_t)));
        BOA_CUDA(cudaMalloc(&ix->hd2, (size_t)nq * nk * sizeof(float)));
        ix->ws_host_Q = nq; ix->ws_host_k = nk;
    }
    BOA_CUDA(cudaMemcpyAsync(ix->hq, queries, (size_t)Q * ix->D * sizeof(float), cudaMemcpyHostToDevice, st));
    BOA_CUDA(cudaMemcpyAsync(ix->hlo, lo, (size_t)Q * ix->m * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    BOA_CUDA(cudaMemcpyAsync(ix->hhi, hi, (size_t)Q * ix->m * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    const int rc = boa_search(ix, ix->hq, Q, ix->hlo, ix->hhi, k, L0, Lmax, ix->hids, ix->hd2, stream);
    if (rc != BOA_OK) {
        cudaStreamSynchronize(st);                   // the caller may free its host buffers right after an error
        return rc;
    }
    BOA_CUDA(cudaMemcpyAsync(out_ids, ix->hids, (size_t)Q * k * sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
    BOA_CUDA(cudaMemcpyAsync(out_dists, ix->hd2, (size_t)Q * k * sizeof(float), cudaMemcpyDeviceToHost, st));
    BOA_CUDA(cudaStreamSynchronize(st));
    return BOA_OK;
}

int boa_search_noalloc(boa_index* ix, const float* queries, int64_t Q, const void* lo, const void* hi,
                       int k, int L0, int Lmax, uint32_t* out_ids, float* out_dists, void* stream)
{
    if (!ix) return BOA_EINVAL;
    if (Q > kNoAllocMaxQ || Lmax > kNoAllocMaxWidth) return BOA_ETOOBIG;
    if (!on_device(ix->device)) return BOA_EINVAL;
    if (ix->metric != BOA_METRIC_L2) return BOA_EINVAL;       // the unit-length query copies need scratch of Q*D floats
    unsigned char* base = nullptr;
    const int rc0 = noalloc_scratch(&base);
    if (rc0 != BOA_OK) return rc0;
    // Point the index at the fixed buffer for the length of this call, run the ordinary
    // driver (which then finds its scratch large enough and allocates nothing), and put
    // the index's own buffers back.
    struct Saved {
        uint32_t *lists, *counters; int32_t *stats, *spill_size; uint64_t* spill;
        int64_t ws_Q; int ws_spill;
        int64_t last_Q; int last_phases, last_launches, last_split; int last_widths[BOA_MAX_PHASES];
    } sv = {ix->lists, ix->counters, ix->stats, ix->spill_size, ix->spill, ix->ws_Q, ix->ws_spill,
            ix->last_Q, ix->last_phases, ix->last_launches, ix->last_split, {0}};
    memcpy(sv.last_widths, ix->last_widths, sizeof(sv.last_widths));
    ix->counters = reinterpret_cast<uint32_t*>(base + kNaCounters);
    ix->lists = reinterpret_cast<uint32_t*>(base + kNaLists);
    ix->stats = reinterpret_cast<int32_t*>(base + kNaStats);
    ix->spill_size = reinterpret_cast<int32_t*>(base + kNaSpillSize);
    ix->spill = reinterpret_cast<uint64_t*>(base + kNaSpill);
    ix->ws_Q = kNoAllocMaxQ;
    ix->ws_spill = kNoAllocMaxWidth;
    const int rc = boa_search(ix, queries, Q, lo, hi, k, L0, Lmax, out_ids, out_dists, stream);
    ix->lists = sv.lists; ix->counters = sv.counters; ix->stats = sv.stats;
    ix->spill_size = sv.spill_size; ix->spill = sv.spill; ix->ws_Q = sv.ws_Q; ix->ws_spill = sv.ws_spill;
    // boa_get_stats / boa_get_phase_counts keep describing the last boa_search: this call's
    // statistics sit in the shared array, which the next call overwrites
    ix->last_Q = sv.last_Q; ix->last_phases = sv.last_phases; ix->last_launches = sv.last_launches;
    ix->last_split = sv.last_split;
    memcpy(ix->last_widths, sv.last_widths, sizeof(sv.last_widths));
    return rc;
}

#ifdef BOA_SECTION_TIMERS
// Debug builds only: cycles per kernel section, summed over warps (12 values, HOST array).
int boa_debug_timers(boa_index* ix, unsigned long long* out, int reset)
{
    if (!ix || !out || !ix->counters) return BOA_EINVAL;
    unsigned long long* d = reinterpret_cast<unsigned long long*>(ix->counters + kCntWords);
    BOA_CUDA(cudaDeviceSynchronize());
    BOA_CUDA(cudaMemcpy(out, d, 12 * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
    if (reset) BOA_CUDA(cudaMemset(d, 0, 12 * sizeof(unsigned long long)));
    return BOA_OK;
}
#endif

int boa_device_status(boa_index* ix, int* status, void* stream)
{
    if (!ix || !status) return BOA_EINVAL;
    *status = 0;
    if (!ix->counters) return BOA_OK;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    uint32_t h = 0;
    BOA_CUDA(cudaMemcpyAsync(&h, ix->counters + kCntStatus, sizeof(h), cudaMemcpyDeviceToHost, st));
    BOA_CUDA(cudaStreamSynchronize(st));
    *status = (int)h;
    return BOA_OK;
}

}  // extern "C"

// Graph construction on the GPU: a batched Vamana build with alpha-dominance pruning run once
// per attribute threshold (the paper's Background section, "Graph construction").  Not part of
// the search hot path; it produces the graph boa_index_create takes.  sm_100a only.
//
// Per batch of new points: (a) the library's own filter-aware beam search over the graph built
// so far collects candidates for every point of the batch, once per attribute threshold with
// the predicate "attribute position within the threshold of the point's own", (b) one warp per point prunes candidates +
// current row down to R neighbours, (c) every selected edge p -> n asks for n -> p: the
// requests are sorted by (target, requester) and one warp per target appends them or, when the
// row overflows, prunes row + requesters.  Everything that decides the result is fixed
// (batch sizes, orders, tie-breaks, the fp32 order of every distance), so the same inputs give
// the same graph every time.
#include "../../include/boa.h"

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include <cub/device/device_radix_sort.cuh>

namespace {

thread_local int g_build_cuda = 0;
#define BUILD_CUDA(expr)                                  \
    do {                                                  \
        cudaError_t e__ = (expr);                         \
        if (e__ != cudaSuccess) {                         \
            g_build_cuda = (int)e__;                      \
            rc = e__ == cudaErrorMemoryAllocation ? BOA_ENOMEM : BOA_ECUDA; \
            goto done;                                    \
        }                                                 \
    } while (0)

constexpr int kMaxCand = 256;          // candidates of one pruning run: Lb + R or R + cap_in, rounded up
constexpr uint32_t kNone = 0xFFFFFFFFu;

struct BuildParams {
    const uint8_t* vec;       // [N][row_bytes] the vectors as given (float or uint8_t)
    int vec_u8, D, row_bytes;
    const float* pos;         // [N][m_pos] attribute positions
    int m_pos;
    uint32_t* graph;          // [N][R] the graph being built (the search index's own copy)
    int R, T;
    float alpha2;
    float thr[8][BOA_MAX_ATTRS];   // [T][m_pos] per-attribute thresholds
};

// Squared L2 distance of two rows by one 8-lane group (g = lane & 7), in the fixed fp32 order of
// the search: the row is cut into 16-byte chunks, chunk c belongs to lane c mod 8, each lane adds
// fmaf(x-y, x-y, acc) over its chunks and elements in ascending order, and the eight sums meet
// as ((p0+p4)+(p2+p6))+((p1+p5)+(p3+p7)).  All eight lanes return the sum.
__device__ __forceinline__ float group_dist2(const uint8_t* a, const uint8_t* b, int row_bytes, bool u8, int g,
                                             bool active)
{
    float acc = 0.0f;
    if (active) {
        for (int off = 16 * g; off < row_bytes; off += 128) {
            const uint4 xa = *reinterpret_cast<const uint4*>(a + off);
            const uint4 xb = *reinterpret_cast<const uint4*>(b + off);
            if (!u8) {
                float d;
                d = __uint_as_float(xa.x) - __uint_as_float(xb.x); acc = fmaf(d, d, acc);
                d = __uint_as_float(xa.y) - __uint_as_float(xb.y); acc = fmaf(d, d, acc);
                d = __uint_as_float(xa.z) - __uint_as_float(xb.z); acc = fmaf(d, d, acc);
                d = __uint_as_float(xa.w) - __uint_as_float(xb.w); acc = fmaf(d, d, acc);
            } else {
                const uint32_t wa[4] = {xa.x, xa.y, xa.z, xa.w}, wb[4] = {xb.x, xb.y, xb.z, xb.w};
#pragma unroll
                for (int w = 0; w < 4; ++w)
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const float d = (float)((wa[w] >> (8 * t)) & 0xFFu) - (float)((wb[w] >> (8 * t)) & 0xFFu);
                        acc = fmaf(d, d, acc);
                    }
            }
        }
    }
    acc += __shfl_xor_sync(0xffffffffu, acc, 4);
    acc += __shfl_xor_sync(0xffffffffu, acc, 2);
    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
    return acc;
}

// b within the threshold vector t of a in every attribute
__device__ __forceinline__ bool attr_within(const float* pos, int m, int64_t a, int64_t b, const float* t)
{
    bool ok = true;
    for (int j = 0; j < m; ++j) ok = ok && !(fabsf(pos[a * m + j] - pos[b * m + j]) > t[j]);
    return ok;
}

// Warp-wide bitonic sort of n <= kMaxCand 64-bit keys in shared memory (ascending); slots
// [n, cap) must hold all-ones keys, cap a power of two.
__device__ void sort_keys_smem(unsigned long long* keys, int cap, int lane)
{
    for (int k = 2; k <= cap; k <<= 1)
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = lane; i < cap; i += 32) {
                const int l = i ^ j;
                if (l > i) {
                    const unsigned long long a = keys[i], b = keys[l];
                    const bool up = (i & k) == 0;
                    if ((a > b) == up) { keys[i] = b; keys[l] = a; }
                }
            }
            __syncwarp();
        }
}

// The pruning step for point p over the ids in cand[0..n) (repeats, kNone and p itself allowed).
// Shared memory of the warp: keys[kMaxCand], flags[kMaxCand], live[kMaxCand].  Writes row[0..R).
// Work is kept to what decides the result: repeats are dropped before any distance is
// computed, and a threshold pass walks a compacted list of the candidates that are still
// unselected, inside its threshold and not yet dominated.
__device__ void prune_point(const BuildParams& bp, int64_t p, const uint32_t* cand, int n, unsigned long long* keys,
                            uint8_t* flags, uint16_t* live, uint32_t* row, int lane)
{
    const int g = lane & 7, gi = lane >> 3;
    const unsigned lt = (1u << lane) - 1u;
    const uint8_t* xp = bp.vec + (size_t)p * bp.row_bytes;
    int cap = 32;
    while (cap < n) cap <<= 1;
    // distinct candidate ids: sort the ids, keep the first of every run
    for (int i = lane; i < cap; i += 32) {
        const uint32_t id = i < n ? cand[i] : kNone;
        keys[i] = (id != kNone && (int64_t)id != p) ? (unsigned long long)id : ~0ull;
    }
    __syncwarp();
    sort_keys_smem(keys, cap, lane);
    int nc = 0;
    for (int i0 = 0; i0 < cap; i0 += 32) {
        const int i = i0 + lane;
        const unsigned long long k = keys[i];
        const bool keep = k != ~0ull && (i == 0 || keys[i - 1] != k);
        const unsigned bal = __ballot_sync(0xffffffffu, keep);
        __syncwarp();
        if (keep) keys[nc + __popc(bal & lt)] = k;
        nc += __popc(bal);
        __syncwarp();
    }
    cap = 32;
    while (cap < nc) cap <<= 1;
    // distance of every candidate to p (four candidates per step, one 8-lane group each), then
    // the order of the pruning: ascending (distance, id)
    for (int i0 = 0; i0 < cap; i0 += 4) {
        const int i = i0 + gi;
        const bool ok = i < nc;
        const uint32_t id = ok ? (uint32_t)keys[i] : 0u;
        const float d = group_dist2(xp, bp.vec + (size_t)id * bp.row_bytes, bp.row_bytes, bp.vec_u8 != 0, g, ok);
        __syncwarp();
        if (g == 0) keys[i] = ok ? (((unsigned long long)__float_as_uint(d) << 32) | id) : ~0ull;
    }
    __syncwarp();
    sort_keys_smem(keys, cap, lane);
    for (int i = lane; i < nc; i += 32) flags[i] = 0;                      // 1 = selected
    __syncwarp();
    int total = 0;
    for (int ti = 0; ti < bp.T && total < bp.R; ++ti) {
        const int budget = bp.R * (ti + 1) / bp.T - bp.R * ti / bp.T;
        int taken = 0;
        // the pass's list: unselected candidates within its threshold, in pruning order
        int nl = 0;
        for (int i0 = 0; i0 < nc; i0 += 32) {
            const int i = i0 + lane;
            const bool in = i < nc && !flags[i] && attr_within(bp.pos, bp.m_pos, p, (uint32_t)keys[i], bp.thr[ti]);
            const unsigned bal = __ballot_sync(0xffffffffu, in);
            if (in) live[nl + __popc(bal & lt)] = (uint16_t)i;
            nl += __popc(bal);
        }
        __syncwarp();
        while (nl > 0 && taken < budget) {
            // the head of the list is the nearest candidate nothing selected in this pass dominates
            const int i = live[0];
            const uint32_t ci = (uint32_t)keys[i];
            __syncwarp();
            if (lane == 0) { flags[i] = 1; row[total] = ci; }
            total++; taken++;
            if (taken == budget) break;
            const uint8_t* xc = bp.vec + (size_t)ci * bp.row_bytes;
            // drop what the new neighbour dominates: 32 list entries per round, four distances per step
            int nn = 0;
            for (int j0 = 1; j0 < nl; j0 += 32) {
                bool dom_mine = false;
                for (int sub = 0; sub < 8 && j0 + 4 * sub < nl; ++sub) {
                    const int jj = j0 + 4 * sub + gi;
                    const bool ok = jj < nl;
                    const unsigned long long kj = keys[ok ? live[jj] : 0];
                    const float dcc = group_dist2(xc, bp.vec + (size_t)(ok ? (uint32_t)kj : 0u) * bp.row_bytes, bp.row_bytes,
                                                  bp.vec_u8 != 0, g, ok);
                    const bool dom = ok && __fmul_rn(bp.alpha2, dcc) <= __uint_as_float((uint32_t)(kj >> 32));
                    const unsigned bal = __ballot_sync(0xffffffffu, dom);       // bit 8*gi: entry j0 + 4*sub + gi
                    if ((lane >> 2) == sub) dom_mine = (bal >> (8 * (lane & 3))) & 1u;
                }
                const bool keep = j0 + lane < nl && !dom_mine;
                const uint16_t mine = live[j0 + lane < nl ? j0 + lane : 0];
                const unsigned bal = __ballot_sync(0xffffffffu, keep);
                __syncwarp();
                if (keep) live[nn + __popc(bal & lt)] = mine;
                nn += __popc(bal);
                __syncwarp();
            }
            nl = nn;
        }
        __syncwarp();
    }
    for (int i = total + lane; i < bp.R; i += 32) row[i] = kNone;
    __syncwarp();
}

// (b) one warp per batch point: candidates of the T searches + the point's current row
__global__ void prune_batch_kernel(BuildParams bp, int64_t start, int bsz, const uint32_t* cand_ids, int Lb, int B)
{
    __shared__ unsigned long long keys[kMaxCand];
    __shared__ uint32_t cand[kMaxCand];
    __shared__ uint8_t flags[kMaxCand];
    __shared__ uint16_t live[kMaxCand];
    const int lane = threadIdx.x;
    for (int b = blockIdx.x; b < bsz; b += gridDim.x) {
        const int64_t p = start + b;
        uint32_t* row = bp.graph + (size_t)p * bp.R;
        for (int ti = 0; ti < bp.T; ++ti)
            for (int i = lane; i < Lb; i += 32) cand[ti * Lb + i] = cand_ids[((size_t)ti * B + b) * Lb + i];
        for (int i = lane; i < bp.R; i += 32) cand[bp.T * Lb + i] = row[i];
        __syncwarp();
        prune_point(bp, p, cand, bp.T * Lb + bp.R, keys, flags, live, row, lane);
    }
}

// bounds of the build's searches: lo = pos - t[j], hi = pos + t[j] per attribute j (one fp32 operation each)
struct ThresholdRow { float t[BOA_MAX_ATTRS]; };
__global__ void window_bounds_kernel(const float* pos, int m, int64_t start, int bsz, ThresholdRow tr, float* lo, float* hi)
{
    const int64_t n = (int64_t)bsz * m;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const float v = pos[start * m + i];
        float t = tr.t[0];
#pragma unroll
        for (int j = 1; j < BOA_MAX_ATTRS; ++j) t = (int)(i % m) == j ? tr.t[j] : t;
        lo[i] = __fsub_rn(v, t);
        hi[i] = __fadd_rn(v, t);
    }
}

// (c1) the requests of a batch: key = target << 32 | requester for every edge of its rows
__global__ void emit_requests_kernel(const uint32_t* graph, int R, int64_t start, int bsz, unsigned long long* keys)
{
    const int64_t n = (int64_t)bsz * R;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t p = start + i / R;
        const uint32_t t = graph[(size_t)p * R + i % R];
        keys[i] = t == kNone ? ~0ull : (((unsigned long long)t << 32) | (uint32_t)p);
    }
}

// (c2) positions where a new target starts in the sorted requests
__global__ void find_heads_kernel(const unsigned long long* keys, int64_t n, uint32_t* heads, uint32_t* n_heads)
{
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const unsigned long long k = keys[i];
        if (k == ~0ull) continue;
        if (i == 0 || (keys[i - 1] >> 32) != (k >> 32)) heads[atomicAdd(n_heads, 1u)] = (uint32_t)i;
    }
}

// (c3) one warp per target: append its requesters (ascending id, at most cap_in, those not in the
// row yet), or prune row + requesters when they do not fit
__global__ void reverse_edges_kernel(BuildParams bp, const unsigned long long* req, int64_t n_req, const uint32_t* heads,
                                     const uint32_t* n_heads, int cap_in)
{
    __shared__ unsigned long long keys[kMaxCand];
    __shared__ uint32_t cand[kMaxCand];
    __shared__ uint8_t flags[kMaxCand];
    __shared__ uint16_t live[kMaxCand];
    const int lane = threadIdx.x;
    const uint32_t nh = *n_heads;
    for (uint32_t h = blockIdx.x; h < nh; h += gridDim.x) {
        const int64_t i0 = heads[h];
        const uint32_t tgt = (uint32_t)(req[i0] >> 32);
        uint32_t* row = bp.graph + (size_t)tgt * bp.R;
        int deg = 0;
        for (int j0 = 0; j0 < bp.R; j0 += 32) {
            const int j = j0 + lane;
            const uint32_t v = j < bp.R ? row[j] : kNone;
            if (j < bp.R) cand[j] = v;
            deg += __popc(__ballot_sync(0xffffffffu, v != kNone));     // rows are padded at the tail only
        }
        __syncwarp();
        int nm = 0;
        for (int r0 = 0; r0 < cap_in; r0 += 32) {
            const int64_t i = i0 + r0 + lane;
            bool take = false;
            uint32_t rq = kNone;
            if (r0 + lane < cap_in && i < n_req && (uint32_t)(req[i] >> 32) == tgt) {
                rq = (uint32_t)req[i];
                take = true;
                for (int j = 0; j < deg; ++j) take = take && cand[j] != rq;
            }
            const unsigned bal = __ballot_sync(0xffffffffu, take);
            if (take) cand[deg + nm + __popc(bal & ((1u << lane) - 1u))] = rq;
            nm += __popc(bal);
        }
        __syncwarp();
        if (deg + nm <= bp.R) {
            for (int j = lane; j < nm; j += 32) row[deg + j] = cand[deg + j];
        } else {
            prune_point(bp, tgt, cand, deg + nm, keys, flags, live, row, lane);
        }
        __syncwarp();
    }
}

__global__ void bytes_to_float_kernel(const uint8_t* src, float* dst, int64_t n)
{
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        dst[i] = (float)src[i];
}

__global__ void fill_u32_kernel(uint32_t* dst, int64_t n, uint32_t v)
{
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        dst[i] = v;
}

}  // namespace

// the search index's own copy of the graph (defined beside the index, in boa.cu)
extern "C" uint32_t* boa_internal_graph(boa_index* index);

extern "C" int boa_graph_build(const void* vectors, int vec_dtype, int64_t N, int D, const float* attr_pos, int m_pos,
                               int R, int Lb, float alpha, const float* thresholds, int T, int B, int passes,
                               int cap_in, int64_t entry, uint32_t* out_graph, int64_t* n_batches, void* stream)
{
    if (!vectors || !attr_pos || !thresholds || !out_graph) return BOA_EINVAL;
    if (N < 1 || R < 1 || R > BOA_MAX_DEGREE || Lb < 1 || Lb > 128 || T < 1 || T > 8 || m_pos < 1 || m_pos > BOA_MAX_ATTRS)
        return BOA_EINVAL;
    if (B < 1 || B > (1 << 20) || passes < 1 || passes > 4 || cap_in < 1 || cap_in > 64 || !(alpha >= 1.0f)) return BOA_EINVAL;
    if (T * Lb + R > kMaxCand || R + cap_in > kMaxCand) return BOA_EINVAL;
    if (vec_dtype != BOA_F32 && vec_dtype != BOA_U8) return BOA_EINVAL;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int rc = BOA_OK;
    boa_index* ix = nullptr;
    // the searches of one batch (one per threshold) are independent: each runs on a handle and a
    // stream of its own, so the partly empty last wave of one overlaps the others
    boa_index* shares[8] = {nullptr};
    cudaStream_t side[8] = {nullptr};
    cudaEvent_t ev_fork = nullptr, ev_join[8] = {nullptr};
    float *wlo = nullptr, *whi = nullptr;
    int types[BOA_MAX_ATTRS];
    uint32_t *empty = nullptr, *cand_ids = nullptr, *heads = nullptr, *n_heads = nullptr;
    float *cand_d = nullptr, *qf = nullptr;
    unsigned long long *req = nullptr, *req_sorted = nullptr;
    void* cub_tmp = nullptr;
    size_t cub_bytes = 0;
    int64_t batches = 0, inserted = 0;
    int sms = 0, dev = 0;
    BuildParams bp;
    for (int j = 0; j < BOA_MAX_ATTRS; ++j) types[j] = BOA_ATTR_F32;

    BUILD_CUDA(cudaGetDevice(&dev));
    BUILD_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    BUILD_CUDA(cudaMalloc(&empty, (size_t)N * R * sizeof(uint32_t)));
    fill_u32_kernel<<<sms * 8, 256, 0, st>>>(empty, N * (int64_t)R, kNone);
    BUILD_CUDA(cudaGetLastError());
    // the build's searches see the attribute positions as float attribute columns
    rc = boa_index_create(&ix, vectors, vec_dtype, N, D, attr_pos, types, m_pos, empty, R, entry, st);
    if (rc != BOA_OK) goto done;
    BUILD_CUDA(cudaMalloc(&wlo, (size_t)T * B * m_pos * sizeof(float)));
    BUILD_CUDA(cudaMalloc(&whi, (size_t)T * B * m_pos * sizeof(float)));
    BUILD_CUDA(cudaEventCreateWithFlags(&ev_fork, cudaEventDisableTiming));
    for (int ti = 1; ti < T; ++ti) {
        rc = boa_index_share(&shares[ti], ix);
        if (rc != BOA_OK) goto done;
        BUILD_CUDA(cudaStreamCreateWithFlags(&side[ti], cudaStreamNonBlocking));
        BUILD_CUDA(cudaEventCreateWithFlags(&ev_join[ti], cudaEventDisableTiming));
    }
    BUILD_CUDA(cudaMalloc(&cand_ids, (size_t)T * B * Lb * sizeof(uint32_t)));
    BUILD_CUDA(cudaMalloc(&cand_d, (size_t)T * B * Lb * sizeof(float)));
    BUILD_CUDA(cudaMalloc(&req, (size_t)B * R * sizeof(unsigned long long)));
    BUILD_CUDA(cudaMalloc(&req_sorted, (size_t)B * R * sizeof(unsigned long long)));
    BUILD_CUDA(cudaMalloc(&heads, (size_t)B * R * sizeof(uint32_t)));
    BUILD_CUDA(cudaMalloc(&n_heads, sizeof(uint32_t)));
    if (vec_dtype == BOA_U8) BUILD_CUDA(cudaMalloc(&qf, (size_t)B * D * sizeof(float)));
    BUILD_CUDA(cub::DeviceRadixSort::SortKeys(nullptr, cub_bytes, req, req_sorted, (int)((int64_t)B * R), 0, 64, st));
    BUILD_CUDA(cudaMalloc(&cub_tmp, cub_bytes));

    bp.vec = reinterpret_cast<const uint8_t*>(vectors);
    bp.vec_u8 = vec_dtype == BOA_U8;
    bp.D = D;
    bp.row_bytes = vec_dtype == BOA_U8 ? D : 4 * D;
    bp.pos = attr_pos;
    bp.m_pos = m_pos;
    bp.graph = boa_internal_graph(ix);
    bp.R = R;
    bp.T = T;
    bp.alpha2 = alpha * alpha;
    for (int i = 0; i < 8; ++i)
        for (int j = 0; j < BOA_MAX_ATTRS; ++j) bp.thr[i][j] = i < T && j < m_pos ? thresholds[(size_t)i * m_pos + j] : INFINITY;

    for (int pass = 0; pass < passes; ++pass) {
        int64_t start = 0;
        while (start < N) {
            int64_t bsz = pass == 0 ? (inserted < 1 ? 1 : (inserted < B ? inserted : B)) : B;
            if (start + bsz > N) bsz = N - start;
            // (a) candidates: per threshold, the filter-valid results of a search at width Lb over the
            // graph so far whose ranges are the point's own attribute positions +- the threshold
            const float* q = reinterpret_cast<const float*>(vectors) + (size_t)start * D;
            if (vec_dtype == BOA_U8) {
                bytes_to_float_kernel<<<sms * 4, 256, 0, st>>>(reinterpret_cast<const uint8_t*>(vectors) + (size_t)start * D,
                                                               qf, bsz * (int64_t)D);
                BUILD_CUDA(cudaGetLastError());
                q = qf;
            }
            if (T > 1) BUILD_CUDA(cudaEventRecord(ev_fork, st));
            for (int ti = 0; ti < T; ++ti) {
                cudaStream_t cs = ti == 0 ? st : side[ti];
                boa_index* h = ti == 0 ? ix : shares[ti];
                float* lo_t = wlo + (size_t)ti * B * m_pos;
                float* hi_t = whi + (size_t)ti * B * m_pos;
                if (ti > 0) BUILD_CUDA(cudaStreamWaitEvent(cs, ev_fork, 0));
                ThresholdRow tr;
                for (int j = 0; j < BOA_MAX_ATTRS; ++j) tr.t[j] = bp.thr[ti][j];
                window_bounds_kernel<<<sms, 256, 0, cs>>>(attr_pos, m_pos, start, (int)bsz, tr, lo_t, hi_t);
                BUILD_CUDA(cudaGetLastError());
                rc = boa_search(h, q, bsz, lo_t, hi_t, Lb, Lb, Lb, cand_ids + (size_t)ti * B * Lb,
                                cand_d + (size_t)ti * B * Lb, cs);
                if (rc != BOA_OK) goto done;
                if (ti > 0) BUILD_CUDA(cudaEventRecord(ev_join[ti], cs));
            }
            for (int ti = 1; ti < T; ++ti) BUILD_CUDA(cudaStreamWaitEvent(st, ev_join[ti], 0));
            // (b) prune every point of the batch
            prune_batch_kernel<<<(unsigned)(bsz < sms * 32 ? bsz : sms * 32), 32, 0, st>>>(bp, start, (int)bsz, cand_ids, Lb, B);
            BUILD_CUDA(cudaGetLastError());
            // (c) reverse edges
            {
                const int64_t nreq = bsz * R;
                emit_requests_kernel<<<sms * 2, 256, 0, st>>>(bp.graph, R, start, (int)bsz, req);
                BUILD_CUDA(cudaGetLastError());
                size_t tmp_bytes = cub_bytes;
                BUILD_CUDA(cub::DeviceRadixSort::SortKeys(cub_tmp, tmp_bytes, req, req_sorted, (int)nreq, 0, 64, st));
                BUILD_CUDA(cudaMemsetAsync(n_heads, 0, sizeof(uint32_t), st));
                find_heads_kernel<<<sms * 2, 256, 0, st>>>(req_sorted, nreq, heads, n_heads);
                BUILD_CUDA(cudaGetLastError());
                reverse_edges_kernel<<<sms * 32, 32, 0, st>>>(bp, req_sorted, nreq, heads, n_heads, cap_in);
                BUILD_CUDA(cudaGetLastError());
            }
            start += bsz;
            if (pass == 0) inserted += bsz;
            batches++;
        }
    }
    BUILD_CUDA(cudaMemcpyAsync(out_graph, bp.graph, (size_t)N * R * sizeof(uint32_t), cudaMemcpyDeviceToDevice, st));
    BUILD_CUDA(cudaStreamSynchronize(st));
    if (n_batches) *n_batches = batches;
done:
    if (rc != BOA_OK) cudaStreamSynchronize(st);
    for (int ti = 1; ti < 8; ++ti) {
        if (side[ti]) { cudaStreamSynchronize(side[ti]); cudaStreamDestroy(side[ti]); }
        if (ev_join[ti]) cudaEventDestroy(ev_join[ti]);
        if (shares[ti]) boa_index_destroy(shares[ti]);
    }
    if (ev_fork) cudaEventDestroy(ev_fork);
    if (ix) boa_index_destroy(ix);
    cudaFree(wlo); cudaFree(whi); cudaFree(empty); cudaFree(cand_ids); cudaFree(cand_d); cudaFree(req);
    cudaFree(req_sorted); cudaFree(heads); cudaFree(n_heads); cudaFree(qf); cudaFree(cub_tmp);
    return rc;
}

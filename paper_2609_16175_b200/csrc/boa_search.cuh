// Warp-per-query filter-aware beam search (Algorithm 2) with the confidence test
// (Eq. 3) and survivor compaction (Algorithm 1, "compact active queries") fused
// into its epilogue.  sm_100a only.
//
// One warp (one CTA of 32 threads) owns one query from start to convergence.  Its
// candidate pool, the table of recently scored ids, the query vector and a staging
// area for neighbour records live in shared memory.  A pool entry is one 64-bit key
//     [63:60] phi (violated predicates)  [59:29] fp32 bits of d^2  [28:1] id  [0] expanded
// so that integer order of keys is the lexicographic order (phi, d^2, id): the
// lambda -> infinity reading of the paper's score dist + lambda*phi.
//
// Neighbour records (vector + attribute cells, one contiguous 32-byte-aligned row
// each) are fetched with one bulk asynchronous copy (cp.async.bulk, the TMA engine)
// per row into the staging area; a transaction barrier tells the warp when the bytes
// have landed.  No register holds data in flight, so one warp keeps up to
// `stage_rows` whole rows in flight at once.
//
// Distances are accumulated in a fixed order: a row is cut into 16-byte chunks,
// chunk c belongs to lane (c mod 8) of an 8-lane group, each lane runs
// acc = fmaf(x-q, x-q, acc) over its chunks in ascending order, and the eight
// partial sums meet in a butterfly (xor 4, 2, 1).  Four neighbours are scored per
// warp round, one per 8-lane group.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace boa {

constexpr uint32_t kNoId = 0xFFFFFFFFu;
constexpr int kThreads = 32;           // one warp per CTA
constexpr uint64_t kKeyMax = ~0ull;
constexpr uint32_t kWaitLimit = 1u << 22;   // bounded wait on the transaction barrier

enum : uint32_t { kStatusCopyTimeout = 1u };

struct SearchParams {
    // index
    const uint8_t* rec;       // [N] records: vector, then m attribute cells, padded to rec_stride
    const uint32_t* graph;    // [N][R]
    int64_t N;
    int D, m, R;
    int rec_stride;           // bytes, multiple of 32
    int rec_bytes;            // bytes of a record that are copied (vector + cells, 16-byte multiple)
    int nchunks;              // 16-byte chunks of one vector
    int attr_off;             // byte offset of the attribute cells inside a record
    uint32_t attr_float_mask; // bit j set: column j is float
    uint32_t entry;
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
    int hash_log2;            // size of the table of recently scored ids
    int stage_rows;           // records the staging area holds
    int max_expand;           // expansions after which a phase gives up
    int first_phase;          // statistics start from zero
    int resume_in;            // load the pool a narrower phase spilled
    int spill_out;            // uncertain queries spill their pool for the next phase
    int last_phase;           // nobody is appended to a survivor list
    float c_eps;              // (1-eps)^2 rounded once to fp32
    int eps_mode;             // 0: use c_eps; -1: never confident; 1: confident iff > k valid
    double tau_q;             // tau * Q: a phase runs only while |A| > tau*Q
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
    // per-query state
    int32_t* final_L;
    int32_t* n_expand;
    int32_t* n_scored;
    int32_t* flags;
    uint64_t* spill;          // [Q][spill_stride] pools carried between phases (resume)
    int32_t* spill_size;      // [Q]
    int spill_stride;
};

// ---------------------------------------------------------------- helpers
__device__ __forceinline__ uint64_t pack_key(uint32_t phi, float d2, uint32_t id)
{
    return ((uint64_t)phi << 60) | ((uint64_t)(__float_as_uint(d2) & 0x7FFFFFFFu) << 29) |
           ((uint64_t)id << 1);
}
__device__ __forceinline__ uint32_t key_id(uint64_t k) { return (uint32_t)(k >> 1) & 0x0FFFFFFFu; }
__device__ __forceinline__ float key_d2(uint64_t k)
{
    return __uint_as_float((uint32_t)(k >> 29) & 0x7FFFFFFFu);
}
__device__ __forceinline__ uint32_t key_phi(uint64_t k) { return (uint32_t)(k >> 60); }

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// One row, global -> shared, completion counted in bytes on `bar`.  No multicast.
__device__ __forceinline__ void bulk_load_row(void* dst, const void* src, uint32_t bytes, uint64_t* bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_u32(dst)),
        "l"(src), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void fence_async_proxy()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ float sq_acc4(float acc, float4 x, float4 q)
{
    float d;
    d = x.x - q.x; acc = fmaf(d, d, acc);
    d = x.y - q.y; acc = fmaf(d, d, acc);
    d = x.z - q.z; acc = fmaf(d, d, acc);
    d = x.w - q.w; acc = fmaf(d, d, acc);
    return acc;
}
__device__ __forceinline__ float sq_acc_bytes(float acc, uint32_t w, float4 q)
{
    float d;
    d = (float)(w & 0xFFu) - q.x;         acc = fmaf(d, d, acc);
    d = (float)((w >> 8) & 0xFFu) - q.y;  acc = fmaf(d, d, acc);
    d = (float)((w >> 16) & 0xFFu) - q.z; acc = fmaf(d, d, acc);
    d = (float)(w >> 24) - q.w;           acc = fmaf(d, d, acc);
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
                if (RS == 2) {
                    uint64_t a = x[0], b = x[RS - 1];
                    x[0] = a < b ? a : b;
                    x[RS - 1] = a < b ? b : a;
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
    int pool_off, nk_off, nr_off, cand_off, hash_off, q_off, stage_off, bar_off, total;
};
__host__ __device__ inline WarpSmem warp_smem_layout(int C, int hash_log2, int D, int RS,
                                                     int stage_rows, int rec_bytes)
{
    WarpSmem s;
    int off = 0;
    s.stage_off = off; off += stage_rows * rec_bytes;          // 16-byte multiple
    s.pool_off = off;  off += ((C + 1) & ~1) * 8;
    s.nk_off = off;    off += 32 * RS * 8;
    s.q_off = off;     off += ((D * 4 + 15) & ~15);
    s.hash_off = off;  off += (1 << hash_log2) * 4;
    s.cand_off = off;  off += 32 * RS * 4;
    s.nr_off = off;    off += 32 * RS * 4;
    s.bar_off = off;   off += 16;
    s.total = (off + 127) & ~127;
    return s;
}

// ---------------------------------------------------------------- the kernel
// VT: 0 = float vectors, 1 = uint8 vectors.  RS: adjacency slots per lane (1: R <= 32,
// 2: R <= 64).
template <int VT, int RS>
__global__ void __launch_bounds__(kThreads) boa_search_kernel(const SearchParams p)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    const int lane = threadIdx.x;
    const int g = lane & 7;        // lane inside its 8-lane group
    const int gi = lane >> 3;      // group index 0..3
    const unsigned lt_mask = (1u << lane) - 1u;

    const WarpSmem lay = warp_smem_layout(p.C, p.hash_log2, p.D, RS, p.stage_rows, p.rec_bytes);
    uint8_t* stage = smem_raw + lay.stage_off;
    uint64_t* pool = reinterpret_cast<uint64_t*>(smem_raw + lay.pool_off);
    uint64_t* nk = reinterpret_cast<uint64_t*>(smem_raw + lay.nk_off);
    uint32_t* nr = reinterpret_cast<uint32_t*>(smem_raw + lay.nr_off);
    uint32_t* cand = reinterpret_cast<uint32_t*>(smem_raw + lay.cand_off);
    uint32_t* hash = reinterpret_cast<uint32_t*>(smem_raw + lay.hash_off);
    float4* qs = reinterpret_cast<float4*>(smem_raw + lay.q_off);
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem_raw + lay.bar_off);

    const uint32_t hmask = (1u << p.hash_log2) - 1u;
    const int hshift = 32 - p.hash_log2;

    // work range of this launch
    const uint32_t w_begin = p.in_begin_ptr ? *p.in_begin_ptr : p.in_begin;
    const uint32_t w_end = p.in_end_ptr ? *p.in_end_ptr : p.in_end;
    if (p.active_count) {
        // Algorithm 1: "while |A| > tau * rho"
        if (!((double)(*p.active_count) > p.tau_q)) return;
    }
    const uint32_t n_work = w_end > w_begin ? w_end - w_begin : 0u;

    if (lane == 0) mbar_init(bar, 1u);
    __syncwarp();
    uint32_t bar_parity = 0;
    bool dead = false;             // a copy never completed: stop taking work

    while (!dead) {
        uint32_t t = 0;
        if (lane == 0) t = atomicAdd(p.ticket, 1u);
        t = __shfl_sync(0xffffffffu, t, 0);
        if (t >= n_work) break;
        const uint32_t qi = p.in_list ? p.in_list[w_begin + t] : (w_begin + t);

        // ---- load the query, its bounds; clear the table of scored ids
        {
            const float4* qsrc = reinterpret_cast<const float4*>(p.queries + (size_t)qi * p.D);
            for (int i = lane; i < p.D / 4; i += 32) qs[i] = qsrc[i];
            uint4 ff = make_uint4(kNoId, kNoId, kNoId, kNoId);
            uint4* h4 = reinterpret_cast<uint4*>(hash);
            for (int i = lane; i < (1 << p.hash_log2) / 4; i += 32) h4[i] = ff;
        }
        int32_t my_lo = 0, my_hi = 0;
        if (g < p.m) {
            my_lo = p.lo[(size_t)qi * p.m + g];
            my_hi = p.hi[(size_t)qi * p.m + g];
        }
        const bool my_float = (p.attr_float_mask >> g) & 1u;
        __syncwarp();

        // Scores cand[0..cnt): fetch the records, distance + violated predicates -> nk[0..cnt).
        auto score = [&](int cnt) {
            for (int b0 = 0; b0 < cnt && !dead; b0 += p.stage_rows) {
                const int nb = (cnt - b0 < p.stage_rows) ? cnt - b0 : p.stage_rows;
                fence_async_proxy();
                if (lane == 0) mbar_expect_tx(bar, (uint32_t)(nb * p.rec_bytes));
                __syncwarp();
                for (int j = lane; j < nb; j += 32) {
                    const uint32_t n = cand[b0 + j];
                    bulk_load_row(stage + (size_t)j * p.rec_bytes, p.rec + (size_t)n * p.rec_stride,
                                  (uint32_t)p.rec_bytes, bar);
                }
                uint32_t spins = 0;
                while (!mbar_try_wait(bar, bar_parity)) {
                    if (++spins > kWaitLimit) { dead = true; break; }
                }
                dead = __any_sync(0xffffffffu, dead);
                bar_parity ^= 1u;
                if (dead) {
                    if (lane == 0) atomicOr(p.status, kStatusCopyTimeout);
                    break;
                }
                for (int r0 = 0; r0 < nb; r0 += 4) {
                    const int j = r0 + gi;
                    const bool act = j < nb;
                    const uint8_t* row = stage + (size_t)(act ? j : 0) * p.rec_bytes;
                    float acc = 0.0f;
                    if (act) {
                        if (VT == 0) {
                            const float4* r4 = reinterpret_cast<const float4*>(row);
#pragma unroll 4
                            for (int c = g; c < p.nchunks; c += 8) acc = sq_acc4(acc, r4[c], qs[c]);
                        } else {
                            const uint4* r4 = reinterpret_cast<const uint4*>(row);
                            for (int c = g; c < p.nchunks; c += 8) {
                                const uint4 x = r4[c];
                                acc = sq_acc_bytes(acc, x.x, qs[4 * c + 0]);
                                acc = sq_acc_bytes(acc, x.y, qs[4 * c + 1]);
                                acc = sq_acc_bytes(acc, x.z, qs[4 * c + 2]);
                                acc = sq_acc_bytes(acc, x.w, qs[4 * c + 3]);
                            }
                        }
                    }
                    acc += __shfl_xor_sync(0xffffffffu, acc, 4);
                    acc += __shfl_xor_sync(0xffffffffu, acc, 2);
                    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
                    bool viol = false;
                    if (act && g < p.m) {
                        const uint32_t av = *reinterpret_cast<const uint32_t*>(row + p.attr_off + 4 * g);
                        if (my_float) {
                            const float x = __uint_as_float(av);
                            viol = !(x >= __int_as_float(my_lo) && x <= __int_as_float(my_hi));
                        } else {
                            const int32_t x = (int32_t)av;
                            viol = x < my_lo || x > my_hi;
                        }
                    }
                    const unsigned bal = __ballot_sync(0xffffffffu, viol);
                    const uint32_t phi = __popc((bal >> (8 * gi)) & 0xFFu);
                    if (act && g == 0) nk[b0 + j] = pack_key(phi, acc, cand[b0 + j]);
                }
                __syncwarp();
            }
        };

        // Returns true when id was not in the table; records it either way.
        auto hash_test_and_set = [&](uint32_t id) -> bool {
            const uint32_t h = (id * 0x9E3779B1u) >> hshift;
            int empty = -1;
#pragma unroll
            for (int pr = 0; pr < 4; ++pr) {
                const uint32_t s = (h + pr) & hmask;
                const uint32_t v = hash[s];
                if (v == id) return false;
                if (v == kNoId && empty < 0) empty = (int)s;
            }
            hash[empty >= 0 ? (uint32_t)empty : h] = id;
            return true;
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
                hash_test_and_set(key_id(e));
            }
            __syncwarp();
        } else {
            if (lane == 0) cand[0] = p.entry;
            __syncwarp();
            score(1);
            if (lane == 0) {
                pool[0] = nk[0];
                hash_test_and_set(p.entry);
            }
            n = 1;
            __syncwarp();
        }

        // ---- Algorithm 2 main loop
        while (!dead) {
            // nearest unexpanded entry among the first L
            const int lim = n < p.L ? n : p.L;
            int pos = -1;
            for (int b0 = cur & ~31; b0 < lim; b0 += 32) {
                const int i = b0 + lane;
                const bool un = (i >= cur) && (i < lim) && ((pool[i] & 1ull) == 0ull);
                const unsigned bal = __ballot_sync(0xffffffffu, un);
                if (bal) { pos = b0 + __ffs(bal) - 1; break; }
            }
            if (pos < 0) break;                                   // converged
            if (n_exp >= p.max_expand) { capped = true; break; }
            const uint32_t u_id = key_id(pool[pos]);
            __syncwarp();
            if (lane == 0) pool[pos] |= 1ull;
            cur = pos + 1;
            n_exp++;

            // adjacency row, drop ids scored before, compact the rest
            uint32_t nb[RS];
            const uint32_t* grow = p.graph + (size_t)u_id * p.R;
#pragma unroll
            for (int s = 0; s < RS; ++s) {
                const int j = lane + 32 * s;
                nb[s] = (j < p.R) ? __ldg(grow + j) : kNoId;
            }
            int cnt = 0;
#pragma unroll
            for (int s = 0; s < RS; ++s) {
                const bool fresh = (nb[s] != kNoId) && hash_test_and_set(nb[s]);
                const unsigned bal = __ballot_sync(0xffffffffu, fresh);
                if (fresh) cand[cnt + __popc(bal & lt_mask)] = nb[s];
                cnt += __popc(bal);
            }
            __syncwarp();
            if (cnt == 0) continue;
            n_sc += cnt;

            // gather + distance + range check (fused)
            score(cnt);
            if (dead) break;

            // new keys that cannot enter a full pool are dropped right away; sort the rest
            const uint64_t worst = (n == p.C) ? (pool[n - 1] >> 1) : (kKeyMax >> 1);
            uint64_t x[RS];
            int live = 0;
#pragma unroll
            for (int s = 0; s < RS; ++s) {
                const int j = lane + 32 * s;
                x[s] = (j < cnt) ? nk[j] : kKeyMax;
                if (x[s] != kKeyMax && (x[s] >> 1) >= worst) x[s] = kKeyMax;
                live += __popc(__ballot_sync(0xffffffffu, x[s] != kKeyMax));
            }
            if (live == 0) continue;
            if (live > 1) sort_keys<RS>(x, lane);
            __syncwarp();

            // rank of every new key in the pool; drop keys the pool already holds
            int steps = 0;
            while ((1 << steps) <= n) ++steps;
            bool keep[RS];
            int kept = 0;
            int pos_new[RS];
#pragma unroll
            for (int s = 0; s < RS; ++s) {
                const uint64_t xs = x[s] >> 1;
                const bool valid = x[s] != kKeyMax;
                int lo_i = 0, hi_i = valid ? n : 0;
                for (int it = 0; it < steps; ++it) {
                    if (lo_i < hi_i) {
                        const int mid = (lo_i + hi_i) >> 1;
                        if ((pool[mid] >> 1) < xs) lo_i = mid + 1; else hi_i = mid;
                    }
                }
                const bool dup = valid && (lo_i < n) && ((pool[lo_i] >> 1) == xs);
                const bool nd = valid && !dup;
                const unsigned bal = __ballot_sync(0xffffffffu, nd);
                const int pidx = kept + __popc(bal & lt_mask);
                pos_new[s] = lo_i + pidx;
                keep[s] = nd && (pos_new[s] < p.C);
                const unsigned kb = __ballot_sync(0xffffffffu, keep[s]);
                if (keep[s]) nr[pidx] = (uint32_t)lo_i;
                kept += __popc(kb);
            }
            __syncwarp();
            if (kept == 0) continue;
            const int rmin = (int)nr[0];

            // shift pool entries right by the number of new keys ranked at or before them
            for (int b0 = (n - 1) & ~31; b0 >= (rmin & ~31); b0 -= 32) {
                const int i = b0 + lane;
                uint64_t e = 0;
                int sh = 0;
                if (i < n && i >= rmin) {
                    e = pool[i];
                    if (kept <= 8) {
                        for (int j = 0; j < kept; ++j) sh += ((int)nr[j] <= i) ? 1 : 0;
                    } else {
                        int a = 0, b = kept;             // upper_bound(nr, i)
                        while (a < b) {
                            const int mid = (a + b) >> 1;
                            if ((int)nr[mid] <= i) a = mid + 1; else b = mid;
                        }
                        sh = a;
                    }
                }
                __syncwarp();
                if (sh > 0 && i + sh < p.C) pool[i + sh] = e;
                __syncwarp();
            }
#pragma unroll
            for (int s = 0; s < RS; ++s)
                if (keep[s]) pool[pos_new[s]] = x[s];
            n = (n + kept < p.C) ? n + kept : p.C;
            if (rmin < cur) cur = rmin;
            __syncwarp();
        }
        if (dead) break;

        // ---- result: the k nearest filter-valid entries (valid ones sort first)
        const int lim = n < p.L ? n : p.L;
        int nv_beam = 0;            // filter-valid entries among the first L
        for (int b0 = 0; b0 < lim; b0 += 32) {
            const int i = b0 + lane;
            const bool ok = (i < lim) && (key_phi(pool[i]) == 0u);
            nv_beam += __popc(__ballot_sync(0xffffffffu, ok));
        }
        for (int i = lane; i < p.k; i += 32) {
            uint32_t id = kNoId;
            float d2 = __int_as_float(0x7f800000);
            if (i < n) {
                const uint64_t e = pool[i];
                if (key_phi(e) == 0u) { id = key_id(e); d2 = key_d2(e); }
            }
            p.out_ids[(size_t)qi * p.k + i] = id;
            p.out_d2[(size_t)qi * p.k + i] = d2;
        }

        // ---- confidence test (Eq. 3) and compaction of the uncertain
        bool uncertain = true;
        if (nv_beam > p.k) {
            if (p.eps_mode < 0) uncertain = true;
            else if (p.eps_mode > 0) uncertain = false;
            else {
                const float d2k = key_d2(pool[p.k - 1]);
                const float d2max = key_d2(pool[nv_beam - 1]);
                uncertain = !(d2k >= p.c_eps * d2max);
            }
        }
        if (lane == 0) {
            p.final_L[qi] = p.L;
            if (p.first_phase) {
                p.n_expand[qi] = n_exp;
                p.n_scored[qi] = n_sc;
                p.flags[qi] = capped ? 1 : 0;
            } else {
                p.n_expand[qi] += n_exp;
                p.n_scored[qi] += n_sc;
                if (capped) p.flags[qi] |= 1;
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
    }
}

}  // namespace boa

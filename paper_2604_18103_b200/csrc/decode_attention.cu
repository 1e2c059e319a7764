// Decode-step attention: one new token per sequence attends over that sequence's packed KV cache
// (the cache of the deeper layers holds only the tokens that stayed active; it simply has fewer rows).
// HBM-bound: every cached key/value row is read once, and in the order it lies in memory: a tile is KT = 128 / Hkv
// consecutive cached tokens with all their KV heads -- 128 (token, KV head) rows, one contiguous piece of the cache.
// All Hq query heads form the rows of the 128-row Q operand, so S = Q K_tile^T holds, for query head r, the scores
// of its own KV head in the columns (token, r / G) and scores it has no use for in the others; P is written with
// zeros there, which makes O += P V_tile the per-head sum.  (The tensor pipe computes 128 rows whatever their
// number: the unused products cost nothing.)  The keys of a sequence are split over persistent CTAs, one per SM
// (flash-decoding); after a grid-wide barrier the CTAs share the merge of the splits.  One cooperative kernel per call
// for batches of up to 32 sequences (larger ones: a one-CTA plan kernel in front).
//   items      : (sequence, tile range), sized so that one item exists per CTA where that keeps the CTAs busy
//   per item   : S = Q K_j^T -> masked online softmax (one thread per query head) -> O += P V_j
//   merge      : O = sum_i 2^((m_i - m) c) O_i / sum_i 2^((m_i - m) c) l_i
#include <cooperative_groups.h>
#include <math.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace dash {

using namespace ptx;

constexpr int kDecRows = 128;                // rows of a tile: (token, KV head) pairs of K and V, query heads of Q
constexpr int kDecThreads = 256;             // warps 0..3: softmax (thread = query head), warp 4: TMA + MMA issue, all eight: merge
constexpr int kDecIssueWarp = 4;
constexpr int kDecRing = 5;                  // K / V tile buffers
constexpr long long kDecWaitCycles = 4000000000LL;
constexpr uint32_t kDecTmemCols = 512;       // S_0 | S_1 | O (| unused)

struct DecItem { int s, b0, b1; };           // tiles b0 .. b1 - 1 of sequence s

struct DecParams {
    const int32_t* cu;
    int S, Hq, G;
    float scale_log2, scale;
    float* partial;             // [item][Hq][D + 4]: unnormalised O row, then m, l
    const DecItem* plan;        // null: the CTAs plan for themselves (S <= kSelfPlanSeqs)
    const int2* seg;            // with a plan: first item and number of items of every sequence
    const int* n_items;
    int target;                 // items aimed at (self-planning)
    int* status;
    void* out; int64_t ldo; float* lse;
};

// Batches of up to kSelfPlanSeqs sequences need no plan kernel: every CTA derives the chunk length and its items
// (item i -> CTA i mod grid; the items are equally long) from cu_seqlens itself.
constexpr int kSelfPlanSeqs = 32;
// The plan of a self-planning launch, built once per CTA in shared memory: thread s fetches sequence s, thread 0 does the few
// serial steps over at most kSelfPlanSeqs numbers.
struct SelfPlan {
    int nb[kSelfPlanSeqs];        // tiles of sequence s
    int first[kSelfPlanSeqs];     // first item of sequence s
    int per[kSelfPlanSeqs];       // items of sequence s
    int chunk, n_items;
};
__device__ __forceinline__ int self_plan_count(const SelfPlan& sp, int S, int chunk) {
    int k = 0;
    for (int s = 0; s < S; ++s) k += (sp.nb[s] + chunk - 1) / chunk;
    return k;
}
// Called by all threads of the CTA (it synchronises).  `target` is twice the number of CTAs.  Chunk length (tiles per item):
// preferred is one item per CTA -- the shortest chunk with at most target / 2 items (the last chunk of every sequence is an
// item of its own, so the first guess can overshoot, and a CTA with a second item would double the kernel's time).  Taken when
// it keeps at least 17 of 20 CTAs busy; otherwise about `target` items.
__device__ __forceinline__ void self_plan_build(SelfPlan& sp, const int32_t* cu, int S, int KT, int target) {
    if ((int)threadIdx.x < S) sp.nb[threadIdx.x] = (cu[threadIdx.x + 1] - cu[threadIdx.x] + KT - 1) / KT;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long all = 0;
        for (int s = 0; s < S; ++s) all += sp.nb[s];
        long long chunk = (all + target - 1) / target;
        if (chunk < 1) chunk = 1;
        const int ctas = target / 2;
        if (ctas > 0) {
            long long c1 = (all + ctas - 1) / ctas;
            if (c1 < 1) c1 = 1;
            int cnt = self_plan_count(sp, S, (int)c1);
            for (int tries = 0; tries < 8 && cnt > ctas; ++tries) cnt = self_plan_count(sp, S, (int)++c1);
            if (cnt <= ctas && cnt * 20 >= ctas * 17) chunk = c1;
        }
        int k = 0;
        for (int s = 0; s < S; ++s) {
            sp.first[s] = k;
            sp.per[s] = (sp.nb[s] + (int)chunk - 1) / (int)chunk;
            k += sp.per[s];
        }
        sp.chunk = (int)chunk;
        sp.n_items = k;
    }
    __syncthreads();
}
__device__ __forceinline__ DecItem self_plan_item(const SelfPlan& sp, int S, int item) {
    DecItem it = {0, 0, 0};
    for (int s = 0; s < S; ++s) {
        if (item < sp.first[s] + sp.per[s]) {
            const int i = item - sp.first[s];
            it.s = s; it.b0 = i * sp.chunk; it.b1 = min((i + 1) * sp.chunk, sp.nb[s]);
            return it;
        }
    }
    return it;
}

// One CTA: per sequence the number of tiles, a common chunk length (tiles per item) so that about `target` items exist,
// then the items of every sequence written next to each other.
__global__ void __launch_bounds__(256)
decode_plan_kernel(const int32_t* __restrict__ cu, int S, int KT, int target, DecItem* __restrict__ plan, int2* __restrict__ seg,
                   int* __restrict__ n_items, int max_items) {
    __shared__ unsigned long long s_total;
    __shared__ int s_chunk;
    if (threadIdx.x == 0) s_total = 0;
    __syncthreads();
    unsigned long long mine = 0;
    for (int s = threadIdx.x; s < S; s += blockDim.x) mine += (unsigned long long)((cu[s + 1] - cu[s] + KT - 1) / KT);
    atomicAdd(&s_total, mine);
    __syncthreads();
    if (threadIdx.x == 0) {
        const long long all = (long long)s_total;
        const long long chunk = (all + target - 1) / target;
        s_chunk = (int)(chunk < 1 ? 1 : chunk);
        // first item of every sequence: one short serial pass over the sequences
        int k = 0;
        for (int s = 0; s < S; ++s) {
            const int nb = (cu[s + 1] - cu[s] + KT - 1) / KT;
            int per = (nb + s_chunk - 1) / s_chunk;
            if (k + per > max_items) per = max_items - k;          // cannot happen: max_items >= target + S
            seg[s] = make_int2(k, per);
            k += per;
        }
        *n_items = k;
    }
    __syncthreads();
    const int chunk = s_chunk;
    for (int s = threadIdx.x; s < S; s += blockDim.x) {
        const int nb = (cu[s + 1] - cu[s] + KT - 1) / KT;
        const int2 sg = seg[s];
        for (int i = 0; i < sg.y; ++i) {
            DecItem it = {s, i * chunk, min((i + 1) * chunk, nb)};
            plan[sg.x + i] = it;
        }
    }
}

template <int D>
struct DecSmem {
    static constexpr int kTileBytes = kDecRows * D * 2;
    static constexpr int kQ = 0, kRing = kTileBytes, kBars = (1 + kDecRing) * kTileBytes;
    static constexpr int kTotal = kBars + 256;
};

// no cached key anywhere: zeros and -inf (what the sum over no keys is)
__global__ void __launch_bounds__(128)
decode_empty_kernel(int Hq, int D, __nv_bfloat16* out, int64_t ldo, float* lse) {
    const int s = (int)blockIdx.x;
    for (int i = threadIdx.x; i < Hq * D; i += blockDim.x) out[(int64_t)s * ldo + i] = __float2bfloat16(0.f);
    if (lse) for (int h = threadIdx.x; h < Hq; h += blockDim.x) lse[(int64_t)s * Hq + h] = -INFINITY;
}

// The merge, shared by all CTAs behind the grid barrier.  A unit is 32 output columns of one (sequence, query head); it goes to a
// group of k warps (k = 1, 2, 4 or 8: as many as there are warps per unit, so that few units with many splits and many units
// with few splits both spread over the machine).  Every warp of the group finds the common maximum and the denominator (one
// round of loads over the splits' m and l), then sums its share of the splits, lane = column; the group meets in shared memory.
template <int D>
__device__ __forceinline__ void decode_merge_units(const DecParams& p, const SelfPlan& sp, bool self_plan, float (*s_acc)[32]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int NW = kDecThreads / 32, CH = D / 32, kRow = D + 4;
    const long long n_units = (long long)p.S * p.Hq * CH;
    const long long warps = (long long)gridDim.x * NW;
    int k = 1;
    while (k < NW && n_units * (2 * k) <= warps) k *= 2;
    const int sub = warp % k;
    const long long n_groups = (long long)gridDim.x * (NW / k), gid = (long long)blockIdx.x * (NW / k) + warp / k;
    const size_t stride = (size_t)p.Hq * kRow;
    for (long long u = gid; u < n_units; u += n_groups) {
        const int ch = (int)(u % CH), hd = (int)((u / CH) % p.Hq), s = (int)(u / ((long long)CH * p.Hq));
        int first, cnt;
        if (self_plan) { first = sp.first[s]; cnt = sp.per[s]; }
        else { const int2 sg = p.seg[s]; first = sg.x; cnt = sg.y; }
        const float* base = p.partial + ((size_t)first * p.Hq + hd) * kRow;
        // the first splits of this warp's share: their loads go out before anything is waited for
        constexpr int B = 8;
        float dv[B], dm[B];
#pragma unroll
        for (int b = 0; b < B; ++b) {
            const int i = sub + b * k;
            dv[b] = 0.f; dm[b] = -INFINITY;
            if (i < cnt) { dv[b] = __ldcg(base + i * stride + ch * 32 + lane); dm[b] = __ldcg(base + i * stride + D); }
        }
        float m0 = -INFINITY, l0 = 0.f, m1 = -INFINITY, l1 = 0.f;
        if (lane < cnt) { m0 = __ldcg(base + lane * stride + D); l0 = __ldcg(base + lane * stride + D + 1); }
        if (lane + 32 < cnt) { m1 = __ldcg(base + (lane + 32) * stride + D); l1 = __ldcg(base + (lane + 32) * stride + D + 1); }
        float mx = fmaxf(m0, m1);
        for (int i = lane + 64; i < cnt; i += 32) mx = fmaxf(mx, __ldcg(base + i * stride + D));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float ls = 0.f;
        if (lane < cnt) ls += exp2f((m0 - mx) * p.scale_log2) * l0;
        if (lane + 32 < cnt) ls += exp2f((m1 - mx) * p.scale_log2) * l1;
        for (int i = lane + 64; i < cnt; i += 32) ls += exp2f((__ldcg(base + i * stride + D) - mx) * p.scale_log2) * __ldcg(base + i * stride + D + 1);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, o);
        float acc = 0.f;
#pragma unroll
        for (int b = 0; b < B; ++b)
            if (sub + b * k < cnt) acc = fmaf(exp2f((dm[b] - mx) * p.scale_log2), dv[b], acc);
        for (int i0 = sub + B * k; i0 < cnt; i0 += B * k) {
#pragma unroll
            for (int b = 0; b < B; ++b) {
                const int i = i0 + b * k;
                dv[b] = 0.f; dm[b] = -INFINITY;
                if (i < cnt) { dv[b] = __ldcg(base + i * stride + ch * 32 + lane); dm[b] = __ldcg(base + i * stride + D); }
            }
#pragma unroll
            for (int b = 0; b < B; ++b)
                if (i0 + b * k < cnt) acc = fmaf(exp2f((dm[b] - mx) * p.scale_log2), dv[b], acc);
        }
        if (k > 1) {
            s_acc[warp][lane] = acc;
            asm volatile("bar.sync %0, %1;" ::"r"(1 + warp / k), "r"(k * 32) : "memory");
            if (sub == 0) {
                acc = 0.f;
                for (int j = 0; j < k; ++j) acc += s_acc[warp + j][lane];
            }
            asm volatile("bar.sync %0, %1;" ::"r"(1 + warp / k), "r"(k * 32) : "memory");
        }
        if (sub == 0) {
            const float v = cnt > 0 ? acc / ls : 0.f;
            reinterpret_cast<__nv_bfloat16*>(p.out)[(int64_t)s * p.ldo + (int64_t)hd * D + ch * 32 + lane] = __float2bfloat16(v);
            if (p.lse && ch == 0 && lane == 0) p.lse[(int64_t)s * p.Hq + hd] = cnt > 0 ? mx * p.scale + logf(ls) : -INFINITY;
        }
    }
}

// One CTA per SM (cooperative launch).  Warp 4 (one lane) streams the K and V tiles of the CTA's items, in order K_0 V_0 K_1 V_1 ..
// across the items, through a ring of kDecRing tile buffers -- the loads run up to kDecRing tiles ahead of the MMAs, whatever item
// they belong to -- and issues the MMAs: S_g = Q K_g^T into one of two TMEM buffers (so S_{g+1} runs while the softmax warps form
// P_g), then O += P_g V_g.  Softmax warp w holds query heads 32 w .. 32 w + 31, one per thread.
template <int D, int HKV>
__global__ void __launch_bounds__(kDecThreads, 1)
decode_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
              const __grid_constant__ CUtensorMap mapV, const DecParams p) {
    extern __shared__ uint8_t smem_raw[];
    using L = DecSmem<D>;
    constexpr int KT = kDecRows / HKV;       // cached tokens per tile
    constexpr int KCH = D / 64;
    constexpr int kChunkBytes = kDecRows * 128;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base + L::kQ, sRing = smem_base + L::kRing;
    const uint32_t bars = smem_base + L::kBars;
    const uint32_t bar_q = bars, bar_full = bars + 8 /* kDecRing of them */, bar_s = bars + 64 /* 2 */, bar_o = bars + 80 /* 2 */,
                   bar_p0 = bars + 96 /* 2 */, bar_p1 = bars + 112 /* 2 */;
    const uint32_t tmem_slot = bars + 128;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_gen + L::kBars + 128);
    volatile uint32_t* abort_gen = reinterpret_cast<volatile uint32_t*>(smem_gen + L::kBars + 132);
    __shared__ SelfPlan sp;
    __shared__ float s_acc[kDecThreads / 32][32];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nsw = (p.Hq + 31) / 32;        // softmax warps at work

    // rows of the Q tile that no load ever writes must not hold NaN patterns: clear the tile once
    for (int i = tid * 16; i < L::kTileBytes; i += kDecThreads * 16) *reinterpret_cast<uint4*>(smem_gen + L::kQ + i) = make_uint4(0, 0, 0, 0);
    fence_proxy_async_smem();
    if (warp == kDecIssueWarp) {
        if (lane == 0) {
            mbar_init(bar_q, 1);
            for (int i = 0; i < kDecRing; ++i) mbar_init(bar_full + 8 * i, 1);
            for (int i = 0; i < 2; ++i) {
                mbar_init(bar_s + 8 * i, 1); mbar_init(bar_o + 8 * i, 1);
                mbar_init(bar_p0 + 8 * i, 32 * nsw); mbar_init(bar_p1 + 8 * i, 32 * nsw);
            }
            *abort_gen = 0;
            fence_barrier_init();
            fence_proxy_async_smem();
            prefetch_tensormap(&mapQ); prefetch_tensormap(&mapK); prefetch_tensormap(&mapV);
        }
        __syncwarp();
        tmem_alloc(tmem_slot, kDecTmemCols);
        tmem_relinquish();
    }
    const bool self_plan = (p.plan == nullptr);
    if (self_plan) self_plan_build(sp, p.cu, p.S, KT, p.target);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_gen;
    const uint32_t tO = tmem + 256;          // S_0 / P_0 at column 0, S_1 / P_1 at 128, O at 256
    constexpr uint32_t idesc_s = idesc_bf16_f32(128, kDecRows, false, false);
    constexpr uint32_t idesc_o = idesc_bf16_f32(128, D, false, true);
    const int n_items = self_plan ? sp.n_items : *p.n_items;
    auto get_item = [&](int item) -> DecItem { return self_plan ? self_plan_item(sp, p.S, item) : p.plan[item]; };

    // ---- state of the issuing lane (warp 4, lane 0); g counts the tiles of this CTA across its items ----
    uint32_t loaded = 0;                     // tile loads issued (load 2g: K of tile g, 2g + 1: V)
    uint32_t s_issued = 0, pv_issued = 0;    // tiles whose S / PV MMAs have been issued
    uint32_t s_conf = 0, o_conf = 0;         // tiles whose S / PV MMAs are known to be complete (barrier phases taken in order)
    int ld_round = 0, ld_j = 0, ld_nblk = 0, ld_row0 = 0;   // load cursor: item blockIdx.x + ld_round * gridDim.x, tile ld_j of it
    bool ld_more = false, prod_ok = true;
    const bool issuer = (warp == kDecIssueWarp && lane == 0);
    auto ld_open = [&]() {                   // point the cursor at the first tile of item ld_round (if there is one)
        const int item = (int)blockIdx.x + ld_round * (int)gridDim.x;
        ld_more = item < n_items;
        if (ld_more) {
            const DecItem it = get_item(item);
            ld_j = 0; ld_nblk = it.b1 - it.b0;
            ld_row0 = p.cu[it.s] + it.b0 * KT;
        }
    };
    // tile h's S MMAs are complete (each phase of bar_s[h & 1] is taken exactly once, in order: S_{h+2} is not issued before)
    auto confirm_s = [&](uint32_t h) -> bool {
        while (s_conf <= h) {
            if (!mbar_wait(bar_s + 8 * (s_conf & 1), (s_conf >> 1) & 1, kDecWaitCycles)) return false;
            ++s_conf;
        }
        return true;
    };
    auto confirm_o = [&](uint32_t h) -> bool {
        while (o_conf <= h) {
            if (!mbar_wait(bar_o + 8 * (o_conf & 1), (o_conf >> 1) & 1, kDecWaitCycles)) return false;
            ++o_conf;
        }
        return true;
    };
    // issue loads while a ring buffer is free: load t takes the buffer of load t - kDecRing, free once the MMAs that read it are done
    auto pump = [&]() -> bool {
        while (ld_more) {
            const uint32_t t = loaded;
            if (t >= (uint32_t)kDecRing) {
                const uint32_t prev = t - kDecRing, gp = prev >> 1;
                if (prev & 1) { if (gp >= pv_issued) return true; if (!confirm_o(gp)) return false; }
                else          { if (gp >= s_issued) return true;  if (!confirm_s(gp)) return false; }
            }
            const uint32_t slot = t % kDecRing, dst = sRing + slot * L::kTileBytes, bar = bar_full + 8 * slot;
            mbar_arrive_expect_tx(bar, L::kTileBytes);
            const CUtensorMap* map = (t & 1) ? &mapV : &mapK;
            for (int c = 0; c < KCH; ++c) tma_load_3d(dst + c * kChunkBytes, map, bar, c * 64, 0, ld_row0 + ld_j * KT);
            ++loaded;
            if (t & 1) {                     // V of the tile: on to the next tile, or the next item
                if (++ld_j == ld_nblk) { ++ld_round; ld_open(); }
            }
        }
        return true;
    };
    auto wait_full = [&](uint32_t t) -> bool { return mbar_wait(bar_full + 8 * (t % kDecRing), (t / kDecRing) & 1, kDecWaitCycles); };
    auto issue_q = [&](const DecItem& it) {
        mbar_arrive_expect_tx(bar_q, (uint32_t)(KCH * p.Hq * 128));
        for (int c = 0; c < KCH; ++c) tma_load_3d(sQ + c * kChunkBytes, &mapQ, bar_q, c * 64, 0, it.s);
    };
    // O += P_h V_h (first of the item: O = ..); the first half of P's columns starts while the rest is still being formed
    auto issue_pv = [&](uint32_t h, bool accumulate) -> bool {
        const uint32_t b = h & 1, php = (h >> 1) & 1, tP = tmem + b * 128;
        if (h >= 2 && !confirm_o(h - 2)) return false;                     // keeps the phases of bar_o[b] from running ahead of this lane
        if (!mbar_wait(bar_p0 + 8 * b, php, kDecWaitCycles) || !wait_full(2 * h + 1)) return false;
        const uint32_t sV = sRing + ((2 * h + 1) % kDecRing) * L::kTileBytes;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < kDecRows / 32; ++kk)
            mma_ts(tO, tP + kk * 8, smem_desc_sw128(sV + kk * 2048, kChunkBytes, 1024), idesc_o, accumulate || (kk > 0));
        if (!mbar_wait(bar_p1 + 8 * b, php, kDecWaitCycles)) return false;
        tc_fence_after();
#pragma unroll
        for (int kk = kDecRows / 32; kk < kDecRows / 16; ++kk)
            mma_ts(tO, tP + kk * 8, smem_desc_sw128(sV + kk * 2048, kChunkBytes, 1024), idesc_o, 1);
        tc_commit(bar_o + 8 * b);
        pv_issued = h + 1;
        return true;
    };
    if (issuer) {
        ld_open();
        if (ld_more) issue_q(get_item((int)blockIdx.x));
        prod_ok = pump();
    }

    uint32_t g0 = 0, items_done = 0;         // first tile of the current item in the CTA's count; items finished
    for (;;) {
        const int item = (int)blockIdx.x + (int)items_done * (int)gridDim.x;
        if (item >= n_items || *abort_gen) break;
        const DecItem it = get_item(item);
        const int len = p.cu[it.s + 1] - p.cu[it.s];
        const int nblk = it.b1 - it.b0;
        const int last_blk = (len + KT - 1) / KT - 1;               // the tile of the sequence with a ragged end
        if (warp == kDecIssueWarp) {
            if (lane == 0) {
                bool ok = prod_ok && mbar_wait(bar_q, items_done & 1, kDecWaitCycles);
                for (int j = 0; j < nblk && ok; ++j) {
                    const uint32_t g = g0 + j, b = g & 1;
                    // S_g goes where S_{g-2} and P_{g-2} were: PV_{g-2} is in front of it in issue order
                    if (g >= 2) ok = confirm_s(g - 2);
                    ok = ok && wait_full(2 * g);
                    if (!ok) break;
                    const uint32_t sK = sRing + ((2 * g) % kDecRing) * L::kTileBytes;
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t off = (kk >> 2) * kChunkBytes + (kk & 3) * 32;
                        mma_ss(tmem + b * 128, smem_desc_sw128(sQ + off, 16, 1024), smem_desc_sw128(sK + off, 16, 1024), idesc_s, kk > 0);
                    }
                    tc_commit(bar_s + 8 * b);
                    s_issued = g + 1;
                    if (j > 0) ok = issue_pv(g - 1, j > 1);
                    ok = ok && pump();
                }
                if (ok) ok = issue_pv(g0 + nblk - 1, nblk > 1);
                // the item's last S is complete: the Q tile may take the next item's rows while this item's O is read out
                if (ok) ok = confirm_s(g0 + nblk - 1);
                const int next = item + (int)gridDim.x;
                if (ok && next < n_items) issue_q(get_item(next));
                if (ok) ok = pump();
                if (!ok) { prod_ok = false; *abort_gen = 1; atomicExch(p.status, DASH_ERR_TIMEOUT); }
            }
            __syncwarp();
        } else if (warp < nsw) {
            // ---- softmax warp: thread = query head r.  Of the 128 columns (token k, KV head h') of S the thread uses those of
            // its own KV head h = r / G: 32 columns at a time come out of TMEM, the own ones are picked by selects (the column's
            // head is a compile-time number), and P goes back with zeros in the other heads' columns. ----
            const int r = warp * 32 + lane;
            const int h = (HKV == 1 || r >= p.Hq) ? 0 : r / p.G;
            const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
            constexpr int OWN = 32 / HKV;                       // own columns per 32
            float m = -INFINITY, l = 0.f;
            bool ok = true;
            for (int j = 0; j < nblk; ++j) {
                const uint32_t g = g0 + j, b = g & 1, ph = (g >> 1) & 1;
                const uint32_t tS = tmem + b * 128 + lane_base, tP = tS;
                ok = mbar_wait(bar_s + 8 * b, ph, kDecWaitCycles);
                if (!ok || *abort_gen) { ok = false; break; }
                tc_fence_after();
                const bool ragged = (it.b0 + j == last_blk);
                const int valid = ragged ? len - (it.b0 + j) * KT : KT;     // cached tokens of this tile that exist (>= 1)
                auto own_of = [&](const uint32_t* reg, float* own, int q) {
#pragma unroll
                    for (int e = 0; e < OWN; ++e) {
                        uint32_t v = reg[e * HKV];
#pragma unroll
                        for (int hh = 1; hh < HKV; ++hh) v = (h == hh) ? reg[e * HKV + hh] : v;
                        own[e] = (q * OWN + e < valid) ? __uint_as_float(v) : -INFINITY;      // past the end of the sequence's cache
                    }
                };
                float mx = -INFINITY;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint32_t reg[32];
                    float own[OWN];
                    tmem_ld32(tS + q * 32, reg);
                    tmem_wait_ld();
                    own_of(reg, own, q);
#pragma unroll
                    for (int e = 0; e < OWN; ++e) mx = fmaxf(mx, own[e]);
                }
                // the reference max only moves when the tile's max exceeds it by more than 2^8 (then O is rescaled)
                const bool grow = (mx - m) * p.scale_log2 > 8.0f;
                const float m_new = grow ? mx : m;
                const float msl = m_new * p.scale_log2;
                const float alpha = grow ? ex2((m - m_new) * p.scale_log2) : 1.0f;
                if (j > 0 && __any_sync(0xffffffffu, grow)) {
                    ok = mbar_wait(bar_o + 8 * ((g - 1) & 1), ((g - 1) >> 1) & 1, kDecWaitCycles);     // PV_{g-1} done
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(tO + lane_base + c * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                        tmem_st32(tO + lane_base + c * 32, o);
                    }
                    tmem_wait_st();
                }
                if (ragged && warp == 0) {
                    // cached rows past the end of the sequence may hold anything: zero them (0 * garbage must not make a NaN)
                    ok = wait_full(2 * g + 1);
                    if (!ok) break;
                    uint8_t* vt = smem_gen + L::kRing + ((2 * g + 1) % kDecRing) * L::kTileBytes;
                    for (int row = valid * HKV + lane; row < kDecRows; row += 32) {
#pragma unroll
                        for (int c = 0; c < KCH; ++c) {
                            uint4* rowp = reinterpret_cast<uint4*>(vt + c * kChunkBytes + row * 128);
#pragma unroll
                            for (int e = 0; e < 8; ++e) rowp[e] = make_uint4(0, 0, 0, 0);
                        }
                    }
                    fence_proxy_async_smem();
                }
                float sum = 0.f;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint32_t reg[32], pk[16];
                    float own[OWN];
                    tmem_ld32(tS + q * 32, reg);
                    tmem_wait_ld();
                    own_of(reg, own, q);
#pragma unroll
                    for (int e = 0; e < OWN; ++e) {
                        own[e] = ex2(fmaf(own[e], p.scale_log2, -msl));         // 0 for the columns past the end
                        sum += own[e];
                    }
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        if (HKV == 1) {
                            pk[i] = pack_bf16(own[(2 * i) % OWN], own[(2 * i + 1) % OWN]);
                        } else {
                            const float v = own[(2 * i) / HKV];
                            pk[i] = pack_bf16(((2 * i) % HKV == h) ? v : 0.f, ((2 * i + 1) % HKV == h) ? v : 0.f);
                        }
                    }
                    // columns 0..63 of P go out (and their PV steps start) while the rest is still being formed
                    tmem_st16(tP + q * 16, pk);
                    if (q == 1 || q == 3) {
                        tmem_wait_st();
                        tc_fence_before();
                        mbar_arrive((q == 1 ? bar_p0 : bar_p1) + 8 * b);
                    }
                }
                l = l * alpha + sum;
                m = m_new;
            }
            const uint32_t gl = g0 + nblk - 1;
            if (ok) ok = mbar_wait(bar_o + 8 * (gl & 1), (gl >> 1) & 1, kDecWaitCycles);
            if (ok && !*abort_gen) {
                tc_fence_after();
                float* dst = p.partial + ((size_t)item * p.Hq + r) * (D + 4);
#pragma unroll 1
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tO + lane_base + c * 32, o);
                    tmem_wait_ld();
                    if (r < p.Hq) {
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            *reinterpret_cast<float4*>(dst + c * 32 + e) =
                                make_float4(__uint_as_float(o[e]), __uint_as_float(o[e + 1]), __uint_as_float(o[e + 2]), __uint_as_float(o[e + 3]));
                    }
                }
                if (r < p.Hq) { dst[D] = m; dst[D + 1] = l; }
            } else if (!ok && lane == 0) {
                *abort_gen = 1;
                atomicExch(p.status, DASH_ERR_TIMEOUT);
            }
        }
        // end of the item: O has been read out; the softmax warps and the issuing lane go on together
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        g0 += (uint32_t)nblk;
        ++items_done;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kDecIssueWarp) {
        tc_fence_after();
        tmem_dealloc(tmem, kDecTmemCols);
    }
    // every CTA's partial results are in memory behind the grid barrier; then the CTAs share the merge
    __threadfence();
    cooperative_groups::this_grid().sync();
    if (!*abort_gen) decode_merge_units<D>(p, sp, self_plan, s_acc);
}

static int decode_grid() { return sm_count(); }
static int decode_target(bool self_plan) {               // items aimed at: two per CTA when the CTAs plan (they go down to one each where
    return (self_plan ? 2 : 4) * decode_grid();          // that keeps them all busy), four per CTA with a plan kernel
}
static int decode_max_items(int S) { return 4 * decode_grid() + S; }

size_t decode_ws_bytes(int64_t n, int S, int Hq, int Hkv, int D) {
    (void)n; (void)Hkv;
    const size_t items = (size_t)decode_max_items(S);
    return 256 + align_up(items * sizeof(DecItem), 256) + align_up((size_t)S * sizeof(int2), 256) +
           align_up(items * (size_t)Hq * (size_t)(D + 4) * sizeof(float), 256);
}

// bf16 tensor [rows, heads, D]: box = 64 x box_heads x box_rows, 128-byte swizzle
static int make_map_heads_box(CUtensorMap* map, const void* base, int64_t rows, int heads, int D, int64_t ld, int box_heads, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return DASH_ERR_CUDA;
    cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)heads, (cuuint64_t)rows};
    cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)ld * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)box_heads, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DASH_OK : DASH_ERR_CUDA;
}

// cooperative launch: the CTAs meet at a grid-wide barrier, so all of them must be resident (one per SM, grid <= SMs)
template <int D, int HKV>
static int launch_decode(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const DecParams& p, int grid, cudaStream_t st) {
    using L = DecSmem<D>;
    const int smem = L::kTotal + 1024;
    static std::atomic<uint64_t> configured{0};
    if (!set_max_smem_once(decode_kernel<D, HKV>, smem, configured)) return DASH_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(kDecThreads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, decode_kernel<D, HKV>, mq, mk, mv, p) == cudaSuccess ? DASH_OK : DASH_ERR_CUDA;
}

template <int D>
static int launch_decode_hkv(int Hkv, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const DecParams& p, int grid,
                             cudaStream_t st) {
    switch (Hkv) {
        case 1: return launch_decode<D, 1>(mq, mk, mv, p, grid, st);
        case 2: return launch_decode<D, 2>(mq, mk, mv, p, grid, st);
        case 4: return launch_decode<D, 4>(mq, mk, mv, p, grid, st);
        case 8: return launch_decode<D, 8>(mq, mk, mv, p, grid, st);
        default: return DASH_ERR_UNSUPPORTED;
    }
}

}  // namespace dash

using namespace dash;

extern "C" int dash_decode_attention(const void* q, const void* Kc, const void* Vc, void* out, float* lse,
                                     int64_t ldq, int64_t ldk, int64_t ldv, int64_t ldo,
                                     const int32_t* cu_seqlens, int S, int64_t n, int Hq, int Hkv, int D, float scale,
                                     dash_dtype dt, void* ws, size_t ws_bytes, void* stream) {
    if (n < 0 || S < 1 || Hq < 1 || Hkv < 1 || !cu_seqlens) return DASH_ERR_INVALID_ARG;
    if (dt != DASH_F32 && dt != DASH_BF16) return DASH_ERR_INVALID_ARG;
    if (dt != DASH_BF16) return DASH_ERR_UNSUPPORTED;                 // the cache is read as stored: bf16 only
    if (D != 64 && D != 128) return DASH_ERR_UNSUPPORTED;
    if (Hq % Hkv) return DASH_ERR_INVALID_ARG;
    if (Hq > kDecRows || (Hkv != 1 && Hkv != 2 && Hkv != 4 && Hkv != 8)) return DASH_ERR_UNSUPPORTED;
    if (n > 0x7fffffffLL || S > 0x7fffffff / Hq) return DASH_ERR_INVALID_ARG;
    if (!q || !out || (n > 0 && (!Kc || !Vc))) return DASH_ERR_INVALID_ARG;
    if (ldq < (int64_t)Hq * D || ldo < (int64_t)Hq * D || ldk < (int64_t)Hkv * D || ldv < (int64_t)Hkv * D) return DASH_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || (n > 0 && (!aligned16(Kc) || !aligned16(Vc)))) return DASH_ERR_INVALID_ARG;
    if ((ldq * 2) % 16 || (ldk * 2) % 16 || (ldv * 2) % 16 || (ldo * 2) % 16) return DASH_ERR_INVALID_ARG;
    if (!(scale > 0.f)) return DASH_ERR_INVALID_ARG;
    if (!ws || ((uintptr_t)ws % 256) || ws_bytes < decode_ws_bytes(n, S, Hq, Hkv, D)) return DASH_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    if (n == 0) {
        decode_empty_kernel<<<S, 128, 0, st>>>(Hq, D, (__nv_bfloat16*)out, ldo, lse);
        DASH_CUDA_TRY(cudaGetLastError());
        return DASH_OK;
    }
    const int max_items = decode_max_items(S);
    const int KT = kDecRows / Hkv;
    char* w = (char*)ws;
    DecItem* plan = (DecItem*)(w + 256);
    int2* seg = (int2*)((char*)plan + align_up((size_t)max_items * sizeof(DecItem), 256));
    float* partial = (float*)((char*)seg + align_up((size_t)S * sizeof(int2), 256));
    const bool self_plan = S <= kSelfPlanSeqs;
    const int target = decode_target(self_plan);
    if (!self_plan) {
        decode_plan_kernel<<<1, 256, 0, st>>>(cu_seqlens, S, KT, target, plan, seg, (int*)(w + 4), max_items);
        DASH_CUDA_TRY(cudaGetLastError());
    }
    CUtensorMap mq, mk, mv;
    int rc;
    if ((rc = make_map_heads_box(&mq, q, S, Hq, D, ldq, Hq, 1)) != DASH_OK) return rc;
    if ((rc = make_map_heads_box(&mk, Kc, n, Hkv, D, ldk, Hkv, KT)) != DASH_OK) return rc;
    if ((rc = make_map_heads_box(&mv, Vc, n, Hkv, D, ldv, Hkv, KT)) != DASH_OK) return rc;
    DecParams p;
    p.cu = cu_seqlens; p.S = S; p.Hq = Hq; p.G = Hq / Hkv;
    p.scale = scale; p.scale_log2 = scale * 1.4426950408889634f;
    p.partial = partial; p.plan = self_plan ? nullptr : plan; p.seg = seg; p.n_items = (const int*)(w + 4);
    p.target = target;
    p.status = status_word_ptr();
    if (!p.status) return DASH_ERR_CUDA;
    p.out = out; p.ldo = ldo; p.lse = lse;
    const int grid = decode_grid();
    return D == 128 ? launch_decode_hkv<128>(Hkv, mq, mk, mv, p, grid, st) : launch_decode_hkv<64>(Hkv, mq, mk, mv, p, grid, st);
}

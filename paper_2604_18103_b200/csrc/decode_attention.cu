// Decode-step attention: one new token per sequence attends over that sequence's packed KV cache
// (the cache of the deeper layers holds only the tokens that stayed active; it simply has fewer rows).
// HBM-bound: every cached key/value row is read once.  The G = Hq / Hkv query heads that share one KV
// head form the (mostly empty) 128-row operand of the tcgen05 MMAs, so K and V tiles stream through
// shared memory once per KV head; the keys of a sequence are split over persistent CTAs (flash-decoding),
// whose partial (max, sum, O) results a merge kernel spread over all SMs combines.
//   plan kernel   : items (sequence, KV head, key-block range), sized so that one item exists per CTA (batches of up to 32 sequences: the CTAs plan for themselves) or four per SM (handed out by ticket)
//   decode kernel : per item  S = Q K_j^T -> masked online softmax (one warp: the rows that exist) -> O += P V_j
//   merge kernel  : O = sum_i 2^((m_i - m) c) O_i / sum_i 2^((m_i - m) c) l_i
#include <math.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace dash {

using namespace ptx;

constexpr int kDecBN = 128;                  // keys per block
constexpr int kDecThreads = 64;              // warp 0: softmax (rows 0..31 of the tile, G of them real), warp 1: TMA + MMA issue
constexpr int kDecRows = 8;                  // query heads per KV head the tile can hold (box of the Q load)
constexpr long long kDecWaitCycles = 4000000000LL;
constexpr uint32_t kDecTmemCols = 256;       // S | O

struct DecItem { int s, kvh, b0, b1; };

struct DecParams {
    const int32_t* cu;
    int S, Hq, Hkv, G;
    float scale_log2, scale;
    float* partial;             // [item][kDecRows][D]: unnormalised O rows
    float2* ml;                 // [Hq][max_items]: their (m, l); the splits of one head lie next to each other
    int max_items;
    const DecItem* plan;        // null: the CTAs plan for themselves (S <= kSelfPlanSeqs)
    const int* n_items;
    unsigned int* ticket;
    int target;                 // items aimed at (self-planning)
    int* status;
};

// Batches of up to kSelfPlanSeqs sequences need no plan kernel, no ticket and no scratch clear: every CTA derives the chunk
// length and its items (item i -> CTA i mod grid; the items are equally long) from cu_seqlens itself, and so does the merge.
constexpr int kSelfPlanSeqs = 32;
__device__ __forceinline__ int dec_blocks(const int32_t* cu, int s) { return (cu[s + 1] - cu[s] + kDecBN - 1) / kDecBN; }
// The plan of a self-planning launch, built once per CTA in shared memory: thread s fetches sequence s, thread 0 does the few
// serial steps over at most kSelfPlanSeqs numbers.  (Every thread deriving it on its own from cu_seqlens cost the merge kernel of a
// 32-sequence batch more than its merging.)
struct SelfPlan {
    int nb[kSelfPlanSeqs];        // key blocks of sequence s
    int first[kSelfPlanSeqs];     // first item of sequence s (its Hkv heads follow each other, `per` items each)
    int per[kSelfPlanSeqs];       // items per (sequence, KV head)
    int chunk, n_items;
};
__device__ __forceinline__ int self_plan_count(const SelfPlan& sp, int S, int Hkv, int chunk) {
    int k = 0;
    for (int s = 0; s < S; ++s) k += ((sp.nb[s] + chunk - 1) / chunk) * Hkv;
    return k;
}
// Called by all threads of the CTA (it synchronises).  `target` is twice the number of CTAs.  Chunk length (key blocks per item):
// preferred is one item per CTA -- the shortest chunk with at most target / 2 items (the last chunk of every sequence and head is an
// item of its own, so the first guess can overshoot, and a CTA with a second item would double the kernel's time); half the pipeline
// ramps and half the partial results to merge.  Taken when it keeps at least 17 of 20 CTAs busy; otherwise about `target` items.
__device__ __forceinline__ void self_plan_build(SelfPlan& sp, const int32_t* cu, int S, int Hkv, int target) {
    if ((int)threadIdx.x < S) sp.nb[threadIdx.x] = dec_blocks(cu, (int)threadIdx.x);
    __syncthreads();
    if (threadIdx.x == 0) {
        long long all = 0;
        for (int s = 0; s < S; ++s) all += sp.nb[s];
        all *= Hkv;
        long long chunk = (all + target - 1) / target;
        if (chunk < 1) chunk = 1;
        const int ctas = target / 2;
        if (ctas > 0) {
            long long c1 = (all + ctas - 1) / ctas;
            if (c1 < 1) c1 = 1;
            int cnt = self_plan_count(sp, S, Hkv, (int)c1);
            for (int tries = 0; tries < 8 && cnt > ctas; ++tries) cnt = self_plan_count(sp, S, Hkv, (int)++c1);
            if (cnt <= ctas && cnt * 20 >= ctas * 17) chunk = c1;
        }
        int k = 0;
        for (int s = 0; s < S; ++s) {
            sp.first[s] = k;
            sp.per[s] = (sp.nb[s] + (int)chunk - 1) / (int)chunk;
            k += sp.per[s] * Hkv;
        }
        sp.chunk = (int)chunk;
        sp.n_items = k;
    }
    __syncthreads();
}
__device__ __forceinline__ DecItem self_plan_item(const SelfPlan& sp, int S, int Hkv, int item) {
    DecItem it = {0, 0, 0, 0};
    for (int s = 0; s < S; ++s) {
        const int per = sp.per[s];
        if (item < sp.first[s] + per * Hkv) {
            const int r = item - sp.first[s], h = r / per, i = r - h * per;
            it.s = s; it.kvh = h; it.b0 = i * sp.chunk; it.b1 = min((i + 1) * sp.chunk, sp.nb[s]);
            return it;
        }
    }
    return it;
}

// One CTA: per sequence the number of key blocks, a common chunk length (blocks per item) so that about
// `target` items exist, then the items of every (sequence, KV head) written next to each other.
__global__ void __launch_bounds__(256)
decode_plan_kernel(const int32_t* __restrict__ cu, int S, int Hkv, int target, DecItem* __restrict__ plan, int2* __restrict__ seg,
                   int* __restrict__ n_items, unsigned int* __restrict__ ticket, int max_items, int* __restrict__ seq_first) {
    __shared__ unsigned long long s_total;
    __shared__ int s_chunk;
    if (threadIdx.x == 0) s_total = 0;
    __syncthreads();
    unsigned long long mine = 0;
    for (int s = threadIdx.x; s < S; s += blockDim.x) mine += (unsigned long long)((cu[s + 1] - cu[s] + kDecBN - 1) / kDecBN);
    atomicAdd(&s_total, mine);
    __syncthreads();
    if (threadIdx.x == 0) {
        const long long all = (long long)s_total * Hkv;
        const long long chunk = (all + target - 1) / target;
        s_chunk = (int)(chunk < 1 ? 1 : chunk);
        // first item of every sequence (its Hkv heads follow each other): one short serial pass over the sequences
        int k = 0;
        for (int s = 0; s < S; ++s) {
            seq_first[s] = k;
            const int nb = (cu[s + 1] - cu[s] + kDecBN - 1) / kDecBN;
            k += ((nb + s_chunk - 1) / s_chunk) * Hkv;
        }
        *n_items = k < max_items ? k : max_items;
        *ticket = 0u;
    }
    __syncthreads();
    const int chunk = s_chunk;
    for (int sh = threadIdx.x; sh < S * Hkv; sh += blockDim.x) {
        const int s = sh / Hkv, h = sh % Hkv;
        const int nb = (cu[s + 1] - cu[s] + kDecBN - 1) / kDecBN;
        const int per = (nb + chunk - 1) / chunk;
        const int first = seq_first[s] + h * per;
        int cnt = 0;
        for (int i = 0; i < per && first + i < max_items; ++i, ++cnt) {
            DecItem it = {s, h, i * chunk, min((i + 1) * chunk, nb)};
            plan[first + i] = it;
        }
        seg[sh] = make_int2(first, cnt);
    }
}

template <int D>
struct DecSmem {
    static constexpr int kTileBytes = kDecBN * D * 2;
    static constexpr int kQ = 0, kK = kTileBytes, kV = 2 * kTileBytes, kBars = 3 * kTileBytes;
    static constexpr int kTotal = kBars + 128;
};

template <int D>
__global__ void __launch_bounds__(kDecThreads)
decode_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
              const __grid_constant__ CUtensorMap mapV, const DecParams p, int q_box_heads) {
    extern __shared__ uint8_t smem_raw[];
    using L = DecSmem<D>;
    constexpr int KCH = D / 64;
    constexpr int kChunkBytes = kDecBN * 128;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base + L::kQ, sK = smem_base + L::kK, sV = smem_base + L::kV;
    const uint32_t bars = smem_base + L::kBars;
    const uint32_t bar_q = bars, bar_k = bars + 8, bar_v = bars + 16, bar_s = bars + 24, bar_o = bars + 32, bar_p0 = bars + 40, bar_p1 = bars + 48;
    const uint32_t tmem_slot = bars + 64;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_gen + L::kBars + 64);
    volatile uint32_t* abort_gen = reinterpret_cast<volatile uint32_t*>(smem_gen + L::kBars + 68);
    volatile int* item_gen = reinterpret_cast<volatile int*>(smem_gen + L::kBars + 72);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    pdl_launch_dependents();                 // the merge kernel may get onto the SMs while this one runs

    // rows of the Q tile that no load ever writes must not hold NaN patterns: clear the tile once
    for (int i = tid * 16; i < L::kTileBytes; i += kDecThreads * 16) *reinterpret_cast<uint4*>(smem_gen + L::kQ + i) = make_uint4(0, 0, 0, 0);
    fence_proxy_async_smem();
    if (warp == 1) {
        if (lane == 0) {
            mbar_init(bar_q, 1); mbar_init(bar_k, 1); mbar_init(bar_v, 1);
            mbar_init(bar_s, 1); mbar_init(bar_o, 1); mbar_init(bar_p0, 32); mbar_init(bar_p1, 32);
            *abort_gen = 0;
            fence_barrier_init();
            fence_proxy_async_smem();
            prefetch_tensormap(&mapQ); prefetch_tensormap(&mapK); prefetch_tensormap(&mapV);
        }
        __syncwarp();
        tmem_alloc(tmem_slot, kDecTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_wait();                              // set-up done; from here on the kernel in front has completed
    const uint32_t tmem = *tmem_slot_gen;
    const uint32_t tS = tmem, tP = tmem, tO = tmem + 128;
    constexpr uint32_t idesc_s = idesc_bf16_f32(128, kDecBN, false, false);
    constexpr uint32_t idesc_o = idesc_bf16_f32(128, D, false, true);
    const bool self_plan = (p.plan == nullptr);
    __shared__ SelfPlan sp;
    if (self_plan) self_plan_build(sp, p.cu, p.S, p.Hkv, p.target);
    const int n_items = self_plan ? sp.n_items : *p.n_items;
    uint32_t blk0 = 0, items_done = 0;       // barrier phases run on across the items of this CTA

    for (;;) {
        int item;
        if (self_plan) {
            item = (int)blockIdx.x + (int)items_done * (int)gridDim.x;
        } else {
            if (tid == 0) *item_gen = (int)atomicAdd(p.ticket, 1u);
            __syncthreads();
            item = *item_gen;
        }
        if (item >= n_items || *abort_gen) break;
        tc_fence_after();
        const DecItem it = self_plan ? self_plan_item(sp, p.S, p.Hkv, item) : p.plan[item];
        const int seq_a = p.cu[it.s], len = p.cu[it.s + 1] - seq_a;
        const int nblk = it.b1 - it.b0;
        const int last_blk = (len + kDecBN - 1) / kDecBN - 1;       // the block of the sequence with a ragged end
        if (warp == 1) {
            if (lane == 0) {
                bool ok = true;
                mbar_arrive_expect_tx(bar_q, (uint32_t)(KCH * q_box_heads * 128));
                for (int c = 0; c < KCH; ++c) tma_load_3d(sQ + c * kChunkBytes, &mapQ, bar_q, c * 64, it.kvh * p.G, it.s);
                mbar_arrive_expect_tx(bar_k, L::kTileBytes);
                for (int c = 0; c < KCH; ++c) tma_load_3d(sK + c * kChunkBytes, &mapK, bar_k, c * 64, it.kvh, seq_a + it.b0 * kDecBN);
                mbar_arrive_expect_tx(bar_v, L::kTileBytes);
                for (int c = 0; c < KCH; ++c) tma_load_3d(sV + c * kChunkBytes, &mapV, bar_v, c * 64, it.kvh, seq_a + it.b0 * kDecBN);
                auto issue_s = [&]() {
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t off = (kk >> 2) * kChunkBytes + (kk & 3) * 32;
                        mma_ss(tS, smem_desc_sw128(sQ + off, 16, 1024), smem_desc_sw128(sK + off, 16, 1024), idesc_s, kk > 0);
                    }
                    tc_commit(bar_s);
                };
                ok = mbar_wait(bar_q, items_done & 1, kDecWaitCycles) && mbar_wait(bar_k, blk0 & 1, kDecWaitCycles);
                if (ok) issue_s();
                for (int j = 0; j < nblk && ok; ++j) {
                    const uint32_t ph = (blk0 + j) & 1;
                    ok = mbar_wait(bar_s, ph, kDecWaitCycles);               // S_j done: the K buffer is free
                    if (!ok) break;
                    if (j + 1 < nblk) {
                        mbar_arrive_expect_tx(bar_k, L::kTileBytes);
                        for (int c = 0; c < KCH; ++c) tma_load_3d(sK + c * kChunkBytes, &mapK, bar_k, c * 64, it.kvh, seq_a + (it.b0 + j + 1) * kDecBN);
                    }
                    ok = mbar_wait(bar_p0, ph, kDecWaitCycles) && mbar_wait(bar_v, ph, kDecWaitCycles);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < kDecBN / 32; ++kk)
                        mma_ts(tO, tP + kk * 8, smem_desc_sw128(sV + kk * 2048, kChunkBytes, 1024), idesc_o, (j > 0) || (kk > 0));
                    ok = mbar_wait(bar_p1, ph, kDecWaitCycles);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int kk = kDecBN / 32; kk < kDecBN / 16; ++kk)
                        mma_ts(tO, tP + kk * 8, smem_desc_sw128(sV + kk * 2048, kChunkBytes, 1024), idesc_o, 1);
                    tc_commit(bar_o);
                    if (j + 1 < nblk) {
                        ok = mbar_wait(bar_k, (blk0 + j + 1) & 1, kDecWaitCycles);
                        if (!ok) break;
                        issue_s();                                         // in issue order behind PV_j, which reads P_j from the same columns
                    }
                    ok = mbar_wait(bar_o, ph, kDecWaitCycles);              // PV_j done: the V buffer is free
                    if (!ok) break;
                    if (j + 1 < nblk) {
                        mbar_arrive_expect_tx(bar_v, L::kTileBytes);
                        for (int c = 0; c < KCH; ++c) tma_load_3d(sV + c * kChunkBytes, &mapV, bar_v, c * 64, it.kvh, seq_a + (it.b0 + j + 1) * kDecBN);
                    }
                }
                if (!ok) { *abort_gen = 1; atomicExch(p.status, DASH_ERR_TIMEOUT); }
            }
        } else {
            // ---- softmax warp.  Only rows 0..G-1 of the 128-row tile exist, so the scores are fetched in the 16-row shape
            // (tcgen05.ld.16x256b): thread t holds, of row t / 4, the keys 8u + 2 (t % 4) + {0, 1} of every group u of 8 keys
            // (and the same of row t / 4 + 8, which is not a real head and is ignored).  Four threads share a row: 32 exponentials
            // per thread and block instead of 128.  P goes back in the 16x128b shape, whose 32-bit column 4u + (t % 4) is exactly
            // the pair of keys the thread holds. ----
            const int sub = lane & 3, hrow = lane >> 2;         // position within the row's four threads, row (query head of the group)
            float m = -INFINITY, l = 0.f;                       // m: common to the row's threads, l: this thread's share
            bool ok = true;
            for (int j = 0; j < nblk; ++j) {
                const uint32_t ph = (blk0 + j) & 1;
                ok = mbar_wait(bar_s, ph, kDecWaitCycles);
                if (!ok || *abort_gen) { ok = false; break; }
                tc_fence_after();
                uint32_t raw[64];
                tmem_ld16x256_x8(tS, &raw[0]);
                tmem_ld16x256_x8(tS + 64, &raw[32]);
                tmem_wait_ld();
                float sc[32];                                   // sc[2u + e] = score of key 8u + 2 sub + e
#pragma unroll
                for (int u = 0; u < 16; ++u) { sc[2 * u] = __uint_as_float(raw[4 * u]); sc[2 * u + 1] = __uint_as_float(raw[4 * u + 1]); }
                const bool ragged = (it.b0 + j == last_blk);
                const int valid = len - (it.b0 + j) * kDecBN;               // keys of this block that exist (>= 1)
                if (ragged) {
#pragma unroll
                    for (int u = 0; u < 16; ++u) {
                        if (8 * u + 2 * sub >= valid) sc[2 * u] = -INFINITY;         // past the end of the sequence's cache
                        if (8 * u + 2 * sub + 1 >= valid) sc[2 * u + 1] = -INFINITY;
                    }
                }
                float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
                for (int c = 0; c < 32; c += 4) {
                    mx0 = fmax3(mx0, sc[c], sc[c + 1]);
                    mx1 = fmax3(mx1, sc[c + 2], sc[c + 3]);
                }
                float mx = fmaxf(mx0, mx1);
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                // the reference max only moves when the block max exceeds it by more than 2^8 (then O is rescaled)
                const bool grow = (mx - m) * p.scale_log2 > 8.0f;
                const float m_new = grow ? mx : m;
                const float msl = m_new * p.scale_log2;
                const float alpha = grow ? ex2((m - m_new) * p.scale_log2) : 1.0f;
                if (j > 0 && __any_sync(0xffffffffu, grow)) {
                    ok = mbar_wait(bar_o, (blk0 + j - 1) & 1, kDecWaitCycles);
                    if (!ok) break;
                    tc_fence_after();
                    const float a_row = __shfl_sync(0xffffffffu, alpha, (lane * 4) & 31);   // lane r < 8 rescales row r of O
#pragma unroll 1
                    for (int c = 0; c < D / 8; ++c) {
                        uint32_t o[8];
                        tmem_ld8(tO + c * 8, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 8; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * (lane < 8 ? a_row : 1.0f));
                        tmem_st8(tO + c * 8, o);
                    }
                    tmem_wait_st();
                }
                if (ragged) {
                    // cached rows past the end of the sequence may hold anything: zero them (0 * garbage must not make a NaN)
                    ok = mbar_wait(bar_v, ph, kDecWaitCycles);
                    if (!ok) break;
                    for (int r = lane; r < kDecBN; r += 32) {
                        if (r >= valid) {
#pragma unroll
                            for (int c = 0; c < KCH; ++c) {
                                uint4* rowp = reinterpret_cast<uint4*>(smem_gen + L::kV + c * kChunkBytes + r * 128);
#pragma unroll
                                for (int e = 0; e < 8; ++e) rowp[e] = make_uint4(0, 0, 0, 0);
                            }
                        }
                    }
                    fence_proxy_async_smem();
                }
                float2 sum2 = make_float2(0.f, 0.f);
                const float2 sl2 = make_float2(p.scale_log2, p.scale_log2), nm2 = make_float2(-msl, -msl);
                uint32_t pk[32];                                // pk[2u] = P of (row, keys 8u + 2 sub + {0,1}); pk[2u + 1] = row + 8: nothing
#pragma unroll
                for (int half = 0; half < 2; ++half) {
#pragma unroll
                    for (int u = half * 8; u < half * 8 + 8; ++u) {
                        const float2 x = __ffma2_rn(make_float2(sc[2 * u], sc[2 * u + 1]), sl2, nm2);
                        float2 pe;
                        pe.x = ex2(x.x); pe.y = ex2(x.y);
                        sum2 = __fadd2_rn(sum2, pe);
                        pk[2 * u] = pack_bf16(pe.x, pe.y);
                        pk[2 * u + 1] = 0u;
                    }
                    // the first 64 keys of P go out (and their PV steps start) while the rest is still being formed
                    tmem_st16x128_x8(tP + half * 32, &pk[half * 16]);
                    tmem_wait_st();
                    tc_fence_before();
                    mbar_arrive(half == 0 ? bar_p0 : bar_p1);
                }
                l = l * alpha + (sum2.x + sum2.y);
                m = m_new;
            }
            if (ok) ok = mbar_wait(bar_o, (blk0 + nblk - 1) & 1, kDecWaitCycles);
            // row sum: the four threads' shares; then lane r < G writes row r (its m and l sit in thread 4 r)
            l += __shfl_xor_sync(0xffffffffu, l, 1);
            l += __shfl_xor_sync(0xffffffffu, l, 2);
            const float m_row = __shfl_sync(0xffffffffu, m, (lane * 4) & 31), l_row = __shfl_sync(0xffffffffu, l, (lane * 4) & 31);
            (void)hrow;
            if (ok && !*abort_gen) {
                tc_fence_after();
                float* dst = p.partial + ((size_t)item * kDecRows + lane) * D;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tO + c * 32, o);
                    tmem_wait_ld();
                    if (lane < p.G) {
#pragma unroll
                        for (int e = 0; e < 32; e += 2)
                            *reinterpret_cast<float2*>(dst + c * 32 + e) = make_float2(__uint_as_float(o[e]), __uint_as_float(o[e + 1]));
                    }
                }
                if (lane < p.G) p.ml[(size_t)(it.kvh * p.G + lane) * p.max_items + item] = make_float2(m_row, l_row);
            } else if (!ok && lane == 0) {
                *abort_gen = 1;
                atomicExch(p.status, DASH_ERR_TIMEOUT);
            }
        }
        tc_fence_before();
        __syncthreads();                      // end of the item: O read out, every tile buffer free
        blk0 += (uint32_t)nblk;
        ++items_done;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, kDecTmemCols);
    }
}

// The merge of the key splits, spread over the whole machine.  A unit is 32 output columns of one (sequence, query head); it goes to a
// group of K warps (K = 1, 2, 4 or 8: as many as there are warps per unit, so that few units with many splits and many units with
// few splits both fill the SMs).  Every warp of the group loads the splits' (m, l) pairs, lane = split (they lie next to each other:
// coalesced), and forms the common maximum, the splits' weights and the denominator; then it sums its share of the splits, lane =
// column, with the weights handed round by shuffles.  All loads of a unit go out before the first is waited for; the group meets in
// shared memory.
constexpr int kMergeThreads = 256;
struct MergeParams {
    const float* partial; const float2* ml; int max_items;
    const int2* seg;            // with a plan: first item and number of items of every (sequence, KV head); else the CTAs plan for themselves
    const int32_t* cu; int S, target, Hq, Hkv, G;
    float scale_log2, scale;
    __nv_bfloat16* out; int64_t ldo; float* lse;
};
template <int D, int K>
__device__ __forceinline__ void decode_merge_units(const MergeParams& p, const SelfPlan& sp, float (*s_acc)[32]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int NW = kMergeThreads / 32, CH = D / 32;
    constexpr int B = 32, ML = B * K / 32;               // splits of one round: B per warp, their (m, l) in ML registers per lane
    const int n_units = p.S * p.Hq * CH;
    const int sub = warp % K;
    const int n_groups = (int)gridDim.x * (NW / K), gid = (int)blockIdx.x * (NW / K) + warp / K;
    const size_t stride = (size_t)kDecRows * D;
    for (int u = gid; u < n_units; u += n_groups) {
        const int ch = u % CH, hd = (u / CH) % p.Hq, s = u / (CH * p.Hq);
        const int kvh = hd / p.G, row = hd % p.G;
        int first, cnt;
        if (!p.seg) { cnt = sp.per[s]; first = sp.first[s] + kvh * cnt; }
        else { const int2 sg = p.seg[s * p.Hkv + kvh]; first = sg.x; cnt = sg.y; }
        const float* base = p.partial + ((size_t)first * kDecRows + row) * D + ch * 32 + lane;
        const float2* mlb = p.ml + (size_t)hd * p.max_items + first;
        float dv[B];
        float2 ml[ML];
#pragma unroll
        for (int b = 0; b < B; ++b) { const int i = sub + b * K; dv[b] = (i < cnt) ? __ldcg(base + i * stride) : 0.f; }
#pragma unroll
        for (int j = 0; j < ML; ++j) { const int i = lane + 32 * j; ml[j] = (i < cnt) ? __ldcg(mlb + i) : make_float2(-INFINITY, 0.f); }
        float mx = -INFINITY;
#pragma unroll
        for (int j = 0; j < ML; ++j) mx = fmaxf(mx, ml[j].x);
        for (int i = lane + 32 * ML; i < cnt; i += 32) mx = fmaxf(mx, __ldcg(mlb + i).x);          // more than B * K splits: further rounds
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float ls = 0.f;
#pragma unroll
        for (int j = 0; j < ML; ++j) {
            ml[j].x = exp2f((ml[j].x - mx) * p.scale_log2);     // the split's weight (0 where there is no split)
            ls = fmaf(ml[j].x, ml[j].y, ls);
        }
        for (int i = lane + 32 * ML; i < cnt; i += 32) { const float2 v = __ldcg(mlb + i); ls = fmaf(exp2f((v.x - mx) * p.scale_log2), v.y, ls); }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, o);
        float acc = 0.f;
#pragma unroll
        for (int b = 0; b < B; ++b) acc = fmaf(__shfl_sync(0xffffffffu, ml[(b * K) / 32].x, (sub + b * K) & 31), dv[b], acc);
        for (int i = sub + B * K; i < cnt; i += K) acc = fmaf(exp2f((__ldcg(mlb + i).x - mx) * p.scale_log2), __ldcg(base + i * stride), acc);
        if (K > 1) {
            s_acc[warp][lane] = acc;
            asm volatile("bar.sync %0, %1;" ::"r"(1 + warp / K), "n"(K * 32) : "memory");
            if (sub == 0) {
                acc = 0.f;
#pragma unroll
                for (int j = 0; j < K; ++j) acc += s_acc[warp + j][lane];
            }
            asm volatile("bar.sync %0, %1;" ::"r"(1 + warp / K), "n"(K * 32) : "memory");
        }
        if (sub == 0) {
            const float v = cnt > 0 ? acc / ls : 0.f;
            p.out[(int64_t)s * p.ldo + (int64_t)hd * D + ch * 32 + lane] = __float2bfloat16(v);
            if (p.lse && ch == 0 && lane == 0) p.lse[(int64_t)s * p.Hq + hd] = cnt > 0 ? mx * p.scale + logf(ls) : -INFINITY;
        }
    }
}

template <int D>
__global__ void __launch_bounds__(kMergeThreads)
decode_merge_kernel(const MergeParams p) {
    __shared__ SelfPlan sp;
    __shared__ float s_acc[kMergeThreads / 32][32];
    pdl_launch_dependents();
    pdl_wait();                              // started while the decode kernel drains: its partial results are complete from here on
    if (!p.seg) self_plan_build(sp, p.cu, p.S, p.Hkv, p.target);
    // warps per unit: as many as the machine has per unit, at most the CTA's eight
    const long long n_units = (long long)p.S * p.Hq * (D / 32), warps = (long long)gridDim.x * (kMergeThreads / 32);
    if (n_units * 16 <= warps) decode_merge_units<D, 8>(p, sp, s_acc);
    else if (n_units * 8 <= warps) decode_merge_units<D, 4>(p, sp, s_acc);
    else if (n_units * 4 <= warps) decode_merge_units<D, 2>(p, sp, s_acc);
    else decode_merge_units<D, 1>(p, sp, s_acc);
}

static int decode_max_items(int S, int Hkv) { return 4 * sm_count() + S * Hkv; }

size_t decode_ws_bytes(int64_t n, int S, int Hq, int Hkv, int D) {
    (void)n; (void)Hq;
    const size_t items = (size_t)decode_max_items(S, Hkv);
    return 256 + align_up(items * sizeof(DecItem), 256) + align_up((size_t)S * Hkv * sizeof(int2), 256) + align_up((size_t)S * sizeof(int), 256) +
           align_up(items * kDecRows * (size_t)D * sizeof(float), 256) + align_up(items * (size_t)Hq * sizeof(float2), 256);
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

template <int D>
static int launch_decode(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const DecParams& p, int box_heads, int grid,
                         cudaStream_t st) {
    using L = DecSmem<D>;
    const int smem = L::kTotal + 1024;
    static std::atomic<uint64_t> configured{0};
    if (!set_max_smem_once(decode_kernel<D>, smem, configured)) return DASH_ERR_CUDA;
    return launch_pdl(decode_kernel<D>, grid, kDecThreads, (size_t)smem, st, mq, mk, mv, p, box_heads) == cudaSuccess ? DASH_OK : DASH_ERR_CUDA;
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
    const int G = Hq / Hkv;
    if (G > kDecRows) return DASH_ERR_UNSUPPORTED;
    if (n > 0x7fffffffLL || S > 0x7fffffff / (Hq * 4)) return DASH_ERR_INVALID_ARG;      // the merge counts its units in an int
    if (!q || !out || (n > 0 && (!Kc || !Vc))) return DASH_ERR_INVALID_ARG;
    if (ldq < (int64_t)Hq * D || ldo < (int64_t)Hq * D || ldk < (int64_t)Hkv * D || ldv < (int64_t)Hkv * D) return DASH_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || (n > 0 && (!aligned16(Kc) || !aligned16(Vc)))) return DASH_ERR_INVALID_ARG;
    if ((ldq * 2) % 16 || (ldk * 2) % 16 || (ldv * 2) % 16 || (ldo * 2) % 16) return DASH_ERR_INVALID_ARG;
    if (!(scale > 0.f)) return DASH_ERR_INVALID_ARG;
    if (!ws || ((uintptr_t)ws % 256) || ws_bytes < decode_ws_bytes(n, S, Hq, Hkv, D)) return DASH_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const int max_items = decode_max_items(S, Hkv);
    char* w = (char*)ws;
    DecItem* plan = (DecItem*)(w + 256);
    int2* seg = (int2*)(w + 256 + align_up((size_t)max_items * sizeof(DecItem), 256));
    int* seq_first = (int*)((char*)seg + align_up((size_t)S * Hkv * sizeof(int2), 256));
    float* partial = (float*)((char*)seq_first + align_up((size_t)S * sizeof(int), 256));
    float2* ml = (float2*)((char*)partial + align_up((size_t)max_items * kDecRows * D * sizeof(float), 256));
    const bool self_plan = S <= kSelfPlanSeqs;
    const int target = 4 * sm_count();        // items aimed at: four per SM (self-planning CTAs go down to one item each where that keeps them all busy)
    if (!self_plan) {
        decode_plan_kernel<<<1, 256, 0, st>>>(cu_seqlens, S, Hkv, target, plan, seg, (int*)(w + 4), (unsigned int*)w, max_items, seq_first);
        DASH_CUDA_TRY(cudaGetLastError());
    }
    const float scale_log2 = scale * 1.4426950408889634f;
    if (n > 0) {
        CUtensorMap mq, mk, mv;
        int rc;
        const int box_heads = Hq < kDecRows ? Hq : kDecRows;
        if ((rc = make_map_heads_box(&mq, q, S, Hq, D, ldq, box_heads, 1)) != DASH_OK) return rc;
        if ((rc = make_map_heads_box(&mk, Kc, n, Hkv, D, ldk, 1, kDecBN)) != DASH_OK) return rc;
        if ((rc = make_map_heads_box(&mv, Vc, n, Hkv, D, ldv, 1, kDecBN)) != DASH_OK) return rc;
        DecParams p;
        p.cu = cu_seqlens; p.S = S; p.Hq = Hq; p.Hkv = Hkv; p.G = G;
        p.scale = scale; p.scale_log2 = scale_log2;
        p.partial = partial; p.ml = ml; p.max_items = max_items; p.plan = self_plan ? nullptr : plan; p.n_items = (const int*)(w + 4); p.ticket = (unsigned int*)w;
        p.target = target;
        p.status = status_word_ptr();
        if (!p.status) return DASH_ERR_CUDA;
        int grid = 2 * sm_count();
        if (grid > max_items) grid = max_items;
        rc = D == 128 ? launch_decode<128>(mq, mk, mv, p, box_heads, grid, st) : launch_decode<64>(mq, mk, mv, p, box_heads, grid, st);
        if (rc != DASH_OK) return rc;
    }
    MergeParams mp;
    mp.partial = partial; mp.ml = ml; mp.max_items = max_items; mp.seg = self_plan ? nullptr : seg;
    mp.cu = cu_seqlens; mp.S = S; mp.target = target; mp.Hq = Hq; mp.Hkv = Hkv; mp.G = G;
    mp.scale_log2 = scale_log2; mp.scale = scale;
    mp.out = (__nv_bfloat16*)out; mp.ldo = ldo; mp.lse = lse;
    // one warp per unit at least, never more CTAs than SMs
    const long long units = (long long)S * Hq * (D / 32);
    long long mgrid = (units * 8 + kMergeThreads / 32 - 1) / (kMergeThreads / 32);
    if (mgrid > sm_count()) mgrid = sm_count();
    if (mgrid < 1) mgrid = 1;
    if (D == 128) DASH_CUDA_TRY(launch_pdl(decode_merge_kernel<128>, (int)mgrid, kMergeThreads, 0, st, mp));
    else DASH_CUDA_TRY(launch_pdl(decode_merge_kernel<64>, (int)mgrid, kMergeThreads, 0, st, mp));
    return DASH_OK;
}

// Causal grouped-query attention over a packed (varlen) batch of active tokens,
// on tcgen05 tensor cores with TMEM accumulators, operands staged by TMA.
//
// Work item: 128 consecutive query rows of one head of one sequence.  A small plan kernel lists the
// items that exist (from cu_seqlens, on the device), heaviest first; persistent CTAs (two per SM) take
// them by ticket, so that no CTA is spent on query tiles that a shorter sequence does not have.
// Thread roles: warps 0-3 own one query row each (TMEM lane = row) and do the
// online softmax; warp 4 allocates TMEM and its lane 0 issues every TMA load and
// every tcgen05.mma.  Two CTAs share an SM (256 TMEM columns and < 113 KB of
// shared memory each), so one CTA's softmax overlaps the other's MMAs.
//
// Per key block j (128 keys), with S and P aliasing the same TMEM columns:
//   S = Q K_j^T  (SS MMA, fp32 in TMEM)  ->  softmax warps: mask, running max,
//   exp2, row sum, P (bf16) back into TMEM, rescale O if the max moved  ->
//   O += P V_j  (TS MMA: A operand read from TMEM)
// Causal tile skipping: a query tile only visits key blocks 0..its own index.
//
// The kernel is launched to start while the kernel in front of it in the stream drains (barriers, TMEM and descriptor prefetch are
// set up before griddepcontrol.wait).  A second instantiation (GATHER) takes the query rows -- and, optionally, the key / value
// rows -- of the packed set by index from full-length tensors (TMA gather4 loads) instead of from packed copies.
#include <math.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace dash {

using namespace ptx;

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = (EncodeTiledFn)p;
    }
    return fn;
}

int make_map_rows_heads(CUtensorMap* map, const void* base, int64_t rows, int heads, int D, int64_t ld, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return DASH_ERR_CUDA;
    cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)heads, (cuuint64_t)rows};
    cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)ld * 2};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DASH_OK : DASH_ERR_CUDA;
}

// bf16 tensor [rows, cols] (cols = heads * D), box = 64 columns of one row: the map of the four-row gather loads
int make_map_rows_gather(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return DASH_ERR_CUDA;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {64, 1};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DASH_OK : DASH_ERR_CUDA;
}

constexpr int kBM = 128;                 // query rows per CTA
constexpr int kBN = 128;                 // keys per block
constexpr int kAttnThreads = 160;
constexpr long long kWaitCycles = 4000000000LL;   // ~2 s: a wait that long is reported, not retried
constexpr uint32_t kTmemCols = 256;

struct AttnParams {
    const int32_t* cu;
    int S, Hq, Hkv, n_qtiles;
    float scale_log2;       // softmax scale * log2(e)
    float scale;
    void* O;
    int64_t ldo;            // elements
    float* lse;             // [Hq, n] or null
    int64_t n;
    int* status;
    const int4* plan;           // (sequence, query tile, first row, end row of the sequence) of every item group, heaviest first; Hq items (heads) per entry
    const int* n_items;         // device: entries * Hq
    unsigned int* ticket;       // device: next item to hand out
    const int32_t* idx;         // GATHER: packed row i is row idx[i] of the full-length Q (and of K, V unless kv_packed)
    int kv_packed;              // GATHER: K and V are packed already ([n, Hkv, D], tiled loads); only Q is fetched by index
};

// ---- plan: which (sequence, query tile) pairs exist, ordered by falling number of key blocks ----
__global__ void __launch_bounds__(1024)
attention_plan_kernel(const int32_t* __restrict__ cu, int S, int Hq, int4* __restrict__ plan, int* __restrict__ n_items,
                      unsigned int* __restrict__ ticket, int64_t max_entries) {
    __shared__ int s_warp[33];
    __shared__ int s_max;
    const int tid = threadIdx.x;
    pdl_launch_dependents();
    if (tid == 0) s_max = 0;
    __syncthreads();
    int mx = 0;
    for (int s = tid; s < S; s += blockDim.x) mx = max(mx, (cu[s + 1] - cu[s] + kBM - 1) / kBM);
    atomicMax(&s_max, mx);
    __syncthreads();
    const int max_nq = s_max;
    int64_t offset = 0;
    for (int top = max_nq - 1; top >= 0; top -= (int)blockDim.x) {
        const int qt = top - tid;                           // thread 0 takes the heaviest level of this chunk
        int cnt = 0;
        if (qt >= 0)
            for (int s = 0; s < S; ++s) cnt += ((cu[s + 1] - cu[s] + kBM - 1) / kBM > qt);
        // exclusive scan over the block
        const int lane = tid & 31, w = tid >> 5;
        int inc = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { int t = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += t; }
        if (lane == 31) s_warp[w] = inc;
        __syncthreads();
        if (w == 0) {
            int x = s_warp[lane], xi = x;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { int t = __shfl_up_sync(0xffffffffu, xi, o); if (lane >= o) xi += t; }
            s_warp[lane] = xi - x;
            if (lane == 31) s_warp[32] = xi;
        }
        __syncthreads();
        int64_t k = offset + s_warp[w] + inc - cnt;
        const int chunk_total = s_warp[32];
        if (qt >= 0)
            for (int s = 0; s < S; ++s)
                if ((cu[s + 1] - cu[s] + kBM - 1) / kBM > qt) { if (k < max_entries) plan[k] = make_int4(s, qt, cu[s], cu[s + 1]); ++k; }
        offset += chunk_total;
        __syncthreads();
    }
    if (tid == 0) {
        if (offset > max_entries) offset = max_entries;     // cannot happen for cu_seqlens[S] <= n; keeps every read in bounds
        *n_items = (int)(offset * Hq);
        *ticket = 0u;
    }
}

template <int D>
struct AttnSmem {
    static constexpr int kTileBytes = kBM * D * 2;
    static constexpr int kQ = 0, kK = kTileBytes, kV = 2 * kTileBytes, kBars = 3 * kTileBytes;
    static constexpr int kTotal = kBars + 128;
};

// GATHER: Q, K and V are full-length [rows, heads * D] tensors and the packed active set is given by p.idx; tiles are fetched four
// rows per instruction (TMA gather4, issued by all lanes of warp 4: lane l brings rows 4l .. 4l+3 of the tile), so the active rows
// of Q, K, V are never copied into packed buffers.  Everything else -- and the packed O -- is the same.
template <int D, bool OUT_F32, bool GATHER>
__global__ void __launch_bounds__(kAttnThreads, 2)
attention_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                 const __grid_constant__ CUtensorMap mapV, const AttnParams p) {
    extern __shared__ uint8_t smem_raw[];
    using L = AttnSmem<D>;
    constexpr int KCH = D / 64;              // 64-element (128-byte) chunks along D
    constexpr int kChunkBytes = kBM * 128;   // one chunk: 128 rows x 128 B
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base + L::kQ, sK = smem_base + L::kK, sV = smem_base + L::kV;
    const uint32_t bars = smem_base + L::kBars;
    const uint32_t bar_q = bars, bar_k = bars + 8, bar_v = bars + 16, bar_s = bars + 24, bar_o = bars + 32, bar_p0 = bars + 40, bar_p1 = bars + 48, bar_o0 = bars + 56;
    const uint32_t tmem_slot = bars + 64;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_gen + L::kBars + 64);
    volatile uint32_t* abort_gen = reinterpret_cast<volatile uint32_t*>(smem_gen + L::kBars + 68);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    pdl_launch_dependents();                               // the kernel behind may set itself up while this one drains
    volatile int* item_gen = reinterpret_cast<volatile int*>(smem_gen + L::kBars + 72);

    if (warp == 4) {
        if (lane == 0) {
            mbar_init(bar_q, 1); mbar_init(bar_k, 1); mbar_init(bar_v, 1);
            mbar_init(bar_s, 1); mbar_init(bar_o, 1); mbar_init(bar_o0, 1); mbar_init(bar_p0, 128); mbar_init(bar_p1, 128);
            *abort_gen = 0;
            fence_barrier_init();
            fence_proxy_async_smem();
            prefetch_tensormap(&mapQ); prefetch_tensormap(&mapK); prefetch_tensormap(&mapV);
        }
        __syncwarp();
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_wait();                                            // set-up done; from here on the kernel in front (plan, projection) has completed
    const uint32_t tmem = *tmem_slot_gen;
    const uint32_t tS = tmem, tP = tmem, tO = tmem + 128;

    constexpr uint32_t idesc_s = idesc_bf16_f32(kBM, kBN, false, false);
    constexpr uint32_t idesc_o = idesc_bf16_f32(kBM, D, false, true);
    const int n_items = *p.n_items;
    const int G = p.Hq / p.Hkv;
    // Barrier phases run on across the items of this CTA: blk0 = key blocks of its earlier items, items_done = their number.
    uint32_t blk0 = 0, items_done = 0;

    for (;;) {
    if (tid == 0) *item_gen = (int)atomicAdd(p.ticket, 1u);
    __syncthreads();
    const int item = *item_gen;
    if (item >= n_items || *abort_gen) break;
    tc_fence_after();
    // the heads of one KV group run next to each other, so their K/V tiles are shared through L2
    const int4 e = p.plan[item / p.Hq];                      // one load: the sequence's bounds ride along with the entry
    const int h = item % p.Hq, qt = e.y;
    const int kvh = h / G;
    const int seq_a = e.z, seq_b = e.w;
    const int len = seq_b - seq_a;
    const int q0 = qt * kBM;
    const int nblk = qt + 1;                                 // causal: key blocks 0..qt
    const uint32_t qph = items_done & 1;

    // tile of 128 packed rows starting at row0, fetched by index: lane l of warp 4 brings rows 4l .. 4l+3
    auto gather_tile = [&](uint32_t sT, const CUtensorMap* map, uint32_t bar, int head, int row0) {
        if (GATHER) {
            if (lane == 0) mbar_arrive_expect_tx(bar, L::kTileBytes);
            __syncwarp();
            int r[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int pr = row0 + 4 * lane + k;                  // rows past the sequence's end: its last row again (masked / zeroed later)
                r[k] = p.idx[pr < seq_b ? pr : seq_b - 1];
            }
#pragma unroll
            for (int c = 0; c < KCH; ++c) tma_gather4(sT + c * kChunkBytes + lane * 512, map, bar, head * D + c * 64, r[0], r[1], r[2], r[3]);
        }
    };
    if (warp == 4 && GATHER && !p.kv_packed) {
        // K and V by index as well: the schedule of the branch below with the whole warp in step -- lane 0 issues the MMAs, every
        // lane its share of the loads (the waits of 32 lanes and their votes cost about 500 cycles per key block)
        bool ok = true;
        auto all_ok = [&](bool v) { return __all_sync(0xffffffffu, v) != 0; };
        auto issue_s = [&]() {
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t off = (kk >> 2) * kChunkBytes + (kk & 3) * 32;
                mma_ss(tS, smem_desc_sw128(sQ + off, 16, 1024), smem_desc_sw128(sK + off, 16, 1024), idesc_s, kk > 0);
            }
            tc_commit(bar_s);
        };
        auto load_kv = [&](uint32_t sT, const CUtensorMap* map, uint32_t bar, int row0) { gather_tile(sT, map, bar, kvh, row0); };
        gather_tile(sQ, &mapQ, bar_q, h, seq_a + q0);
        load_kv(sK, &mapK, bar_k, seq_a);
        load_kv(sV, &mapV, bar_v, seq_a);
        ok = all_ok(mbar_wait(bar_q, qph, kWaitCycles) && mbar_wait(bar_k, blk0 & 1, kWaitCycles));
        if (ok && lane == 0) issue_s();
        __syncwarp();
        for (int j = 0; j < nblk && ok; ++j) {
            const uint32_t ph = (blk0 + j) & 1;
            ok = all_ok(mbar_wait(bar_s, ph, kWaitCycles));                   // S_j done: the K buffer is free
            if (!ok) break;
            if (j + 1 < nblk) load_kv(sK, &mapK, bar_k, seq_a + (j + 1) * kBN);
            ok = all_ok(mbar_wait(bar_v, ph, kWaitCycles) && mbar_wait(bar_p0, ph, kWaitCycles));
            if (!ok) break;
            if (lane == 0) {
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < kBN / 32; ++kk)
                    mma_ts(tO, tP + kk * 8, smem_desc_sw128(sV + kk * 2048, kChunkBytes, 1024), idesc_o, (j > 0) || (kk > 0));
                tc_commit(bar_o0);
            }
            if (j + 1 < nblk) ok = all_ok(mbar_wait(bar_k, (blk0 + j + 1) & 1, kWaitCycles));     // (ahead of the wait for P, as below)
            ok = ok && all_ok(mbar_wait(bar_p1, ph, kWaitCycles));
            if (!ok) break;
            if (lane == 0) {
                tc_fence_after();
#pragma unroll
                for (int kk = kBN / 32; kk < kBN / 16; ++kk)
                    mma_ts(tO, tP + kk * 8, smem_desc_sw128(sV + kk * 2048, kChunkBytes, 1024), idesc_o, 1);
                if (j + 1 < nblk) issue_s();
                tc_commit(bar_o);
            }
            ok = all_ok(mbar_wait(bar_o, ph, kWaitCycles));                   // PV_j done: the V buffer is free
            if (!ok) break;
            if (j + 1 < nblk) load_kv(sV, &mapV, bar_v, seq_a + (j + 1) * kBN);
        }
        if (!ok && lane == 0) { *abort_gen = 1; atomicExch(p.status, DASH_ERR_TIMEOUT); }
    } else if (warp == 4) {
        // Q by index (K and V packed): the whole warp fetches the query tile, then lane 0 runs the item as for packed tensors
        if (GATHER) gather_tile(sQ, &mapQ, bar_q, h, seq_a + q0);
        if (lane == 0) {
            bool ok = true;
            if (!GATHER) {
                mbar_arrive_expect_tx(bar_q, L::kTileBytes);
                for (int c = 0; c < KCH; ++c) tma_load_3d(sQ + c * kChunkBytes, &mapQ, bar_q, c * 64, h, seq_a + q0);
            }
            mbar_arrive_expect_tx(bar_k, L::kTileBytes);
            for (int c = 0; c < KCH; ++c) tma_load_3d(sK + c * kChunkBytes, &mapK, bar_k, c * 64, kvh, seq_a);
            mbar_arrive_expect_tx(bar_v, L::kTileBytes);
            for (int c = 0; c < KCH; ++c) tma_load_3d(sV + c * kChunkBytes, &mapV, bar_v, c * 64, kvh, seq_a);
            auto issue_s = [&]() {
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * kChunkBytes + (kk & 3) * 32;
                    mma_ss(tS, smem_desc_sw128(sQ + off, 16, 1024), smem_desc_sw128(sK + off, 16, 1024), idesc_s, kk > 0);
                }
                tc_commit(bar_s);
            };
            ok = mbar_wait(bar_q, qph, kWaitCycles) && mbar_wait(bar_k, blk0 & 1, kWaitCycles);
            if (ok) { tc_fence_after(); issue_s(); }
            for (int j = 0; j < nblk && ok; ++j) {
                const uint32_t ph = (blk0 + j) & 1;
                // S_j done: the K buffer is free for the next block
                ok = mbar_wait(bar_s, ph, kWaitCycles);
                if (!ok) break;
                if (j + 1 < nblk) {
                    mbar_arrive_expect_tx(bar_k, L::kTileBytes);
                    for (int c = 0; c < KCH; ++c) tma_load_3d(sK + c * kChunkBytes, &mapK, bar_k, c * 64, kvh, seq_a + (j + 1) * kBN);
                }
                // O += P_j V_j, started as soon as the first 64 keys of P are in TMEM.  (The waits for the tiles come before the
                // waits for P: a wait holds this thread for some 70 cycles even when its barrier is complete, and behind a
                // hand-over of P those cycles are on the chain to the next S.)
                ok = mbar_wait(bar_v, ph, kWaitCycles) && mbar_wait(bar_p0, ph, kWaitCycles);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < kBN / 32; ++kk)
                    mma_ts(tO, tP + kk * 8, smem_desc_sw128(sV + kk * 2048, kChunkBytes, 1024), idesc_o, (j > 0) || (kk > 0));
                tc_commit(bar_o0);                            // for a softmax thread that has to rescale O in the middle of the block
                if (j + 1 < nblk) ok = mbar_wait(bar_k, (blk0 + j + 1) & 1, kWaitCycles);      // K_{j+1}, asked for at the top of this block
                ok = ok && mbar_poll(bar_p1, ph, kWaitCycles);                                 // polled: what follows is the chain to S_{j+1}
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int kk = kBN / 32; kk < kBN / 16; ++kk)
                    mma_ts(tO, tP + kk * 8, smem_desc_sw128(sV + kk * 2048, kChunkBytes, 1024), idesc_o, 1);
                // S_{j+1} goes into the pipe right behind PV_j: tcgen05.mma of one thread execute in issue
                // order, so PV_j has read P_j before S_{j+1} overwrites the columns they share.  The commit that reports PV_j
                // comes behind the S products (a commit holds this thread as long as a product does, and S_{j+1} is what the
                // softmax warps wait for): the V buffer is given free that much later, which costs less.
                if (j + 1 < nblk) issue_s();
                tc_commit(bar_o);
                // PV_j done: the V buffer is free
                ok = mbar_wait(bar_o, ph, kWaitCycles);
                if (!ok) break;
                if (j + 1 < nblk) {
                    mbar_arrive_expect_tx(bar_v, L::kTileBytes);
                    for (int c = 0; c < KCH; ++c) tma_load_3d(sV + c * kChunkBytes, &mapV, bar_v, c * 64, kvh, seq_a + (j + 1) * kBN);
                }
            }
            if (!ok) { *abort_gen = 1; atomicExch(p.status, DASH_ERR_TIMEOUT); }
        }
    } else {
        // ---- softmax warps: thread <-> query row ----
        const int row = tid;                               // 0..127
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        const bool row_valid = (q0 + row) < len;
        float m = -INFINITY, l = 0.f;
        bool ok = true;
        for (int j = 0; j < nblk; ++j) {
            const uint32_t ph = (blk0 + j) & 1;
            ok = mbar_wait(bar_s, ph, kWaitCycles);
            if (!ok || *abort_gen) { ok = false; break; }
            tc_fence_after();
            uint32_t sreg[128];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld32(tS + lane_base + c * 32, &sreg[c * 32]);
            tmem_wait_ld();
            const bool diag = (j == qt);
            auto mask_diag = [&](int c0, int c1) {
#pragma unroll
                for (int c = c0; c < c1; ++c)
                    if (c > row) sreg[c] = 0xff800000u;     // -inf: keys after the query (and past the sequence end)
            };
            if (diag) mask_diag(0, 128);
            // The reference m of the row (exponentials are taken of s - m) is the first block's row maximum and stays unless a later
            // block towers over it: a block's exponentials are formed against the m at hand without looking for the block's maximum,
            // and their sum tells whether that was safe.  Sums below 2^64 are (P up to 2^64 is exact in bf16's range and harmless in
            // the fp32 sums of P V and l); a larger or non-finite sum sends the warp through the rescaling path below.
            if (j == 0) {
                // four independent chains of three-input max keep the reduction short and off the latency-bound path
                float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                for (int c = 0; c < 128; c += 8) {
                    mx0 = fmax3(mx0, __uint_as_float(sreg[c]), __uint_as_float(sreg[c + 1]));
                    mx1 = fmax3(mx1, __uint_as_float(sreg[c + 2]), __uint_as_float(sreg[c + 3]));
                    mx2 = fmax3(mx2, __uint_as_float(sreg[c + 4]), __uint_as_float(sreg[c + 5]));
                    mx3 = fmax3(mx3, __uint_as_float(sreg[c + 6]), __uint_as_float(sreg[c + 7]));
                }
                m = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));          // finite: key 0 is visible to every query row
            }
            if (diag) {
                // keys past the end of the sequence: their V rows may hold anything (another
                // sequence, or never-written memory); zero them so 0 * garbage cannot make a NaN
                ok = mbar_wait(bar_v, ph, kWaitCycles);
                if (!ok) break;
                if (j * kBN + row >= len) {
#pragma unroll
                    for (int c = 0; c < KCH; ++c) {
                        uint4* rowp = reinterpret_cast<uint4*>(smem_gen + L::kV + c * kChunkBytes + row * 128);
#pragma unroll
                        for (int e = 0; e < 8; ++e) rowp[e] = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async_smem();
                }
            }
            const float2 sl2 = make_float2(p.scale_log2, p.scale_log2);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                // scale-subtract and row sums on packed fp32 pairs (two lanes per FMA-pipe instruction); P is packed in place
                auto exps = [&]() -> float {
                    float2 sumA = make_float2(0.f, 0.f), sumB = make_float2(0.f, 0.f);
                    const float msl = m * p.scale_log2;
                    const float2 nm2 = make_float2(-msl, -msl);
#pragma unroll
                    for (int c = half * 64; c < half * 64 + 64; c += 4) {
                        const float2 xa = __ffma2_rn(make_float2(__uint_as_float(sreg[c]), __uint_as_float(sreg[c + 1])), sl2, nm2);
                        const float2 xb = __ffma2_rn(make_float2(__uint_as_float(sreg[c + 2]), __uint_as_float(sreg[c + 3])), sl2, nm2);
                        float2 pa, pb;
                        pa.x = ex2(xa.x);
                        pa.y = ex2(xa.y);
                        pb.x = ex2(xb.x);
                        pb.y = ex2(xb.y);
                        sumA = __fadd2_rn(sumA, pa);
                        sumB = __fadd2_rn(sumB, pb);
                        sreg[c >> 1] = pack_bf16(pa.x, pa.y);
                        sreg[(c >> 1) + 1] = pack_bf16(pb.x, pb.y);
                    }
                    return (sumA.x + sumA.y) + (sumB.x + sumB.y);
                };
                float hs = exps();
                if (__any_sync(0xffffffffu, row_valid && !(hs < 1.8446744e19f))) {     // (rows past the sequence's end may hold anything and are never written)
                    // rare: some row of the warp met scores far above its reference.  The half's scores are still in TMEM (P has not
                    // been stored over them): fetch them again, move m where the half's maximum asks for it (the rows that need not
                    // move keep theirs), bring O and l to the new m -- O once every product issued so far has landed -- and redo.
                    tmem_ld32(tS + lane_base + half * 64, &sreg[half * 64]);
                    tmem_ld32(tS + lane_base + half * 64 + 32, &sreg[half * 64 + 32]);
                    tmem_wait_ld();
                    if (diag) mask_diag(half * 64, half * 64 + 64);
                    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
                    for (int c = half * 64; c < half * 64 + 64; c += 4) {
                        mx0 = fmax3(mx0, __uint_as_float(sreg[c]), __uint_as_float(sreg[c + 1]));
                        mx1 = fmax3(mx1, __uint_as_float(sreg[c + 2]), __uint_as_float(sreg[c + 3]));
                    }
                    const float mx = fmaxf(mx0, mx1);
                    const bool grow = (mx - m) * p.scale_log2 > 8.0f;
                    const float m_new = grow ? mx : m;
                    const float alpha = grow ? ex2((m - m_new) * p.scale_log2) : 1.0f;
                    if (half == 1) ok = mbar_wait(bar_o0, ph, kWaitCycles);                       // the first half's products of this block
                    else if (j > 0) ok = mbar_wait(bar_o, (blk0 + j - 1) & 1, kWaitCycles);       // the blocks before
                    if (!ok) break;
                    if (half == 1 || j > 0) {
                        tc_fence_after();
#pragma unroll 1
                        for (int c = 0; c < D / 8; ++c) {
                            uint32_t o[8];
                            tmem_ld8(tO + lane_base + c * 8, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < 8; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                            tmem_st8(tO + lane_base + c * 8, o);
                        }
                    }
                    l *= alpha;
                    m = m_new;
                    hs = exps();
                }
                // the first 64 keys of P go out (and their PV steps start) while the rest is still being formed
                tmem_st32(tP + lane_base + half * 32, &sreg[half * 32]);
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(half == 0 ? bar_p0 : bar_p1);
                l += hs;
            }
            if (!ok) break;
        }
        if (ok) ok = mbar_wait(bar_o, (blk0 + nblk - 1) & 1, kWaitCycles);
        if (ok && !*abort_gen) {
            tc_fence_after();
            const float inv = 1.0f / l;
            const int64_t grow = (int64_t)seq_a + q0 + row;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t o[32];
                tmem_ld32(tO + lane_base + c * 32, o);
                tmem_wait_ld();
                if (row_valid) {
                    if (OUT_F32) {
                        float* dst = reinterpret_cast<float*>(p.O) + grow * p.ldo + (int64_t)h * D + c * 32;
#pragma unroll
                        for (int e = 0; e < 32; e += 4) {
                            uint4 v;
                            v.x = __float_as_uint(__uint_as_float(o[e]) * inv); v.y = __float_as_uint(__uint_as_float(o[e + 1]) * inv);
                            v.z = __float_as_uint(__uint_as_float(o[e + 2]) * inv); v.w = __float_as_uint(__uint_as_float(o[e + 3]) * inv);
                            st_v4(dst + e, v);
                        }
                    } else {
                        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.O) + grow * p.ldo + (int64_t)h * D + c * 32;
#pragma unroll
                        for (int e = 0; e < 32; e += 8) {
                            uint4 v;
                            v.x = pack_bf16(__uint_as_float(o[e]) * inv, __uint_as_float(o[e + 1]) * inv);
                            v.y = pack_bf16(__uint_as_float(o[e + 2]) * inv, __uint_as_float(o[e + 3]) * inv);
                            v.z = pack_bf16(__uint_as_float(o[e + 4]) * inv, __uint_as_float(o[e + 5]) * inv);
                            v.w = pack_bf16(__uint_as_float(o[e + 6]) * inv, __uint_as_float(o[e + 7]) * inv);
                            st_v4(dst + e, v);
                        }
                    }
                }
            }
            if (row_valid && p.lse) p.lse[(int64_t)h * p.n + grow] = m * p.scale + logf(l);
        } else if (!ok && lane == 0) {
            *abort_gen = 1;
            atomicExch(p.status, DASH_ERR_TIMEOUT);
        }
    }
    // end of the item: O has been read out, every tile buffer is free
    tc_fence_before();
    __syncthreads();
    blk0 += (uint32_t)nblk;
    ++items_done;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

__global__ void f32_to_bf16_rows_kernel(const float* __restrict__ src, int64_t ld_src, __nv_bfloat16* __restrict__ dst, int64_t ld_dst,
                                        int64_t rows, int cols) {
    const int64_t total = rows * (cols / 4);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        int64_t r = i / (cols / 4);
        int c = (int)(i % (cols / 4)) * 4;
        float4 v = *reinterpret_cast<const float4*>(src + r * ld_src + c);
        uint2 o = make_uint2(pack_bf16(v.x, v.y), pack_bf16(v.z, v.w));
        *reinterpret_cast<uint2*>(dst + r * ld_dst + c) = o;
    }
}

int launch_f32_to_bf16(const float* src, int64_t ld_src, void* dst, int64_t ld_dst, int64_t rows, int64_t cols, cudaStream_t st) {
    if (rows <= 0 || cols <= 0) return DASH_OK;
    int64_t grid = (rows * (cols / 4) + 255) / 256, cap = (int64_t)sm_count() * 8;
    if (grid > cap) grid = cap;
    f32_to_bf16_rows_kernel<<<(int)grid, 256, 0, st>>>(src, ld_src, (__nv_bfloat16*)dst, ld_dst, rows, (int)cols);
    return cudaGetLastError() == cudaSuccess ? DASH_OK : DASH_ERR_CUDA;
}

// workspace: [0,256) ticket + item count; then the plan (one int4 per existing (sequence, query tile));
// then, for fp32 tensors, their bf16 copies
static size_t plan_entries(int64_t n, int S) { return (size_t)(n / kBM) + (size_t)S + 1; }
static size_t plan_bytes(int64_t n, int S) { return align_up(plan_entries(n, S) * sizeof(int4), 256); }
size_t attention_ws_bytes(int64_t n, int S, int Hq, int Hkv, int D, dash_dtype dt) {
    size_t b = 256 + plan_bytes(n, S);
    if (dt != DASH_BF16) b += align_up((size_t)n * (Hq + 2 * Hkv) * D * 2, 256);
    return b;
}

template <int D, bool OUT_F32, bool GATHER>
static int launch_attention(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const AttnParams& p, int grid, cudaStream_t st) {
    using L = AttnSmem<D>;
    const int smem = L::kTotal + 1024;
    static std::atomic<uint64_t> configured{0};
    if (!set_max_smem_once(attention_kernel<D, OUT_F32, GATHER>, smem, configured)) return DASH_ERR_CUDA;
    return launch_pdl(attention_kernel<D, OUT_F32, GATHER>, grid, kAttnThreads, (size_t)smem, st, mq, mk, mv, p) == cudaSuccess ? DASH_OK : DASH_ERR_CUDA;
}

// The item list of a call (see attention_plan_kernel) into the head of its workspace.  A caller that knows cu_seqlens early
// launches it ahead of the work that produces Q, K, V and then calls attention_planned().
int attention_plan(const int32_t* cu_seqlens, int S, int64_t n, int Hq, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (!cu_seqlens || S < 1 || n < 0 || n > 0x7fffffffLL || Hq < 1) return DASH_ERR_INVALID_ARG;
    if (n == 0) return DASH_OK;
    if (!ws || ((uintptr_t)ws % 256) || ws_bytes < 256 + plan_bytes(n, S)) return DASH_ERR_WORKSPACE;
    if ((int64_t)plan_entries(n, S) * Hq > 0x7fffffffLL) return DASH_ERR_UNSUPPORTED;
    attention_plan_kernel<<<1, 1024, 0, st>>>(cu_seqlens, S, Hq, (int4*)((char*)ws + 256), (int*)((char*)ws + 4), (unsigned int*)ws,
                                              (int64_t)plan_entries(n, S));
    return cudaGetLastError() == cudaSuccess ? DASH_OK : DASH_ERR_CUDA;
}

static int attention_impl(const void* Q, const void* K, const void* V, void* O, float* lse,
                          int64_t ldq, int64_t ldk, int64_t ldv, int64_t ldo,
                          const int32_t* cu_seqlens, int S, int64_t n, int64_t max_seqlen,
                          int Hq, int Hkv, int D, float scale, int causal, dash_dtype dt,
                          void* ws, size_t ws_bytes, void* stream, bool planned, const int32_t* idx = nullptr, int64_t n_full = 0,
                          bool kv_packed = false) {
    if (n < 0 || S < 1 || max_seqlen < 0 || Hq < 1 || Hkv < 1 || !cu_seqlens) return DASH_ERR_INVALID_ARG;
    if (dt != DASH_F32 && dt != DASH_BF16) return DASH_ERR_INVALID_ARG;
    if (D != 64 && D != 128) return DASH_ERR_UNSUPPORTED;
    if (Hq % Hkv) return DASH_ERR_INVALID_ARG;
    if (causal != 1) return DASH_ERR_UNSUPPORTED;
    if (n > 0x7fffffffLL || max_seqlen > n) return DASH_ERR_INVALID_ARG;
    if (n == 0 || max_seqlen == 0) return DASH_OK;
    if (!Q || !K || !V || !O) return DASH_ERR_INVALID_ARG;
    const int es = (dt == DASH_BF16) ? 2 : 4;
    if (ldq < (int64_t)Hq * D || ldo < (int64_t)Hq * D || ldk < (int64_t)Hkv * D || ldv < (int64_t)Hkv * D) return DASH_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return DASH_ERR_INVALID_ARG;
    if ((ldq * es) % 16 || (ldk * es) % 16 || (ldv * es) % 16 || (ldo * es) % 16) return DASH_ERR_INVALID_ARG;
    if (!(scale > 0.f)) return DASH_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;

    const void *q = Q, *k = K, *v = V;
    int64_t lq = ldq, lk = ldk, lv = ldv;
    if (!ws || ((uintptr_t)ws % 256) || ws_bytes < attention_ws_bytes(n, S, Hq, Hkv, D, dt)) return DASH_ERR_WORKSPACE;
    if (idx && (dt != DASH_BF16 || n_full < 1 || n_full > 0x7fffffffLL)) return dt != DASH_BF16 ? DASH_ERR_UNSUPPORTED : DASH_ERR_INVALID_ARG;
    if (dt == DASH_F32) {
        __nv_bfloat16* qb = (__nv_bfloat16*)((char*)ws + 256 + plan_bytes(n, S));
        __nv_bfloat16* kb = qb + (size_t)n * Hq * D;
        __nv_bfloat16* vb = kb + (size_t)n * Hkv * D;
        const int cap = sm_count() * 8;
        auto cvt = [&](const void* src, int64_t ld, __nv_bfloat16* dst, int cols) {
            int64_t total = n * (cols / 4);
            int grid = (int)((total + 255) / 256);
            if (grid > cap) grid = cap;
            f32_to_bf16_rows_kernel<<<grid, 256, 0, st>>>((const float*)src, ld, dst, cols, n, cols);
        };
        cvt(Q, ldq, qb, Hq * D); cvt(K, ldk, kb, Hkv * D); cvt(V, ldv, vb, Hkv * D);
        DASH_CUDA_TRY(cudaGetLastError());
        q = qb; k = kb; v = vb;
        lq = (int64_t)Hq * D; lk = lv = (int64_t)Hkv * D;
    }
    CUtensorMap mq, mk, mv;
    int rc;
    if (idx) {
        if ((rc = make_map_rows_gather(&mq, q, n_full, (int64_t)Hq * D, lq)) != DASH_OK) return rc;
        if (kv_packed) {
            if ((rc = make_map_rows_heads(&mk, k, n, Hkv, D, lk, kBN)) != DASH_OK) return rc;
            if ((rc = make_map_rows_heads(&mv, v, n, Hkv, D, lv, kBN)) != DASH_OK) return rc;
        } else {
            if ((rc = make_map_rows_gather(&mk, k, n_full, (int64_t)Hkv * D, lk)) != DASH_OK) return rc;
            if ((rc = make_map_rows_gather(&mv, v, n_full, (int64_t)Hkv * D, lv)) != DASH_OK) return rc;
        }
    } else {
        if ((rc = make_map_rows_heads(&mq, q, n, Hq, D, lq, kBM)) != DASH_OK) return rc;
        if ((rc = make_map_rows_heads(&mk, k, n, Hkv, D, lk, kBN)) != DASH_OK) return rc;
        if ((rc = make_map_rows_heads(&mv, v, n, Hkv, D, lv, kBN)) != DASH_OK) return rc;
    }

    AttnParams p;
    p.cu = cu_seqlens; p.S = S; p.Hq = Hq; p.Hkv = Hkv;
    p.n_qtiles = (int)((max_seqlen + kBM - 1) / kBM);
    p.scale = scale;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.O = O; p.ldo = ldo; p.lse = lse; p.n = n; p.idx = idx; p.kv_packed = kv_packed ? 1 : 0;
    p.status = status_word_ptr();
    if (!p.status) return DASH_ERR_CUDA;
    p.ticket = (unsigned int*)ws;
    p.n_items = (const int*)((char*)ws + 4);
    p.plan = (const int4*)((char*)ws + 256);
    if (!planned && (rc = attention_plan(cu_seqlens, S, n, Hq, ws, ws_bytes, st)) != DASH_OK) return rc;
    // persistent CTAs, two per SM, never more than there can be items
    int64_t grid64 = (int64_t)p.n_qtiles * Hq * S;
    if (grid64 > 2LL * sm_count()) grid64 = 2LL * sm_count();
    const int grid = (int)grid64;
    if (idx) return D == 128 ? launch_attention<128, false, true>(mq, mk, mv, p, grid, st) : launch_attention<64, false, true>(mq, mk, mv, p, grid, st);
    if (D == 128) return dt == DASH_F32 ? launch_attention<128, true, false>(mq, mk, mv, p, grid, st) : launch_attention<128, false, false>(mq, mk, mv, p, grid, st);
    return dt == DASH_F32 ? launch_attention<64, true, false>(mq, mk, mv, p, grid, st) : launch_attention<64, false, false>(mq, mk, mv, p, grid, st);
}

// same as dash_varlen_attention for a workspace whose item list attention_plan() has already been asked for on this stream
int attention_planned(const void* Q, const void* K, const void* V, void* O, float* lse, int64_t ldq, int64_t ldk, int64_t ldv, int64_t ldo,
                      const int32_t* cu_seqlens, int S, int64_t n, int64_t max_seqlen, int Hq, int Hkv, int D, float scale, dash_dtype dt,
                      void* ws, size_t ws_bytes, cudaStream_t st) {
    return attention_impl(Q, K, V, O, lse, ldq, ldk, ldv, ldo, cu_seqlens, S, n, max_seqlen, Hq, Hkv, D, scale, 1, dt, ws, ws_bytes, (void*)st, true);
}

}  // namespace dash

extern "C" int dash_varlen_attention(const void* Q, const void* K, const void* V, void* O, float* lse,
                                     int64_t ldq, int64_t ldk, int64_t ldv, int64_t ldo,
                                     const int32_t* cu_seqlens, int S, int64_t n, int64_t max_seqlen,
                                     int Hq, int Hkv, int D, float scale, int causal, dash_dtype dt,
                                     void* ws, size_t ws_bytes, void* stream) {
    return dash::attention_impl(Q, K, V, O, lse, ldq, ldk, ldv, ldo, cu_seqlens, S, n, max_seqlen, Hq, Hkv, D, scale, causal, dt, ws, ws_bytes,
                                stream, false);
}

extern "C" int dash_varlen_attention_indexed(const void* Q, const void* K, const void* V, void* O, float* lse,
                                             int64_t ldq, int64_t ldk, int64_t ldv, int64_t ldo,
                                             const int32_t* idx, int64_t n_full, int kv_packed,
                                             const int32_t* cu_seqlens, int S, int64_t n, int64_t max_seqlen,
                                             int Hq, int Hkv, int D, float scale, int causal, dash_dtype dt,
                                             void* ws, size_t ws_bytes, void* stream) {
    if ((!idx && n > 0) || (kv_packed != 0 && kv_packed != 1)) return DASH_ERR_INVALID_ARG;
    if (n > n_full) return DASH_ERR_INVALID_ARG;
    return dash::attention_impl(Q, K, V, O, lse, ldq, ldk, ldv, ldo, cu_seqlens, S, n, max_seqlen, Hq, Hkv, D, scale, causal, dt, ws, ws_bytes,
                                stream, false, idx, n_full, kv_packed != 0);
}

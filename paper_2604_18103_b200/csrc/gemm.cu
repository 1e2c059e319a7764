// Projections of the block as persistent tcgen05 GEMMs: C[n, N] = A[n, K] W[K, N], bf16 operands, fp32 accumulation in
// TMEM, with the element-wise work that follows each projection done on the accumulators before anything is written:
//   PLAIN  : C = A W (bf16 or fp32 out; any N, K that keep rows 16-byte aligned: tiles past the edge of W or along K are
//            zero-filled by the loads, columns past N are not stored)   (down projection of the FFN; every projection of the
//            path that runs the norm, the rotary embedding and the residual as passes of their own; fp32 tensors, whose
//            operands are rounded to bf16 copies first)
//   ROPE   : Q | K | V = Hn Wqkv with the rotary embedding applied to the Q and K heads    (Eq. 1, inside Attn)
//   RESID  : U = O Wo is never stored: H~ = H + U goes straight to x_full[tok[row]], and the per-row partial sums of
//            u^2, h^2 and (h+u)^2 of this tile's columns go to a small buffer (the score of Eq. 2 and the next norm's row factor are
//            finished from them)
//   SWIGLU : one tile holds 128 gate and the matching 128 up columns: act = silu(g) * u      (FFN of Alg. 1)
// One CTA per SM, in clusters of two: a pair computes a 256 x 256 tile with tcgen05.mma.cta_group::2 -- CTA r holds rows
// 128 r .. of the A tile and columns 128 r .. of the W tile, so every SM loads only half of the W operand.  K in steps of 64
// through a 6-stage TMA ring; warp 0 of each CTA issues its loads (their bytes are counted on the pair's even CTA), warp 1 of
// the even CTA issues the MMAs and releases stages / hands over accumulators in both CTAs with multicast commits, warps 2-5
// of each CTA read their 128 accumulator rows (two TMEM buffers, so a tile's epilogue overlaps the next tile's MMAs).
#include <math.h>

#include "common.cuh"
#include "gemm.cuh"
#include "sm100_ptx.cuh"

namespace dash {

using namespace ptx;

constexpr int kGM = 128, kGN = 256, kGK = 64, kGStages = 6;      // kGM: rows per CTA (256 per pair)
constexpr int kGABytes = kGM * kGK * 2, kGBBytes = kGK * (kGN / 2) * 2, kGStageBytes = kGABytes + kGBBytes;   // per CTA
constexpr int kGThreads = 192;
constexpr int kGGroupN = 16;                 // n tiles per group of the tile order
constexpr long long kGWait = 4000000000LL;

constexpr uint32_t kPeerMask = 0xFEFFFFFFu;   // clears the CTA-rank bit of a shared::cluster address: the pair's even CTA

__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// tiled load into this CTA's shared memory whose bytes are counted on the barrier of the pair's even CTA
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst_smem, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar & kPeerMask), "r"(c0), "r"(c1) : "memory");
}
// arrives, once every tcgen05 operation issued so far has completed, on the barrier at this offset in both CTAs of the pair
__device__ __forceinline__ void commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void arrive_on_leader(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar & kPeerMask) : "memory");
}
// The low word of a shared-memory descriptor holds the start address (>> 4) and the leading offset, the high word
// everything that does not change inside a tile: stepping through a tile is a 32-bit add.
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t saddr, uint32_t lbo_bytes) {
    return ((saddr & 0x3FFFFu) >> 4) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
__device__ __forceinline__ constexpr uint32_t smem_desc_hi_sw128(uint32_t sbo_bytes) {
    return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
}
__device__ __forceinline__ void mma_ss_lh(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %6, 0;\n\tmov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %5, {%7, %7, %7, %7, %7, %7, %7, %7}, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}

// tile t -> (m tile of 256 rows, n tile): the n tiles come in groups of kGGroupN; within a group the m tiles run one after the other and
// each visits the group's n tiles, so that the CTAs of a wave share a few A row-blocks and a few W column-blocks in L2
__device__ __forceinline__ void tile_coords(int t, int m_tiles, int n_tiles, int& mt, int& nt) {
    const int per_group = m_tiles * kGGroupN;
    const int g = t / per_group, r = t - g * per_group;
    const int gw = min(kGGroupN, n_tiles - g * kGGroupN);        // the last group may be narrower
    mt = r / gw;
    nt = g * kGGroupN + r % gw;
}

struct GemmArgs {
    int n, N, K;                 // rows (upper bound), columns of W that one tile row of the output spans, depth
    int n_tiles;                 // tiles along the output columns
    void* C; int64_t ldc;        // PLAIN / ROPE / SWIGLU output (elements)
    int out_f32;                 // PLAIN: C is fp32 (else bf16)
    const int32_t* n_dev;        // device: true number of rows (<= n), or null
    int* status;
    GemmEpilogue e;
};

template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapW, const GemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bars = base + kGStages * kGStageBytes;
    auto full = [&](int s) { return bars + 8 * s; };
    auto empty = [&](int s) { return bars + 8 * (kGStages + s); };
    auto acc_full = [&](int b) { return bars + 8 * (2 * kGStages + b); };
    auto acc_empty = [&](int b) { return bars + 8 * (2 * kGStages + 2 + b); };
    const uint32_t slot = bars + 8 * (2 * kGStages + 4);
    volatile uint32_t* slot_gen = reinterpret_cast<volatile uint32_t*>(smem_raw + (slot - smem_u32(smem_raw)));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // the kernel behind (attention, tail pass) may set itself up while this one drains; this kernel itself is launched in plain
    // stream order: started early behind the attention or row kernels it measured 15 us slower per launch
    pdl_launch_dependents();
    const int rank = (int)cluster_rank();                  // 0: the pair's even CTA (issues the MMAs, owns the full / acc_empty barriers)
    if (warp == 1) {
        if (lane == 0) {
            for (int s = 0; s < kGStages; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
            for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 256); }
            fence_barrier_init();
            fence_proxy_async_smem();
        }
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else if (warp == 0 && lane == 0) {
        prefetch_tensormap(&mapA); prefetch_tensormap(&mapW);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                    // the peer's barriers exist before anything is signalled across
    tc_fence_after();
    const uint32_t tmem = *slot_gen;
    const int m_tiles = (g.n + 2 * kGM - 1) / (2 * kGM), n_tiles = g.n_tiles, tiles = m_tiles * n_tiles, ksteps = (g.K + kGK - 1) / kGK;
    const int n_pairs = (int)gridDim.x / 2, pair = (int)blockIdx.x / 2;
    constexpr uint32_t idesc = idesc_bf16_f32(2 * kGM, kGN, false, true);
    constexpr uint32_t hi = smem_desc_hi_sw128(1024);

    if (warp == 0) {
        // ---- loads of this CTA: its 128 x 64 half of the A tile (K-major), its 64 x 128 half of the W tile as two 64-column chunks ----
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int t = pair; t < tiles && ok; t += n_pairs) {
                int mt, nt;
                tile_coords(t, m_tiles, n_tiles, mt, nt);
                const int m0 = mt * 2 * kGM + rank * kGM;
                for (int k = 0; k < ksteps && ok; ++k, ++it) {
                    const int s = it % kGStages;
                    if (it >= kGStages) ok = mbar_wait(empty(s), ((it / kGStages) - 1) & 1, kGWait);
                    if (!ok) break;
                    const uint32_t sA = base + s * kGStageBytes, sB = sA + kGABytes;
                    if (rank == 0) mbar_arrive_expect_tx(full(s), 2 * kGStageBytes);     // both CTAs' bytes land on this barrier
                    tma_load_2d_pair(sA, &mapA, full(s), k * kGK, m0);
#pragma unroll
                    for (int c = 0; c < kGN / 2 / 64; ++c) {
                        // SWIGLU: columns 0-127 of the tile (the even CTA's half) are gate features nt * 128 .., columns 128-255 the same features of "up"
                        const int col = (EPI == GEMM_SWIGLU) ? (rank * g.e.m + nt * 128 + c * 64) : (nt * kGN + rank * (kGN / 2) + c * 64);
                        tma_load_2d_pair(sB + c * (kGK * 128), &mapW, full(s), col, k * kGK);
                    }
                }
            }
            if (!ok) atomicExch(g.status, DASH_ERR_TIMEOUT);
        }
    } else if (warp == 1) {
        // ---- MMAs (even CTA only): four 256 x 256 x 16 steps per stage into the tile's TMEM buffer of both CTAs ----
        if (lane == 0 && rank == 0) {
            uint32_t it = 0, tl = 0;
            bool ok = true;
            for (int t = pair; t < tiles && ok; t += n_pairs, ++tl) {
                const int b = tl & 1;
                if (tl >= 2) ok = mbar_wait(acc_empty(b), ((tl >> 1) - 1) & 1, kGWait);
                if (!ok) break;
                tc_fence_after();
                const uint32_t tD = tmem + b * kGN;
                for (int k = 0; k < ksteps && ok; ++k, ++it) {
                    const int s = it % kGStages;
                    ok = mbar_wait(full(s), (it / kGStages) & 1, kGWait);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sA = base + s * kGStageBytes, sB = sA + kGABytes;
                    const uint32_t a_lo = smem_desc_lo(sA, 16), b_lo = smem_desc_lo(sB, kGK * 128);
#pragma unroll
                    for (int kk = 0; kk < kGK / 16; ++kk)
                        mma_ss_lh(tD, a_lo + ((kk * 32) >> 4), hi, b_lo + ((kk * 2048) >> 4), hi, idesc, (k > 0) || (kk > 0));
                    commit_pair(empty(s));
                }
                commit_pair(acc_full(b));
            }
            if (!ok) atomicExch(g.status, DASH_ERR_TIMEOUT);
        }
    } else {
        // ---- epilogue: thread <-> row of the tile (TMEM lane), 256 fp32 accumulators read 32 at a time ----
        const int q = warp & 3;                                   // TMEM lane quarter this warp may read
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        int n_true = g.n;
        if (g.n_dev) { const int nd = *g.n_dev; if (nd < n_true) n_true = nd; }
        uint32_t tl = 0;
        bool ok = true;
        for (int t = pair; t < tiles; t += n_pairs, ++tl) {
            const int b = tl & 1;
            int mt, nt;
            tile_coords(t, m_tiles, n_tiles, mt, nt);
            ok = mbar_wait(acc_full(b), (tl >> 1) & 1, kGWait);
            if (!ok) break;
            tc_fence_after();
            const int row = mt * 2 * kGM + rank * kGM + q * 32 + lane;
            const bool live = row < n_true;
            const uint32_t tD = tmem + b * kGN + lane_base;
            if (EPI == GEMM_PLAIN) {
                // columns at or past N (a last, partial tile) are not stored; N is a multiple of 8 (bf16) / 4 (fp32)
                const int col0 = nt * kGN;
#pragma unroll
                for (int c = 0; c < kGN / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tD + c * 32, o);
                    tmem_wait_ld();
                    if (live && g.out_f32) {
                        float* dst = reinterpret_cast<float*>(g.C) + (int64_t)row * g.ldc + col0 + c * 32;
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            if (col0 + c * 32 + e < g.N) st_v4(dst + e, make_uint4(o[e], o[e + 1], o[e + 2], o[e + 3]));
                    } else if (live) {
                        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(g.C) + (int64_t)row * g.ldc + col0 + c * 32;
#pragma unroll
                        for (int e = 0; e < 32; e += 8)
                            if (col0 + c * 32 + e < g.N)
                                st_v4(dst + e, make_uint4(pack_bf16(__uint_as_float(o[e]), __uint_as_float(o[e + 1])),
                                                          pack_bf16(__uint_as_float(o[e + 2]), __uint_as_float(o[e + 3])),
                                                          pack_bf16(__uint_as_float(o[e + 4]), __uint_as_float(o[e + 5])),
                                                          pack_bf16(__uint_as_float(o[e + 6]), __uint_as_float(o[e + 7]))));
                    }
                }
            } else if (EPI == GEMM_ROPE) {
                // heads of D columns; inside a head of Q or K the pair (i, i + D/2) is rotated by the angle of (row, i)
                __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(g.C) + (int64_t)row * g.ldc + nt * kGN;
                const int D = g.e.D, half = D >> 1;
                int64_t trow = row;                                            // (cos, sin) of this row: its own entry, or its position's
                if (g.e.rope_pos) { trow = live ? g.e.rope_pos[row] : 0; if (trow >= g.e.rope_len) trow = g.e.rope_len - 1; if (trow < 0) trow = 0; }
                const float2* cs = g.e.rope_table + trow * half;
                const float rsc = (g.e.row_scale && live) ? g.e.row_scale[row] : 1.0f;
                for (int h0 = 0; h0 < kGN; h0 += D) {
                    const bool rotate = (nt * kGN + h0) < g.e.n_rot_cols;
                    // D = 128: two 32-column chunks per half; D = 64: one
                    for (int c = 0; c < half; c += 32) {
                        uint32_t x1[32], x2[32];
                        tmem_ld32(tD + h0 + c, x1);
                        tmem_ld32(tD + h0 + half + c, x2);
                        tmem_wait_ld();
                        if (live) {
                            float y1[32], y2[32];
#pragma unroll
                            for (int e = 0; e < 32; ++e) {
                                const float a = __uint_as_float(x1[e]) * rsc, bb = __uint_as_float(x2[e]) * rsc;
                                if (rotate) {
                                    const float2 t2 = cs[c + e];
                                    y1[e] = a * t2.x - bb * t2.y;
                                    y2[e] = bb * t2.x + a * t2.y;
                                } else { y1[e] = a; y2[e] = bb; }
                            }
#pragma unroll
                            for (int e = 0; e < 32; e += 8) {
                                st_v4(dst + h0 + c + e, make_uint4(pack_bf16(y1[e], y1[e + 1]), pack_bf16(y1[e + 2], y1[e + 3]),
                                                                   pack_bf16(y1[e + 4], y1[e + 5]), pack_bf16(y1[e + 6], y1[e + 7])));
                                st_v4(dst + h0 + half + c + e, make_uint4(pack_bf16(y2[e], y2[e + 1]), pack_bf16(y2[e + 2], y2[e + 3]),
                                                                          pack_bf16(y2[e + 4], y2[e + 5]), pack_bf16(y2[e + 6], y2[e + 7])));
                            }
                        }
                    }
                }
            } else if (EPI == GEMM_RESID) {
                // H~ = H + U (U in fp32, one rounding) to x_full[tok[row]]; sums of u^2 and h^2 over this tile's 256 columns
                const __nv_bfloat16* hsrc = reinterpret_cast<const __nv_bfloat16*>(g.e.H) + (int64_t)row * g.e.ldh + nt * kGN;
                __nv_bfloat16* dst = live ? reinterpret_cast<__nv_bfloat16*>(g.e.x_full) + (int64_t)(g.e.tok_index ? g.e.tok_index[row] : row) * g.e.ldx + nt * kGN : nullptr;
                float su = 0.f, sh = 0.f, st2 = 0.f;
#pragma unroll
                for (int c = 0; c < kGN / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tD + c * 32, o);
                    tmem_wait_ld();
                    if (live) {
#pragma unroll
                        for (int e = 0; e < 32; e += 8) {
                            const uint4 hv = ld_v4(hsrc + c * 32 + e);        // coherent: x_full may be H itself (identity token rows)
                            const float hf[8] = {bf16lo(hv.x), bf16hi(hv.x), bf16lo(hv.y), bf16hi(hv.y), bf16lo(hv.z), bf16hi(hv.z), bf16lo(hv.w), bf16hi(hv.w)};
                            float y[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                const float u = __uint_as_float(o[e + i]);
                                su += u * u;
                                sh += hf[i] * hf[i];
                                y[i] = hf[i] + u;
                                st2 += y[i] * y[i];
                            }
                            st_v4(dst + c * 32 + e, make_uint4(pack_bf16(y[0], y[1]), pack_bf16(y[2], y[3]), pack_bf16(y[4], y[5]), pack_bf16(y[6], y[7])));
                        }
                    }
                }
                if (live) g.e.sums[(int64_t)row * n_tiles + nt] = make_float4(su, sh, st2, 0.f);
            } else {
                // SWIGLU: columns 0-127 gate, 128-255 up of the same 128 features
                __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(g.C) + (int64_t)row * g.ldc + nt * 128;
                const float rsc = (g.e.row_scale && live) ? g.e.row_scale[row] : 1.0f;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t gt[32], up[32];
                    tmem_ld32(tD + c * 32, gt);
                    tmem_ld32(tD + 128 + c * 32, up);
                    tmem_wait_ld();
                    if (live) {
                        float a[32];
#pragma unroll
                        for (int e = 0; e < 32; ++e) {
                            const float z = __uint_as_float(gt[e]) * rsc;
                            a[e] = z / (1.0f + __expf(-z)) * (__uint_as_float(up[e]) * rsc);
                        }
#pragma unroll
                        for (int e = 0; e < 32; e += 8)
                            st_v4(dst + c * 32 + e, make_uint4(pack_bf16(a[e], a[e + 1]), pack_bf16(a[e + 2], a[e + 3]),
                                                               pack_bf16(a[e + 4], a[e + 5]), pack_bf16(a[e + 6], a[e + 7])));
                    }
                }
            }
            tc_fence_before();
            arrive_on_leader(acc_empty(b));
        }
        if (!ok && lane == 0) atomicExch(g.status, DASH_ERR_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                    // nobody leaves while the peer may still signal its barriers or read its tiles
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

// Per row (one warp): (cos, sin) of pos[t] * base^(-2i/D) for i < D/2, angles formed and reduced in fp64 (positions reach 1e5 rad
// at i = 0: fp32 would lose the angle), evaluated in fp32 on the reduced angle; and, when asked, the row factor of the RMSNorm, 1 / sqrt(mean(h^2) + eps), from one pass over the bf16 row
struct RopeFreqs { double inv_freq[64]; };
__global__ void __launch_bounds__(256)
row_prep_kernel(const int32_t* __restrict__ pos, int64_t n, int half, RopeFreqs fr, float2* __restrict__ table, const char* __restrict__ H,
                int64_t ldh_b, int nvec, float inv_d, float eps, float* __restrict__ inv_rms, const int32_t* __restrict__ n_dev) {
    pdl_launch_dependents();
    if (n_dev) { int64_t nd = *n_dev; if (nd < n) n = nd; }
    const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
    for (int64_t t = (int64_t)blockIdx.x * wpb + (threadIdx.x >> 5); t < n; t += (int64_t)gridDim.x * wpb) {
        float ss = 0.f;
        if (inv_rms) {
            const char* h = H + t * ldh_b;
            for (int base = 0; base < nvec; base += 128) {
                uint4 x[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) { const int v = base + k * 32 + lane; if (v < nvec) x[k] = ld_nc_v4(h + ((int64_t)v << 4)); }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int v = base + k * 32 + lane;
                    if (v < nvec) {
                        const float f[8] = {bf16lo(x[k].x), bf16hi(x[k].x), bf16lo(x[k].y), bf16hi(x[k].y), bf16lo(x[k].z), bf16hi(x[k].z), bf16lo(x[k].w), bf16hi(x[k].w)};
#pragma unroll
                        for (int e = 0; e < 8; ++e) ss += f[e] * f[e];
                    }
                }
            }
        }
        if (table) {
            const double ps = pos ? (double)pos[t] : (double)t;
            for (int i = lane; i < half; i += 32) {
                // angle formed and reduced to [-pi, pi] in fp64 (three operations), sine and cosine of the reduced angle in fp32
                const double ang = ps * fr.inv_freq[i];
                const double red = fma(-6.283185307179586476925286766559, rint(ang * 0.15915494309189533576888376337251), ang);
                float sn, cs;
                sincosf((float)red, &sn, &cs);
                table[t * half + i] = make_float2(cs, sn);
            }
        }
        if (inv_rms) {
            ss = warp_sum(ss);
            if (lane == 0) inv_rms[t] = rsqrtf(ss * inv_d + eps);
        }
    }
}

static int make_map_2d_bf16(CUtensorMap* map, const void* basep, uint64_t inner, uint64_t outer, uint64_t ld_elems, uint32_t box_inner,
                            uint32_t box_outer) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return DASH_ERR_CUDA;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {ld_elems * 2};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(basep), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS
               ? DASH_OK : DASH_ERR_CUDA;
}

template <int EPI>
static int launch_gemm(const CUtensorMap& ma, const CUtensorMap& mw, const GemmArgs& g, cudaStream_t st) {
    const int smem = kGStages * kGStageBytes + 1024 + 256;
    static std::atomic<uint64_t> configured{0};
    if (!set_max_smem_once(gemm_kernel<EPI>, smem, configured)) return DASH_ERR_CUDA;
    const int tiles = ((g.n + 2 * kGM - 1) / (2 * kGM)) * g.n_tiles;
    int pairs = sm_count() / 2;
    if (pairs > tiles) pairs = tiles;
    gemm_kernel<EPI><<<2 * pairs, kGThreads, smem, st>>>(ma, mw, g);
    return cudaGetLastError() == cudaSuccess ? DASH_OK : DASH_ERR_CUDA;
}

bool gemm_shape_ok(GemmEpilogueKind kind, int64_t n, int64_t N, int64_t K, int64_t lda, int64_t ldw, const GemmEpilogue& e) {
    if (n < 1 || n > 0x7fffffffLL || N < 1 || N > 0x7fffffffLL || K < 1 || K > 0x7fffffffLL || (lda % 8) || (ldw % 8)) return false;
    if (kind == GEMM_PLAIN) return (N % 4) == 0 && (K % 8) == 0;      // rows of A, W and C start on 16-byte boundaries
    // the fused epilogues work on whole 256-column tiles and whole K steps
    if (K < kGK || (K % kGK)) return false;
    if (kind == GEMM_SWIGLU) return e.m >= 128 && (e.m % 128) == 0 && N == 2 * (int64_t)e.m;
    if (N < kGN || (N % kGN)) return false;
    if (kind == GEMM_ROPE) return (e.D == 64 || e.D == 128) && (e.n_rot_cols % kGN) == 0 && e.n_rot_cols <= N;
    return true;
}

int gemm_bf16(GemmEpilogueKind kind, const void* A, int64_t lda, const void* W, int64_t ldw, void* C, int64_t ldc, int64_t n, int64_t N,
              int64_t K, const GemmEpilogue& e, const int32_t* n_dev, cudaStream_t st, bool out_f32) {
    if (!gemm_shape_ok(kind, n, N, K, lda, ldw, e)) return DASH_ERR_UNSUPPORTED;
    if (!aligned16(A) || !aligned16(W)) return DASH_ERR_INVALID_ARG;
    if (out_f32 && kind != GEMM_PLAIN) return DASH_ERR_UNSUPPORTED;
    if (kind == GEMM_PLAIN && (!aligned16(C) || (ldc * (out_f32 ? 4 : 2)) % 16 || (!out_f32 && (N % 8)))) return DASH_ERR_UNSUPPORTED;
    CUtensorMap ma, mw;
    int rc;
    if ((rc = make_map_2d_bf16(&ma, A, (uint64_t)K, (uint64_t)n, (uint64_t)lda, 64, kGM)) != DASH_OK) return rc;
    if ((rc = make_map_2d_bf16(&mw, W, (uint64_t)N, (uint64_t)K, (uint64_t)ldw, 64, kGK)) != DASH_OK) return rc;
    GemmArgs g;
    g.n = (int)n; g.N = (int)N; g.K = (int)K;
    g.n_tiles = kind == GEMM_SWIGLU ? e.m / 128 : (int)((N + kGN - 1) / kGN);
    g.C = C; g.ldc = ldc; g.n_dev = n_dev; g.e = e; g.out_f32 = out_f32 ? 1 : 0;
    g.status = status_word_ptr();
    if (!g.status) return DASH_ERR_CUDA;
    switch (kind) {
        case GEMM_PLAIN: return launch_gemm<GEMM_PLAIN>(ma, mw, g, st);
        case GEMM_ROPE: return launch_gemm<GEMM_ROPE>(ma, mw, g, st);
        case GEMM_RESID: return launch_gemm<GEMM_RESID>(ma, mw, g, st);
        default: return launch_gemm<GEMM_SWIGLU>(ma, mw, g, st);
    }
}

int launch_row_prep(const int32_t* pos, int64_t n, int D, double rope_base, float2* table, const void* H, int64_t ldh, int d, float rms_eps,
                    float* inv_rms, const int32_t* n_dev, cudaStream_t st, bool beside_front) {
    RopeFreqs fr;
    for (int i = 0; i < D / 2; ++i) fr.inv_freq[i] = pow(rope_base, -2.0 * i / D);
    int64_t blocks = (n + 7) / 8, cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    // beside_front: the kernel in front in the stream is one whose output this kernel does not read and that was itself an ordinary
    // launch (the block step's attention item list): launched to start beside it -- the kernel has no griddepcontrol.wait, and its
    // inputs were complete before the kernel in front started.
    if (beside_front)
        return launch_pdl(row_prep_kernel, (int)blocks, 256, 0, st, pos, n, D / 2, fr, table, (const char*)H, ldh * 2, d * 2 / 16, 1.0f / d,
                          rms_eps, inv_rms, n_dev) == cudaSuccess ? DASH_OK : DASH_ERR_CUDA;
    row_prep_kernel<<<(int)blocks, 256, 0, st>>>(pos, n, D / 2, fr, table, (const char*)H, ldh * 2, d * 2 / 16, 1.0f / d, rms_eps, inv_rms, n_dev);
    return cudaGetLastError() == cudaSuccess ? DASH_OK : DASH_ERR_CUDA;
}

}  // namespace dash

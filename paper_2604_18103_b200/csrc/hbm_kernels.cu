// HBM-bound kernels of the halted-prefill path: delta-attention score (+ fused
// residual and threshold), halting rule, single-pass compaction, scatter.
#include "common.cuh"
#include "dash_testing.h"
#include "sm100_ptx.cuh"

namespace dash {

// ---------------------------------------------------------------------------
// step 1: r_t = ||U_t|| / max(||H_t||, eps)   (Eq. 2; "relative" form of Fig. 1)
// One warp per row, 128-bit loads, 8 loads in flight per lane, fp32 sums,
// shuffle reduction.  Optional: H~ = H + U written in the same pass (optionally
// to an indexed row), and the threshold rule applied to r.
// ---------------------------------------------------------------------------
struct FusedThreshold {
    float tau;
    int keep_first, keep_last;
    const int32_t* cu;
    int S;
    uint8_t* mask_out;
};

template <bool BF16>
__device__ __forceinline__ float sumsq_vec(uint4 v) {
    if (BF16) {
        float a0 = bf16lo(v.x), a1 = bf16hi(v.x), a2 = bf16lo(v.y), a3 = bf16hi(v.y);
        float a4 = bf16lo(v.z), a5 = bf16hi(v.z), a6 = bf16lo(v.w), a7 = bf16hi(v.w);
        return a0 * a0 + a1 * a1 + a2 * a2 + a3 * a3 + a4 * a4 + a5 * a5 + a6 * a6 + a7 * a7;
    } else {
        float a0 = __uint_as_float(v.x), a1 = __uint_as_float(v.y), a2 = __uint_as_float(v.z), a3 = __uint_as_float(v.w);
        return a0 * a0 + a1 * a1 + a2 * a2 + a3 * a3;
    }
}
template <bool BF16>
__device__ __forceinline__ uint4 add_vec(uint4 a, uint4 b) {
    uint4 o;
    if (BF16) {
        o.x = pack_bf16(bf16lo(a.x) + bf16lo(b.x), bf16hi(a.x) + bf16hi(b.x));
        o.y = pack_bf16(bf16lo(a.y) + bf16lo(b.y), bf16hi(a.y) + bf16hi(b.y));
        o.z = pack_bf16(bf16lo(a.z) + bf16lo(b.z), bf16hi(a.z) + bf16hi(b.z));
        o.w = pack_bf16(bf16lo(a.w) + bf16lo(b.w), bf16hi(a.w) + bf16hi(b.w));
    } else {
        o.x = __float_as_uint(__uint_as_float(a.x) + __uint_as_float(b.x));
        o.y = __float_as_uint(__uint_as_float(a.y) + __uint_as_float(b.y));
        o.z = __float_as_uint(__uint_as_float(a.z) + __uint_as_float(b.z));
        o.w = __float_as_uint(__uint_as_float(a.w) + __uint_as_float(b.w));
    }
    return o;
}

template <bool BF16>
__global__ void __launch_bounds__(256)
delta_norm_kernel(const char* __restrict__ U, const char* __restrict__ H, int64_t n, int nvec,
                  int64_t ldU_b, int64_t ldH_b, int mode, float eps, float* __restrict__ r_out,
                  char* Hres, int64_t ldR_b, const int32_t* __restrict__ res_index,
                  FusedThreshold ft, const int32_t* __restrict__ n_dev, int aliased) {
    const int lane = threadIdx.x & 31;
    const int wpb = blockDim.x >> 5;
    if (n_dev) { int64_t nd = *n_dev; if (nd < n) n = nd; }
    const bool need_h = (mode == DASH_NORM_REL) || (Hres != nullptr);
    constexpr int CH = 4;
    for (int64_t row = (int64_t)blockIdx.x * wpb + (threadIdx.x >> 5); row < n; row += (int64_t)gridDim.x * wpb) {
        const char* u = U + row * ldU_b;
        const char* h = H + row * ldH_b;
        char* o = nullptr;
        if (Hres) o = Hres + (res_index ? (int64_t)res_index[row] : row) * ldR_b;
        float su = 0.f, sh = 0.f;
        for (int base = 0; base < nvec; base += 32 * CH) {
            uint4 a[CH], b[CH];
#pragma unroll
            for (int k = 0; k < CH; ++k) {
                int v = base + k * 32 + lane;
                if (v < nvec) {
                    // the read-only path only where the residual output overlaps neither input (each vector is read before it is
                    // written, by the same thread, so an output that is H itself is well defined -- through coherent loads)
                    a[k] = aliased ? ld_v4(u + ((int64_t)v << 4)) : ld_nc_v4(u + ((int64_t)v << 4));
                    if (need_h) b[k] = aliased ? ld_v4(h + ((int64_t)v << 4)) : ld_nc_v4(h + ((int64_t)v << 4));
                }
            }
#pragma unroll
            for (int k = 0; k < CH; ++k) {
                int v = base + k * 32 + lane;
                if (v < nvec) {
                    su += sumsq_vec<BF16>(a[k]);
                    if (need_h) {
                        sh += sumsq_vec<BF16>(b[k]);
                        if (o) st_v4(o + ((int64_t)v << 4), add_vec<BF16>(a[k], b[k]));
                    }
                }
            }
        }
        su = warp_sum(su);
        sh = warp_sum(sh);
        if (lane == 0) {
            float num = sqrtf(su);
            float r = (mode == DASH_NORM_ABS) ? num : num / fmaxf(sqrtf(sh), eps);
            r_out[row] = r;
            if (ft.mask_out) {
                int s = find_seq(ft.cu, ft.S, (int)row);
                int local = (int)row - ft.cu[s], len = ft.cu[s + 1] - ft.cu[s];
                bool prot = (local < ft.keep_first) || (local >= len - ft.keep_last);
                ft.mask_out[row] = (prot || !(r < ft.tau)) ? 1 : 0;
            }
        }
    }
}

// ---------------------------------------------------------------------------
// step 2: halting rule
// ---------------------------------------------------------------------------
__global__ void select_threshold_kernel(const float* __restrict__ r, int64_t n, const int32_t* __restrict__ cu, int S,
                                        float tau, int keep_first, int keep_last, uint8_t* __restrict__ mask, int halt_high) {
    int64_t total = cu[S];
    if (total < n) n = total;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < n; t += (int64_t)gridDim.x * blockDim.x) {
        int s = find_seq(cu, S, (int)t);
        int local = (int)t - cu[s], len = cu[s + 1] - cu[s];
        bool prot = (local < keep_first) || (local >= len - keep_last);
        const bool halted = halt_high ? (r[t] > tau) : (r[t] < tau);      // NaN compares false: stays
        mask[t] = (prot || !halted) ? 1 : 0;
    }
}

// monotone map fp32 -> u32 (larger value = larger key); NaN -> max; -0 -> +0
__device__ __forceinline__ uint32_t order_key(float f) {
    uint32_t b = __float_as_uint(f);
    if ((b & 0x7fffffffu) > 0x7f800000u) return 0xffffffffu;
    if (b == 0x80000000u) b = 0;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// exclusive scan of one int per thread over a 1024-thread block; total returned to all
__device__ __forceinline__ int block_excl_scan_1024(int v, int* s_warp, int* total) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) s_warp[w] = inc;
    __syncthreads();
    if (w == 0) {
        int x = s_warp[lane];
        int xi = x;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, xi, o);
            if (lane >= o) xi += t;
        }
        s_warp[lane] = xi - x;
        if (lane == 31) s_warp[32] = xi;
    }
    __syncthreads();
    int res = s_warp[w] + inc - v;
    *total = s_warp[32];
    __syncthreads();
    return res;
}

// One 1024-thread CTA per sequence: 4-pass MSB radix select of the k-th largest
// key among the eligible (unprotected) tokens, then one ordered pass that keeps
// keys above the cut and the lowest-index ties.
__global__ void __launch_bounds__(1024)
select_keep_count_kernel(const float* __restrict__ r, const int32_t* __restrict__ cu, int S,
                         const int32_t* __restrict__ keep_counts, int keep_first, int keep_last,
                         uint8_t* __restrict__ mask, int halt_high) {
    __shared__ int hist[256];
    __shared__ int s_warp[33];
    __shared__ uint32_t s_prefix;
    __shared__ int s_remaining;
    const int s = blockIdx.x;
    const int a = cu[s], b = cu[s + 1], ns = b - a;
    if (ns <= 0) return;
    const int kf = min(max(keep_first, 0), ns);
    const int kl = min(max(keep_last, 0), ns - kf);
    const int e0 = a + kf, e1 = b - kl;          // eligible range [e0, e1)
    const int n_el = e1 - e0;
    int k_el = keep_counts[s] - (kf + kl);
    k_el = min(max(k_el, 0), n_el);
    for (int t = a + threadIdx.x; t < e0; t += blockDim.x) mask[t] = 1;
    for (int t = e1 + threadIdx.x; t < b; t += blockDim.x) mask[t] = 1;
    if (k_el == 0 || k_el == n_el) {
        uint8_t v = k_el ? 1 : 0;
        for (int t = e0 + threadIdx.x; t < e1; t += blockDim.x) mask[t] = v;
        return;
    }
    uint32_t prefix = 0, pmask = 0;
    int remaining = k_el;                         // rank (from the top) inside the current bucket
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0;
        __syncthreads();
        for (int t = e0 + threadIdx.x; t < e1; t += blockDim.x) {
            uint32_t key = order_key(halt_high ? -r[t] : r[t]);
            if ((key & pmask) == prefix) atomicAdd(&hist[(key >> shift) & 255], 1);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int acc = 0, bsel = 0;
            for (int bk = 255; bk >= 0; --bk) {
                if (acc + hist[bk] >= remaining) { bsel = bk; break; }
                acc += hist[bk];
            }
            s_prefix = prefix | ((uint32_t)bsel << shift);
            s_remaining = remaining - acc;
        }
        __syncthreads();
        prefix = s_prefix;
        remaining = s_remaining;
        pmask |= (0xffu << shift);
        __syncthreads();
    }
    // prefix = key of the k-th largest; `remaining` of the tokens that tie with it stay
    const uint32_t cut = prefix;
    const int per = (n_el + blockDim.x - 1) / blockDim.x;
    const int t0 = min(e0 + (int)threadIdx.x * per, e1), t1 = min(t0 + per, e1);
    int ties = 0;
    for (int t = t0; t < t1; ++t) ties += (order_key(halt_high ? -r[t] : r[t]) == cut);
    int total;
    int rank = block_excl_scan_1024(ties, s_warp, &total);
    for (int t = t0; t < t1; ++t) {
        uint32_t key = order_key(halt_high ? -r[t] : r[t]);
        uint8_t v = 0;
        if (key > cut) v = 1;
        else if (key == cut) { v = rank < remaining; ++rank; }
        mask[t] = v;
    }
}

// ---------------------------------------------------------------------------
// step 3: compaction.  Single pass: each CTA takes a tile of TILE tokens, ballots
// its mask, finds its output base, then its 16 warps move the tile's active rows
// in 4 KB pieces (128-bit accesses, 8 per lane in flight).
// Output base of a tile = number of active tokens before it:
//  - DIRECT (small inputs): counted straight from the mask bytes in front of the
//    tile (a few KB from L2) -- no scratch, no ordering between CTAs;
//  - otherwise: ticketed tiles publish their counts and look back over the
//    preceding tiles (decoupled look-back, bounded spin).
// ---------------------------------------------------------------------------
struct RowStreams {
    const char* src[DASH_MAX_ROW_STREAMS];
    char* dst[DASH_MAX_ROW_STREAMS];
    int64_t row_bytes[DASH_MAX_ROW_STREAMS], src_ld[DASH_MAX_ROW_STREAMS], dst_ld[DASH_MAX_ROW_STREAMS];
    int vec16[DASH_MAX_ROW_STREAMS];
    int count;
};

constexpr unsigned long long kFlagAgg = 1ull << 32, kFlagPrefix = 2ull << 32;
constexpr int kCompactThreads = 512;
constexpr int kPieceBytes = 4096;                       // one warp moves one piece at a time

__device__ __forceinline__ unsigned long long ld_state(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_state(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ int nonzero_bytes(uint32_t w) { return __popc(__vcmpne4(w, 0u)) >> 3; }

template <int TILE, bool DIRECT>
__global__ void __launch_bounds__(kCompactThreads)
compact_kernel(const uint8_t* __restrict__ mask, int64_t n_upper, const int32_t* __restrict__ cu_in, int S,
               RowStreams rs, const int32_t* __restrict__ pos_in, int32_t* __restrict__ pos_out,
               const int32_t* __restrict__ tok_in, int32_t* __restrict__ tok_out,
               int32_t* __restrict__ idx_out, int32_t* __restrict__ cu_out, int32_t* __restrict__ n_out_dev,
               unsigned long long* tile_state, unsigned int* ticket, int* status, int mask_vec16, uint32_t spin_limit) {
    constexpr int NW = TILE / 32;                       // warps that ballot
    constexpr int NWARPS = kCompactThreads / 32;
    __shared__ unsigned int s_ballot[NW];
    __shared__ int s_wprefix[NW + 1];
    __shared__ int s_src[TILE];
    __shared__ int s_base;
    __shared__ int s_part[NWARPS];
    __shared__ unsigned int s_tile;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int tile;
    if (DIRECT) {
        tile = (int)blockIdx.x;
    } else {
        if (threadIdx.x == 0) s_tile = atomicAdd(ticket, 1u);
        __syncthreads();
        tile = (int)s_tile;
    }
    int64_t n = cu_in[S];
    if (n > n_upper) n = n_upper;
    const int64_t t_start = (int64_t)tile * TILE;
    if (t_start >= n && tile != 0) return;              // nothing depends on tiles past the end
    const int64_t t_end = (t_start + TILE < n) ? t_start + TILE : n;
    const bool last_tile = (t_end >= n);

    int my = 0;
    if (warp < NW) {
        int64_t t = t_start + threadIdx.x;
        my = (t < n) ? (mask[t] != 0) : 0;
        unsigned int bal = __ballot_sync(0xffffffffu, my);
        if (lane == 0) s_ballot[warp] = bal;
    }
    if (DIRECT) {
        // active tokens in front of this tile, straight from the mask (t_start is a multiple of 32)
        int cnt = 0;
        if (mask_vec16) {
            const uint4* mv = reinterpret_cast<const uint4*>(mask);
            for (int64_t v = threadIdx.x; v < (t_start >> 4); v += kCompactThreads) {
                const uint4 w = ld_nc_v4(mv + v);
                cnt += nonzero_bytes(w.x) + nonzero_bytes(w.y) + nonzero_bytes(w.z) + nonzero_bytes(w.w);
            }
        } else {
            for (int64_t t = threadIdx.x; t < t_start; t += kCompactThreads) cnt += (mask[t] != 0);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
        if (lane == 0) s_part[warp] = cnt;
    }
    __syncthreads();
    if (warp == 0) {
        int c = (lane < NW) ? __popc(s_ballot[lane]) : 0;
        int inc = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int x = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += x;
        }
        if (lane < NW) s_wprefix[lane] = inc - c;
        const int agg = __shfl_sync(0xffffffffu, inc, 31);
        if (lane == 0) s_wprefix[NW] = agg;
        int base = 0;
        if (DIRECT) {
            int v = (lane < NWARPS) ? s_part[lane] : 0;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            base = v;
        } else if (tile == 0) {
            if (lane == 0) st_state(&tile_state[0], kFlagPrefix | (unsigned int)agg);
        } else {
            // publish this tile's count, then look back
            if (lane == 0) st_state(&tile_state[tile], kFlagAgg | (unsigned int)agg);
            int look = tile - 1;
            bool done = false, timed_out = false;
            while (!done) {
                const int j = look - lane;
                unsigned long long st = kFlagPrefix;    // virtual tiles before 0: prefix 0
                uint32_t spins = 0;
                if (j >= 0) {
                    st = ld_state(&tile_state[j]);
                    while ((st >> 32) == 0) {
                        if (++spins > spin_limit) { timed_out = true; break; }
                        __nanosleep(32);
                        st = ld_state(&tile_state[j]);
                    }
                }
                if (__any_sync(0xffffffffu, timed_out)) { timed_out = true; break; }
                const unsigned int has_prefix = __ballot_sync(0xffffffffu, (st >> 32) == 2);
                const int first = has_prefix ? (__ffs(has_prefix) - 1) : 32;   // nearest tile with a full prefix
                int v = (lane <= first) ? (int)(unsigned int)(st & 0xffffffffu) : 0;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                base += v;
                if (has_prefix) done = true; else look -= 32;
            }
            if (timed_out) { if (lane == 0) atomicExch(status, DASH_ERR_TIMEOUT); base = 0; }
            if (lane == 0) st_state(&tile_state[tile], kFlagPrefix | (unsigned int)(base + agg));
        }
        if (lane == 0) s_base = base;
    }
    __syncthreads();
    const int base = s_base;
    const int count = s_wprefix[NW];
    if (warp < NW && my) {
        int local = s_wprefix[warp] + __popc(s_ballot[warp] & ((1u << lane) - 1u));
        int t = (int)(t_start + threadIdx.x);
        s_src[local] = t;
        if (idx_out) idx_out[base + local] = t;
        if (pos_out) pos_out[base + local] = pos_in[t];
        if (tok_out) tok_out[base + local] = tok_in[t];
    }
    // new sequence boundaries: cu_out[s] = number of active tokens before cu_in[s]
    for (int s = threadIdx.x; s <= S; s += blockDim.x) {
        int64_t c = cu_in[s];
        if (c > n) c = n;
        bool mine = (c >= t_start && c < t_start + TILE && c < t_end) || (last_tile && c == t_end);
        if (tile == 0 && n == 0) mine = true;
        if (mine) {
            int p = (int)(c - t_start);
            int v = base;
            if (p >= TILE || c >= t_end) v += count;
            else v += s_wprefix[p >> 5] + __popc(s_ballot[p >> 5] & ((1u << (p & 31)) - 1u));
            cu_out[s] = v;
            if (s == S && n_out_dev) *n_out_dev = v;
        }
    }
    __syncthreads();
    // move the rows: the tile's (row, piece) items are dealt round-robin to the warps, across all row tensors
    int first_warp = 0;                                 // warp that takes item 0 of the current tensor
    for (int q = 0; q < rs.count; ++q) {
        const int64_t rb = rs.row_bytes[q];
        if (rs.vec16[q]) {
            const int pieces = (int)((rb + kPieceBytes - 1) / kPieceBytes);
            const int items = count * pieces;
            for (int it = (warp - first_warp + NWARPS) % NWARPS; it < items; it += NWARPS) {
                const int k = it / pieces, pc = it - k * pieces;
                const int64_t off = (int64_t)pc * kPieceBytes;
                const int64_t len = (rb - off < kPieceBytes) ? rb - off : kPieceBytes;
                warp_copy_row16(rs.src[q] + (int64_t)s_src[k] * rs.src_ld[q] + off, rs.dst[q] + (int64_t)(base + k) * rs.dst_ld[q] + off, len, lane);
            }
            first_warp = (first_warp + items) % NWARPS;
        } else {
            for (int k = (warp - first_warp + NWARPS) % NWARPS; k < count; k += NWARPS)
                warp_copy_row4(rs.src[q] + (int64_t)s_src[k] * rs.src_ld[q], rs.dst[q] + (int64_t)(base + k) * rs.dst_ld[q], rb, lane);
            first_warp = (first_warp + count) % NWARPS;
        }
    }
}

__global__ void __launch_bounds__(256)
scatter_kernel(const char* __restrict__ src, int64_t n, int64_t row_bytes, int64_t src_ld, const int32_t* __restrict__ tok_index,
               const uint8_t* __restrict__ sel, int which, const int32_t* __restrict__ n_dev, char* __restrict__ dst,
               int64_t dst_ld, int vec16) {
    const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
    if (n_dev) { int64_t nd = *n_dev; if (nd < n) n = nd; }
    for (int64_t i = (int64_t)blockIdx.x * wpb + (threadIdx.x >> 5); i < n; i += (int64_t)gridDim.x * wpb) {
        if (which != 2 && (int)(sel[i] != 0) != which) continue;
        int64_t drow = tok_index ? (int64_t)tok_index[i] : i;
        if (vec16) warp_copy_row16(src + i * src_ld, dst + drow * dst_ld, row_bytes, lane);
        else warp_copy_row4(src + i * src_ld, dst + drow * dst_ld, row_bytes, lane);
    }
}

// ---------------------------------------------------------------------------
// Steps 1-3 of the block step in one pass (threshold rule, every row's H~ written to the full-length
// buffer): per tile of 32 tokens the 16 warps form r, the keep decision and H~ = H + U, stream H~ to
// x_full[tok[row]], then the tile finds its output base by decoupled look-back and copies its active
// rows (just written, still in L2) into the next block's packed buffer.  Reads U and H once, writes
// x_full and H_next once: no separate scatter and compaction passes over H~.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint4 ld_cg_v4(const void* p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

struct TailArgs {
    const char* U; const char* H; int64_t ldU_b, ldH_b; int nvec; int mode; float eps;
    const uint8_t* mask_in;       // non-null: keep decisions are given (r and the mask are not formed), U is any update to add to H
    const float4* sums; int n_sum_tiles;   // non-null: per-row partial (sum u^2, sum h^2, ..) from the output-projection epilogue; with U null
                                           // the rows are already in x_full and only the score, the decision and the compaction remain
    float tau; int keep_first, keep_last; const int32_t* cu_in; int S;
    const int32_t* tok_in; const int32_t* pos_in;
    char* x_full; int64_t ldx_b; char* H_next; int64_t ldn_b;
    float* r_out; uint8_t* mask_out; int32_t* tok_next; int32_t* pos_next; int32_t* cu_next; int32_t* n_next;
    unsigned long long* tile_state; unsigned int* ticket; int* status;
    float* inv_next; float inv_d, rms_eps;     // non-null: 1 / sqrt(mean(row^2) + rms_eps) of every row that goes to H_next, in its order
};

template <bool BF16>
__global__ void __launch_bounds__(kCompactThreads, 2)
delta_tail_kernel(const TailArgs a, int64_t n_upper) {
    constexpr int TILE = 32, NWARPS = kCompactThreads / 32, RPW = TILE / NWARPS;   // 2 rows per warp
    __shared__ int s_keep[TILE];
    __shared__ int s_src[TILE];
    __shared__ float s_inv[TILE];
    __shared__ int s_base, s_count;
    __shared__ unsigned int s_tile, s_ballot;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    ptx::pdl_wait();                                       // launched to start early: nothing global is touched before the kernel in front is done
    if (threadIdx.x == 0) s_tile = atomicAdd(a.ticket, 1u);
    __syncthreads();
    const int tile = (int)s_tile;
    int64_t n = a.cu_in[a.S];
    if (n > n_upper) n = n_upper;
    const int64_t t_start = (int64_t)tile * TILE;
    if (t_start >= n && tile != 0) return;
    const int64_t t_end = (t_start + TILE < n) ? t_start + TILE : n;
    const bool last_tile = (t_end >= n);
    constexpr int CH = 4;
#pragma unroll 1
    for (int rr = 0; rr < RPW; ++rr) {
        const int local = warp * RPW + rr;
        const int64_t row = t_start + local;
        int keep = 0;
        float ss = 0.f;                                  // sum of squares of the row as it goes on (H~ or H')
        if (row < n) {
            float su = 0.f, sh = 0.f;
            if (a.U) {
                const char* u = a.U + row * a.ldU_b;
                const char* h = a.H + row * a.ldH_b;
                char* o = a.x_full + (int64_t)a.tok_in[row] * a.ldx_b;
                for (int base = 0; base < a.nvec; base += 32 * CH) {
                    uint4 x[CH], y[CH];
#pragma unroll
                    for (int k = 0; k < CH; ++k) {
                        const int v = base + k * 32 + lane;
                        if (v < a.nvec) { x[k] = ld_nc_v4(u + ((int64_t)v << 4)); y[k] = ld_nc_v4(h + ((int64_t)v << 4)); }
                    }
#pragma unroll
                    for (int k = 0; k < CH; ++k) {
                        const int v = base + k * 32 + lane;
                        if (v < a.nvec) {
                            su += sumsq_vec<BF16>(x[k]);
                            sh += sumsq_vec<BF16>(y[k]);
                            const uint4 z = add_vec<BF16>(x[k], y[k]);
                            if (a.inv_next) ss += sumsq_vec<BF16>(z);
                            st_v4(o + ((int64_t)v << 4), z);
                        }
                    }
                }
            }
            if (a.mask_in) {
                keep = a.mask_in[row] != 0;
            } else {
                if (a.sums) {
                    // the projection's column tiles, summed in a fixed order (lane i takes tiles i, i + 32, ...)
                    su = 0.f; sh = 0.f;
                    for (int i = lane; i < a.n_sum_tiles; i += 32) { const float4 p2 = a.sums[(int64_t)row * a.n_sum_tiles + i]; su += p2.x; sh += p2.y; ss += p2.z; }
                }
                su = warp_sum(su);
                sh = warp_sum(sh);
                const float num = sqrtf(su);
                const float r = (a.mode == DASH_NORM_ABS) ? num : num / fmaxf(sqrtf(sh), a.eps);
                const int s = find_seq(a.cu_in, a.S, (int)row);
                const int lp = (int)row - a.cu_in[s], len = a.cu_in[s + 1] - a.cu_in[s];
                const bool prot = (lp < a.keep_first) || (lp >= len - a.keep_last);
                keep = (prot || !(r < a.tau)) ? 1 : 0;
                if (lane == 0) { a.r_out[row] = r; a.mask_out[row] = (uint8_t)keep; }
            }
        }
        if (a.inv_next) ss = warp_sum(ss);
        if (lane == 0) { s_keep[local] = keep; s_inv[local] = rsqrtf(ss * a.inv_d + a.rms_eps); }
    }
    __syncthreads();                                    // also orders this CTA's x_full rows before the copies below
    if (warp == 0) {
        const int my = s_keep[lane];
        const unsigned int bal = __ballot_sync(0xffffffffu, my);
        const int agg = __popc(bal);
        int base = 0;
        if (tile == 0) {
            if (lane == 0) st_state(&a.tile_state[0], kFlagPrefix | (unsigned int)agg);
        } else {
            if (lane == 0) st_state(&a.tile_state[tile], kFlagAgg | (unsigned int)agg);
            int look = tile - 1;
            bool done = false, timed_out = false;
            while (!done) {
                const int j = look - lane;
                unsigned long long st = kFlagPrefix;
                uint32_t spins = 0;
                if (j >= 0) {
                    st = ld_state(&a.tile_state[j]);
                    while ((st >> 32) == 0) {
                        if (++spins > kSpinLimit) { timed_out = true; break; }
                        __nanosleep(32);
                        st = ld_state(&a.tile_state[j]);
                    }
                }
                if (__any_sync(0xffffffffu, timed_out)) { timed_out = true; break; }
                const unsigned int has_prefix = __ballot_sync(0xffffffffu, (st >> 32) == 2);
                const int first = has_prefix ? (__ffs(has_prefix) - 1) : 32;
                int v = (lane <= first) ? (int)(unsigned int)(st & 0xffffffffu) : 0;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                base += v;
                if (has_prefix) done = true; else look -= 32;
            }
            if (timed_out) { if (lane == 0) atomicExch(a.status, DASH_ERR_TIMEOUT); base = 0; }
            if (lane == 0) st_state(&a.tile_state[tile], kFlagPrefix | (unsigned int)(base + agg));
        }
        if (my) {
            const int k = __popc(bal & ((1u << lane) - 1u));
            const int t = (int)t_start + lane;
            s_src[k] = t;
            a.tok_next[base + k] = a.tok_in[t];
            a.pos_next[base + k] = a.pos_in[t];
            if (a.inv_next) a.inv_next[base + k] = s_inv[lane];
        }
        if (lane == 0) { s_base = base; s_count = agg; s_ballot = bal; }
    }
    __syncthreads();
    const int base = s_base, count = s_count;
    const unsigned int bal = s_ballot;
    for (int s = threadIdx.x; s <= a.S; s += blockDim.x) {
        int64_t c = a.cu_in[s];
        if (c > n) c = n;
        bool mine = (c >= t_start && c < t_start + TILE && c < t_end) || (last_tile && c == t_end);
        if (tile == 0 && n == 0) mine = true;
        if (mine) {
            const int p = (int)(c - t_start);
            int v = base;
            if (p >= TILE || c >= t_end) v += count;
            else v += __popc(bal & ((1u << p) - 1u));
            a.cu_next[s] = v;
            if (s == a.S && a.n_next) *a.n_next = v;
        }
    }
    // copy the tile's active rows x_full[tok] -> H_next[base + k], 4 KB pieces dealt to the warps
    const int64_t rb = (int64_t)a.nvec << 4;
    const int pieces = (int)((rb + kPieceBytes - 1) / kPieceBytes);
    const int items = count * pieces;
    for (int it = warp; it < items; it += NWARPS) {
        const int k = it / pieces, pc = it - k * pieces;
        const int64_t off = (int64_t)pc * kPieceBytes;
        const int nv = (int)(((rb - off < kPieceBytes) ? rb - off : kPieceBytes) >> 4);
        const char* src = a.x_full + (int64_t)a.tok_in[s_src[k]] * a.ldx_b + off;
        char* dst = a.H_next + (int64_t)(base + k) * a.ldn_b + off;
        uint4 r[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) { const int v = q * 32 + lane; if (v < nv) r[q] = ld_cg_v4(src + ((int64_t)v << 4)); }
#pragma unroll
        for (int q = 0; q < 8; ++q) { const int v = q * 32 + lane; if (v < nv) st_v4(dst + ((int64_t)v << 4), r[q]); }
    }
}

static int rows_grid(int64_t n, int wpb) {
    int64_t blocks = (n + wpb - 1) / wpb;
    int64_t cap = (int64_t)sm_count() * 8;     // 8 CTAs of 256 threads fill an SM
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

}  // namespace dash

using namespace dash;

extern "C" int dash_delta_norm(const void* U, const void* H, int64_t n, int d, int64_t ldU, int64_t ldH,
                               dash_dtype dt, dash_norm_mode mode, float eps, float* r_out,
                               void* Hres_out, int64_t ldHres, const int32_t* res_index,
                               const dash_threshold* fused, const int32_t* n_dev, void* stream) {
    if (n < 0 || d <= 0 || (d % 8) != 0) return DASH_ERR_INVALID_ARG;
    if (dt != DASH_F32 && dt != DASH_BF16) return DASH_ERR_INVALID_ARG;
    if (mode != DASH_NORM_REL && mode != DASH_NORM_ABS) return DASH_ERR_INVALID_ARG;
    if (n == 0) return DASH_OK;
    const int es = (dt == DASH_BF16) ? 2 : 4;
    const bool need_h = (mode == DASH_NORM_REL) || Hres_out;
    if (!U || !r_out || (need_h && !H)) return DASH_ERR_INVALID_ARG;
    if (ldU < d || (need_h && ldH < d) || (Hres_out && ldHres < d)) return DASH_ERR_INVALID_ARG;
    if (!aligned16(U) || (need_h && !aligned16(H)) || (Hres_out && !aligned16(Hres_out))) return DASH_ERR_INVALID_ARG;
    if ((ldU * es) % 16 || (need_h && (ldH * es) % 16) || (Hres_out && (ldHres * es) % 16)) return DASH_ERR_INVALID_ARG;
    if (n > 0x7fffffffLL) return DASH_ERR_UNSUPPORTED;
    FusedThreshold ft = {0.f, 0, 0, nullptr, 0, nullptr};
    if (fused) {
        if (!fused->cu_seqlens || fused->S < 1 || !fused->mask_out || fused->keep_first < 0 || fused->keep_last < 0)
            return DASH_ERR_INVALID_ARG;
        ft = {fused->tau, fused->keep_first, fused->keep_last, fused->cu_seqlens, fused->S, fused->mask_out};
    }
    const int nvec = d * es / 16;
    cudaStream_t st = (cudaStream_t)stream;
    const int grid = rows_grid(n, 8);
    // does the residual output overlap an input?  (H~ written over H is allowed when row t goes to row t)
    auto overlaps = [&](const void* a, int64_t lda) {
        if (!Hres_out || !a) return false;
        const char *a0 = (const char*)a, *a1 = a0 + n * lda * es, *o0 = (const char*)Hres_out, *o1 = o0 + n * ldHres * es;
        return a0 < o1 && o0 < a1;
    };
    const int aliased = (overlaps(U, ldU) || overlaps(H, ldH)) ? 1 : 0;
    if (aliased && res_index) return DASH_ERR_INVALID_ARG;      // an indexed destination inside an input would be read after it was written
    if (dt == DASH_BF16)
        delta_norm_kernel<true><<<grid, 256, 0, st>>>((const char*)U, (const char*)H, n, nvec, ldU * es, ldH * es, (int)mode, eps,
                                                      r_out, (char*)Hres_out, ldHres * es, res_index, ft, n_dev, aliased);
    else
        delta_norm_kernel<false><<<grid, 256, 0, st>>>((const char*)U, (const char*)H, n, nvec, ldU * es, ldH * es, (int)mode, eps,
                                                       r_out, (char*)Hres_out, ldHres * es, res_index, ft, n_dev, aliased);
    DASH_CUDA_TRY(cudaGetLastError());
    return DASH_OK;
}

extern "C" int dash_select(const float* r, int64_t n, const int32_t* cu_seqlens, int S, dash_sel_mode mode, float tau,
                           const int32_t* keep_counts, int keep_first, int keep_last, uint8_t* mask_out, void* stream) {
    if (n < 0 || S < 1 || !cu_seqlens || keep_first < 0 || keep_last < 0) return DASH_ERR_INVALID_ARG;
    if (mode < DASH_SEL_THRESHOLD || mode > DASH_SEL_KEEP_COUNT_HALT_HIGH) return DASH_ERR_INVALID_ARG;
    const int halt_high = (mode == DASH_SEL_THRESHOLD_HALT_HIGH || mode == DASH_SEL_KEEP_COUNT_HALT_HIGH) ? 1 : 0;
    if (n > 0x7fffffffLL) return DASH_ERR_UNSUPPORTED;
    if (n == 0) return DASH_OK;
    if (!r || !mask_out) return DASH_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (mode == DASH_SEL_THRESHOLD || mode == DASH_SEL_THRESHOLD_HALT_HIGH) {
        int grid = (int)((n + 255) / 256);
        int cap = sm_count() * 8;
        if (grid > cap) grid = cap;
        select_threshold_kernel<<<grid, 256, 0, st>>>(r, n, cu_seqlens, S, tau, keep_first, keep_last, mask_out, halt_high);
    } else {
        if (!keep_counts) return DASH_ERR_INVALID_ARG;
        select_keep_count_kernel<<<S, 1024, 0, st>>>(r, cu_seqlens, S, keep_counts, keep_first, keep_last, mask_out, halt_high);
    }
    DASH_CUDA_TRY(cudaGetLastError());
    return DASH_OK;
}

// keep_counts[s] from the length of sequence s as it stands on the device: the arithmetic of dash_keep_count, in fp64
__global__ void __launch_bounds__(256)
keep_counts_kernel(const int32_t* __restrict__ cu, int S, double rho, int keep_first, int keep_last, int mode, int32_t* __restrict__ out) {
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= S) return;
    const long long n = (long long)cu[s + 1] - cu[s];
    long long k;
    if (mode == 0) {
        k = (long long)floor(__dmul_rn(__dsub_rn(1.0, rho), (double)n));
    } else {
        long long n_fix = (long long)keep_first + keep_last;
        if (n_fix > n) n_fix = n;
        k = n - (long long)floor(rint(__dmul_rn(rho, (double)(n - n_fix))));      // rint: to nearest, ties to even
    }
    out[s] = (int32_t)(k < 0 ? 0 : (k > n ? n : k));
}

extern "C" int dash_keep_counts_device(const int32_t* cu_seqlens, int S, double rho, int keep_first, int keep_last, int mode,
                                       int32_t* keep_counts_out, void* stream) {
    if (!cu_seqlens || !keep_counts_out || S < 1 || !(rho >= 0.0) || !(rho < 1.0) || keep_first < 0 || keep_last < 0 || (mode != 0 && mode != 1))
        return DASH_ERR_INVALID_ARG;
    keep_counts_kernel<<<(S + 255) / 256, 256, 0, (cudaStream_t)stream>>>(cu_seqlens, S, rho, keep_first, keep_last, mode, keep_counts_out);
    return cudaGetLastError() == cudaSuccess ? DASH_OK : DASH_ERR_CUDA;
}

// Tokens per CTA.  Small tiles keep the CTAs balanced when the active rows cluster (a packed batch whose
// image blocks halt almost entirely while its text blocks stay); larger ones only bound the look-back chain.
static int compact_tile_for(int64_t n) {
    if (n <= 16384) return 32;
    if (n <= 262144) return 64;
    if (n <= 1048576) return 128;
    return 256;
}
// up to this many rows the output base of a tile is counted straight from the mask (no scratch, no look-back)
constexpr int64_t kCompactDirectMaxRows = 32768;

static size_t compact_ws_bytes(int64_t n) {
    int64_t tiles = (n + 31) / 32 + 1;
    return align_up(256 + (size_t)tiles * 8, 256);
}

// stall: test hook (see dash_testing.h) -- look-back path whatever the size, tile ticket started at 1, spin limit as given
static int compact_impl(const uint8_t* mask, int64_t n, const int32_t* cu_in, int S,
                        const dash_rows* rows, int n_rows,
                        const int32_t* pos_in, int32_t* pos_out, const int32_t* tok_in, int32_t* tok_out,
                        int32_t* idx_out, int32_t* cu_out, int32_t* n_out_dev,
                        void* ws, size_t ws_bytes, void* stream, bool stall, uint32_t spin_limit) {
    if (n < 0 || S < 1 || !cu_in || !cu_out || n_rows < 0 || n_rows > DASH_MAX_ROW_STREAMS) return DASH_ERR_INVALID_ARG;
    if (n > 0 && !mask) return DASH_ERR_INVALID_ARG;
    if (n_rows > 0 && !rows) return DASH_ERR_INVALID_ARG;
    if (n > 0x7fffffffLL) return DASH_ERR_UNSUPPORTED;
    if ((pos_out && !pos_in) || (tok_out && !tok_in)) return DASH_ERR_INVALID_ARG;
    RowStreams rs;
    rs.count = n_rows;
    for (int q = 0; q < n_rows; ++q) {
        const dash_rows& x = rows[q];
        if (!x.src || !x.dst || x.row_bytes <= 0 || (x.row_bytes % 4) || x.src_ld_bytes < x.row_bytes || x.dst_ld_bytes < x.row_bytes)
            return DASH_ERR_INVALID_ARG;
        if ((x.src_ld_bytes % 4) || (x.dst_ld_bytes % 4) || ((uintptr_t)x.src % 4) || ((uintptr_t)x.dst % 4)) return DASH_ERR_INVALID_ARG;
        rs.src[q] = (const char*)x.src; rs.dst[q] = (char*)x.dst;
        rs.row_bytes[q] = x.row_bytes; rs.src_ld[q] = x.src_ld_bytes; rs.dst_ld[q] = x.dst_ld_bytes;
        rs.vec16[q] = aligned16(x.src) && aligned16(x.dst) && !(x.row_bytes % 16) && !(x.src_ld_bytes % 16) && !(x.dst_ld_bytes % 16);
    }
    if (!ws || ((uintptr_t)ws % 256) || ws_bytes < compact_ws_bytes(n)) return DASH_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const int TILE = compact_tile_for(n);
    const int tiles = (int)((n + TILE - 1) / TILE) > 0 ? (int)((n + TILE - 1) / TILE) : 1;
    const bool direct = n <= kCompactDirectMaxRows && !stall;
    unsigned int* ticket = (unsigned int*)ws;
    unsigned long long* state = (unsigned long long*)((char*)ws + 256);
    if (!direct) DASH_CUDA_TRY(cudaMemsetAsync(ws, 0, 256 + (size_t)tiles * 8, st));
    if (stall) DASH_CUDA_TRY(cudaMemsetAsync(ws, 1, 1, st));          // ticket = 1: tile 0 is never taken, tile 1 waits for it in vain
    int* status = status_word_ptr();
    if (!status) return DASH_ERR_CUDA;
    const int mask_vec16 = aligned16(mask) ? 1 : 0;
#define DASH_LAUNCH_COMPACT(T, DIRECT)                                                                                       \
    compact_kernel<T, DIRECT><<<tiles, kCompactThreads, 0, st>>>(mask, n, cu_in, S, rs, pos_in, pos_out, tok_in, tok_out, \
                                                                 idx_out, cu_out, n_out_dev, state, ticket, status, mask_vec16, spin_limit)
    if (direct) {
        switch (TILE) {
            case 256: DASH_LAUNCH_COMPACT(256, true); break;
            case 128: DASH_LAUNCH_COMPACT(128, true); break;
            case 64: DASH_LAUNCH_COMPACT(64, true); break;
            default: DASH_LAUNCH_COMPACT(32, true); break;
        }
    } else {
        switch (TILE) {
            case 256: DASH_LAUNCH_COMPACT(256, false); break;
            case 128: DASH_LAUNCH_COMPACT(128, false); break;
            case 64: DASH_LAUNCH_COMPACT(64, false); break;
            default: DASH_LAUNCH_COMPACT(32, false); break;
        }
    }
#undef DASH_LAUNCH_COMPACT
    DASH_CUDA_TRY(cudaGetLastError());
    return DASH_OK;
}

extern "C" int dash_compact(const uint8_t* mask, int64_t n, const int32_t* cu_in, int S,
                            const dash_rows* rows, int n_rows,
                            const int32_t* pos_in, int32_t* pos_out, const int32_t* tok_in, int32_t* tok_out,
                            int32_t* idx_out, int32_t* cu_out, int32_t* n_out_dev,
                            void* ws, size_t ws_bytes, void* stream) {
    return compact_impl(mask, n, cu_in, S, rows, n_rows, pos_in, pos_out, tok_in, tok_out, idx_out, cu_out, n_out_dev, ws, ws_bytes, stream, false,
                        kSpinLimit);
}

extern "C" int dash_testing_compact_stalled(const uint8_t* mask, int64_t n, const int32_t* cu_in, int S, int32_t* idx_out, int32_t* cu_out,
                                            int32_t* n_out_dev, uint32_t spin_limit, void* ws, size_t ws_bytes, void* stream) {
    if (n < 64 || spin_limit < 1 || spin_limit > kSpinLimit) return DASH_ERR_INVALID_ARG;
    return compact_impl(mask, n, cu_in, S, nullptr, 0, nullptr, nullptr, nullptr, nullptr, idx_out, cu_out, n_out_dev, ws, ws_bytes, stream, true,
                        spin_limit);
}

extern "C" int dash_scatter(const void* src, int64_t n, int64_t row_bytes, int64_t src_ld_bytes,
                            const int32_t* tok_index, const uint8_t* sel, int which, const int32_t* n_dev,
                            void* dst_full, int64_t dst_ld_bytes, void* stream) {
    if (n < 0 || row_bytes <= 0 || (row_bytes % 4) || which < 0 || which > 2) return DASH_ERR_INVALID_ARG;
    if (n == 0) return DASH_OK;
    if (!src || !dst_full || (which != 2 && !sel)) return DASH_ERR_INVALID_ARG;
    if (src_ld_bytes < row_bytes || dst_ld_bytes < row_bytes || (src_ld_bytes % 4) || (dst_ld_bytes % 4)) return DASH_ERR_INVALID_ARG;
    if (((uintptr_t)src % 4) || ((uintptr_t)dst_full % 4)) return DASH_ERR_INVALID_ARG;
    int vec16 = aligned16(src) && aligned16(dst_full) && !(row_bytes % 16) && !(src_ld_bytes % 16) && !(dst_ld_bytes % 16);
    scatter_kernel<<<rows_grid(n, 8), 256, 0, (cudaStream_t)stream>>>((const char*)src, n, row_bytes, src_ld_bytes, tok_index, sel, which,
                                                                       n_dev, (char*)dst_full, dst_ld_bytes, vec16);
    DASH_CUDA_TRY(cudaGetLastError());
    return DASH_OK;
}

// ---------------------------------------------------------------------------
// Compaction for callers that may not allocate: the look-back scratch (ticket word
// + one 64-bit state per 32-token tile) is a fixed array in the library image.
// ---------------------------------------------------------------------------
constexpr size_t kStaticScratchBytes = 256 + (size_t)(DASH_COMPACT_STATIC_MAX_ROWS / 32 + 1) * 8;
static __device__ __align__(256) unsigned char g_compact_scratch[(kStaticScratchBytes + 255) / 256 * 256];

// Host code cannot use the array's name as a pointer (on the host it is only a handle for
// the runtime): ask for its device address once per device, with that device current.
static void* compact_scratch_ptr() {
    static std::atomic<void*> ptrs[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    void* p = ptrs[dev].load(std::memory_order_acquire);
    if (!p) {
        if (cudaGetSymbolAddress((void**)&p, g_compact_scratch) != cudaSuccess) return nullptr;
        ptrs[dev].store(p, std::memory_order_release);      // two threads that race here store the same address
    }
    return p;
}

extern "C" int dash_compact_static(const uint8_t* mask, int64_t n, const int32_t* cu_in, int S,
                                   const dash_rows* rows, int n_rows,
                                   const int32_t* pos_in, int32_t* pos_out, const int32_t* tok_in, int32_t* tok_out,
                                   int32_t* idx_out, int32_t* cu_out, int32_t* n_out_dev, void* stream) {
    if (n > DASH_COMPACT_STATIC_MAX_ROWS) return DASH_ERR_TOO_LARGE;
    void* scratch = compact_scratch_ptr();
    if (!scratch) return DASH_ERR_CUDA;
    // same kernel and launch as dash_compact; it clears the part of the scratch it uses first
    return dash_compact(mask, n, cu_in, S, rows, n_rows, pos_in, pos_out, tok_in, tok_out, idx_out, cu_out, n_out_dev,
                        scratch, sizeof(g_compact_scratch), stream);
}

namespace dash {

// r (and, with ft.mask_out set, the threshold decision) from the per-row partial sums of the output-projection epilogue; with
// inv_rms_out set also the row factor of the next RMSNorm, 1 / sqrt(mean((h+u)^2) + rms_eps)
__global__ void __launch_bounds__(256)
sums_to_score_kernel(const float4* __restrict__ sums, int n_sum_tiles, int64_t n, int mode, float eps, float* __restrict__ r_out,
                     FusedThreshold ft, const int32_t* __restrict__ n_dev, float* __restrict__ inv_rms_out, float inv_d, float rms_eps) {
    if (n_dev) { int64_t nd = *n_dev; if (nd < n) n = nd; }
    for (int64_t row = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; row < n; row += (int64_t)gridDim.x * blockDim.x) {
        float su = 0.f, sh = 0.f;
        float st2 = 0.f;
        for (int i = 0; i < n_sum_tiles; ++i) { const float4 p2 = sums[row * n_sum_tiles + i]; su += p2.x; sh += p2.y; st2 += p2.z; }
        if (inv_rms_out) inv_rms_out[row] = rsqrtf(st2 * inv_d + rms_eps);
        const float num = sqrtf(su);
        const float r = (mode == DASH_NORM_ABS) ? num : num / fmaxf(sqrtf(sh), eps);
        r_out[row] = r;
        if (ft.mask_out) {
            const int s = find_seq(ft.cu, ft.S, (int)row);
            const int local = (int)row - ft.cu[s], len = ft.cu[s + 1] - ft.cu[s];
            const bool prot = (local < ft.keep_first) || (local >= len - ft.keep_last);
            ft.mask_out[row] = (prot || !(r < ft.tau)) ? 1 : 0;
        }
    }
}

int launch_sums_to_score(const float4* sums, int n_sum_tiles, int64_t n, dash_norm_mode mode, float eps, float* r_out, const dash_threshold* fused,
                         const int32_t* n_dev, float* inv_rms_out, int d, float rms_eps, cudaStream_t st) {
    FusedThreshold ft = {0.f, 0, 0, nullptr, 0, nullptr};
    if (fused) ft = {fused->tau, fused->keep_first, fused->keep_last, fused->cu_seqlens, fused->S, fused->mask_out};
    int64_t blocks = (n + 255) / 256, cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    sums_to_score_kernel<<<(int)blocks, 256, 0, st>>>(sums, n_sum_tiles, n, (int)mode, eps, r_out, ft, n_dev, inv_rms_out, 1.0f / d, rms_eps);
    return cudaGetLastError() == cudaSuccess ? DASH_OK : DASH_ERR_CUDA;
}

// Fused tail of the block step (see delta_tail_kernel).  Preconditions checked by the caller: threshold rule, every row
// scattered, 16-byte aligned rows.  ws: the compaction workspace (ticket + one state word per 32-token tile); ws_is_clear: the
// caller has already zeroed it on this stream with clear_tail_ws (ahead of the kernels in front, so that this launch follows a
// kernel directly and may start while that one drains).
static size_t tail_ws_clear_bytes(int64_t n) { return 256 + (size_t)((n + 31) / 32 > 0 ? (n + 31) / 32 : 1) * 8; }
int clear_tail_ws(void* ws, size_t ws_bytes, int64_t n, cudaStream_t st) {
    if (!ws || ((uintptr_t)ws % 256) || ws_bytes < compact_ws_bytes(n)) return DASH_ERR_WORKSPACE;
    DASH_CUDA_TRY(cudaMemsetAsync(ws, 0, tail_ws_clear_bytes(n), st));
    return DASH_OK;
}
int launch_delta_tail(const void* U, const void* H, const uint8_t* mask_in, const float4* sums, int n_sum_tiles, int64_t n, int d, dash_dtype dt, dash_norm_mode mode, float eps, float tau,
                      int keep_first, int keep_last, const int32_t* cu_in, int S, const int32_t* tok_in, const int32_t* pos_in,
                      void* x_full, void* H_next, float* r_out, uint8_t* mask_out, int32_t* tok_next, int32_t* pos_next,
                      int32_t* cu_next, int32_t* n_next, void* ws, size_t ws_bytes, bool ws_is_clear, cudaStream_t st, float* inv_next,
                      float rms_eps) {
    const int es = dt == DASH_BF16 ? 2 : 4;
    if (!ws || ((uintptr_t)ws % 256) || ws_bytes < compact_ws_bytes(n)) return DASH_ERR_WORKSPACE;
    const int tiles = (int)((n + 31) / 32) > 0 ? (int)((n + 31) / 32) : 1;
    if (!ws_is_clear) DASH_CUDA_TRY(cudaMemsetAsync(ws, 0, tail_ws_clear_bytes(n), st));
    TailArgs a;
    a.mask_in = mask_in; a.sums = sums; a.n_sum_tiles = n_sum_tiles;
    a.U = (const char*)U; a.H = (const char*)H; a.ldU_b = a.ldH_b = (int64_t)d * es; a.nvec = d * es / 16; a.mode = (int)mode; a.eps = eps;
    a.tau = tau; a.keep_first = keep_first; a.keep_last = keep_last; a.cu_in = cu_in; a.S = S; a.tok_in = tok_in; a.pos_in = pos_in;
    a.x_full = (char*)x_full; a.ldx_b = (int64_t)d * es; a.H_next = (char*)H_next; a.ldn_b = (int64_t)d * es;
    a.r_out = r_out; a.mask_out = mask_out; a.tok_next = tok_next; a.pos_next = pos_next; a.cu_next = cu_next; a.n_next = n_next;
    a.ticket = (unsigned int*)ws; a.tile_state = (unsigned long long*)((char*)ws + 256);
    a.inv_next = inv_next; a.inv_d = 1.0f / (float)d; a.rms_eps = rms_eps;
    a.status = status_word_ptr();
    if (!a.status) return DASH_ERR_CUDA;
    if (dt == DASH_BF16) DASH_CUDA_TRY(launch_pdl(delta_tail_kernel<true>, tiles, kCompactThreads, 0, st, a, n));
    else DASH_CUDA_TRY(launch_pdl(delta_tail_kernel<false>, tiles, kCompactThreads, 0, st, a, n));
    return DASH_OK;
}
size_t compact_ws_bytes_pub(int64_t n) { return compact_ws_bytes(n); }
}  // namespace dash

// dash_layer_step: the body of the prefill loop for one block (without the FFN),
// on the packed active tokens: RMSNorm -> QKV projection -> rotary embedding ->
// causal attention -> output projection -> delta score / residual / halting rule
// -> scatter of the updated states -> compaction of the tokens that stay active.
// Every step runs in this library's own kernels; the projections are the tcgen05 GEMMs of gemm.cu -- with the norm's row
// factor, the rotary embedding, the residual and the score's row sums on their accumulators where the shapes allow it (bf16,
// whole 256-column tiles), as plain GEMMs between passes of their own otherwise.  One stream, no host synchronisation.
#include <math.h>

#include "common.cuh"
#include "gemm.cuh"

namespace dash {

// y = x / sqrt(mean(x^2) + eps) * w ; one warp per row, second read served by L1/L2
template <bool BF16>
__global__ void __launch_bounds__(256)
rmsnorm_kernel(const char* __restrict__ X, int64_t ldx_b, const char* __restrict__ W, char* __restrict__ Y, int64_t ldy_b,
               int64_t n, int nvec, float inv_d, float eps, const int32_t* __restrict__ n_dev) {
    const int lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
    if (n_dev) { int64_t nd = *n_dev; if (nd < n) n = nd; }
    for (int64_t row = (int64_t)blockIdx.x * wpb + (threadIdx.x >> 5); row < n; row += (int64_t)gridDim.x * wpb) {
        const uint4* x = reinterpret_cast<const uint4*>(X + row * ldx_b);
        const uint4* w = reinterpret_cast<const uint4*>(W);
        uint4* y = reinterpret_cast<uint4*>(Y + row * ldy_b);
        float ss = 0.f;
        for (int v = lane; v < nvec; v += 32) {
            uint4 a = x[v];
            if (BF16) {
                float f[8] = {bf16lo(a.x), bf16hi(a.x), bf16lo(a.y), bf16hi(a.y), bf16lo(a.z), bf16hi(a.z), bf16lo(a.w), bf16hi(a.w)};
#pragma unroll
                for (int e = 0; e < 8; ++e) ss += f[e] * f[e];
            } else {
                float f[4] = {__uint_as_float(a.x), __uint_as_float(a.y), __uint_as_float(a.z), __uint_as_float(a.w)};
#pragma unroll
                for (int e = 0; e < 4; ++e) ss += f[e] * f[e];
            }
        }
        ss = warp_sum(ss);
        const float rs = rsqrtf(ss * inv_d + eps);
        for (int v = lane; v < nvec; v += 32) {
            uint4 a = x[v], g = w[v], o;
            if (BF16) {
                o.x = pack_bf16(bf16lo(a.x) * rs * bf16lo(g.x), bf16hi(a.x) * rs * bf16hi(g.x));
                o.y = pack_bf16(bf16lo(a.y) * rs * bf16lo(g.y), bf16hi(a.y) * rs * bf16hi(g.y));
                o.z = pack_bf16(bf16lo(a.z) * rs * bf16lo(g.z), bf16hi(a.z) * rs * bf16hi(g.z));
                o.w = pack_bf16(bf16lo(a.w) * rs * bf16lo(g.w), bf16hi(a.w) * rs * bf16hi(g.w));
            } else {
                o.x = __float_as_uint(__uint_as_float(a.x) * rs * __uint_as_float(g.x));
                o.y = __float_as_uint(__uint_as_float(a.y) * rs * __uint_as_float(g.y));
                o.z = __float_as_uint(__uint_as_float(a.z) * rs * __uint_as_float(g.z));
                o.w = __float_as_uint(__uint_as_float(a.w) * rs * __uint_as_float(g.w));
            }
            y[v] = o;
        }
    }
}

// Rotary embedding in place on the first `heads` heads of every row of the fused
// QKV buffer: pair (i, i + D/2) rotated by pos * inv_freq[i].  One warp per token;
// the angles are formed and reduced in fp64 (positions reach 1e5 rad at i = 0).
struct RopeFreq { double inv_freq[64]; };

template <bool BF16, int D>
__global__ void __launch_bounds__(256)
rope_kernel(char* __restrict__ X, int64_t ldx_b, const int32_t* __restrict__ pos, int64_t n, int heads, RopeFreq fr,
            const int32_t* __restrict__ n_dev) {
    constexpr int HALF = D / 2;
    __shared__ float s_cos[8][HALF], s_sin[8][HALF];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, wpb = blockDim.x >> 5;
    if (n_dev) { int64_t nd = *n_dev; if (nd < n) n = nd; }
    constexpr int ES = BF16 ? 2 : 4;
    constexpr int EPV = 16 / ES;                 // elements per 16-byte vector
    constexpr int VPH = HALF / EPV;              // vectors per half head
    for (int64_t t = (int64_t)blockIdx.x * wpb + w; t < n; t += (int64_t)gridDim.x * wpb) {
        const double ps = (double)pos[t];
        for (int i = lane; i < HALF; i += 32) {
            double sn, cs;
            sincos(ps * fr.inv_freq[i], &sn, &cs);
            s_cos[w][i] = (float)cs; s_sin[w][i] = (float)sn;
        }
        __syncwarp();
        char* row = X + t * ldx_b;
        for (int q = lane; q < heads * VPH; q += 32) {
            const int hd = q / VPH, v = q % VPH;
            uint4* p1 = reinterpret_cast<uint4*>(row + (int64_t)hd * D * ES) + v;
            uint4* p2 = p1 + VPH;
            uint4 a = *p1, b = *p2, oa, ob;
            const float* c = &s_cos[w][v * EPV];
            const float* s = &s_sin[w][v * EPV];
            if (BF16) {
                float x1[8] = {bf16lo(a.x), bf16hi(a.x), bf16lo(a.y), bf16hi(a.y), bf16lo(a.z), bf16hi(a.z), bf16lo(a.w), bf16hi(a.w)};
                float x2[8] = {bf16lo(b.x), bf16hi(b.x), bf16lo(b.y), bf16hi(b.y), bf16lo(b.z), bf16hi(b.z), bf16lo(b.w), bf16hi(b.w)};
                float y1[8], y2[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) { y1[e] = x1[e] * c[e] - x2[e] * s[e]; y2[e] = x2[e] * c[e] + x1[e] * s[e]; }
                oa = make_uint4(pack_bf16(y1[0], y1[1]), pack_bf16(y1[2], y1[3]), pack_bf16(y1[4], y1[5]), pack_bf16(y1[6], y1[7]));
                ob = make_uint4(pack_bf16(y2[0], y2[1]), pack_bf16(y2[2], y2[3]), pack_bf16(y2[4], y2[5]), pack_bf16(y2[6], y2[7]));
            } else {
                float x1[4] = {__uint_as_float(a.x), __uint_as_float(a.y), __uint_as_float(a.z), __uint_as_float(a.w)};
                float x2[4] = {__uint_as_float(b.x), __uint_as_float(b.y), __uint_as_float(b.z), __uint_as_float(b.w)};
                float y1[4], y2[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) { y1[e] = x1[e] * c[e] - x2[e] * s[e]; y2[e] = x2[e] * c[e] + x1[e] * s[e]; }
                oa = make_uint4(__float_as_uint(y1[0]), __float_as_uint(y1[1]), __float_as_uint(y1[2]), __float_as_uint(y1[3]));
                ob = make_uint4(__float_as_uint(y2[0]), __float_as_uint(y2[1]), __float_as_uint(y2[2]), __float_as_uint(y2[3]));
            }
            *p1 = oa; *p2 = ob;
        }
        __syncwarp();
    }
}

int launch_sums_to_score(const float4* sums, int n_sum_tiles, int64_t n, dash_norm_mode mode, float eps, float* r_out, const dash_threshold* fused,
                         const int32_t* n_dev, float* inv_rms_out, int d, float rms_eps, cudaStream_t st);
int launch_delta_tail(const void* U, const void* H, const uint8_t* mask_in, const float4* sums, int n_sum_tiles, int64_t n, int d, dash_dtype dt, dash_norm_mode mode, float eps, float tau,
                      int keep_first, int keep_last, const int32_t* cu_in, int S, const int32_t* tok_in, const int32_t* pos_in,
                      void* x_full, void* H_next, float* r_out, uint8_t* mask_out, int32_t* tok_next, int32_t* pos_next,
                      int32_t* cu_next, int32_t* n_next, void* ws, size_t ws_bytes, bool ws_is_clear, cudaStream_t st, float* inv_next,
                      float rms_eps);
int clear_tail_ws(void* ws, size_t ws_bytes, int64_t n, cudaStream_t st);
int attention_plan(const int32_t* cu_seqlens, int S, int64_t n, int Hq, void* ws, size_t ws_bytes, cudaStream_t st);
int attention_planned(const void* Q, const void* K, const void* V, void* O, float* lse, int64_t ldq, int64_t ldk, int64_t ldv, int64_t ldo,
                      const int32_t* cu_seqlens, int S, int64_t n, int64_t max_seqlen, int Hq, int Hkv, int D, float scale, dash_dtype dt,
                      void* ws, size_t ws_bytes, cudaStream_t st);

// Room for the bf16 copies of the operands of a projection on fp32 tensors
struct ConvScratch { char* a; size_t a_bytes; char* w; size_t w_bytes; };
static size_t conv_a_bytes(int64_t n, int64_t k_max) { return align_up((size_t)n * align_up((size_t)k_max, 8) * 2, 256); }
static size_t conv_w_bytes(int64_t k, int64_t n_cols) { return align_up((size_t)k * align_up((size_t)n_cols, 8) * 2, 256); }

// C = A W (plain).  bf16: the GEMM of gemm.cu as it is.  fp32: its operands are rounded to bf16 copies first (what the
// attention kernel does with Q, K, V), the product accumulates in fp32 and is stored as fp32.
static int project(dash_dtype dt, const void* A, int64_t lda, const void* W, int64_t ldw, void* C, int64_t ldc, int64_t n, int64_t N, int64_t K,
                   const int32_t* n_dev, const ConvScratch& cs, cudaStream_t st) {
    GemmEpilogue e;
    if (dt == DASH_BF16) return gemm_bf16(GEMM_PLAIN, A, lda, W, ldw, C, ldc, n, N, K, e, n_dev, st);
    if ((K % 8) || (N % 4)) return DASH_ERR_UNSUPPORTED;
    const int64_t lda_b = K, ldw_b = (int64_t)align_up((size_t)N, 8);
    if ((size_t)n * lda_b * 2 > cs.a_bytes || (size_t)K * ldw_b * 2 > cs.w_bytes) return DASH_ERR_WORKSPACE;
    int rc;
    if ((rc = launch_f32_to_bf16((const float*)A, lda, cs.a, lda_b, n, K, st)) != DASH_OK) return rc;
    if ((rc = launch_f32_to_bf16((const float*)W, ldw, cs.w, ldw_b, K, N, st)) != DASH_OK) return rc;
    return gemm_bf16(GEMM_PLAIN, cs.a, lda_b, cs.w, ldw_b, C, ldc, n, N, K, e, n_dev, st, true);
}

static int rows_grid8(int64_t n) {
    int64_t blocks = (n + 7) / 8, cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    return (int)(blocks < 1 ? 1 : blocks);
}


// act[t, j] = silu(GU[t, j]) * GU[t, m + j]   (gated feed-forward; silu(z) = z / (1 + exp(-z))), 8 (bf16) or 4 (fp32) columns per thread
template <bool BF16>
__global__ void __launch_bounds__(256)
swiglu_kernel(const char* __restrict__ GU, int64_t ldgu_b, char* __restrict__ ACT, int64_t lda_b, int64_t n, int m,
              const int32_t* __restrict__ n_dev) {
    constexpr int ES = BF16 ? 2 : 4, EPV = 16 / ES;
    if (n_dev) { int64_t nd = *n_dev; if (nd < n) n = nd; }
    const int vpr = m / EPV;                              // 16-byte vectors per output row
    const int64_t total = n * vpr;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t t = i / vpr;
        const int v = (int)(i - t * vpr);
        const uint4 g = ld_nc_v4(GU + t * ldgu_b + ((int64_t)v << 4));
        const uint4 u = ld_nc_v4(GU + t * ldgu_b + (int64_t)m * ES + ((int64_t)v << 4));
        auto act = [](float a, float b) { return a / (1.0f + __expf(-a)) * b; };
        uint4 o;
        if (BF16) {
            o.x = pack_bf16(act(bf16lo(g.x), bf16lo(u.x)), act(bf16hi(g.x), bf16hi(u.x)));
            o.y = pack_bf16(act(bf16lo(g.y), bf16lo(u.y)), act(bf16hi(g.y), bf16hi(u.y)));
            o.z = pack_bf16(act(bf16lo(g.z), bf16lo(u.z)), act(bf16hi(g.z), bf16hi(u.z)));
            o.w = pack_bf16(act(bf16lo(g.w), bf16lo(u.w)), act(bf16hi(g.w), bf16hi(u.w)));
        } else {
            o.x = __float_as_uint(act(__uint_as_float(g.x), __uint_as_float(u.x)));
            o.y = __float_as_uint(act(__uint_as_float(g.y), __uint_as_float(u.y)));
            o.z = __float_as_uint(act(__uint_as_float(g.z), __uint_as_float(u.z)));
            o.w = __float_as_uint(act(__uint_as_float(g.w), __uint_as_float(u.w)));
        }
        st_v4(ACT + t * lda_b + ((int64_t)v << 4), o);
    }
}

// W_out[i, :] = w[i] * W[i, :]: the norm's weight folded into the projection behind it (one 16-byte vector per thread)
template <bool BF16>
__global__ void __launch_bounds__(256)
fold_norm_weight_kernel(const char* __restrict__ W, int64_t ldw_b, const char* __restrict__ w, char* __restrict__ Wout, int64_t ldo_b, int d, int vpr) {
    const int64_t total = (int64_t)d * vpr;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int row = (int)(i / vpr), v = (int)(i - (int64_t)row * vpr);
        const uint4 a = *reinterpret_cast<const uint4*>(W + row * ldw_b + ((int64_t)v << 4));
        uint4 o;
        if (BF16) {
            const float g = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(w)[row]);
            o.x = pack_bf16(bf16lo(a.x) * g, bf16hi(a.x) * g); o.y = pack_bf16(bf16lo(a.y) * g, bf16hi(a.y) * g);
            o.z = pack_bf16(bf16lo(a.z) * g, bf16hi(a.z) * g); o.w = pack_bf16(bf16lo(a.w) * g, bf16hi(a.w) * g);
        } else {
            const float g = reinterpret_cast<const float*>(w)[row];
            o.x = __float_as_uint(__uint_as_float(a.x) * g); o.y = __float_as_uint(__uint_as_float(a.y) * g);
            o.z = __float_as_uint(__uint_as_float(a.z) * g); o.w = __float_as_uint(__uint_as_float(a.w) * g);
        }
        *reinterpret_cast<uint4*>(Wout + row * ldo_b + ((int64_t)v << 4)) = o;
    }
}

static bool cfg_ok(const dash_layer_cfg* c) {
    if (!c || c->d <= 0 || c->Hq < 1 || c->Hkv < 1 || (c->D != 64 && c->D != 128)) return false;
    if ((c->d % 8) || (c->Hq % c->Hkv)) return false;
    if (c->dt != DASH_F32 && c->dt != DASH_BF16) return false;
    if (!c->Wqkv || !c->Wo || (!c->rms_weight && !c->rms_folded)) return false;
    if (c->rms_folded != 0 && c->rms_folded != 1) return false;
    if (c->sel_mode < DASH_SEL_THRESHOLD || c->sel_mode > DASH_SEL_KEEP_COUNT_HALT_HIGH) return false;
    if ((c->sel_mode == DASH_SEL_KEEP_COUNT || c->sel_mode == DASH_SEL_KEEP_COUNT_HALT_HIGH) && !c->keep_counts) return false;
    if (c->keep_first < 0 || c->keep_last < 0) return false;
    if (c->scatter_which != 0 && c->scatter_which != 2) return false;
    if (!(c->rope_base > 0.0)) return false;
    if ((c->k_cache == nullptr) != (c->v_cache == nullptr)) return false;
    if (c->rope_table && (c->rope_table_len < 1 || ((uintptr_t)c->rope_table % 8))) return false;
    return true;
}

}  // namespace dash

using namespace dash;

extern "C" int dash_fold_norm_weight(const void* W, const void* rms_weight, int d, int64_t N, int64_t ldw, dash_dtype dt,
                                     void* W_out, int64_t ldo, void* stream) {
    if (dt != DASH_F32 && dt != DASH_BF16) return DASH_ERR_INVALID_ARG;
    const int es = dt == DASH_BF16 ? 2 : 4, epv = 16 / es;
    if (!W || !rms_weight || !W_out || d < 1 || N < 1 || (N % epv) || ldw < N || ldo < N) return DASH_ERR_INVALID_ARG;
    if (!aligned16(W) || !aligned16(W_out) || (ldw * es) % 16 || (ldo * es) % 16 || ((uintptr_t)rms_weight % es)) return DASH_ERR_INVALID_ARG;
    const int64_t vpr = N / epv;
    if (vpr > 0x7fffffffLL) return DASH_ERR_UNSUPPORTED;
    int64_t blocks = ((int64_t)d * vpr + 255) / 256, cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    cudaStream_t st = (cudaStream_t)stream;
    if (dt == DASH_BF16) fold_norm_weight_kernel<true><<<(int)blocks, 256, 0, st>>>((const char*)W, ldw * es, (const char*)rms_weight, (char*)W_out, ldo * es, d, (int)vpr);
    else fold_norm_weight_kernel<false><<<(int)blocks, 256, 0, st>>>((const char*)W, ldw * es, (const char*)rms_weight, (char*)W_out, ldo * es, d, (int)vpr);
    DASH_CUDA_TRY(cudaGetLastError());
    return DASH_OK;
}

extern "C" int dash_rope_table(double rope_base, int D, int64_t n_pos, void* table, void* stream) {
    if (!table || ((uintptr_t)table % 8) || n_pos < 1 || n_pos > 0x7fffffffLL || !(rope_base > 0.0) || (D != 64 && D != 128)) return DASH_ERR_INVALID_ARG;
    return launch_row_prep(nullptr, n_pos, D, rope_base, (float2*)table, nullptr, 0, 0, 0.f, nullptr, nullptr, (cudaStream_t)stream);
}

extern "C" int dash_layer_workspace(const dash_layer_cfg* cfg, int64_t n, int S, dash_layer_ws_layout* out) {
    if (!cfg_ok(cfg) || n < 0 || S < 1 || !out) return DASH_ERR_INVALID_ARG;
    const size_t es = cfg->dt == DASH_BF16 ? 2 : 4;
    const size_t nq = (size_t)(cfg->Hq + 2 * cfg->Hkv) * cfg->D;
    size_t off = 0;
    out->Hn = off;  off += align_up((size_t)n * cfg->d * es, 256);
    out->QKV = off; off += align_up((size_t)n * nq * es, 256);
    out->O = off;   off += align_up((size_t)n * cfg->Hq * cfg->D * es, 256);
    out->U = off;   off += align_up((size_t)n * cfg->d * es, 256);
    out->Ht = off;  off += align_up((size_t)n * cfg->d * es, 256);
    out->scratch = off;                    // fp32 tensors: bf16 copies of a projection's operands (activations, then weights)
    if (cfg->dt == DASH_F32) {
        const int64_t hd = (int64_t)cfg->Hq * cfg->D;
        off += conv_a_bytes(n, cfg->d > hd ? cfg->d : hd);
        off += conv_w_bytes(cfg->d, (int64_t)nq > cfg->d ? (int64_t)nq : cfg->d) > conv_w_bytes(hd, cfg->d) ? conv_w_bytes(cfg->d, (int64_t)nq > cfg->d ? (int64_t)nq : cfg->d) : conv_w_bytes(hd, cfg->d);
    }
    off += align_up(dash_workspace_bytes(DASH_WS_COMPACT, n, S, 0, 0, 0, cfg->dt), 256);
    off += align_up(dash_workspace_bytes(DASH_WS_ATTENTION, n, S, cfg->Hq, cfg->Hkv, cfg->D, cfg->dt), 256);
    off += align_up((size_t)n * (cfg->D / 2) * sizeof(float2), 256);              // (cos, sin) of every row for the QKV epilogue
    off += align_up((size_t)n * ((cfg->d + 255) / 256) * sizeof(float4), 256);    // per-row partial sums of the output-projection epilogue
    off += 2 * align_up((size_t)n * sizeof(float), 256);                          // row factors of the two folded norms
    out->total = off;
    return DASH_OK;
}

namespace dash {

struct StepWs {
    dash_layer_ws_layout L;
    char *Hn, *QKV, *O, *U, *Ht, *compact_ws, *attn_ws;
    ConvScratch conv;
    size_t compact_bytes, attn_bytes;
    float2* rope_tab;
    float4* sums;
    float *inv_rms, *inv_rms2;
};

static int carve_ws(const dash_layer_cfg* cfg, int64_t n, int S, void* ws, StepWs* out) {
    int rc = dash_layer_workspace(cfg, n, S, &out->L);
    if (rc != DASH_OK) return rc;
    char* w = (char*)ws;
    out->Hn = w + out->L.Hn; out->QKV = w + out->L.QKV; out->O = w + out->L.O; out->U = w + out->L.U; out->Ht = w + out->L.Ht;
    out->conv = {nullptr, 0, nullptr, 0};
    char* after = w + out->L.scratch;
    if (cfg->dt == DASH_F32) {
        const int64_t hd = (int64_t)cfg->Hq * cfg->D, nq = (int64_t)(cfg->Hq + 2 * cfg->Hkv) * cfg->D;
        const size_t ab = conv_a_bytes(n, cfg->d > hd ? cfg->d : hd);
        const size_t w1 = conv_w_bytes(cfg->d, nq > cfg->d ? nq : cfg->d), w2 = conv_w_bytes(hd, cfg->d);
        const size_t wb = w1 > w2 ? w1 : w2;
        out->conv = {after, ab, after + ab, wb};
        after += ab + wb;
    }
    out->compact_ws = after;
    out->compact_bytes = align_up(dash_workspace_bytes(DASH_WS_COMPACT, n, S, 0, 0, 0, cfg->dt), 256);
    out->attn_ws = out->compact_ws + out->compact_bytes;
    out->attn_bytes = dash_workspace_bytes(DASH_WS_ATTENTION, n, S, cfg->Hq, cfg->Hkv, cfg->D, cfg->dt);
    out->rope_tab = (float2*)(out->attn_ws + align_up(out->attn_bytes, 256));
    out->sums = (float4*)((char*)out->rope_tab + align_up((size_t)n * (cfg->D / 2) * sizeof(float2), 256));
    out->inv_rms = (float*)((char*)out->sums + align_up((size_t)n * ((cfg->d + 255) / 256) * sizeof(float4), 256));
    out->inv_rms2 = (float*)((char*)out->inv_rms + align_up((size_t)n * sizeof(float), 256));
    return DASH_OK;
}

static int launch_rmsnorm(dash_dtype dt, const void* X, const void* weight, void* Y, int64_t n, int d, float eps, const int32_t* n_dev,
                          cudaStream_t st) {
    const int es = dt == DASH_BF16 ? 2 : 4, nvec = d * es / 16;
    if (dt == DASH_BF16) rmsnorm_kernel<true><<<rows_grid8(n), 256, 0, st>>>((const char*)X, (int64_t)d * es, (const char*)weight, (char*)Y, (int64_t)d * es, n, nvec, 1.f / d, eps, n_dev);
    else rmsnorm_kernel<false><<<rows_grid8(n), 256, 0, st>>>((const char*)X, (int64_t)d * es, (const char*)weight, (char*)Y, (int64_t)d * es, n, nvec, 1.f / d, eps, n_dev);
    DASH_CUDA_TRY(cudaGetLastError());
    return DASH_OK;
}

// O = attention(rotary(LN(H) Wqkv)) into W.O: RMSNorm -> Q | K | V projection (rotary embedding in the GEMM epilogue when this
// library's GEMM takes the shape, else a pass of its own) -> causal attention over the packed active set
static int attention_to_O(const dash_layer_cfg* cfg, const void* H_in, const int32_t* pos_in, const int32_t* cu_in, int S, int64_t n,
                          int64_t max_seqlen, const StepWs& W, cudaStream_t st) {
    const int es = cfg->dt == DASH_BF16 ? 2 : 4;
    const bool bf = cfg->dt == DASH_BF16;
    const int d = cfg->d, Hq = cfg->Hq, Hkv = cfg->Hkv, D = cfg->D;
    const int64_t nq = (int64_t)(Hq + 2 * Hkv) * D;
    const int32_t* n_dev = cu_in + S;            // true number of entering tokens lives on the device
    int rc;
    // the attention kernel's item list needs only cu_seqlens: asked for first, so that the attention kernel directly follows the
    // projection in the stream (and may set itself up while that one drains)
    if ((rc = attention_plan(cu_in, S, n, Hq, W.attn_ws, W.attn_bytes, st)) != DASH_OK) return rc;
    GemmEpilogue e;
    e.D = D; e.n_rot_cols = (Hq + Hkv) * D; e.rope_table = W.rope_tab;
    const bool fused = bf && gemm_shape_ok(GEMM_ROPE, n, nq, d, d, nq, e);
    if ((cfg->rope_table || cfg->inv_rms_in || cfg->inv_rms_next) && !(fused && cfg->rms_folded)) return DASH_ERR_UNSUPPORTED;
    if (fused && cfg->rms_folded) {
        // LN folded into the projection: its weight sits in Wqkv, its row factor 1 / rms is applied to the accumulators.
        // One pass over H gives the row factors and the rotary angles -- unless the caller hands them in (a table of the angles
        // by position, made once per prefill; the row factors as the previous block left them): Q | K | V = (H Wqkv) / rms, Q and
        // K rotated.
        if (cfg->rope_table) { e.rope_table = (const float2*)cfg->rope_table; e.rope_pos = pos_in; e.rope_len = cfg->rope_table_len; }
        if (!cfg->rope_table || !cfg->inv_rms_in) {
            rc = launch_row_prep(pos_in, n, D, cfg->rope_base, cfg->rope_table ? nullptr : W.rope_tab, H_in, d, d, cfg->rms_eps,
                                 cfg->inv_rms_in ? nullptr : W.inv_rms, n_dev, st, true);      // beside the item list in front
            if (rc != DASH_OK) return rc;
        }
        e.row_scale = cfg->inv_rms_in ? cfg->inv_rms_in : W.inv_rms;
        if ((rc = gemm_bf16(GEMM_ROPE, H_in, d, cfg->Wqkv, nq, W.QKV, nq, n, nq, d, e, n_dev, st)) != DASH_OK) return rc;
    } else if (fused) {
        // LN (read as RMSNorm), then Q | K | V = Hn Wqkv with the Q and K heads rotated on the accumulators
        if ((rc = launch_rmsnorm(cfg->dt, H_in, cfg->rms_weight, W.Hn, n, d, cfg->rms_eps, n_dev, st)) != DASH_OK) return rc;
        if ((rc = launch_row_prep(pos_in, n, D, cfg->rope_base, W.rope_tab, nullptr, 0, d, 0.f, nullptr, n_dev, st)) != DASH_OK) return rc;
        if ((rc = gemm_bf16(GEMM_ROPE, W.Hn, d, cfg->Wqkv, nq, W.QKV, nq, n, nq, d, e, n_dev, st)) != DASH_OK) return rc;
    } else {
        if (cfg->rms_folded) return DASH_ERR_UNSUPPORTED;      // folded weights need the fused projection (bf16, 256-column tiles)
        if ((rc = launch_rmsnorm(cfg->dt, H_in, cfg->rms_weight, W.Hn, n, d, cfg->rms_eps, n_dev, st)) != DASH_OK) return rc;
        if ((rc = project(cfg->dt, W.Hn, d, cfg->Wqkv, nq, W.QKV, nq, n, nq, d, n_dev, W.conv, st)) != DASH_OK) return rc;
        // rotary embedding on the Q and K heads
        RopeFreq fr;
        for (int i = 0; i < D / 2; ++i) fr.inv_freq[i] = pow(cfg->rope_base, -2.0 * i / D);
        const int heads = Hq + Hkv;
        if (bf && D == 128) rope_kernel<true, 128><<<rows_grid8(n), 256, 0, st>>>(W.QKV, nq * es, pos_in, n, heads, fr, n_dev);
        else if (bf) rope_kernel<true, 64><<<rows_grid8(n), 256, 0, st>>>(W.QKV, nq * es, pos_in, n, heads, fr, n_dev);
        else if (D == 128) rope_kernel<false, 128><<<rows_grid8(n), 256, 0, st>>>(W.QKV, nq * es, pos_in, n, heads, fr, n_dev);
        else rope_kernel<false, 64><<<rows_grid8(n), 256, 0, st>>>(W.QKV, nq * es, pos_in, n, heads, fr, n_dev);
        DASH_CUDA_TRY(cudaGetLastError());
    }
    if (cfg->k_cache) {
        // this depth's KV cache rows: keys (rotary applied) and values of the entering tokens, packed [n, Hkv, D]
        const int64_t kvb = (int64_t)Hkv * D * es;
        if ((rc = dash_scatter(W.QKV + (int64_t)Hq * D * es, n, kvb, nq * es, nullptr, nullptr, 2, n_dev, cfg->k_cache, kvb, st)) != DASH_OK) return rc;
        if ((rc = dash_scatter(W.QKV + (int64_t)(Hq + Hkv) * D * es, n, kvb, nq * es, nullptr, nullptr, 2, n_dev, cfg->v_cache, kvb, st)) != DASH_OK) return rc;
    }
    // attention over the packed active set
    return attention_planned(W.QKV, W.QKV + (int64_t)Hq * D * es, W.QKV + (int64_t)(Hq + Hkv) * D * es, W.O, nullptr, nq, nq, nq,
                             (int64_t)Hq * D, cu_in, S, n, max_seqlen, Hq, Hkv, D, 1.0f / sqrtf((float)D), cfg->dt,
                             W.attn_ws, W.attn_bytes, st);
}

// U = O Wo  (pre-residual attention output, Eq. 1) into W.U
static int out_proj_U(const dash_layer_cfg* cfg, const int32_t* cu_in, int S, int64_t n, const StepWs& W, cudaStream_t st) {
    const int64_t hd = (int64_t)cfg->Hq * cfg->D;
    return project(cfg->dt, W.O, hd, cfg->Wo, cfg->d, W.U, cfg->d, n, cfg->d, hd, cu_in + S, W.conv, st);
}

// Output projection with the residual in its epilogue: dst[idx[row]] = H + O Wo (idx null: row), per-row sums of u^2, h^2 into W.sums.
// Returns DASH_ERR_UNSUPPORTED when this library's GEMM does not take the shape (the caller then goes through U).
static int out_proj_residual(const dash_layer_cfg* cfg, const void* H_in, const int32_t* idx, void* dst, const int32_t* cu_in, int S, int64_t n,
                             const StepWs& W, cudaStream_t st) {
    const int64_t hd = (int64_t)cfg->Hq * cfg->D;
    GemmEpilogue e;
    e.H = H_in; e.ldh = cfg->d; e.tok_index = idx; e.x_full = dst; e.ldx = cfg->d; e.sums = W.sums;
    if (cfg->dt != DASH_BF16 || !gemm_shape_ok(GEMM_RESID, n, cfg->d, hd, hd, cfg->d, e)) return DASH_ERR_UNSUPPORTED;
    return gemm_bf16(GEMM_RESID, W.O, hd, cfg->Wo, cfg->d, nullptr, 0, n, cfg->d, hd, e, cu_in + S, st);
}

// r (and, threshold rule, the keep mask) from U and H, H~ = H + U into W.Ht; keep-count rule: the radix select on r
static int score_and_select(const dash_layer_cfg* cfg, const void* H_in, const int32_t* cu_in, int S, int64_t n, float* r_out,
                            uint8_t* mask_out, const StepWs& W, cudaStream_t st) {
    const int d = cfg->d;
    dash_threshold ft = {cfg->tau, cfg->keep_first, cfg->keep_last, cu_in, S, mask_out};
    int rc = dash_delta_norm(W.U, H_in, n, d, d, d, cfg->dt, cfg->norm_mode, cfg->norm_eps, r_out, W.Ht, d, nullptr,
                             cfg->sel_mode == DASH_SEL_THRESHOLD ? &ft : nullptr, cu_in + S, st);
    if (rc != DASH_OK) return rc;
    if (cfg->sel_mode != DASH_SEL_THRESHOLD)
        rc = dash_select(r_out, n, cu_in, S, cfg->sel_mode, cfg->tau, cfg->keep_counts, cfg->keep_first, cfg->keep_last, mask_out, st);
    return rc;
}

static bool block_cfg_ok(const dash_block_cfg* c) {
    if (!c || !cfg_ok(&c->attn)) return false;
    const int epv = c->attn.dt == DASH_BF16 ? 8 : 4;
    if (c->m <= 0 || (c->m % epv) || !c->Wgu || !c->Wd || (!c->rms2_weight && !c->rms2_folded)) return false;
    if (c->rms2_folded != 0 && c->rms2_folded != 1) return false;
    if (c->signal != DASH_SIGNAL_ATTN && c->signal != DASH_SIGNAL_BLOCK) return false;
    if (c->signal == DASH_SIGNAL_BLOCK && 2 * c->m < c->attn.d) return false;      // U + F is formed in the gate | up buffer
    return c->attn.scatter_which == 2;
}

}  // namespace dash

extern "C" int dash_layer_step(const dash_layer_cfg* cfg, const void* H_in, const int32_t* tok_index_in,
                               const int32_t* pos_in, const int32_t* cu_in, int S, int64_t n, int64_t max_seqlen,
                               void* x_full, void* H_next, int32_t* tok_index_next, int32_t* pos_next,
                               int32_t* cu_next, int32_t* n_next_dev, float* r_out, uint8_t* mask_out,
                               void* ws, size_t ws_bytes, void* stream) {
    if (!cfg_ok(cfg) || n < 0 || S < 1 || max_seqlen < 0 || max_seqlen > n) return DASH_ERR_INVALID_ARG;
    if (!cu_in || !cu_next) return DASH_ERR_INVALID_ARG;
    if (n > 0 && (!H_in || !pos_in || !tok_index_in || !x_full || !H_next || !tok_index_next || !pos_next || !r_out || !mask_out))
        return DASH_ERR_INVALID_ARG;
    StepWs W;
    int rc = carve_ws(cfg, n, S, ws, &W);
    if (rc != DASH_OK) return rc;
    if (!ws || ((uintptr_t)ws % 256) || ws_bytes < W.L.total) return DASH_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const int es = cfg->dt == DASH_BF16 ? 2 : 4;
    const int d = cfg->d;
    if (n > 0) {
        if (!aligned16(H_in) || !aligned16(x_full) || !aligned16(H_next) || !aligned16(cfg->Wqkv) || !aligned16(cfg->Wo) ||
            (cfg->rms_weight && !aligned16(cfg->rms_weight)))
            return DASH_ERR_INVALID_ARG;
        const bool tail_pass = cfg->sel_mode == DASH_SEL_THRESHOLD && cfg->scatter_which == 2;
        // the tail pass's look-back words are cleared up front: its launch then follows the output projection directly
        if (tail_pass && (rc = clear_tail_ws(W.compact_ws, W.compact_bytes, n, st)) != DASH_OK) return rc;
        if ((rc = attention_to_O(cfg, H_in, pos_in, cu_in, S, n, max_seqlen, W, st)) != DASH_OK) return rc;
        if (tail_pass) {
            // output projection with H~ = H + U written straight to x_full and the row sums of u^2, h^2 beside it; then the score, the
            // halting rule and the compaction of the rows that stay (from x_full) in one pass
            rc = out_proj_residual(cfg, H_in, tok_index_in, x_full, cu_in, S, n, W, st);
            if (rc == DASH_OK)
                return launch_delta_tail(nullptr, nullptr, nullptr, W.sums, d / 256, n, d, cfg->dt, cfg->norm_mode, cfg->norm_eps, cfg->tau,
                                         cfg->keep_first, cfg->keep_last, cu_in, S, tok_index_in, pos_in, x_full, H_next, r_out, mask_out,
                                         tok_index_next, pos_next, cu_next, n_next_dev, W.compact_ws, W.compact_bytes, true, st,
                                         cfg->inv_rms_next, cfg->rms_eps);
            if (rc != DASH_ERR_UNSUPPORTED) return rc;
            // fp32, or shapes without whole 256-column tiles: U through the plain GEMM, then r, H~, the rule, scatter and compaction in one pass
            if ((rc = out_proj_U(cfg, cu_in, S, n, W, st)) != DASH_OK) return rc;
            return launch_delta_tail(W.U, H_in, nullptr, nullptr, 0, n, d, cfg->dt, cfg->norm_mode, cfg->norm_eps, cfg->tau, cfg->keep_first,
                                     cfg->keep_last, cu_in, S, tok_index_in, pos_in, x_full, H_next, r_out, mask_out, tok_index_next,
                                     pos_next, cu_next, n_next_dev, W.compact_ws, W.compact_bytes, true, st, nullptr, cfg->rms_eps);
        }
        if (cfg->inv_rms_next) return DASH_ERR_UNSUPPORTED;      // the row factors come out of the fused tail pass (threshold rule, every row scattered)
        if ((rc = out_proj_U(cfg, cu_in, S, n, W, st)) != DASH_OK) return rc;
        if ((rc = score_and_select(cfg, H_in, cu_in, S, n, r_out, mask_out, W, st)) != DASH_OK) return rc;
        // updated states reach the full-length output (halted tokens stay frozen there from now on)
        rc = dash_scatter(W.Ht, n, (int64_t)d * es, (int64_t)d * es, tok_index_in, mask_out, cfg->scatter_which, cu_in + S, x_full,
                          (int64_t)d * es, st);
        if (rc != DASH_OK) return rc;
    }
    dash_rows rows = {W.Ht, H_next, (int64_t)d * es, (int64_t)d * es, (int64_t)d * es};
    return dash_compact(mask_out, n, cu_in, S, &rows, n > 0 ? 1 : 0, pos_in, pos_next, tok_index_in, tok_index_next, nullptr,
                        cu_next, n_next_dev, W.compact_ws, W.compact_bytes, st);
}

extern "C" int dash_block_workspace(const dash_block_cfg* cfg, int64_t n, int S, dash_block_ws_layout* out) {
    if (!block_cfg_ok(cfg) || n < 0 || S < 1 || !out) return DASH_ERR_INVALID_ARG;
    int rc = dash_layer_workspace(&cfg->attn, n, S, &out->attn);
    if (rc != DASH_OK) return rc;
    const size_t es = cfg->attn.dt == DASH_BF16 ? 2 : 4;
    size_t off = align_up(out->attn.total, 256);
    out->GU = off;  off += align_up((size_t)n * 2 * cfg->m * es, 256);
    out->ACT = off; off += align_up((size_t)n * cfg->m * es, 256);
    out->F = off;   off += align_up((size_t)n * cfg->attn.d * es, 256);
    if (cfg->attn.dt == DASH_F32) {        // bf16 copies of the operands of the feed-forward's projections
        off += conv_a_bytes(n, cfg->m > cfg->attn.d ? cfg->m : cfg->attn.d);
        off += conv_w_bytes(cfg->attn.d, 2 * (int64_t)cfg->m) > conv_w_bytes(cfg->m, cfg->attn.d) ? conv_w_bytes(cfg->attn.d, 2 * (int64_t)cfg->m) : conv_w_bytes(cfg->m, cfg->attn.d);
    }
    out->total = off;
    return DASH_OK;
}

extern "C" int dash_block_step(const dash_block_cfg* cfg, const void* H_in, const int32_t* tok_index_in,
                               const int32_t* pos_in, const int32_t* cu_in, int S, int64_t n, int64_t max_seqlen,
                               void* x_full, void* H_next, int32_t* tok_index_next, int32_t* pos_next,
                               int32_t* cu_next, int32_t* n_next_dev, float* r_out, uint8_t* mask_out,
                               void* ws, size_t ws_bytes, void* stream) {
    if (!block_cfg_ok(cfg) || n < 0 || S < 1 || max_seqlen < 0 || max_seqlen > n) return DASH_ERR_INVALID_ARG;
    if (!cu_in || !cu_next) return DASH_ERR_INVALID_ARG;
    if (n > 0 && (!H_in || !pos_in || !tok_index_in || !x_full || !H_next || !tok_index_next || !pos_next || !r_out || !mask_out))
        return DASH_ERR_INVALID_ARG;
    const dash_layer_cfg* a = &cfg->attn;
    dash_block_ws_layout BL;
    int rc = dash_block_workspace(cfg, n, S, &BL);
    if (rc != DASH_OK) return rc;
    if (!ws || ((uintptr_t)ws % 256) || ws_bytes < BL.total) return DASH_ERR_WORKSPACE;
    StepWs W;
    if ((rc = carve_ws(a, n, S, ws, &W)) != DASH_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const int es = a->dt == DASH_BF16 ? 2 : 4;
    const int d = a->d, m = cfg->m;
    char *GU = (char*)ws + BL.GU, *ACT = (char*)ws + BL.ACT, *F = (char*)ws + BL.F;
    ConvScratch conv = {nullptr, 0, nullptr, 0};
    if (a->dt == DASH_F32) {
        char* c0 = F + align_up((size_t)n * d * es, 256);
        const size_t ab = conv_a_bytes(n, m > d ? m : d);
        const size_t w1 = conv_w_bytes(d, 2 * (int64_t)m), w2 = conv_w_bytes(m, d);
        conv = {c0, ab, c0 + ab, w1 > w2 ? w1 : w2};
    }
    if (n == 0) {
        return dash_compact(mask_out, 0, cu_in, S, nullptr, 0, pos_in, pos_next, tok_index_in, tok_index_next, nullptr, cu_next, n_next_dev,
                            W.compact_ws, W.compact_bytes, st);
    }
    if (!aligned16(H_in) || !aligned16(x_full) || !aligned16(H_next) || !aligned16(a->Wqkv) || !aligned16(a->Wo) || (a->rms_weight && !aligned16(a->rms_weight)) ||
        !aligned16(cfg->Wgu) || !aligned16(cfg->Wd) || (cfg->rms2_weight && !aligned16(cfg->rms2_weight)))
        return DASH_ERR_INVALID_ARG;
    const int32_t* n_dev = cu_in + S;
    // the tail pass's look-back words are cleared up front: its launch then follows the down projection directly
    if ((rc = clear_tail_ws(W.compact_ws, W.compact_bytes, n, st)) != DASH_OK) return rc;
    // U = Attn(LN(H)); score and selection from U; H~ = H + U
    if ((rc = attention_to_O(a, H_in, pos_in, cu_in, S, n, max_seqlen, W, st)) != DASH_OK) return rc;
    bool have_inv_rms2 = false;
    rc = cfg->signal == DASH_SIGNAL_ATTN ? out_proj_residual(a, H_in, nullptr, W.Ht, cu_in, S, n, W, st) : DASH_ERR_UNSUPPORTED;
    if (rc == DASH_OK) {
        // H~ came out of the projection's epilogue (into W.Ht) with the row sums: finish the score, then the rule
        dash_threshold ft = {a->tau, a->keep_first, a->keep_last, cu_in, S, mask_out};
        have_inv_rms2 = cfg->rms2_folded != 0;
        if ((rc = launch_sums_to_score(W.sums, d / 256, n, a->norm_mode, a->norm_eps, r_out, a->sel_mode == DASH_SEL_THRESHOLD ? &ft : nullptr,
                                       n_dev, have_inv_rms2 ? W.inv_rms2 : nullptr, d, a->rms_eps, st)) != DASH_OK) return rc;
        if (a->sel_mode != DASH_SEL_THRESHOLD &&
            (rc = dash_select(r_out, n, cu_in, S, a->sel_mode, a->tau, a->keep_counts, a->keep_first, a->keep_last, mask_out, st)) != DASH_OK)
            return rc;
    } else if (rc == DASH_ERR_UNSUPPORTED) {
        if ((rc = out_proj_U(a, cu_in, S, n, W, st)) != DASH_OK) return rc;
        if ((rc = score_and_select(a, H_in, cu_in, S, n, r_out, mask_out, W, st)) != DASH_OK) return rc;   // also leaves H~ in W.Ht
    } else {
        return rc;
    }
    // F = FFN(LN(H~)): gate | up projection, silu(gate) * up, down projection
    GemmEpilogue eg;
    eg.m = m;
    const bool fused_ffn = a->dt == DASH_BF16 && gemm_shape_ok(GEMM_SWIGLU, n, 2 * (int64_t)m, d, d, 2 * (int64_t)m, eg);
    if (cfg->rms2_folded && !(fused_ffn && have_inv_rms2)) return DASH_ERR_UNSUPPORTED;   // folded weights need the fused projections
    if (!cfg->rms2_folded && (rc = launch_rmsnorm(a->dt, W.Ht, cfg->rms2_weight, W.Hn, n, d, a->rms_eps, n_dev, st)) != DASH_OK) return rc;
    if (fused_ffn) {
        // gate | up projection with silu(gate) * up on the accumulators: the [n, 2m] intermediate is never stored; with the norm
        // folded in, the operand is H~ itself and the accumulators take the row factor 1 / rms first
        eg.row_scale = cfg->rms2_folded ? W.inv_rms2 : nullptr;
        if ((rc = gemm_bf16(GEMM_SWIGLU, cfg->rms2_folded ? W.Ht : W.Hn, d, cfg->Wgu, 2 * (int64_t)m, ACT, m, n, 2 * (int64_t)m, d, eg, n_dev, st)) != DASH_OK) return rc;
    } else {
        if ((rc = project(a->dt, W.Hn, d, cfg->Wgu, 2 * (int64_t)m, GU, 2 * (int64_t)m, n, 2 * (int64_t)m, d, n_dev, conv, st)) != DASH_OK) return rc;
        const int64_t total = n * (int64_t)(m / (16 / es));
        int64_t blocks = (total + 255) / 256, cap = (int64_t)sm_count() * 16;
        if (blocks > cap) blocks = cap;
        if (a->dt == DASH_BF16) swiglu_kernel<true><<<(int)blocks, 256, 0, st>>>(GU, 2 * (int64_t)m * es, ACT, (int64_t)m * es, n, m, n_dev);
        else swiglu_kernel<false><<<(int)blocks, 256, 0, st>>>(GU, 2 * (int64_t)m * es, ACT, (int64_t)m * es, n, m, n_dev);
        DASH_CUDA_TRY(cudaGetLastError());
    }
    if ((rc = project(a->dt, ACT, m, cfg->Wd, d, F, d, n, d, m, n_dev, conv, st)) != DASH_OK) return rc;
    if (cfg->signal == DASH_SIGNAL_BLOCK) {
        // ablation: score = change over the whole block, H' - H = U + F (formed in the gate | up buffer, free by now)
        if ((rc = dash_delta_norm(F, W.U, n, d, d, d, a->dt, DASH_NORM_ABS, a->norm_eps, r_out, GU, d, nullptr, nullptr, n_dev, st)) != DASH_OK) return rc;
        dash_threshold ft = {a->tau, a->keep_first, a->keep_last, cu_in, S, mask_out};
        rc = dash_delta_norm(GU, H_in, n, d, d, d, a->dt, a->norm_mode, a->norm_eps, r_out, nullptr, d, nullptr,
                             a->sel_mode == DASH_SEL_THRESHOLD ? &ft : nullptr, n_dev, st);
        if (rc != DASH_OK) return rc;
        if (a->sel_mode != DASH_SEL_THRESHOLD &&
            (rc = dash_select(r_out, n, cu_in, S, a->sel_mode, a->tau, a->keep_counts, a->keep_first, a->keep_last, mask_out, st)) != DASH_OK)
            return rc;
    }
    // H' = H~ + F to x_full (every entering token: H' is also the last updated value of the tokens that halt here) and,
    // for the tokens that stay, to the next block's packed buffer -- one pass, keep decisions taken from mask_out
    return launch_delta_tail(F, W.Ht, mask_out, nullptr, 0, n, d, a->dt, a->norm_mode, a->norm_eps, a->tau, a->keep_first, a->keep_last, cu_in, S,
                             tok_index_in, pos_in, x_full, H_next, nullptr, nullptr, tok_index_next, pos_next, cu_next, n_next_dev,
                             W.compact_ws, W.compact_bytes, true, st, a->inv_rms_next, a->rms_eps);
}

// dash_layer_step: the body of the prefill loop for one block (without the FFN),
// on the packed active tokens: RMSNorm -> QKV projection -> rotary embedding ->
// causal attention -> output projection -> delta score / residual / halting rule
// -> scatter of the updated states -> compaction of the tokens that stay active.
// The two projections are plain library GEMMs (cuBLASLt); everything else runs in
// this library's own kernels.  One stream, no host synchronisation.
#include <cublasLt.h>
#include <math.h>

#include <map>
#include <mutex>
#include <tuple>

#include "common.cuh"

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

// ---- library GEMM: C[n, N] = A[n, K] * W[K, N], all row-major ---------------------
struct LtState {
    cublasLtHandle_t handle = nullptr;
    std::mutex mu;
    std::map<std::tuple<int, int64_t, int64_t, int64_t, int64_t, int64_t, int64_t>, cublasLtMatmulAlgo_t> algos;
};
static LtState& lt() { static LtState s; return s; }
constexpr size_t kLtWorkspace = 64ull << 20;

static int gemm_rowmajor(dash_dtype dt, const void* A, int64_t lda, const void* W, int64_t ldw, void* C, int64_t ldc,
                         int64_t n, int64_t N, int64_t K, void* lt_ws, cudaStream_t st) {
    LtState& s = lt();
    std::lock_guard<std::mutex> g(s.mu);
    if (!s.handle && cublasLtCreate(&s.handle) != CUBLAS_STATUS_SUCCESS) return DASH_ERR_CUDA;
    const cudaDataType_t ty = (dt == DASH_BF16) ? CUDA_R_16BF : CUDA_R_32F;
    cublasLtMatmulDesc_t op = nullptr;
    cublasLtMatrixLayout_t la = nullptr, lb = nullptr, lc = nullptr;
    int rc = DASH_ERR_CUDA;
    const float alpha = 1.f, beta = 0.f;
    do {
        if (cublasLtMatmulDescCreate(&op, CUBLAS_COMPUTE_32F, CUDA_R_32F) != CUBLAS_STATUS_SUCCESS) break;
        // row-major C = A W  <=>  column-major C^T[N,n] = W^T[N,K] A^T[K,n]
        if (cublasLtMatrixLayoutCreate(&la, ty, N, K, ldw) != CUBLAS_STATUS_SUCCESS) break;
        if (cublasLtMatrixLayoutCreate(&lb, ty, K, n, lda) != CUBLAS_STATUS_SUCCESS) break;
        if (cublasLtMatrixLayoutCreate(&lc, ty, N, n, ldc) != CUBLAS_STATUS_SUCCESS) break;
        auto key = std::make_tuple((int)dt, n, N, K, lda, ldw, ldc);
        auto it = s.algos.find(key);
        if (it == s.algos.end()) {
            cublasLtMatmulPreference_t pref = nullptr;
            if (cublasLtMatmulPreferenceCreate(&pref) != CUBLAS_STATUS_SUCCESS) break;
            size_t wsz = kLtWorkspace;
            cublasLtMatmulPreferenceSetAttribute(pref, CUBLASLT_MATMUL_PREF_MAX_WORKSPACE_BYTES, &wsz, sizeof(wsz));
            cublasLtMatmulHeuristicResult_t res;
            int found = 0;
            cublasStatus_t hs = cublasLtMatmulAlgoGetHeuristic(s.handle, op, la, lb, lc, lc, pref, 1, &res, &found);
            cublasLtMatmulPreferenceDestroy(pref);
            if (hs != CUBLAS_STATUS_SUCCESS || found < 1) break;
            it = s.algos.emplace(key, res.algo).first;
        }
        if (cublasLtMatmul(s.handle, op, &alpha, W, la, A, lb, &beta, C, lc, C, lc, &it->second, lt_ws, kLtWorkspace, st) !=
            CUBLAS_STATUS_SUCCESS)
            break;
        rc = DASH_OK;
    } while (0);
    if (la) cublasLtMatrixLayoutDestroy(la);
    if (lb) cublasLtMatrixLayoutDestroy(lb);
    if (lc) cublasLtMatrixLayoutDestroy(lc);
    if (op) cublasLtMatmulDescDestroy(op);
    return rc;
}

int launch_delta_tail(const void* U, const void* H, int64_t n, int d, dash_dtype dt, dash_norm_mode mode, float eps, float tau,
                      int keep_first, int keep_last, const int32_t* cu_in, int S, const int32_t* tok_in, const int32_t* pos_in,
                      void* x_full, void* H_next, float* r_out, uint8_t* mask_out, int32_t* tok_next, int32_t* pos_next,
                      int32_t* cu_next, int32_t* n_next, void* ws, size_t ws_bytes, cudaStream_t st);

static int rows_grid8(int64_t n) {
    int64_t blocks = (n + 7) / 8, cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    return (int)(blocks < 1 ? 1 : blocks);
}

static bool cfg_ok(const dash_layer_cfg* c) {
    if (!c || c->d <= 0 || c->Hq < 1 || c->Hkv < 1 || (c->D != 64 && c->D != 128)) return false;
    if ((c->d % 8) || (c->Hq % c->Hkv)) return false;
    if (c->dt != DASH_F32 && c->dt != DASH_BF16) return false;
    if (!c->Wqkv || !c->Wo || !c->rms_weight) return false;
    if (c->sel_mode != DASH_SEL_THRESHOLD && c->sel_mode != DASH_SEL_KEEP_COUNT) return false;
    if (c->sel_mode == DASH_SEL_KEEP_COUNT && !c->keep_counts) return false;
    if (c->keep_first < 0 || c->keep_last < 0) return false;
    if (c->scatter_which != 0 && c->scatter_which != 2) return false;
    if (!(c->rope_base > 0.0)) return false;
    return true;
}

}  // namespace dash

using namespace dash;

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
    out->scratch = off;
    off += kLtWorkspace;
    off += align_up(dash_workspace_bytes(DASH_WS_COMPACT, n, S, 0, 0, 0, cfg->dt), 256);
    off += align_up(dash_workspace_bytes(DASH_WS_ATTENTION, n, S, cfg->Hq, cfg->Hkv, cfg->D, cfg->dt), 256);
    out->total = off;
    return DASH_OK;
}

extern "C" int dash_layer_step(const dash_layer_cfg* cfg, const void* H_in, const int32_t* tok_index_in,
                               const int32_t* pos_in, const int32_t* cu_in, int S, int64_t n, int64_t max_seqlen,
                               void* x_full, void* H_next, int32_t* tok_index_next, int32_t* pos_next,
                               int32_t* cu_next, int32_t* n_next_dev, float* r_out, uint8_t* mask_out,
                               void* ws, size_t ws_bytes, void* stream) {
    if (!cfg_ok(cfg) || n < 0 || S < 1 || max_seqlen < 0 || max_seqlen > n) return DASH_ERR_INVALID_ARG;
    if (!cu_in || !cu_next) return DASH_ERR_INVALID_ARG;
    if (n > 0 && (!H_in || !pos_in || !tok_index_in || !x_full || !H_next || !tok_index_next || !pos_next || !r_out || !mask_out))
        return DASH_ERR_INVALID_ARG;
    dash_layer_ws_layout L;
    int rc = dash_layer_workspace(cfg, n, S, &L);
    if (rc != DASH_OK) return rc;
    if (!ws || ((uintptr_t)ws % 256) || ws_bytes < L.total) return DASH_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char* w = (char*)ws;
    const int es = cfg->dt == DASH_BF16 ? 2 : 4;
    const bool bf = cfg->dt == DASH_BF16;
    const int d = cfg->d, Hq = cfg->Hq, Hkv = cfg->Hkv, D = cfg->D;
    const int64_t nq = (int64_t)(Hq + 2 * Hkv) * D;
    char *Hn = w + L.Hn, *QKV = w + L.QKV, *O = w + L.O, *U = w + L.U, *Ht = w + L.Ht;
    char* lt_ws = w + L.scratch;
    char* compact_ws = lt_ws + kLtWorkspace;
    const size_t compact_bytes = align_up(dash_workspace_bytes(DASH_WS_COMPACT, n, S, 0, 0, 0, cfg->dt), 256);
    char* attn_ws = compact_ws + compact_bytes;
    const size_t attn_bytes = dash_workspace_bytes(DASH_WS_ATTENTION, n, S, Hq, Hkv, D, cfg->dt);
    const int32_t* n_dev = cu_in + S;            // true number of entering tokens lives on the device

    if (n > 0) {
        if (!aligned16(H_in) || !aligned16(x_full) || !aligned16(H_next) || !aligned16(cfg->Wqkv) || !aligned16(cfg->Wo) ||
            !aligned16(cfg->rms_weight))
            return DASH_ERR_INVALID_ARG;
        // LN (read as RMSNorm)
        const int nvec = d * es / 16;
        if (bf) rmsnorm_kernel<true><<<rows_grid8(n), 256, 0, st>>>((const char*)H_in, (int64_t)d * es, (const char*)cfg->rms_weight, Hn, (int64_t)d * es, n, nvec, 1.f / d, cfg->rms_eps, n_dev);
        else rmsnorm_kernel<false><<<rows_grid8(n), 256, 0, st>>>((const char*)H_in, (int64_t)d * es, (const char*)cfg->rms_weight, Hn, (int64_t)d * es, n, nvec, 1.f / d, cfg->rms_eps, n_dev);
        DASH_CUDA_TRY(cudaGetLastError());
        // Q | K | V = Hn Wqkv
        if ((rc = gemm_rowmajor(cfg->dt, Hn, d, cfg->Wqkv, nq, QKV, nq, n, nq, d, lt_ws, st)) != DASH_OK) return rc;
        // rotary embedding on the Q and K heads
        RopeFreq fr;
        for (int i = 0; i < D / 2; ++i) fr.inv_freq[i] = pow(cfg->rope_base, -2.0 * i / D);
        const int heads = Hq + Hkv;
        if (bf && D == 128) rope_kernel<true, 128><<<rows_grid8(n), 256, 0, st>>>(QKV, nq * es, pos_in, n, heads, fr, n_dev);
        else if (bf) rope_kernel<true, 64><<<rows_grid8(n), 256, 0, st>>>(QKV, nq * es, pos_in, n, heads, fr, n_dev);
        else if (D == 128) rope_kernel<false, 128><<<rows_grid8(n), 256, 0, st>>>(QKV, nq * es, pos_in, n, heads, fr, n_dev);
        else rope_kernel<false, 64><<<rows_grid8(n), 256, 0, st>>>(QKV, nq * es, pos_in, n, heads, fr, n_dev);
        DASH_CUDA_TRY(cudaGetLastError());
        // attention over the packed active set
        rc = dash_varlen_attention(QKV, QKV + (int64_t)Hq * D * es, QKV + (int64_t)(Hq + Hkv) * D * es, O, nullptr, nq, nq, nq,
                                   (int64_t)Hq * D, cu_in, S, n, max_seqlen, Hq, Hkv, D, 1.0f / sqrtf((float)D), 1, cfg->dt,
                                   attn_ws, attn_bytes, st);
        if (rc != DASH_OK) return rc;
        // U = O Wo  (pre-residual attention output, Eq. 1)
        if ((rc = gemm_rowmajor(cfg->dt, O, (int64_t)Hq * D, cfg->Wo, d, U, d, n, d, (int64_t)Hq * D, lt_ws, st)) != DASH_OK) return rc;
        if (cfg->sel_mode == DASH_SEL_THRESHOLD && cfg->scatter_which == 2) {
            // r, H~ = H + U, the halting rule, the scatter of H~ and the compaction of the rows that stay, in one pass
            return launch_delta_tail(U, H_in, n, d, cfg->dt, cfg->norm_mode, cfg->norm_eps, cfg->tau, cfg->keep_first, cfg->keep_last,
                                     cu_in, S, tok_index_in, pos_in, x_full, H_next, r_out, mask_out, tok_index_next, pos_next,
                                     cu_next, n_next_dev, compact_ws, compact_bytes, st);
        }
        // r, H~ = H + U, and (threshold mode) the halting rule in the same pass
        dash_threshold ft = {cfg->tau, cfg->keep_first, cfg->keep_last, cu_in, S, mask_out};
        rc = dash_delta_norm(U, H_in, n, d, d, d, cfg->dt, cfg->norm_mode, cfg->norm_eps, r_out, Ht, d, nullptr,
                             cfg->sel_mode == DASH_SEL_THRESHOLD ? &ft : nullptr, n_dev, st);
        if (rc != DASH_OK) return rc;
        if (cfg->sel_mode == DASH_SEL_KEEP_COUNT) {
            rc = dash_select(r_out, n, cu_in, S, DASH_SEL_KEEP_COUNT, 0.f, cfg->keep_counts, cfg->keep_first, cfg->keep_last,
                             mask_out, nullptr, 0, st);
            if (rc != DASH_OK) return rc;
        }
        // updated states reach the full-length output (halted tokens stay frozen there from now on)
        rc = dash_scatter(Ht, n, (int64_t)d * es, (int64_t)d * es, tok_index_in, mask_out, cfg->scatter_which, n_dev, x_full,
                          (int64_t)d * es, st);
        if (rc != DASH_OK) return rc;
    }
    dash_rows rows = {Ht, H_next, (int64_t)d * es, (int64_t)d * es, (int64_t)d * es};
    return dash_compact(mask_out, n, cu_in, S, &rows, n > 0 ? 1 : 0, pos_in, pos_next, tok_index_in, tok_index_next, nullptr,
                        cu_next, n_next_dev, compact_ws, compact_bytes, st);
}

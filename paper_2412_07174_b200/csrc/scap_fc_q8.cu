// Sparse FC on 8-bit weights (Table 4 applies SCAP to 8-bit models).  Storage: Wq[K,N] signed 8-bit, input-channel-
// major like the 16-bit layout, one binary32 scale per input channel, W[k,n] = wscale[k] * Wq[k,n].  Because the
// scale belongs to the input channel it is folded into the pruned activation once per kept channel (d * wscale),
// and the streaming loop multiplies by the raw integers.  A kept row of a 128-column tile is 128 bytes, so a
// thread's 16-byte load covers 16 columns and 8 lanes cover the row.  The kernel is the FC kernel of scap_fc.cuh
// instantiated for one byte per weight: same prologue, compaction, register double buffer and asynchronous cluster
// exchange.
#include <string.h>

#include "scap_fc.cuh"

namespace scap {

constexpr int Q8_TN = 128;   // columns per CTA

// Split-K factor: the most CTAs (tiles of 128 columns x S) that are all resident; ties: the larger cluster.
static int q8_split(int K, int N) {
    const int tiles = (N + Q8_TN - 1) / Q8_TN;
    int best_S = 1;
    long long best = -1;
    for (int S = 1; S <= MAX_CLUSTER; ++S) {
        if (g_tune.split_k > 0 && S > g_tune.split_k) continue;
        if (S > 1 && K / S < 64) continue;
        const long long ctas = (long long)tiles * S;
        if (S > 1 && ctas > resident_ctas(S)) continue;
        if (ctas >= best) { best = ctas; best_S = S; }
    }
    return best_S;
}

template <int BT, int MODE, typename XT, int PUT>
static cudaError_t launch_q8_pu(const FcArgs &a, cudaStream_t st) {
    static SmemOptIn opt_in;
    auto kern = fc_kernel<true, BT, MODE, XT, EPI_BIAS, Q8_TN, PUT, 1>;
    cudaError_t e0 = ensure_dynamic_smem(kern, fc_smem_bytes(BT), opt_in);
    if (e0 != cudaSuccess) return e0;
    return launch_cluster(kern, dim3((a.Nh + Q8_TN - 1) / Q8_TN, a.S), dim3(FC_THREADS), fc_smem_bytes(BT), a.S, st, g_tune.pdl != 0, a);
}

// The threshold code comes unrolled for 2, 4, 6 or 8 chunk slots per warp: the smallest that takes the rank's channels in one fill.
template <int BT, int MODE, typename XT>
static cudaError_t launch_q8_t(const FcArgs &a, cudaStream_t st) {
    const int per_rank = ((a.K + 31) / 32 + a.S - 1) / a.S, need = (per_rank + FC_WARPS - 1) / FC_WARPS;
    // (two rows, sparse call: the 8-slot form is the faster one whatever the count - measured, 15.7 against 18.0 us)
    if (BT == 2 && MODE == MODE_GATHER) return launch_q8_pu<BT, MODE, XT, fc_pu(BT)>(a, st);
    if (need <= 2) return launch_q8_pu<BT, MODE, XT, 2>(a, st);
    if (need <= 4) return launch_q8_pu<BT, MODE, XT, 4>(a, st);
    if (need <= 6) return launch_q8_pu<BT, MODE, XT, 6>(a, st);
    return launch_q8_pu<BT, MODE, XT, fc_pu(BT)>(a, st);
}

// xkind: 0 fp16, 1 bf16, 2 float activations.  Batches beyond two rows run two rows at a time (row results are
// independent; the union mask then spans two rows).
static cudaError_t launch_q8(int mode, int xkind, FcArgs a, cudaStream_t st) {
    const int B = a.B;
    const size_t xsz = xkind == 2 ? 4 : 2;
    const unsigned char *x0 = static_cast<const unsigned char *>(a.x);
    float *y0 = a.y;
    for (int b0 = 0; b0 < B; b0 += 2) {
        a.B = B - b0 >= 2 ? 2 : 1;
        a.x = x0 + (size_t)b0 * a.x_ld * xsz;
        a.y = y0 + (size_t)b0 * a.y_ld;
        cudaError_t e;
        if (a.B == 1) {
            if (mode == MODE_DENSE) e = xkind == 2 ? launch_q8_t<1, MODE_DENSE, float>(a, st) : xkind == 1 ? launch_q8_t<1, MODE_DENSE, __nv_bfloat16>(a, st) : launch_q8_t<1, MODE_DENSE, __half>(a, st);
            else e = xkind == 1 ? launch_q8_t<1, MODE_GATHER, __nv_bfloat16>(a, st) : launch_q8_t<1, MODE_GATHER, __half>(a, st);
        } else {
            if (mode == MODE_DENSE) e = xkind == 1 ? launch_q8_t<2, MODE_DENSE, __nv_bfloat16>(a, st) : launch_q8_t<2, MODE_DENSE, __half>(a, st);
            else e = xkind == 1 ? launch_q8_t<2, MODE_GATHER, __nv_bfloat16>(a, st) : launch_q8_t<2, MODE_GATHER, __half>(a, st);
        }
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace scap

using namespace scap;

extern "C" {

static scap_status q8_check(const void *x, const void *Wq, const float *wscale, const float *m, const float *b, float *y, int B, int K,
                            int N, scap_dtype xdt, const void *ws, size_t ws_bytes) {
    if (!x || !Wq || !wscale || !y || !ws) return SCAP_ERR_INVALID_ARG;
    if (xdt != SCAP_F16 && xdt != SCAP_BF16) return SCAP_ERR_DTYPE;
    if (B < 1 || B > SCAP_MAX_BATCH || K < 1 || N < 1 || K > SCAP_MAX_K) return SCAP_ERR_SHAPE;
    if (N % 16 != 0 || !aligned16(x) || !aligned16(Wq) || !aligned16(y) || !aligned16(ws) || (m && !aligned16(m)) || (b && !aligned16(b)))
        return SCAP_ERR_ALIGN;
    if (ws_bytes < scap_fc_workspace(B, K, N)) return SCAP_ERR_WORKSPACE;
    return check_device();
}

scap_status scap_sparse_fc_q8(const void *x, scap_dtype xdt, const signed char *Wq, const float *wscale, const float *m,
                              const float *tau, const float *b_fused, float *y, int B, int K, int N, uint32_t *idx_out,
                              int *nnz_out, void *ws, size_t ws_bytes, scap_stream_t stream) {
    if (!tau) return SCAP_ERR_INVALID_ARG;
    scap_status stt = q8_check(x, Wq, wscale, m, b_fused, y, B, K, N, xdt, ws, ws_bytes);
    if (stt != SCAP_OK) return stt;
    if ((idx_out || nnz_out) && B > 2) return SCAP_ERR_SHAPE;  // the kept list describes one launch (at most two rows)
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    FcArgs a;
    memset(&a, 0, sizeof(a));
    a.W = Wq; a.wscale = wscale; a.K = K; a.ldw = N; a.Nh = N; a.B = B; a.tn = Q8_TN; a.S = q8_split(K, N);
    a.x = x; a.x_ld = K; a.m = m; a.tau = tau; a.bias = b_fused; a.y = y; a.y_ld = N;
    a.l2_hints = g_tune.l2_hints; a.head_rows = g_tune.head_rows; a.status = tc_status_ptr();
    const bool inspect = idx_out || nnz_out;
    if (inspect) a.bits = reinterpret_cast<uint32_t *>(ws);
    cudaError_t e = launch_q8(MODE_GATHER, xdt == SCAP_BF16 ? 1 : 0, a, st);
    if (e != cudaSuccess) return cuda_status(e);
    if (inspect) e = launch_expand_bits(a.bits, K, idx_out, nnz_out, st);
    return cuda_status(e);
}

scap_status scap_dense_fc_q8(const void *x, scap_dtype xdt, const signed char *Wq, const float *wscale, const float *b, float *y,
                             int B, int K, int N, void *ws, size_t ws_bytes, scap_stream_t stream) {
    scap_status stt = q8_check(x, Wq, wscale, nullptr, b, y, B, K, N, xdt, ws, ws_bytes);
    if (stt != SCAP_OK) return stt;
    FcArgs a;
    memset(&a, 0, sizeof(a));
    a.W = Wq; a.wscale = wscale; a.K = K; a.ldw = N; a.Nh = N; a.B = B; a.tn = Q8_TN; a.S = q8_split(K, N);
    a.x = x; a.x_ld = K; a.bias = b; a.y = y; a.y_ld = N;
    a.l2_hints = g_tune.l2_hints; a.head_rows = g_tune.head_rows > 0 ? g_tune.head_rows : 4; a.status = tc_status_ptr();
    return cuda_status(launch_q8(MODE_DENSE, xdt == SCAP_BF16 ? 1 : 0, a, reinterpret_cast<cudaStream_t>(stream)));
}

scap_status scap_fold_bias_q8(const signed char *Wq, const float *wscale, const float *m, const float *b, int K, int N,
                              float *b_fused, void *ws, size_t ws_bytes, scap_stream_t stream) {
    if (!m) return SCAP_ERR_INVALID_ARG;
    scap_status stt = q8_check(m, Wq, wscale, nullptr, b, b_fused, 1, K, N, SCAP_BF16, ws, ws_bytes);
    if (stt != SCAP_OK) return stt;
    FcArgs a;
    memset(&a, 0, sizeof(a));
    a.W = Wq; a.wscale = wscale; a.K = K; a.ldw = N; a.Nh = N; a.B = 1; a.tn = Q8_TN; a.S = q8_split(K, N);
    a.x = m; a.x_ld = K; a.bias = b; a.y = b_fused; a.y_ld = N;
    a.l2_hints = g_tune.l2_hints; a.status = tc_status_ptr();
    a.hold_dependents = 1;  // it writes a parameter: ordinary stream order on both sides
    return cuda_status(launch_q8(MODE_DENSE, 2, a, reinterpret_cast<cudaStream_t>(stream)));
}

}  // extern "C"

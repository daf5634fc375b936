// Entry points of the decode-time sparse FC, the dense baseline, bias folding and the host-buffer
// variant, plus the launch plumbing shared with the SwiGLU and MoE entry points.
#include <string.h>

#include "scap_fc.cuh"

namespace scap {

Tuning g_tune = {0, 1};

scap_status check_device() {
    static int cached[64];  // 0 unknown, 1 ok, 2 unsupported
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return SCAP_ERR_CUDA;
    }
    if (dev >= 0 && dev < 64 && cached[dev]) return cached[dev] == 1 ? SCAP_OK : SCAP_ERR_UNSUPPORTED_ARCH;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return SCAP_ERR_CUDA;
    }
    if (dev >= 0 && dev < 64) cached[dev] = major == 10 ? 1 : 2;
    return major == 10 ? SCAP_OK : SCAP_ERR_UNSUPPORTED_ARCH;
}

int sm_count() {
    static int cached = 0;
    if (cached) return cached;
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        n <= 0) {
        cudaGetLastError();
        return 148;  // B200; used only so that workspace queries work on a machine without a GPU
    }
    cached = n;
    return n;
}

// Split-K factor: fill every SM with four resident CTAs in a single wave, but keep at least 32 rows
// per slice at full density.
int choose_split(int K, int tiles_total) {
    if (g_tune.split_k > 0) return g_tune.split_k < MAX_SPLIT ? g_tune.split_k : MAX_SPLIT;
    const int target = sm_count() * 4;
    int S = (target + tiles_total / 2) / tiles_total;
    const int by_rows = (K + 31) / 32;
    if (S > by_rows) S = by_rows;
    if (S > MAX_SPLIT) S = MAX_SPLIT;
    if (S < 1) S = 1;
    return S;
}

FcLayout fc_layout(int B, int K, int N, int halves, size_t base) {
    FcLayout L;
    const int Nh = N / halves;
    L.nchunks = (K + CH - 1) / CH;
    L.Kpad = L.nchunks * CH;
    L.tiles = halves * ((Nh + TN - 1) / TN);
    L.S = choose_split(K, L.tiles);
    size_t off = align_up(base, 256);
    L.counts = off;
    off = align_up(off + sizeof(int) * L.nchunks, 256);
    L.tickets = off;
    off = align_up(off + sizeof(int) * L.tiles, 256);
    L.idx_local = off;
    off = align_up(off + sizeof(uint32_t) * L.Kpad, 256);
    L.xs_local = off;
    off = align_up(off + sizeof(float) * (size_t)B * L.Kpad, 256);
    L.partials = off;
    off = align_up(off + sizeof(float) * (size_t)L.S * B * N, 256);
    L.total = off;
    return L;
}

void bind_layout(GemvArgs &a, const FcLayout &L, unsigned char *ws) {
    a.S = L.S;
    a.counts = reinterpret_cast<const int *>(ws + L.counts);
    a.idx_local = reinterpret_cast<const uint32_t *>(ws + L.idx_local);
    a.xs_local = reinterpret_cast<const float *>(ws + L.xs_local);
    a.Kpad = L.Kpad;
    a.nchunks = L.nchunks;
    a.partials = reinterpret_cast<float *>(ws + L.partials);
    a.tickets = reinterpret_cast<int *>(ws + L.tickets);
}

template <typename XT>
cudaError_t launch_compact(const XT *x, const float *m, const float *tau, int B, int K, const FcLayout &L, unsigned char *ws,
                           int ntickets, cudaStream_t st) {
    return launch(compact_kernel<XT>, dim3(L.nchunks), dim3(CH), 0, st, g_tune.pdl != 0, x, m, tau, B, K,
                  reinterpret_cast<int *>(ws + L.counts), reinterpret_cast<uint32_t *>(ws + L.idx_local),
                  reinterpret_cast<float *>(ws + L.xs_local), L.Kpad, reinterpret_cast<int *>(ws + L.tickets), ntickets);
}
template cudaError_t launch_compact<__half>(const __half *, const float *, const float *, int, int, const FcLayout &,
                                            unsigned char *, int, cudaStream_t);
template cudaError_t launch_compact<__nv_bfloat16>(const __nv_bfloat16 *, const float *, const float *, int, int,
                                                   const FcLayout &, unsigned char *, int, cudaStream_t);

template <bool BF16, int BT, int MODE, typename XT, int EPI>
static cudaError_t launch_gemv_t(const GemvArgs &a, cudaStream_t st) {
    const int tiles = a.halves * ((a.Nh + TN - 1) / TN);
    return launch(gemv_kernel<BF16, BT, MODE, XT, EPI>, dim3(tiles, a.S), dim3(GEMV_THREADS), 0, st, g_tune.pdl != 0, a);
}

template <bool BF16, int MODE, typename XT, int EPI>
static cudaError_t launch_gemv_bt(const GemvArgs &a, cudaStream_t st) {
    switch (batch_tile(a.B)) {
        case 1: return launch_gemv_t<BF16, 1, MODE, XT, EPI>(a, st);
        case 2: return launch_gemv_t<BF16, 2, MODE, XT, EPI>(a, st);
        case 4: return launch_gemv_t<BF16, 4, MODE, XT, EPI>(a, st);
        case 8: return launch_gemv_t<BF16, 8, MODE, XT, EPI>(a, st);
        default: return launch_gemv_t<BF16, 16, MODE, XT, EPI>(a, st);
    }
}

cudaError_t launch_gemv(bool bf16, int mode, int xkind, int epi, const GemvArgs &a, cudaStream_t st) {
    if (mode == MODE_GATHER) {
        if (epi == EPI_GLU)
            return bf16 ? launch_gemv_bt<true, MODE_GATHER, float, EPI_GLU>(a, st)
                        : launch_gemv_bt<false, MODE_GATHER, float, EPI_GLU>(a, st);
        return bf16 ? launch_gemv_bt<true, MODE_GATHER, float, EPI_BIAS>(a, st)
                    : launch_gemv_bt<false, MODE_GATHER, float, EPI_BIAS>(a, st);
    }
    if (xkind == 2)  // fp32 activation (the mode vector when folding the bias): batch 1 only
        return bf16 ? launch_gemv_t<true, 1, MODE_DENSE, float, EPI_BIAS>(a, st)
                    : launch_gemv_t<false, 1, MODE_DENSE, float, EPI_BIAS>(a, st);
    return bf16 ? launch_gemv_bt<true, MODE_DENSE, __nv_bfloat16, EPI_BIAS>(a, st)
                : launch_gemv_bt<false, MODE_DENSE, __half, EPI_BIAS>(a, st);
}

static scap_status validate_fc(const void *x, const void *W, const float *y, int B, int K, int N, int dt) {
    if (!x || !W || !y) return SCAP_ERR_INVALID_ARG;
    if (dt != SCAP_F16 && dt != SCAP_BF16) return SCAP_ERR_DTYPE;
    if (B < 1 || B > SCAP_MAX_BATCH || K < 1 || N < 1 || K > MAX_CHUNKS_SMEM * CH) return SCAP_ERR_SHAPE;
    if (N % 8 != 0 || !aligned16(x) || !aligned16(W) || !aligned16(y)) return SCAP_ERR_ALIGN;
    return SCAP_OK;
}

static scap_status sparse_fc_impl(const void *x, const void *W, const float *m, const float *tau, const float *b_fused,
                                  float *y, int B, int K, int N, scap_dtype dt, uint32_t *idx_out, int *nnz_out,
                                  unsigned char *ws, cudaStream_t st) {
    const FcLayout L = fc_layout(B, K, N, 1, 0);
    cudaError_t e = dt == SCAP_BF16
                        ? launch_compact(reinterpret_cast<const __nv_bfloat16 *>(x), m, tau, B, K, L, ws, L.tiles, st)
                        : launch_compact(reinterpret_cast<const __half *>(x), m, tau, B, K, L, ws, L.tiles, st);
    if (e != cudaSuccess) return cuda_status(e);
    GemvArgs a;
    memset(&a, 0, sizeof(a));
    a.W = W; a.K = K; a.ldw = N; a.halves = 1; a.Nh = N; a.B = B;
    bind_layout(a, L, ws);
    a.bias = b_fused; a.y = y; a.idx_out = idx_out; a.nnz_out = nnz_out;
    return cuda_status(launch_gemv(dt == SCAP_BF16, MODE_GATHER, 0, EPI_BIAS, a, st));
}

// The tickets of a dense call are cleared by a one-CTA kernel (the sparse path clears them in its compaction).
__global__ void clear_tickets_kernel(int *tickets, int n) {
    griddep_wait();
    griddep_launch_dependents();
    for (int i = threadIdx.x; i < n; i += blockDim.x) tickets[i] = 0;
}

static scap_status dense_impl(const void *x, int xkind, const void *W, const float *b, const void *b16, float *y, int B,
                              int K, int N, scap_dtype dt, unsigned char *ws, cudaStream_t st) {
    const FcLayout L = fc_layout(B, K, N, 1, 0);
    if (L.S > 1) {
        cudaError_t e = launch(clear_tickets_kernel, dim3(1), dim3(256), 0, st, g_tune.pdl != 0,
                               reinterpret_cast<int *>(ws + L.tickets), L.tiles);
        if (e != cudaSuccess) return cuda_status(e);
    }
    GemvArgs a;
    memset(&a, 0, sizeof(a));
    a.W = W; a.K = K; a.ldw = N; a.halves = 1; a.Nh = N; a.B = B;
    bind_layout(a, L, ws);
    a.x = x;
    a.bias = b; a.bias16 = b16; a.y = y;
    return cuda_status(launch_gemv(dt == SCAP_BF16, MODE_DENSE, xkind, EPI_BIAS, a, st));
}

}  // namespace scap

using namespace scap;

extern "C" {

const char *scap_status_string(scap_status st) {
    switch (st) {
        case SCAP_OK: return "SCAP_OK";
        case SCAP_ERR_INVALID_ARG: return "SCAP_ERR_INVALID_ARG";
        case SCAP_ERR_SHAPE: return "SCAP_ERR_SHAPE";
        case SCAP_ERR_DTYPE: return "SCAP_ERR_DTYPE";
        case SCAP_ERR_ALIGN: return "SCAP_ERR_ALIGN";
        case SCAP_ERR_WORKSPACE: return "SCAP_ERR_WORKSPACE";
        case SCAP_ERR_CUDA: return "SCAP_ERR_CUDA";
        case SCAP_ERR_TIMEOUT: return "SCAP_ERR_TIMEOUT";
        case SCAP_ERR_UNSUPPORTED_ARCH: return "SCAP_ERR_UNSUPPORTED_ARCH";
    }
    return "SCAP_ERR_UNKNOWN";
}

int scap_version(void) { return 1000; }

scap_status scap_tune(const char *key, int value) {
    if (!key) return SCAP_ERR_INVALID_ARG;
    if (!strcmp(key, "split_k")) {
        if (value < 0 || value > MAX_SPLIT) return SCAP_ERR_INVALID_ARG;
        g_tune.split_k = value;
        return SCAP_OK;
    }
    if (!strcmp(key, "pdl")) {
        g_tune.pdl = value != 0;
        return SCAP_OK;
    }
    return SCAP_ERR_INVALID_ARG;
}

size_t scap_fc_workspace(int B, int K, int N) {
    if (B < 1 || B > SCAP_MAX_BATCH || K < 1 || N < 1 || K > MAX_CHUNKS_SMEM * CH) return 0;
    return fc_layout(B, K, N, 1, 0).total;
}

scap_status scap_sparse_fc(const void *x, const void *W, const float *m, const float *tau, const float *b_fused, float *y,
                           int B, int K, int N, scap_dtype dt, uint32_t *idx_out, int *nnz_out, void *ws, size_t ws_bytes,
                           scap_stream_t stream) {
    scap_status st = validate_fc(x, W, y, B, K, N, dt);
    if (st != SCAP_OK) return st;
    if (!tau || !ws) return SCAP_ERR_INVALID_ARG;
    if (!aligned16(ws) || (m && !aligned16(m)) || (b_fused && !aligned16(b_fused))) return SCAP_ERR_ALIGN;
    if (ws_bytes < scap_fc_workspace(B, K, N)) return SCAP_ERR_WORKSPACE;
    if ((st = check_device()) != SCAP_OK) return st;
    return sparse_fc_impl(x, W, m, tau, b_fused, y, B, K, N, dt, idx_out, nnz_out, static_cast<unsigned char *>(ws),
                          reinterpret_cast<cudaStream_t>(stream));
}

scap_status scap_dense_fc(const void *x, const void *W, const float *b, float *y, int B, int K, int N, scap_dtype dt,
                          void *ws, size_t ws_bytes, scap_stream_t stream) {
    scap_status st = validate_fc(x, W, y, B, K, N, dt);
    if (st != SCAP_OK) return st;
    if (!ws) return SCAP_ERR_INVALID_ARG;
    if (!aligned16(ws) || (b && !aligned16(b))) return SCAP_ERR_ALIGN;
    if (ws_bytes < scap_fc_workspace(B, K, N)) return SCAP_ERR_WORKSPACE;
    if ((st = check_device()) != SCAP_OK) return st;
    return dense_impl(x, dt == SCAP_BF16 ? 1 : 0, W, b, nullptr, y, B, K, N, dt, static_cast<unsigned char *>(ws),
                      reinterpret_cast<cudaStream_t>(stream));
}

size_t scap_fold_bias_workspace(int K, int N) { return scap_fc_workspace(1, K, N); }

scap_status scap_fold_bias(const void *W, const float *m, const void *b, int K, int N, scap_dtype dt, float *b_fused,
                           void *ws, size_t ws_bytes, scap_stream_t stream) {
    scap_status st = validate_fc(m, W, b_fused, 1, K, N, dt);
    if (st != SCAP_OK) return st;
    if (!ws) return SCAP_ERR_INVALID_ARG;
    if (!aligned16(ws) || (b && !aligned16(b))) return SCAP_ERR_ALIGN;
    if (ws_bytes < scap_fold_bias_workspace(K, N)) return SCAP_ERR_WORKSPACE;
    if ((st = check_device()) != SCAP_OK) return st;
    return dense_impl(m, 2, W, nullptr, b, b_fused, 1, K, N, dt, static_cast<unsigned char *>(ws),
                      reinterpret_cast<cudaStream_t>(stream));
}

size_t scap_fc_host_workspace(int B, int K, int N) {
    const size_t fc = scap_fc_workspace(B, K, N);
    if (!fc) return 0;
    return fc + align_up((size_t)B * K * 2, 256) + align_up((size_t)B * N * 4, 256);
}

scap_status scap_sparse_fc_host(const void *x_host, const void *W, const float *m, const float *tau, const float *b_fused,
                                float *y_host, int B, int K, int N, scap_dtype dt, void *ws, size_t ws_bytes,
                                scap_stream_t stream) {
    if (!x_host || !y_host || !W || !tau || !ws) return SCAP_ERR_INVALID_ARG;
    if (dt != SCAP_F16 && dt != SCAP_BF16) return SCAP_ERR_DTYPE;
    if (B < 1 || B > SCAP_MAX_BATCH || K < 1 || N < 1 || K > MAX_CHUNKS_SMEM * CH) return SCAP_ERR_SHAPE;
    if (N % 8 != 0 || !aligned16(W) || !aligned16(ws) || (m && !aligned16(m)) || (b_fused && !aligned16(b_fused)))
        return SCAP_ERR_ALIGN;
    if (ws_bytes < scap_fc_host_workspace(B, K, N)) return SCAP_ERR_WORKSPACE;
    scap_status st = check_device();
    if (st != SCAP_OK) return st;
    unsigned char *w = static_cast<unsigned char *>(ws);
    const size_t fc = scap_fc_workspace(B, K, N);
    unsigned char *x_dev = w + fc;
    float *y_dev = reinterpret_cast<float *>(w + fc + align_up((size_t)B * K * 2, 256));
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(x_dev, x_host, (size_t)B * K * 2, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_status(e);
    st = sparse_fc_impl(x_dev, W, m, tau, b_fused, y_dev, B, K, N, dt, nullptr, nullptr, w, s);
    if (st != SCAP_OK) return st;
    e = cudaMemcpyAsync(y_host, y_dev, (size_t)B * N * 4, cudaMemcpyDeviceToHost, s);
    return cuda_status(e);
}

}  // extern "C"

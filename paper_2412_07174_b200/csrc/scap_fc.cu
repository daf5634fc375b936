// Entry points of the decode-time sparse FC, the dense baseline, bias folding and the host-buffer
// variant, plus the launch plumbing shared with the SwiGLU and MoE entry points.
#include <string.h>

#include <atomic>

#include "scap_fc.cuh"

namespace scap {

Tuning g_tune = {0, 1, 1, 1, 4, 16, 1, 0, 0, 0, 1};

scap_status check_device() {
    static std::atomic<int> cached[64];  // 0 unknown, 1 ok, 2 unsupported
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return SCAP_ERR_CUDA;
    }
    if (dev >= 0 && dev < 64) {
        const int hit = cached[dev].load(std::memory_order_relaxed);
        if (hit) return hit == 1 ? SCAP_OK : SCAP_ERR_UNSUPPORTED_ARCH;
    }
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return SCAP_ERR_CUDA;
    }
    if (dev >= 0 && dev < 64) cached[dev].store(major == 10 ? 1 : 2, std::memory_order_relaxed);
    return major == 10 ? SCAP_OK : SCAP_ERR_UNSUPPORTED_ARCH;
}

int sm_count() {
    static std::atomic<int> cached_by_dev[64];
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) {
        const int hit = cached_by_dev[dev].load(std::memory_order_relaxed);
        if (hit) return hit;
    } else {
        cudaGetLastError();
    }
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        n <= 0) {
        cudaGetLastError();
        return 148;  // B200; used only so that queries work on a machine without a GPU
    }
    if (dev >= 0 && dev < 64) cached_by_dev[dev].store(n, std::memory_order_relaxed);
    return n;
}

// CTAs of clusters of size S that can be resident at once, as the runtime reports it for this device (a cluster
// needs S SMs of one GPC with a free CTA slot, so the figure depends on how the device's SMs are grouped and is a
// little below 2 * SMs for S > 1).  Queried once per size for the batch-1 kernel, which has the launch shape of
// all variants (256 threads, two CTAs per SM); 2 * SMs where the query is not possible.
int resident_ctas(int S) {
    static std::atomic<int> cached_by_dev[64][MAX_CLUSTER + 1];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); dev = -1; }
    if (dev >= 0 && dev < 64) {
        const int hit = cached_by_dev[dev][S].load(std::memory_order_relaxed);
        if (hit) return hit;
    }
    int n = 2 * sm_count();
    if (S > 1) {
        auto kern = fc_kernel<true, 1, MODE_GATHER, __nv_bfloat16, EPI_BIAS, 128>;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(1, S);
        cfg.blockDim = dim3(FC_THREADS);
        cfg.dynamicSmemBytes = fc_smem_for(1);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 1;
        attr[0].val.clusterDim.y = S;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&clusters, kern, &cfg) == cudaSuccess && clusters > 0) n = clusters * S;
        else cudaGetLastError();
    }
    if (dev >= 0 && dev < 64) cached_by_dev[dev][S].store(n, std::memory_order_relaxed);
    return n;
}

// Two CTAs fit on an SM, so up to 2 * SMs CTAs are resident at once (fewer in clusters, see above).  Among tile widths {128, 256} and cluster
// sizes 8 .. 1 pick the pair with the most CTAs within that budget, keeping at least 64 input channels per slice.
// Ties: fewer fills of the kept-channel stage per CTA (B decides the stage capacity), then the narrower tile (its
// smaller cluster exchanges less), then the larger cluster.
void choose_config(int K, int Nh, int epi, int groups, int B, int *tn_out, int *S_out) {
    const int bt = fc_batch_tile(B), cap = is_mma(bt) ? mma_cap(bt) : fc_cap(bt);
    const int nchunks = (K + 31) / 32;
    int best_tn = g_tune.tile ? g_tune.tile : 256, best_S = 1;
    long long best = -1;
    for (int tn = 128; tn <= 256; tn <<= 1) {
        if (g_tune.tile && tn != g_tune.tile) continue;
        const int tiles = fc_tiles(Nh, epi, tn);
        for (int S = MAX_CLUSTER; S >= 1; --S) {
            if (g_tune.split_k > 0 && S > g_tune.split_k) continue;
            if (S > 1 && K / S < 64) continue;
            const long long ctas = (long long)tiles * groups * S;
            const int budget = resident_ctas(S);
            if (ctas > budget && !(S == 1 && tn == (g_tune.tile ? g_tune.tile : 256))) continue;
            const int fills = ((nchunks + S - 1) / S * 32 + cap - 1) / cap;
            const long long score = ctas > budget ? 0 : ctas * 64 + (63 - (fills < 63 ? fills : 63));
            if (score > best) { best = score; best_tn = tn; best_S = S; }
        }
    }
    *tn_out = best_tn;
    *S_out = best_S;
}

template <bool BF16, int BT, int MODE, typename XT, int EPI, int TNT, int PUT>
static cudaError_t launch_fc_pu(const FcArgs &a, cudaStream_t st) {
    static SmemOptIn opt_in;
    auto kern = fc_kernel<BF16, BT, MODE, XT, EPI, TNT, PUT>;
    cudaError_t e0 = ensure_dynamic_smem(kern, fc_smem_for(BT), opt_in);
    if (e0 != cudaSuccess) return e0;
    return launch_cluster(kern, dim3(fc_tiles(a.Nh, EPI, TNT), a.S), dim3(FC_THREADS), fc_smem_for(BT), a.S, st,
                          g_tune.pdl != 0, a);
}

// The fp32-FMA bodies come unrolled for 2, 4, 6 (and, up to batch 2, 8) chunk slots per warp: the smallest one that takes
// the rank's channels in one fill, else the largest (several fills).
template <bool BF16, int BT, int MODE, typename XT, int EPI, int TNT>
static cudaError_t launch_fc_tn(const FcArgs &a, cudaStream_t st) {
    if constexpr (is_mma(BT)) {
        return launch_fc_pu<BF16, BT, MODE, XT, EPI, TNT, fc_pu(BT)>(a, st);
    } else {
        const int per_rank = ((a.K + 31) / 32 + a.S - 1) / a.S, need = (per_rank + FC_WARPS - 1) / FC_WARPS;
        if (need <= 2) return launch_fc_pu<BF16, BT, MODE, XT, EPI, TNT, 2>(a, st);
        if (need <= 4) return launch_fc_pu<BF16, BT, MODE, XT, EPI, TNT, 4>(a, st);
        if (need <= 6 || fc_pu(BT) == 6) return launch_fc_pu<BF16, BT, MODE, XT, EPI, TNT, 6>(a, st);
        return launch_fc_pu<BF16, BT, MODE, XT, EPI, TNT, fc_pu(BT)>(a, st);
    }
}

template <bool BF16, int BT, int MODE, typename XT, int EPI>
static cudaError_t launch_fc_t(const FcArgs &a, cudaStream_t st) {
    return a.tn == 128 ? launch_fc_tn<BF16, BT, MODE, XT, EPI, 128>(a, st) : launch_fc_tn<BF16, BT, MODE, XT, EPI, 256>(a, st);
}

template <bool BF16, int MODE, typename XT, int EPI>
static cudaError_t launch_fc_bt(const FcArgs &a, cudaStream_t st) {
    switch (fc_batch_tile(a.B)) {
        case 1: return launch_fc_t<BF16, 1, MODE, XT, EPI>(a, st);
        case 2: return launch_fc_t<BF16, 2, MODE, XT, EPI>(a, st);
        case 4: return launch_fc_t<BF16, 4, MODE, XT, EPI>(a, st);
        case 8: return launch_fc_t<BF16, 8, MODE, XT, EPI>(a, st);
        default: return launch_fc_t<BF16, 16, MODE, XT, EPI>(a, st);
    }
}

template <bool BF16>
static cudaError_t launch_fc_w(int mode, int xkind, int epi, const FcArgs &a, cudaStream_t st) {
    using ST = typename std::conditional<BF16, __nv_bfloat16, __half>::type;
    if (mode == MODE_DENSE) {
        if (xkind == 2) return launch_fc_t<BF16, 1, MODE_DENSE, float, EPI_BIAS>(a, st);  // bias folding: x = m, batch 1
        return launch_fc_bt<BF16, MODE_DENSE, ST, EPI_BIAS>(a, st);
    }
    if (epi == EPI_GLU) return launch_fc_bt<BF16, MODE_GATHER, ST, EPI_GLU>(a, st);
    if (xkind == 2) return launch_fc_bt<BF16, MODE_GATHER, float, EPI_BIAS>(a, st);  // down projection reading fp32 z
    return launch_fc_bt<BF16, MODE_GATHER, ST, EPI_BIAS>(a, st);
}

cudaError_t launch_fc(bool bf16, int mode, int xkind, int epi, const FcArgs &a, cudaStream_t st) {
    if (ds_applicable(a, epi, bf16)) {
        FcArgs t = a;
        t.tn = 128;
        t.S = ds_choose_split(a.K, a.Nh, epi);
        t.spin = g_tune.tc_spin;
        t.status = tc_status_ptr();
        return launch_fc_ds(bf16, mode, xkind, epi, t, st);
    }
    if (tc_applicable(a, epi, bf16)) {
        FcArgs t = a;
        t.tn = 256;
        t.S = tc_choose_split(a.K, a.Nh, epi, a.B, bf16);
        t.spin = g_tune.tc_spin;
        return launch_fc_tc(bf16, mode, xkind, epi, t, st);
    }
    FcArgs f = a;
    f.l2_hints = g_tune.l2_hints;
    // A dense call needs every row, so the head of its stream is always asked for early (nothing is wasted); a sparse
    // call only on request (tune key "head_rows"): what it asks for and then prunes is extra traffic.
    f.head_rows = g_tune.head_rows > 0 ? g_tune.head_rows : (mode == MODE_DENSE ? 4 : 0);
    f.status = tc_status_ptr();
    return bf16 ? launch_fc_w<true>(mode, xkind, epi, f, st) : launch_fc_w<false>(mode, xkind, epi, f, st);
}

// Copies n16 16-byte words from device-addressable host memory into device memory (one word per thread).
__global__ void __launch_bounds__(256) pull_host_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, long long n16) {
    griddep_wait();               // the previous kernel in the stream may still read dst
    griddep_launch_dependents();  // the FC kernel that follows waits for this grid before it reads dst
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n16) dst[i] = src[i];
}

// One CTA of 1024 threads: popcount prefix over the mask words, then every word's thread writes its set bits.
__global__ void __launch_bounds__(1024) expand_bits_kernel(const uint32_t *__restrict__ bits, int K,
                                                          uint32_t *__restrict__ idx_out, int *__restrict__ nnz_out) {
    __shared__ int s_warp[32];
    __shared__ int s_carry;
    griddep_wait();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nwords = (K + 31) >> 5;
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (int w0 = 0; w0 < nwords; w0 += 1024) {
        const int w = w0 + tid;
        const uint32_t word = w < nwords ? __ldcg(bits + w) : 0u;
        const int c = __popc(word);
        int v = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, v, o);
            if (lane >= o) v += t;
        }
        if (lane == 31) s_warp[warp] = v;
        __syncthreads();
        int base = s_carry;
        for (int q = 0; q < warp; ++q) base += s_warp[q];
        int pos = base + v - c;
        if (idx_out) {
            uint32_t rem = word;
            while (rem) {
                const int bit = __ffs(rem) - 1;
                rem &= rem - 1;
                idx_out[pos++] = (uint32_t)(w * 32 + bit);
            }
        }
        __syncthreads();
        if (tid == 1023) s_carry = base + v;
        __syncthreads();
    }
    if (tid == 0 && nnz_out) *nnz_out = s_carry;
}

cudaError_t launch_expand_bits(const uint32_t *bits, int K, uint32_t *idx_out, int *nnz_out, cudaStream_t st) {
    return launch(expand_bits_kernel, dim3(1), dim3(1024), 0, st, false, bits, K, idx_out, nnz_out);
}

static scap_status validate_fc(const void *x, const void *W, const float *y, int B, int K, int N, int dt) {
    if (!x || !W || !y) return SCAP_ERR_INVALID_ARG;
    if (dt != SCAP_F16 && dt != SCAP_BF16) return SCAP_ERR_DTYPE;
    if (B < 1 || B > SCAP_MAX_BATCH || K < 1 || N < 1 || K > SCAP_MAX_K) return SCAP_ERR_SHAPE;
    if (N % 8 != 0 || !aligned16(x) || !aligned16(W) || !aligned16(y)) return SCAP_ERR_ALIGN;
    return SCAP_OK;
}

static size_t bits_bytes(int K) { return align_up(sizeof(uint32_t) * ((K + 31) / 32), 256); }

static scap_status sparse_fc_impl(const void *x, const void *W, const float *m, const float *tau, const float *b_fused,
                                  float *y, int B, int K, int N, scap_dtype dt, uint32_t *idx_out, int *nnz_out,
                                  unsigned char *ws, cudaStream_t st) {
    FcArgs a;
    memset(&a, 0, sizeof(a));
    a.W = W; a.K = K; a.ldw = N; a.Nh = N; a.B = B;
    choose_config(K, N, EPI_BIAS, 1, B, &a.tn, &a.S);
    a.x = x; a.x_ld = K; a.m = m; a.tau = tau; a.bias = b_fused; a.y = y; a.y_ld = N;
    const bool inspect = idx_out || nnz_out;
    if (inspect) a.bits = reinterpret_cast<uint32_t *>(ws);
    cudaError_t e = launch_fc(dt == SCAP_BF16, MODE_GATHER, dt == SCAP_BF16 ? 1 : 0, EPI_BIAS, a, st);
    if (e != cudaSuccess) return cuda_status(e);
    if (inspect) e = launch_expand_bits(a.bits, K, idx_out, nnz_out, st);
    return cuda_status(e);
}

static scap_status dense_impl(const void *x, int xkind, const void *W, const float *b, const void *b16, float *y, int B,
                              int K, int N, scap_dtype dt, cudaStream_t st, bool writes_parameters) {
    FcArgs a;
    memset(&a, 0, sizeof(a));
    a.W = W; a.K = K; a.ldw = N; a.Nh = N; a.B = B;
    choose_config(K, N, EPI_BIAS, 1, B, &a.tn, &a.S);
    a.x = x; a.x_ld = K; a.bias = b; a.bias16 = b16; a.y = y; a.y_ld = N;
    a.hold_dependents = writes_parameters ? 1 : 0;
    return cuda_status(launch_fc(dt == SCAP_BF16, MODE_DENSE, xkind, EPI_BIAS, a, st));
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

int scap_version(void) { return 1002; }

scap_status scap_device_status(void) {
    const int v = tc_take_status();
    if (v < 0) return SCAP_ERR_CUDA;
    return v == 0 ? SCAP_OK : SCAP_ERR_TIMEOUT;
}

scap_status scap_tune(const char *key, int value) {
    if (!key) return SCAP_ERR_INVALID_ARG;
    if (!strcmp(key, "split_k")) {
        if (value < 0 || value > MAX_CLUSTER) return SCAP_ERR_INVALID_ARG;
        g_tune.split_k = value;
        return SCAP_OK;
    }
    if (!strcmp(key, "pdl")) {
        g_tune.pdl = value != 0;
        return SCAP_OK;
    }
    if (!strcmp(key, "host_direct")) {
        g_tune.host_direct = value != 0;
        return SCAP_OK;
    }
    if (!strcmp(key, "fma_rows")) {
        if (value != 2 && value != 4) return SCAP_ERR_INVALID_ARG;
        g_tune.fma_rows = value;
        return SCAP_OK;
    }
    if (!strcmp(key, "cal_strip")) {
        if (value != 16 && value != 32) return SCAP_ERR_INVALID_ARG;
        g_tune.cal_strip = value;
        return SCAP_OK;
    }
    if (!strcmp(key, "l2_hints")) {
        g_tune.l2_hints = value != 0;
        return SCAP_OK;
    }
    if (!strcmp(key, "head_rows")) {
        if (value < 0 || value > 64) return SCAP_ERR_INVALID_ARG;
        g_tune.head_rows = value;
        return SCAP_OK;
    }
    if (!strcmp(key, "tile")) {
        if (value != 0 && value != 128 && value != 256) return SCAP_ERR_INVALID_ARG;
        g_tune.tile = value;
        return SCAP_OK;
    }
    if (!strcmp(key, "dense_stream")) {
        if (value < 0 || value > 2) return SCAP_ERR_INVALID_ARG;
        g_tune.dense_stream = value;
        return SCAP_OK;
    }
    if (!strcmp(key, "tc_spin")) {
        if (value < 0) return SCAP_ERR_INVALID_ARG;
        g_tune.tc_spin = value;
        return SCAP_OK;
    }
    if (!strcmp(key, "tcgen05")) {
        if (value < 0 || value > 2) return SCAP_ERR_INVALID_ARG;
        g_tune.tc = value;
        return SCAP_OK;
    }
    return SCAP_ERR_INVALID_ARG;
}

size_t scap_fc_workspace(int B, int K, int N) {
    if (B < 1 || B > SCAP_MAX_BATCH || K < 1 || N < 1 || K > SCAP_MAX_K) return 0;
    return bits_bytes(K);
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
    return dense_impl(x, dt == SCAP_BF16 ? 1 : 0, W, b, nullptr, y, B, K, N, dt, reinterpret_cast<cudaStream_t>(stream), false);
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
    return dense_impl(m, 2, W, nullptr, b, b_fused, 1, K, N, dt, reinterpret_cast<cudaStream_t>(stream), true);
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
    if (B < 1 || B > SCAP_MAX_BATCH || K < 1 || N < 1 || K > SCAP_MAX_K) return SCAP_ERR_SHAPE;
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
    // Page-locked buffers that the device can address (cudaHostAlloc / cudaHostRegister memory under unified
    // addressing): a small kernel pulls x across the bus once into the workspace, and the FC kernel writes each
    // element of y straight to host memory - two launches instead of copy, launch, copy.  (Reading x in place from
    // the FC kernel would fetch it once per column tile over the bus; measured slower.)  Anything else goes
    // through the staging copies below.
    if (g_tune.host_direct) {
        cudaPointerAttributes ax, ay;
        const bool okx = cudaPointerGetAttributes(&ax, x_host) == cudaSuccess && ax.type == cudaMemoryTypeHost && ax.devicePointer;
        const bool oky = okx && cudaPointerGetAttributes(&ay, y_host) == cudaSuccess && ay.type == cudaMemoryTypeHost && ay.devicePointer;
        if (!okx || !oky) cudaGetLastError();
        if (okx && oky && aligned16(ax.devicePointer) && aligned16(ay.devicePointer) && ((size_t)B * K * 2) % 16 == 0) {
            const long long n16 = (long long)B * K * 2 / 16;
            const int blocks = (int)((n16 + 255) / 256);
            cudaError_t e = launch(pull_host_kernel, dim3(blocks), dim3(256), 0, s, g_tune.pdl != 0,
                                   static_cast<const uint4 *>(ax.devicePointer), reinterpret_cast<uint4 *>(x_dev), n16);
            if (e != cudaSuccess) return cuda_status(e);
            return sparse_fc_impl(x_dev, W, m, tau, b_fused, static_cast<float *>(ay.devicePointer), B, K, N, dt, nullptr, nullptr, w, s);
        }
    }
    cudaError_t e = cudaMemcpyAsync(x_dev, x_host, (size_t)B * K * 2, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_status(e);
    st = sparse_fc_impl(x_dev, W, m, tau, b_fused, y_dev, B, K, N, dt, nullptr, nullptr, w, s);
    if (st != SCAP_OK) return st;
    e = cudaMemcpyAsync(y_host, y_dev, (size_t)B * N * 4, cudaMemcpyDeviceToHost, s);
    return cuda_status(e);
}

}  // extern "C"

// SwiGLU FFN block (Alg. 2): compaction of h -> gather-GEMV over the packed gate|up weight whose
// second pass also forms z = up * silu(gate) and compacts it -> gather-GEMV over the down weight.
#include <string.h>

#include "scap_fc.cuh"

namespace scap {

// One CTA: prefix over the chunk counts, then every chunk's local list is copied to its global offset.
__global__ void expand_idx_kernel(const int *__restrict__ counts, const uint32_t *__restrict__ idx_local, int nchunks,
                                  uint32_t *__restrict__ idx_out, int *__restrict__ nnz_out) {
    __shared__ int s_prefix[MAX_CHUNKS_SMEM + 1];
    griddep_wait();
    if (threadIdx.x == 0) {
        int acc = 0;
        for (int c = 0; c < nchunks; ++c) {
            s_prefix[c] = acc;
            acc += counts[c];
        }
        s_prefix[nchunks] = acc;
        if (nnz_out) *nnz_out = acc;
    }
    __syncthreads();
    if (!idx_out) return;
    for (int c = 0; c < nchunks; ++c) {
        const int n = s_prefix[c + 1] - s_prefix[c];
        for (int j = threadIdx.x; j < n; j += blockDim.x) idx_out[s_prefix[c] + j] = idx_local[(size_t)c * CH + j];
    }
}

cudaError_t launch_expand_idx(const int *counts, const uint32_t *idx_local, int nchunks, uint32_t *idx_out, int *nnz_out,
                              cudaStream_t st) {
    return launch(expand_idx_kernel, dim3(1), dim3(256), 0, st, false, counts, idx_local, nchunks, idx_out, nnz_out);
}

struct GluLayout {
    FcLayout s1, s2;  // stage 1: K = D, N = 2F (two halves); stage 2: K = F, N = D
    size_t total;
};

static GluLayout glu_layout(int B, int D, int F) {
    GluLayout G;
    G.s1 = fc_layout(B, D, 2 * F, 2, 0);
    G.s2 = fc_layout(B, F, D, 1, G.s1.total);
    G.total = G.s2.total;
    return G;
}

}  // namespace scap

using namespace scap;

extern "C" {

size_t scap_glu_workspace(int B, int D, int F) {
    if (B < 1 || B > SCAP_MAX_BATCH || D < 1 || F < 1 || D > MAX_CHUNKS_SMEM * CH || F > MAX_CHUNKS_SMEM * CH) return 0;
    return glu_layout(B, D, F).total;
}

scap_status scap_glu_ffn(const void *h, const void *Wgu, const void *Wd, const float *m1, const float *tau1,
                         const float *bgu_fused, const float *m2, const float *tau2, const float *bd_fused, float *y, int B,
                         int D, int F, scap_dtype dt, float *z_out, uint32_t *idx1_out, int *nnz1_out, uint32_t *idx2_out,
                         int *nnz2_out, void *ws, size_t ws_bytes, scap_stream_t stream) {
    if (!h || !Wgu || !Wd || !tau1 || !tau2 || !y || !ws) return SCAP_ERR_INVALID_ARG;
    if (dt != SCAP_F16 && dt != SCAP_BF16) return SCAP_ERR_DTYPE;
    if (B < 1 || B > SCAP_MAX_BATCH || D < 1 || F < 1 || D > MAX_CHUNKS_SMEM * CH || F > MAX_CHUNKS_SMEM * CH)
        return SCAP_ERR_SHAPE;
    if (D % 8 != 0 || F % 8 != 0 || !aligned16(h) || !aligned16(Wgu) || !aligned16(Wd) || !aligned16(y) || !aligned16(ws) ||
        (m1 && !aligned16(m1)) || (m2 && !aligned16(m2)) || (bgu_fused && !aligned16(bgu_fused)) ||
        (bd_fused && !aligned16(bd_fused)) || (z_out && !aligned16(z_out)))
        return SCAP_ERR_ALIGN;
    if (ws_bytes < scap_glu_workspace(B, D, F)) return SCAP_ERR_WORKSPACE;
    scap_status stt = check_device();
    if (stt != SCAP_OK) return stt;

    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    unsigned char *w = static_cast<unsigned char *>(ws);
    const GluLayout G = glu_layout(B, D, F);
    const bool bf16 = dt == SCAP_BF16;

    // stage 1: centre + threshold h; the tickets cleared are the per-pair tickets (tiles / 2)
    cudaError_t e = bf16 ? launch_compact(reinterpret_cast<const __nv_bfloat16 *>(h), m1, tau1, B, D, G.s1, w, G.s1.tiles, st)
                         : launch_compact(reinterpret_cast<const __half *>(h), m1, tau1, B, D, G.s1, w, G.s1.tiles, st);
    if (e != cudaSuccess) return cuda_status(e);

    GemvArgs a;
    memset(&a, 0, sizeof(a));
    a.W = Wgu; a.K = D; a.ldw = 2 * F; a.halves = 2; a.Nh = F; a.B = B;
    bind_layout(a, G.s1, w);
    a.bias = bgu_fused;
    a.m2 = m2; a.tau2 = tau2; a.z_out = z_out;
    a.counts2 = reinterpret_cast<int *>(w + G.s2.counts);
    a.idx_local2 = reinterpret_cast<uint32_t *>(w + G.s2.idx_local);
    a.xs_local2 = reinterpret_cast<float *>(w + G.s2.xs_local);
    a.Kpad2 = G.s2.Kpad;
    a.tickets_next = reinterpret_cast<int *>(w + G.s2.tickets);
    a.ntickets_next = G.s2.tiles;
    e = launch_gemv(bf16, MODE_GATHER, 0, EPI_GLU, a, st);
    if (e != cudaSuccess) return cuda_status(e);

    GemvArgs d;
    memset(&d, 0, sizeof(d));
    d.W = Wd; d.K = F; d.ldw = D; d.halves = 1; d.Nh = D; d.B = B;
    bind_layout(d, G.s2, w);
    d.bias = bd_fused; d.y = y; d.idx_out = idx2_out; d.nnz_out = nnz2_out;
    e = launch_gemv(bf16, MODE_GATHER, 0, EPI_BIAS, d, st);
    if (e != cudaSuccess) return cuda_status(e);

    if (idx1_out || nnz1_out) {
        // inspection only: expand the stage-1 chunk-local lists into the global ascending list
        e = launch_expand_idx(reinterpret_cast<const int *>(w + G.s1.counts), reinterpret_cast<const uint32_t *>(w + G.s1.idx_local),
                              G.s1.nchunks, idx1_out, nnz1_out, st);
        if (e != cudaSuccess) return cuda_status(e);
    }
    return SCAP_OK;
}

}  // extern "C"


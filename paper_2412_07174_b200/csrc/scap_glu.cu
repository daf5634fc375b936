// SwiGLU FFN block (Alg. 2): one fused FC kernel over the packed gate|up weight whose cluster
// reduction also forms z = up * silu(gate), then one fused FC kernel over the down weight that
// thresholds z itself.  z (fp32, B x F) is the only intermediate and stays L2-resident.
#include <atomic>
#include <string.h>

#include "scap_fc.cuh"

namespace scap {

struct GluLayout {
    size_t bits1, z, bits2, total;
};

static GluLayout glu_layout(int B, int D, int F) {
    GluLayout G;
    G.bits1 = 0;
    G.z = align_up(sizeof(uint32_t) * ((D + 31) / 32), 256);
    G.bits2 = G.z + align_up(sizeof(float) * (size_t)B * F, 256);
    G.total = G.bits2 + align_up(sizeof(uint32_t) * ((F + 31) / 32), 256);
    return G;
}

}  // namespace scap

using namespace scap;

extern "C" {

size_t scap_glu_workspace(int B, int D, int F) {
    if (B < 1 || B > SCAP_MAX_BATCH || D < 1 || F < 1 || D > SCAP_MAX_K || F > SCAP_MAX_K) return 0;
    return glu_layout(B, D, F).total;
}

// Both two-stage FFN blocks: gated (packed gate|up weight [D, 2F], z = up * silu(gate)) or plain (up weight [D, F],
// z = gelu(up)); the second stage is the sparse down projection on z in either case.
static scap_status ffn_impl(bool gated, const void *h, const void *Wgu, const void *Wd, const float *m1, const float *tau1,
                            const float *bgu_fused, const float *m2, const float *tau2, const float *bd_fused, float *y, int B,
                            int D, int F, scap_dtype dt, float *z_out, uint32_t *idx1_out, int *nnz1_out, uint32_t *idx2_out,
                            int *nnz2_out, void *ws, size_t ws_bytes, scap_stream_t stream) {
    if (!h || !Wgu || !Wd || !tau1 || !tau2 || !y || !ws) return SCAP_ERR_INVALID_ARG;
    if (dt != SCAP_F16 && dt != SCAP_BF16) return SCAP_ERR_DTYPE;
    if (B < 1 || B > SCAP_MAX_BATCH || D < 1 || F < 1 || D > SCAP_MAX_K || F > SCAP_MAX_K) return SCAP_ERR_SHAPE;
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
    float *z = reinterpret_cast<float *>(w + G.z);

    FcArgs a;
    memset(&a, 0, sizeof(a));
    const int epi1 = gated ? EPI_GLU : EPI_BIAS;
    a.W = Wgu; a.K = D; a.ldw = gated ? 2 * F : F; a.Nh = F; a.B = B;
    a.act = gated ? 0 : 1;
    choose_config(D, F, epi1, 1, B, &a.tn, &a.S);
    a.x = h; a.x_ld = D; a.m = m1; a.tau = tau1; a.bias = bgu_fused;
    a.y = z; a.y_ld = F; a.z_copy = z_out;
    if (idx1_out || nnz1_out) a.bits = reinterpret_cast<uint32_t *>(w + G.bits1);
    FcArgs d;
    memset(&d, 0, sizeof(d));
    d.W = Wd; d.K = F; d.ldw = D; d.Nh = D; d.B = B;
    choose_config(F, D, EPI_BIAS, 1, B, &d.tn, &d.S);
    d.x = z; d.x_ld = F; d.m = m2; d.tau = tau2; d.bias = bd_fused; d.y = y; d.y_ld = D;
    if (idx2_out || nnz2_out) d.bits = reinterpret_cast<uint32_t *>(w + G.bits2);
    // The two stages run back to back: either both take the tcgen05 kernel or neither does (measured: a stage on
    // it between two mma.sync stages loses more at the kernel boundaries than it gains).
    // The dense-stream kernel (batches above the FMA limit) takes both stages whenever it takes one.
    const bool ds_both = ds_applicable(a, epi1, bf16) && ds_applicable(d, EPI_BIAS, bf16);
    if (!ds_both && !(tc_applicable(a, epi1, bf16) && tc_applicable(d, EPI_BIAS, bf16))) a.no_tc = d.no_tc = 1;

    cudaError_t e = launch_fc(bf16, MODE_GATHER, bf16 ? 1 : 0, epi1, a, st);
    if (e != cudaSuccess) return cuda_status(e);
    e = launch_fc(bf16, MODE_GATHER, 2, EPI_BIAS, d, st);
    if (e != cudaSuccess) return cuda_status(e);

    if (a.bits) {
        e = launch_expand_bits(a.bits, D, idx1_out, nnz1_out, st);
        if (e != cudaSuccess) return cuda_status(e);
    }
    if (d.bits) {
        e = launch_expand_bits(d.bits, F, idx2_out, nnz2_out, st);
        if (e != cudaSuccess) return cuda_status(e);
    }
    return SCAP_OK;
}

scap_status scap_glu_ffn(const void *h, const void *Wgu, const void *Wd, const float *m1, const float *tau1,
                         const float *bgu_fused, const float *m2, const float *tau2, const float *bd_fused, float *y, int B,
                         int D, int F, scap_dtype dt, float *z_out, uint32_t *idx1_out, int *nnz1_out, uint32_t *idx2_out,
                         int *nnz2_out, void *ws, size_t ws_bytes, scap_stream_t stream) {
    return ffn_impl(true, h, Wgu, Wd, m1, tau1, bgu_fused, m2, tau2, bd_fused, y, B, D, F, dt, z_out, idx1_out, nnz1_out, idx2_out,
                    nnz2_out, ws, ws_bytes, stream);
}

size_t scap_gelu_ffn_workspace(int B, int D, int F) { return scap_glu_workspace(B, D, F); }

scap_status scap_gelu_ffn(const void *h, const void *Wu, const void *Wd, const float *m1, const float *tau1,
                          const float *bu_fused, const float *m2, const float *tau2, const float *bd_fused, float *y, int B,
                          int D, int F, scap_dtype dt, float *z_out, uint32_t *idx1_out, int *nnz1_out, uint32_t *idx2_out,
                          int *nnz2_out, void *ws, size_t ws_bytes, scap_stream_t stream) {
    return ffn_impl(false, h, Wu, Wd, m1, tau1, bu_fused, m2, tau2, bd_fused, y, B, D, F, dt, z_out, idx1_out, nnz1_out, idx2_out,
                    nnz2_out, ws, ws_bytes, stream);
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// SwiGLU block for callers that cannot allocate device memory.
//
// The intermediate z and the mask words of scap_glu_ffn normally live in a caller-provided workspace.
// Here they live in the file-scope array below, which is part of the library image: every GPU that
// loads the library holds these 2 MiB until the process exits.  The array's name is only a host-side
// handle; kernels need its device address, which is looked up once per device with
// cudaGetSymbolAddress (with that device current) and cached.
// ------------------------------------------------------------------------------------------------
namespace scap {

constexpr size_t GLU_STATIC_BYTES = (size_t)2 << 20;
static __device__ __align__(256) unsigned char g_glu_static_scratch[GLU_STATIC_BYTES];

static scap_status glu_static_address(unsigned char **out) {
    static std::atomic<unsigned char *> cached[64];  // first calls may come from several host threads at once
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return SCAP_ERR_CUDA;
    }
    if (dev >= 0 && dev < 64) {
        unsigned char *hit = cached[dev].load(std::memory_order_acquire);
        if (hit) {
            *out = hit;
            return SCAP_OK;
        }
    }
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_glu_static_scratch) != cudaSuccess || p == nullptr) {
        cudaGetLastError();
        return SCAP_ERR_CUDA;
    }
    if (dev >= 0 && dev < 64) cached[dev].store(static_cast<unsigned char *>(p), std::memory_order_release);
    *out = static_cast<unsigned char *>(p);
    return SCAP_OK;
}

}  // namespace scap

extern "C" {

size_t scap_glu_static_capacity(void) { return GLU_STATIC_BYTES; }

scap_status scap_glu_ffn_static(const void *h, const void *Wgu, const void *Wd, const float *m1, const float *tau1,
                                const float *bgu_fused, const float *m2, const float *tau2, const float *bd_fused, float *y,
                                int B, int D, int F, scap_dtype dt, float *z_out, scap_stream_t stream) {
    const size_t need = scap_glu_workspace(B, D, F);
    if (need == 0) return SCAP_ERR_SHAPE;
    if (need > GLU_STATIC_BYTES) return SCAP_ERR_WORKSPACE;  // B * F too large for the built-in scratch
    scap_status st = check_device();
    if (st != SCAP_OK) return st;
    unsigned char *scratch = nullptr;
    if ((st = glu_static_address(&scratch)) != SCAP_OK) return st;
    // Every scratch word that is read is written earlier in the same call (z by the gate|up kernel before the
    // down kernel reads it), so nothing has to be cleared even though the array keeps the previous call's data.
    return scap_glu_ffn(h, Wgu, Wd, m1, tau1, bgu_fused, m2, tau2, bd_fused, y, B, D, F, dt, z_out, nullptr, nullptr, nullptr,
                        nullptr, scratch, GLU_STATIC_BYTES, stream);
}

}  // extern "C"

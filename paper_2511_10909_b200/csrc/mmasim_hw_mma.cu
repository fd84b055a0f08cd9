// The one real MMA interface of this machine (Section 3.2 lists ten; a B200 offers the Blackwell one): single
// warp-level `mma.sync` instructions wrapped as D = MMA(A, B, C), for differential runs of the Blackwell models
// against the hardware they describe (Step 4 of the paper's method, Section 3.1).
//
// One warp owns one tile of 16 rows of A (8 for FP64) and the 8 rows of B^T (B is N x K row-major, N = 8, shared by
// all tiles); K may be a multiple of the instruction's K, in which case the instructions are chained through the
// accumulator exactly like Algorithm 5: d <- MMA(A_t, B_t, d).  Fragments are read straight from global memory with
// the register layouts of the PTX ISA (groupID = lane / 4, tid = lane % 4).
#include <cuda_fp16.h>
#include "mmasim_internal.h"

namespace mmasim {
namespace {

enum HwKind : int {
    HW_F16_F32 = 0,     // m16n8k16  f32 <- f16 x f16 + f32
    HW_F16_F16 = 1,     // m16n8k16  f16 <- f16 x f16 + f16
    HW_BF16_F32 = 2,    // m16n8k16  f32 <- bf16 x bf16 + f32
    HW_TF32_F32 = 3,    // m16n8k8   f32 <- tf32 x tf32 + f32
    HW_E4M3_F32 = 4,    // m16n8k32  f32 <- e4m3 x e4m3 + f32
    HW_E5M2_F32 = 5,    // m16n8k32  f32 <- e5m2 x e5m2 + f32
    HW_F64 = 6,         // m8n8k4    f64 <- f64 x f64 + f64
    HW_F16_F32_K8 = 7,  // m16n8k8   f32 <- f16 x f16 + f32
    HW_TF32_F32_K4 = 8, // m16n8k4   f32 <- tf32 x tf32 + f32
    HW_E4M3_F16 = 9,    // m16n8k32  f16 <- e4m3 x e4m3 + f16
    HW_E5M2_F16 = 10,   // m16n8k32  f16 <- e5m2 x e5m2 + f16
    HW_E4M3_E5M2_F32 = 11,  // m16n8k32  f32 <- e4m3 x e5m2 + f32
    HW_E4M3_F32_K16 = 12,   // m16n8k16  f32 <- e4m3 x e4m3 + f32
    HW_COUNT
};

struct HwShape { int rows, k, in_bytes, acc_bytes; };
__host__ __device__ inline HwShape hw_shape(int kind) {
    switch (kind) {
        case HW_F16_F32: return {16, 16, 2, 4};
        case HW_F16_F16: return {16, 16, 2, 2};
        case HW_BF16_F32: return {16, 16, 2, 4};
        case HW_TF32_F32: return {16, 8, 4, 4};
        case HW_E4M3_F32: return {16, 32, 1, 4};
        case HW_E5M2_F32: return {16, 32, 1, 4};
        case HW_F64: return {8, 4, 8, 8};
        case HW_F16_F32_K8: return {16, 8, 2, 4};
        case HW_E4M3_F16: return {16, 32, 1, 2};
        case HW_E5M2_F16: return {16, 32, 1, 2};
        case HW_E4M3_E5M2_F32: return {16, 32, 1, 4};
        case HW_E4M3_F32_K16: return {16, 16, 1, 4};
        default: return {16, 4, 4, 4};      // HW_TF32_F32_K4
    }
}

template <int KIND>
__global__ void __launch_bounds__(128) hw_mma_kernel(int64_t tiles, int64_t K, const void* A, const void* B, const void* C, void* D) {
    const int lane = threadIdx.x % 32;
    const int64_t tile = int64_t(blockIdx.x) * (blockDim.x / 32) + threadIdx.x / 32;
    if (tile >= tiles) return;                                  // whole warps leave together
    const int gid = lane / 4, tg = lane % 4;
    const HwShape sh = hw_shape(KIND);
    const int64_t row0 = tile * sh.rows;

    if (KIND == HW_F64) {
        const double* a = static_cast<const double*>(A);
        const double* b = static_cast<const double*>(B);
        double d0 = 0.0, d1 = 0.0;
        if (C) { d0 = static_cast<const double*>(C)[(row0 + gid) * 8 + tg * 2]; d1 = static_cast<const double*>(C)[(row0 + gid) * 8 + tg * 2 + 1]; }
        for (int64_t k0 = 0; k0 < K; k0 += 4) {
            const double fa = a[(row0 + gid) * K + k0 + tg], fb = b[int64_t(gid) * K + k0 + tg];
            asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};" : "+d"(d0), "+d"(d1) : "d"(fa), "d"(fb));
        }
        static_cast<double*>(D)[(row0 + gid) * 8 + tg * 2] = d0;
        static_cast<double*>(D)[(row0 + gid) * 8 + tg * 2 + 1] = d1;
        return;
    }

    // accumulator fragment: (row gid, cols 2 tg, 2 tg + 1) and (row gid + 8, same columns)
    uint32_t c[4] = {0u, 0u, 0u, 0u};
    if (C) {
        if (sh.acc_bytes == 4) {
            const uint32_t* cp = static_cast<const uint32_t*>(C);
            c[0] = cp[(row0 + gid) * 8 + tg * 2]; c[1] = cp[(row0 + gid) * 8 + tg * 2 + 1];
            c[2] = cp[(row0 + gid + 8) * 8 + tg * 2]; c[3] = cp[(row0 + gid + 8) * 8 + tg * 2 + 1];
        } else {
            const uint16_t* cp = static_cast<const uint16_t*>(C);
            c[0] = uint32_t(cp[(row0 + gid) * 8 + tg * 2]) | (uint32_t(cp[(row0 + gid) * 8 + tg * 2 + 1]) << 16);
            c[1] = uint32_t(cp[(row0 + gid + 8) * 8 + tg * 2]) | (uint32_t(cp[(row0 + gid + 8) * 8 + tg * 2 + 1]) << 16);
        }
    }
    for (int64_t k0 = 0; k0 < K; k0 += sh.k) {
        uint32_t a[4] = {0u, 0u, 0u, 0u}, b[2] = {0u, 0u};
        if (sh.in_bytes == 2) {
            // 16-bit elements, two per register.  k16: a0 (gid, 2tg..), a1 (gid+8, 2tg..), a2 (gid, 2tg+8..), a3 (gid+8, 2tg+8..);
            // b0 (k 2tg.., n gid), b1 (k 2tg+8.., n gid).  k8: a0, a1 and b0 only.
            const uint16_t* ap = static_cast<const uint16_t*>(A);
            const uint16_t* bp = static_cast<const uint16_t*>(B);
            auto pair = [](const uint16_t* p) { return uint32_t(p[0]) | (uint32_t(p[1]) << 16); };
            a[0] = pair(ap + (row0 + gid) * K + k0 + tg * 2);
            a[1] = pair(ap + (row0 + gid + 8) * K + k0 + tg * 2);
            b[0] = pair(bp + int64_t(gid) * K + k0 + tg * 2);
            if (sh.k == 16) {
                a[2] = pair(ap + (row0 + gid) * K + k0 + tg * 2 + 8);
                a[3] = pair(ap + (row0 + gid + 8) * K + k0 + tg * 2 + 8);
                b[1] = pair(bp + int64_t(gid) * K + k0 + tg * 2 + 8);
            }
        } else if (sh.in_bytes == 4) {
            // TF32.  k8: a0 (gid, tg), a1 (gid+8, tg), a2 (gid, tg+4), a3 (gid+8, tg+4); b0 (k tg, n gid), b1 (k tg+4).  k4: a0, a1, b0.
            const uint32_t* ap = static_cast<const uint32_t*>(A);
            const uint32_t* bp = static_cast<const uint32_t*>(B);
            a[0] = ap[(row0 + gid) * K + k0 + tg];
            a[1] = ap[(row0 + gid + 8) * K + k0 + tg];
            b[0] = bp[int64_t(gid) * K + k0 + tg];
            if (sh.k == 8) {
                a[2] = ap[(row0 + gid) * K + k0 + tg + 4];
                a[3] = ap[(row0 + gid + 8) * K + k0 + tg + 4];
                b[1] = bp[int64_t(gid) * K + k0 + tg + 4];
            }
        } else {
            // 8-bit elements, four per register: a0 (gid, 4tg..), a1 (gid+8, 4tg..), a2 (gid, 4tg+16..), a3 (gid+8, 4tg+16..);
            // b0 (k 4tg.., n gid), b1 (k 4tg+16.., n gid)
            const unsigned char* ap = static_cast<const unsigned char*>(A);
            const unsigned char* bp = static_cast<const unsigned char*>(B);
            auto quad = [](const unsigned char* p) { return uint32_t(p[0]) | (uint32_t(p[1]) << 8) | (uint32_t(p[2]) << 16) | (uint32_t(p[3]) << 24); };
            a[0] = quad(ap + (row0 + gid) * K + k0 + tg * 4);
            a[1] = quad(ap + (row0 + gid + 8) * K + k0 + tg * 4);
            b[0] = quad(bp + int64_t(gid) * K + k0 + tg * 4);
            if (sh.k == 32) {                   // k16: a0, a1 and b0 only
                a[2] = quad(ap + (row0 + gid) * K + k0 + tg * 4 + 16);
                a[3] = quad(ap + (row0 + gid + 8) * K + k0 + tg * 4 + 16);
                b[1] = quad(bp + int64_t(gid) * K + k0 + tg * 4 + 16);
            }
        }
        if (KIND == HW_F16_F32)
            asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
        else if (KIND == HW_F16_F16)
            asm volatile("mma.sync.aligned.m16n8k16.row.col.f16.f16.f16.f16 {%0,%1}, {%2,%3,%4,%5}, {%6,%7}, {%0,%1};"
                         : "+r"(c[0]), "+r"(c[1]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
        else if (KIND == HW_BF16_F32)
            asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
        else if (KIND == HW_TF32_F32)
            asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
        else if (KIND == HW_E4M3_F32)
            asm volatile("mma.sync.aligned.m16n8k32.row.col.f32.e4m3.e4m3.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
        else if (KIND == HW_E5M2_F32)
            asm volatile("mma.sync.aligned.m16n8k32.row.col.f32.e5m2.e5m2.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
        else if (KIND == HW_E4M3_F16)
            asm volatile("mma.sync.aligned.m16n8k32.row.col.f16.e4m3.e4m3.f16 {%0,%1}, {%2,%3,%4,%5}, {%6,%7}, {%0,%1};"
                         : "+r"(c[0]), "+r"(c[1]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
        else if (KIND == HW_E5M2_F16)
            asm volatile("mma.sync.aligned.m16n8k32.row.col.f16.e5m2.e5m2.f16 {%0,%1}, {%2,%3,%4,%5}, {%6,%7}, {%0,%1};"
                         : "+r"(c[0]), "+r"(c[1]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
        else if (KIND == HW_E4M3_E5M2_F32)
            asm volatile("mma.sync.aligned.m16n8k32.row.col.f32.e4m3.e5m2.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
        else if (KIND == HW_E4M3_F32_K16)
            asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.e4m3.e4m3.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                         : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(b[0]));
        else if (KIND == HW_F16_F32_K8)
            asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                         : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(b[0]));
        else if (KIND == HW_TF32_F32_K4)
            asm volatile("mma.sync.aligned.m16n8k4.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                         : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(b[0]));
    }
    if (sh.acc_bytes == 4) {
        uint32_t* dp = static_cast<uint32_t*>(D);
        dp[(row0 + gid) * 8 + tg * 2] = c[0]; dp[(row0 + gid) * 8 + tg * 2 + 1] = c[1];
        dp[(row0 + gid + 8) * 8 + tg * 2] = c[2]; dp[(row0 + gid + 8) * 8 + tg * 2 + 1] = c[3];
    } else {
        uint16_t* dp = static_cast<uint16_t*>(D);
        dp[(row0 + gid) * 8 + tg * 2] = uint16_t(c[0]); dp[(row0 + gid) * 8 + tg * 2 + 1] = uint16_t(c[0] >> 16);
        dp[(row0 + gid + 8) * 8 + tg * 2] = uint16_t(c[1]); dp[(row0 + gid + 8) * 8 + tg * 2 + 1] = uint16_t(c[1] >> 16);
    }
}

template <int KIND>
cudaError_t launch_hw(int64_t tiles, int64_t K, const void* A, const void* B, const void* C, void* D, cudaStream_t st) {
    const unsigned blocks = unsigned((tiles + 3) / 4);
    hw_mma_kernel<KIND><<<blocks, 128, 0, st>>>(tiles, K, A, B, C, D);
    return cudaGetLastError();
}

}  // namespace

int launch_hw_mma(int kind, int64_t M, int64_t K, const void* A, const void* B, const void* C, void* D, cudaStream_t stream) {
    if (kind < 0 || kind >= HW_COUNT) { set_error("mmasim_hw_mma: unknown kind %d", kind); return MMASIM_ERR_INVALID_ARG; }
    const HwShape sh = hw_shape(kind);
    if (M < sh.rows || M % sh.rows || K < sh.k || K % sh.k) {
        set_error("mmasim_hw_mma: M must be a multiple of %d and K a multiple of %d for this instruction", sh.rows, sh.k);
        return MMASIM_ERR_SHAPE;
    }
    const int64_t tiles = M / sh.rows;
    cudaError_t err;
    switch (kind) {
        case HW_F16_F32: err = launch_hw<HW_F16_F32>(tiles, K, A, B, C, D, stream); break;
        case HW_F16_F16: err = launch_hw<HW_F16_F16>(tiles, K, A, B, C, D, stream); break;
        case HW_BF16_F32: err = launch_hw<HW_BF16_F32>(tiles, K, A, B, C, D, stream); break;
        case HW_TF32_F32: err = launch_hw<HW_TF32_F32>(tiles, K, A, B, C, D, stream); break;
        case HW_E4M3_F32: err = launch_hw<HW_E4M3_F32>(tiles, K, A, B, C, D, stream); break;
        case HW_E5M2_F32: err = launch_hw<HW_E5M2_F32>(tiles, K, A, B, C, D, stream); break;
        case HW_F64: err = launch_hw<HW_F64>(tiles, K, A, B, C, D, stream); break;
        case HW_F16_F32_K8: err = launch_hw<HW_F16_F32_K8>(tiles, K, A, B, C, D, stream); break;
        case HW_E4M3_F16: err = launch_hw<HW_E4M3_F16>(tiles, K, A, B, C, D, stream); break;
        case HW_E5M2_F16: err = launch_hw<HW_E5M2_F16>(tiles, K, A, B, C, D, stream); break;
        case HW_E4M3_E5M2_F32: err = launch_hw<HW_E4M3_E5M2_F32>(tiles, K, A, B, C, D, stream); break;
        case HW_E4M3_F32_K16: err = launch_hw<HW_E4M3_F32_K16>(tiles, K, A, B, C, D, stream); break;
        default: err = launch_hw<HW_TF32_F32_K4>(tiles, K, A, B, C, D, stream); break;
    }
    if (err != cudaSuccess) { set_error("mmasim_hw_mma launch failed: %s", cudaGetErrorString(err)); return MMASIM_ERR_CUDA; }
    return MMASIM_OK;
}

}  // namespace mmasim

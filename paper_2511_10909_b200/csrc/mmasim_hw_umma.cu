// The B200's fifth-generation matrix instruction (tcgen05.mma) as an MMA interface D = MMA(A, B, C) (Section 3.2): the
// instruction class behind the paper's Blackwell rows for FP8 / FP6 / FP4 and the block-scaled types (Table 3's UTC*MMA
// rows, Tables 4 and 5).  One CTA of 128 threads per tile of 128 rows of A; the tile's operands are written to shared
// memory with plain stores in the instruction's canonical K-major layout without swizzling (8-row x 16-byte core
// matrices), C goes into tensor memory with tcgen05.st, one thread issues the instruction(s) (a longer K chains
// instructions through the accumulator in tensor memory, ascending k), and D comes back with tcgen05.ld.
//
// Every wait is bounded: the one wait of the kernel (on the mbarrier that tcgen05.commit arrives at) polls
// mbarrier.try_wait until a clock budget runs out, then records MMASIM_ERR_TIMEOUT in the caller's status word, frees
// the tensor memory it holds and returns.  MMASIM_UMMA_SELFTEST_TIMEOUT exercises exactly that path: nothing is issued,
// so nobody ever arrives at the barrier.
#include <cstdlib>
#include "mmasim_internal.h"

namespace mmasim {
namespace {

constexpr int TILE_M = 128, TILE_N = 16, NTHREADS = 128, TMEM_COLS = 64;
constexpr int SFA_COL = 16, SFB_COL = 32, SF_GROUPS = 4;    // tensor-memory columns: D 0..15, scales of A 16..31, of B 32..47

enum UmmaKind : int {
    UK_F16_F32 = 0, UK_BF16_F32, UK_TF32_F32, UK_E4M3_F32, UK_E5M2_F32, UK_E4M3_E5M2_F32, UK_E2M3_F32, UK_E3M2_F32, UK_E2M1_F32,
    UK_SELFTEST_TIMEOUT,
    UK_MXE4M3, UK_MXE5M2, UK_MXE2M3, UK_MXE3M2, UK_MXE2M1, UK_MXF4, UK_NVF4,
    UK_F16_F16, UK_E4M3_F16, UK_E5M2_F16, UK_E2M1_F16, UK_COUNT
};

struct UmmaShape {
    int elem_bytes;     // storage bytes of an A / B element in global memory (sub-byte types: one per byte)
    int k_instr;        // elements of K per instruction (32 bytes of operand per row)
    int mma_kind;       // 0: kind::f16, 1: kind::tf32, 2: kind::f8f6f4, 3: kind::mxf8f6f4 (one scale per 32 elements),
                        // 4: kind::mxf4 (packed FP4, E8M0 per 32), 5: kind::mxf4nvf4 (packed FP4, UE4M3 per 16)
    int a_fmt, b_fmt;   // format codes of the instruction descriptor
    int sf_per_step;    // scale factors per row and instruction (0: unscaled)
    int acc16;          // 1: FP16 accumulator (C and D are 16-bit words)
};

__host__ __device__ inline UmmaShape umma_shape(int kind) {
    switch (kind) {
        case UK_F16_F32: return {2, 16, 0, 0, 0, 0};
        case UK_BF16_F32: return {2, 16, 0, 1, 1, 0};
        case UK_TF32_F32: return {4, 8, 1, 2, 2, 0};
        case UK_E4M3_F32: return {1, 32, 2, 0, 0, 0};
        case UK_E5M2_F32: return {1, 32, 2, 1, 1, 0};
        case UK_E4M3_E5M2_F32: return {1, 32, 2, 0, 1, 0};
        case UK_E2M3_F32: return {1, 32, 2, 3, 3, 0};
        case UK_E3M2_F32: return {1, 32, 2, 4, 4, 0};
        case UK_E2M1_F32: return {1, 32, 2, 5, 5, 0};
        case UK_MXE4M3: return {1, 32, 3, 0, 0, 1};
        case UK_MXE5M2: return {1, 32, 3, 1, 1, 1};
        case UK_MXE2M3: return {1, 32, 3, 3, 3, 1};
        case UK_MXE3M2: return {1, 32, 3, 4, 4, 1};
        case UK_MXE2M1: return {1, 32, 3, 5, 5, 1};
        case UK_MXF4: return {0, 64, 4, 1, 1, 2};           // elem_bytes 0: two elements per byte
        case UK_NVF4: return {0, 64, 5, 1, 1, 4};
        case UK_F16_F16: return {2, 16, 0, 0, 0, 0, 1};
        case UK_E4M3_F16: return {1, 32, 2, 0, 0, 0, 1};
        case UK_E5M2_F16: return {1, 32, 2, 1, 1, 0, 1};
        case UK_E2M1_F16: return {1, 32, 2, 5, 5, 0, 1};
        default: return {1, 32, 2, 0, 0, 0};
    }
}

// Instruction descriptor: D format (bits 4-5: 1 FP32, 0 FP16), A / B formats (bits 7-9, 10-12), both operands K-major (bits 15,
// 16 = 0), N / 8 in bits 17-22, M / 16 in bits 24-28.
__host__ __device__ inline uint32_t instr_desc(const UmmaShape& s) {
    return (s.acc16 ? 0u : (1u << 4)) | (uint32_t(s.a_fmt) << 7) | (uint32_t(s.b_fmt) << 10) | (uint32_t(TILE_N >> 3) << 17) | (uint32_t(TILE_M >> 4) << 24);
}
// Block-scaled kinds: no D format field (the accumulator is FP32); which of the four scale bytes of a tensor-memory word
// the instruction uses in bits 4-5 (B) and 29-30 (A); scale type in bit 23 (1: E8M0, 0: UE4M3).
__host__ __device__ inline uint32_t instr_desc_scaled(const UmmaShape& s, int sf_id, bool e8m0) {
    return (uint32_t(sf_id) << 4) | (uint32_t(s.a_fmt) << 7) | (uint32_t(s.b_fmt) << 10) | (uint32_t(TILE_N >> 3) << 17) |
           (uint32_t(e8m0 ? 1 : 0) << 23) | (uint32_t(TILE_M >> 4) << 24) | (uint32_t(sf_id) << 29);
}

// Shared-memory matrix descriptor, K-major, no swizzle: start address, leading byte offset (between the two 16-byte
// columns of core matrices that one instruction reads along K) and stride byte offset (between 8-row groups), all in
// units of 16 bytes; descriptor version 1 in bits 46-47.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return uint64_t((addr & 0x3FFFFu) >> 4) | (uint64_t(lbo >> 4) << 16) | (uint64_t(sbo >> 4) << 32) | (uint64_t(1) << 46);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }

// The sub-byte types of kind::f8f6f4 sit in shared memory sixteen elements per 16-byte chunk: the codes packed from bit 0
// upwards (4 bits each: 8 bytes; 6 bits each: 12 bytes), the rest of the chunk padding.  `bits` = 8 leaves a chunk as it is.
__device__ __forceinline__ uint4 pack_chunk(uint4 v, int bits) {
    if (bits == 8) return v;
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    unsigned long long lo = 0ull, hi = 0ull;            // up to 96 bits of packed codes
    const uint32_t mask = (1u << bits) - 1u;
    for (int i = 0; i < 16; ++i) {
        const unsigned long long code = (w[i >> 2] >> (8 * (i & 3))) & mask;
        const int pos = bits * i;
        if (pos < 64) { lo |= code << pos; if (pos + bits > 64) hi |= code >> (64 - pos); }
        else hi |= code << (pos - 64);
    }
    return make_uint4(uint32_t(lo), uint32_t(lo >> 32), uint32_t(hi), uint32_t(hi >> 32));
}

// rows x kbytes of a row-major global matrix -> canonical layout: byte (r, b) at (r / 8) * sbo + (b / 16) * 128 + (r % 8) * 16 + b % 16
__device__ __forceinline__ void stage_operand(unsigned char* dst, const unsigned char* src, int rows, int kbytes, int bits, int tid) {
    const int chunks = kbytes / 16, sbo = chunks * 128;
    for (int q = tid; q < rows * chunks; q += NTHREADS) {
        const int r = q / chunks, c = q % chunks;
        const uint4 v = *reinterpret_cast<const uint4*>(src + int64_t(r) * kbytes + 16 * c);
        *reinterpret_cast<uint4*>(dst + (r / 8) * sbo + c * 128 + (r % 8) * 16) = pack_chunk(v, bits);
    }
}

template <int MMA_KIND>
__device__ __forceinline__ void issue_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc) {
    // the accumulator already holds C: every instruction adds to it
    if (MMA_KIND == 0)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     :: "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc) : "memory");
    else if (MMA_KIND == 1)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
                     :: "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
                     :: "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc) : "memory");
}

template <int MMA_KIND>
__device__ __forceinline__ void issue_mma_scaled(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t sfa, uint32_t sfb) {
    if (MMA_KIND == 3)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale.scale_vec::1X [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
                     :: "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(sfa), "r"(sfb) : "memory");
    else if (MMA_KIND == 4)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
                     :: "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(sfa), "r"(sfb) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.scale_vec::4X [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
                     :: "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(sfa), "r"(sfb) : "memory");
}

__global__ void __launch_bounds__(NTHREADS) hw_umma_kernel(int kind, int64_t K, const unsigned char* A, const unsigned char* B,
                                                          const void* Cv, void* Dv, const unsigned char* SFA,
                                                          const unsigned char* SFB, int32_t* status, long long wait_clocks) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) unsigned long long mbar;
    __shared__ uint32_t tmem_base_s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const UmmaShape sh = umma_shape(kind);
    const int kbytes = sh.elem_bytes ? int(K) * sh.elem_bytes : int(K) / 2;
    unsigned char* sA = smem;
    unsigned char* sB = smem + TILE_M * kbytes;
    const int64_t row0 = int64_t(blockIdx.x) * TILE_M;

    const bool container8 = sh.mma_kind == 2 || sh.mma_kind == 3;     // sub-byte types arrive one element per byte
    const int bits_a = !container8 ? 8 : (sh.a_fmt == 5 ? 4 : (sh.a_fmt >= 3 ? 6 : 8));
    const int bits_b = !container8 ? 8 : (sh.b_fmt == 5 ? 4 : (sh.b_fmt >= 3 ? 6 : 8));
    stage_operand(sA, A + row0 * kbytes, TILE_M, kbytes, bits_a, tid);
    stage_operand(sB, B, TILE_N, kbytes, bits_b, tid);
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&tmem_base_s)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&mbar)) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");          // the staged operands, for the instruction's reads
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_s;
    const uint32_t taddr = tmem_base + (uint32_t(32 * warp) << 16);       // this warp's 32 lanes = rows 32 w .. 32 w + 31

    // C into tensor memory: thread (warp, lane) holds row 32 warp + lane, TILE_N columns
    // (FP16 accumulators: 16-bit words; in tensor memory one per 32-bit column, in its low half - found with exact integers)
    const uint32_t* C = static_cast<const uint32_t*>(Cv);
    const uint16_t* C16 = static_cast<const uint16_t*>(Cv);
    uint32_t* D = static_cast<uint32_t*>(Dv);
    uint16_t* D16 = static_cast<uint16_t*>(Dv);
    uint32_t c[TILE_N];
#pragma unroll
    for (int j = 0; j < TILE_N; ++j) {
        const int64_t idx = (row0 + 32 * warp + lane) * TILE_N + j;
        c[j] = !Cv ? 0u : (sh.acc16 ? uint32_t(C16[idx]) : C[idx]);
    }

    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                 :: "r"(taddr), "r"(c[0]), "r"(c[1]), "r"(c[2]), "r"(c[3]), "r"(c[4]), "r"(c[5]), "r"(c[6]), "r"(c[7]),
                    "r"(c[8]), "r"(c[9]), "r"(c[10]), "r"(c[11]), "r"(c[12]), "r"(c[13]), "r"(c[14]), "r"(c[15]) : "memory");
    if (sh.sf_per_step) {
        // Scale factors into tensor memory.  A 32-bit word holds four consecutive scale bytes of one row (four instruction
        // steps' worth at one scale per step); the word of row r lives in column r / 32 of a group of four columns at
        // lane r % 32, and every 32-lane quarter carries a full copy: output row R reads lane R, column R / 32 for A's
        // scale and lane 32 (R / 32) + n, column n / 32 for column n's (found by filling the words with their own
        // position and reading the products of all-ones operands back).  Thread (warp, lane) writes the four words of the
        // rows lane, lane + 32, lane + 64, lane + 96 for each group (B: rows below TILE_N, the rest zero).
        const int nsf = int(K) / sh.k_instr * sh.sf_per_step;            // scale bytes per row
#pragma unroll
        for (int grp = 0; grp < SF_GROUPS; ++grp) {
            uint32_t wa[4], wb[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int r = 32 * j + lane;
                wa[j] = wb[j] = 0u;
                for (int b = 0; b < 4; ++b) {
                    const int idx = 4 * grp + b;
                    if (idx < nsf) {
                        wa[j] |= uint32_t(SFA[(row0 + r) * nsf + idx]) << (8 * b);
                        if (r < TILE_N) wb[j] |= uint32_t(SFB[r * nsf + idx]) << (8 * b);
                    }
                }
            }
            asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1,%2,%3,%4};"
                         :: "r"(taddr + uint32_t(SFA_COL + 4 * grp)), "r"(wa[0]), "r"(wa[1]), "r"(wa[2]), "r"(wa[3]) : "memory");
            asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1,%2,%3,%4};"
                         :: "r"(taddr + uint32_t(SFB_COL + 4 * grp)), "r"(wb[0]), "r"(wb[1]), "r"(wb[2]), "r"(wb[3]) : "memory");
        }
    }
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();

    if (tid == 0 && kind != UK_SELFTEST_TIMEOUT) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t idesc = instr_desc(sh);
        const uint32_t sbo = uint32_t(kbytes / 16) * 128u;
        const int steps = int(K) / sh.k_instr;
        for (int s = 0; s < steps; ++s) {                                 // 32 bytes of K = two core matrices per step
            const uint64_t adesc = smem_desc(smem_u32(sA) + 256u * s, 128u, sbo);
            const uint64_t bdesc = smem_desc(smem_u32(sB) + 256u * s, 128u, sbo);
            if (sh.mma_kind == 0) issue_mma<0>(tmem_base, adesc, bdesc, idesc);
            else if (sh.mma_kind == 1) issue_mma<1>(tmem_base, adesc, bdesc, idesc);
            else if (sh.mma_kind == 2) issue_mma<2>(tmem_base, adesc, bdesc, idesc);
            else {
                const int first = s * sh.sf_per_step;                    // index of this step's first scale byte
                const uint32_t id2 = instr_desc_scaled(sh, first & 3, sh.mma_kind != 5);
                const uint32_t sfa = tmem_base + uint32_t(SFA_COL + 4 * (first >> 2)), sfb = tmem_base + uint32_t(SFB_COL + 4 * (first >> 2));
                if (sh.mma_kind == 3) issue_mma_scaled<3>(tmem_base, adesc, bdesc, id2, sfa, sfb);
                else if (sh.mma_kind == 4) issue_mma_scaled<4>(tmem_base, adesc, bdesc, id2, sfa, sfb);
                else issue_mma_scaled<5>(tmem_base, adesc, bdesc, id2, sfa, sfb);
            }
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(smem_u32(&mbar)) : "memory");
    }

    // the one wait: polls until the commit has arrived or the clock budget is spent
    bool done = false;
    const long long t0 = clock64();
    while (!done) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(smem_u32(&mbar)) : "memory");
        done = ok != 0u;
        if (!done && clock64() - t0 > wait_clocks) break;
    }
    if (!done) {
        if (tid == 0) atomicExch(status, int32_t(MMASIM_ERR_TIMEOUT));
    } else {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        uint32_t d[TILE_N];
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                     : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]), "=r"(d[4]), "=r"(d[5]), "=r"(d[6]), "=r"(d[7]),
                       "=r"(d[8]), "=r"(d[9]), "=r"(d[10]), "=r"(d[11]), "=r"(d[12]), "=r"(d[13]), "=r"(d[14]), "=r"(d[15])
                     : "r"(taddr) : "memory");
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int j = 0; j < TILE_N; ++j) {
            const int64_t idx = (row0 + 32 * warp + lane) * TILE_N + j;
            if (!sh.acc16) D[idx] = d[j];
            else D16[idx] = uint16_t(d[j]);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"(TMEM_COLS) : "memory");
}

}  // namespace

int launch_hw_umma(int kind, int64_t M, int64_t K, const void* A, const void* B, const void* C, void* D, const void* sfa,
                   const void* sfb, int32_t* status, cudaStream_t stream) {
    if (kind < 0 || kind >= UK_COUNT) { set_error("mmasim_hw_umma: unknown kind %d", kind); return MMASIM_ERR_INVALID_ARG; }
    const UmmaShape sh = umma_shape(kind);
    if (M < TILE_M || M % TILE_M || K < sh.k_instr || K % sh.k_instr) {
        set_error("mmasim_hw_umma: M must be a multiple of %d and K a multiple of %d for this instruction", TILE_M, sh.k_instr);
        return MMASIM_ERR_SHAPE;
    }
    const size_t smem = size_t(TILE_M + TILE_N) * (sh.elem_bytes ? size_t(K) * sh.elem_bytes : size_t(K) / 2);
    if (sh.sf_per_step) {
        if (!sfa || !sfb) { set_error("mmasim_hw_umma: this kind needs scale factors"); return MMASIM_ERR_INVALID_ARG; }
        if (K / sh.k_instr * sh.sf_per_step > 4 * SF_GROUPS) {
            set_error("mmasim_hw_umma: at most %d scale factors per row in one call", 4 * SF_GROUPS);
            return MMASIM_ERR_SHAPE;
        }
    }
    if (smem > 200 * 1024) { set_error("mmasim_hw_umma: K too long for one shared-memory tile"); return MMASIM_ERR_SHAPE; }
    cudaError_t err = cudaFuncSetAttribute(hw_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (err == cudaSuccess) {
        // about one second at the SM's top clock; the self-test gives up after about a millisecond
        const long long wait_clocks = kind == UK_SELFTEST_TIMEOUT ? 2000000ll : 2000000000ll;
        hw_umma_kernel<<<unsigned(M / TILE_M), NTHREADS, smem, stream>>>(kind, K, static_cast<const unsigned char*>(A),
                                                                        static_cast<const unsigned char*>(B), C, D,
                                                                        static_cast<const unsigned char*>(sfa),
                                                                        static_cast<const unsigned char*>(sfb), status, wait_clocks);
        err = cudaGetLastError();
    }
    if (err != cudaSuccess) { set_error("mmasim_hw_umma launch failed: %s", cudaGetErrorString(err)); return MMASIM_ERR_CUDA; }
    return MMASIM_OK;
}

}  // namespace mmasim

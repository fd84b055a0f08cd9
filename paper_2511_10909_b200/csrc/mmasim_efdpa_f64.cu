// Tuned E-FDPA (Algorithm 6) kernel: the CDNA1 FP16 / BF16 models - RNE-FP32 of the EXACT sum c + sum_k a_k b_k of
// a block of L = 4 (FP16) or 2 (BF16) products.
//
// Operands come as decoded blocks through bulk copies, as in the FP64 T-FDPA kernel (mmasim_tfdpa_f64.cuh); every
// product of two FP16 / BF16 values is exact in a double.  The sum of a block is formed twice by the FP64 matrix
// instruction, from the same accumulator: once with every multiply-add rounded toward minus infinity, once toward plus
// infinity.  The first chain never exceeds the exact partial sum and the second never falls below it, and once they
// differ they stay apart (RD(x + p) <= x + p < y + p <= RU(y + p) for x < y); so the two results are the same double if
// and only if every partial sum was exact, and then that double is the exact sum and one cvt.rn.f32.f64 is the single
// rounding of Algorithm 6.  No exponent window has to be computed.  Whatever does not pass - terms too far apart for 53
// bits, sums that cancel to zero (the two chains give -0 and +0), a NaN accumulator, an infinity or a NaN in the chunk -
// goes through the by-the-book block function on the raw words (exact 640-bit fixed-point sum), which also produces and
// propagates the special values: the accumulator between blocks is the plain output word.
// The B operands of the decoded blocks carry a small offset in the low word of the double (used by the truncating
// kernels); FP16 and BF16 significands fit the high word, so clearing the low word gives the exact value back.
#include "mmasim_tfdpa_f64.cuh"

namespace mmasim {
namespace fast64 {

namespace {

using fast::EK_F16;
using fast::EK_BF16;

// By the book: decode the L elements of row i of A and row j of B from global memory and run Algorithm 6.
template <int EK, int L>
__device__ __noinline__ uint32_t efdpa_by_the_book(DevModel m, const void* A, const void* B, int64_t ia, int64_t ib, uint32_t c) {
    const FmtDesc fa = fmt_desc(m.fmt_a), fb = fmt_desc(m.fmt_b);
    uint32_t a[L], b[L];
#pragma unroll
    for (int k = 0; k < L; ++k) {
        a[k] = decode_elem(fa, raw_elem<EK>(A, ia + k));
        b[k] = decode_elem(fb, raw_elem<EK>(B, ib + k));
    }
    return efdpa_block(a, b, L, c, m);
}

template <int EK, int L>
__global__ void __launch_bounds__(NT, 1) efdpa64_kernel(DevModel m, GemmArgs g, const Blk64<BM>* __restrict__ wa,
                                                        const Blk64<BN>* __restrict__ wb) {
    constexpr int NBLK = KC / L;
    constexpr bool SCALAR = L == 2;                     // (with blocks of 4 the matrix instruction wins: 12.3 against 15.4 ms at 4096^3)
    static_assert(L == 2 || L == 4, "one matrix instruction (four terms) per block");
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SmemMM& sm = *reinterpret_cast<SmemMM*>(smem_raw);

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int wr = warp >> 2, wc = warp & 3, gq = lane >> 2, tq = lane & 3;      // warp grid 4 x 4, warp tile 32 x 16
    auto row_at = [&](int r) { return wr * 32 + gq + 8 * r; };                   // inside the CTA tile
    auto col_at = [&](int c) { return wc * 16 + 8 * (c >> 1) + 2 * tq + (c & 1); };
    const int64_t row0 = int64_t(blockIdx.y) * BM, col0 = int64_t(blockIdx.x) * BN;

    const int NCH = int(g.K / KC);
    const Blk64<BM>* src_a = wa + int64_t(blockIdx.y) * NCH;
    const Blk64<BN>* src_b = wb + int64_t(blockIdx.x) * NCH;
    auto issue = [&](int n) {                              // one thread: both copies of chunk n into buffer n & 1
        unsigned long long* bar = &sm.full[n & 1];
        fast::mbar_expect_tx(bar, uint32_t(sizeof(Blk64<BM>) + sizeof(Blk64<BN>)));
        fast::bulk_load(&sm.a[n & 1], src_a + n, uint32_t(sizeof(Blk64<BM>)), bar);
        fast::bulk_load(&sm.b[n & 1], src_b + n, uint32_t(sizeof(Blk64<BN>)), bar);
    };
    if (tid == 0) {
        sm.error = 0;
        fast::mbar_init(&sm.full[0], 1u);
        fast::mbar_init(&sm.full[1], 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        issue(0);
        if (NCH > 1) issue(1);
    }

    uint32_t cw[TM][TN];                                // the accumulator of each output: the FP32 word, special values included
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + row_at(r), j = col0 + col_at(c);
            cw[r][c] = (g.C && i < g.M && j < g.N) ? static_cast<const uint32_t*>(g.C)[i * g.ldc + j] : 0u;
        }
    __syncthreads();                                    // the barriers are initialised

    for (int chunk = 0; chunk < NCH; ++chunk) {
        const int64_t k0 = int64_t(chunk) * KC;
        if (!fast::mbar_wait(&sm.full[chunk & 1], uint32_t(chunk >> 1) & 1u)) *reinterpret_cast<volatile int*>(&sm.error) = 1;
        const Blk64<BM>& sa_blk = sm.a[chunk & 1];
        const Blk64<BN>& sb_blk = sm.b[chunk & 1];
        const bool chunk_special = (sa_blk.special | sb_blk.special) != 0u;

#pragma unroll 1
        for (int blk = 0; blk < NBLK; ++blk) {
            const int kb = blk * L;
            uint32_t slow = chunk_special ? 0xFFFFu : 0u;   // bit r * TN + c: this output goes by the book
            if (SCALAR) {
                // blocks of two elements would leave half of a matrix instruction empty: scalar multiply-adds, L per chain
                double av[TM][L], bv[TN][L];
#pragma unroll
                for (int r = 0; r < TM; ++r) {
#pragma unroll
                    for (int q = 0; q < L / 2; ++q) {
                        const double2 t = *reinterpret_cast<const double2*>(&sa_blk.d[row_at(r)][kb + 2 * q]);
                        av[r][2 * q] = t.x; av[r][2 * q + 1] = t.y;
                    }
                }
#pragma unroll
                for (int c = 0; c < TN; ++c) {
#pragma unroll
                    for (int q = 0; q < L / 2; ++q) {
                        const double2 t = *reinterpret_cast<const double2*>(&sb_blk.d[col_at(c)][kb + 2 * q]);
                        bv[c][2 * q] = __hiloint2double(__double2hiint(t.x), 0); bv[c][2 * q + 1] = __hiloint2double(__double2hiint(t.y), 0);
                    }
                }
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c) {
                        // the accumulator as a double; adding +0 turns a -0 (which Algorithm 6 treats like +0) into +0
                        const double c0 = __dadd_rn(double(__uint_as_float(cw[r][c])), 0.0);
                        double lo = c0, hi = c0;
#pragma unroll
                        for (int k = 0; k < L; ++k) { lo = __fma_rd(av[r][k], bv[c][k], lo); hi = __fma_ru(av[r][k], bv[c][k], hi); }
                        const bool fits = !chunk_special && lo == hi && __double2hiint(lo) == __double2hiint(hi);
                        if (!fits) slow |= 1u << (r * TN + c);
                        if (fits) cw[r][c] = __float_as_uint(__double2float_rn(lo));
                    }
            } else {
                // operand fragments of the block's matrix instruction: lane (g, t) holds A[8 r + g][kb + t], B[8 j + g][kb + t];
                // blocks of two elements leave the lanes t = 2, 3 empty
                double af[TM], bf[TN / 2];
                const bool lane_used = L == 4 || tq < 2;
    #pragma unroll
                for (int r = 0; r < TM; ++r) af[r] = lane_used ? sa_blk.d[wr * 32 + 8 * r + gq][kb + (L == 4 ? tq : (tq & 1))] : 0.0;
    #pragma unroll
                for (int j = 0; j < TN / 2; ++j) {
                    const double x = sb_blk.d[wc * 16 + 8 * j + gq][kb + (L == 4 ? tq : (tq & 1))];
                    bf[j] = lane_used ? __hiloint2double(__double2hiint(x), 0) : 0.0;
                }
    #pragma unroll
                for (int r = 0; r < TM; ++r)
    #pragma unroll
                    for (int j = 0; j < TN / 2; ++j) {
                        // the accumulator as a double; adding +0 turns a -0 (which Algorithm 6 treats like +0) into +0
                        double lo0 = __dadd_rn(double(__uint_as_float(cw[r][2 * j])), 0.0);
                        double lo1 = __dadd_rn(double(__uint_as_float(cw[r][2 * j + 1])), 0.0);
                        double hi0 = lo0, hi1 = lo1;
                        asm volatile("mma.sync.aligned.m8n8k4.row.col.rm.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                                     : "+d"(lo0), "+d"(lo1) : "d"(af[r]), "d"(bf[j]));
                        asm volatile("mma.sync.aligned.m8n8k4.row.col.rp.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                                     : "+d"(hi0), "+d"(hi1) : "d"(af[r]), "d"(bf[j]));
                        // the same double (bit for bit: not -0 against +0, not a NaN): the exact sum
                        // (the stand-ins of infinities and NaNs are zeros: in such a chunk the accumulator waits for the by-the-book pass)
                        const bool fits0 = !chunk_special && lo0 == hi0 && __double2hiint(lo0) == __double2hiint(hi0);
                        const bool fits1 = !chunk_special && lo1 == hi1 && __double2hiint(lo1) == __double2hiint(hi1);
                        if (!fits0) slow |= 1u << (r * TN + 2 * j);
                        if (!fits1) slow |= 1u << (r * TN + 2 * j + 1);
                        if (fits0) cw[r][2 * j] = __float_as_uint(__double2float_rn(lo0));
                        if (fits1) cw[r][2 * j + 1] = __float_as_uint(__double2float_rn(lo1));
                    }
            }
            if (slow) {                                        // rare
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int c = 0; c < TN; ++c)
                        if ((slow >> (r * TN + c)) & 1u) {
                            const int64_t i = row0 + row_at(r), j = col0 + col_at(c);
                            cw[r][c] = (i < g.M && j < g.N)
                                           ? efdpa_by_the_book<EK, L>(m, g.A, g.B, i * g.lda + k0 + kb, j * g.ldb + k0 + kb, cw[r][c]) : 0u;
                        }
            }
        }
        __syncthreads();                                // everybody has finished with this buffer
        if (*reinterpret_cast<volatile int*>(&sm.error)) break;
        if (tid == 0 && chunk + 2 < NCH) issue(chunk + 2);
    }

    if (*reinterpret_cast<volatile int*>(&sm.error)) {  // a copy never arrived: count it, give the copies in flight one more
        if (tid == 0) {                                 // bounded wait each, and store nothing
            if (g.copy_timeouts) atomicAdd(g.copy_timeouts, 1u);
            fast::mbar_wait(&sm.full[0], 0u);
            fast::mbar_wait(&sm.full[1], 0u);
        }
        return;
    }
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) {
            const int64_t i = row0 + row_at(r), j = col0 + col_at(c);
            if (i >= g.M || j >= g.N) continue;
            uint32_t w = cw[r][c];
            if (g.row_scale) {
                float sc = __fmul_rn(g.row_scale[i], g.col_scale[j]);
                if (sc != sc) sc = __uint_as_float(0x7FFFFFFFu);
                float v = __fmul_rn(sc, __uint_as_float(w));
                if (v != v) v = __uint_as_float(0x7FFFFFFFu);
                w = __float_as_uint(v);
            }
            static_cast<uint32_t*>(g.D)[i * g.ldd + j] = w;
        }
}

template <int EK, int L>
cudaError_t launch_e_one(const DevModel& m, const GemmArgs& g, cudaStream_t stream) {
    const size_t sh = sizeof(SmemMM);
    cudaError_t err = cudaFuncSetAttribute(efdpa64_kernel<EK, L>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sh));
    if (err != cudaSuccess) return err;
    const size_t dsh_a = 256 * sizeof(LutEntry64) + sizeof(Blk64<BM>), dsh_b = 256 * sizeof(LutEntry64) + sizeof(Blk64<BN>);
    if ((err = cudaFuncSetAttribute(decode64_kernel<EK, BM, true, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(dsh_a))) != cudaSuccess) return err;
    if ((err = cudaFuncSetAttribute(decode64_kernel<EK, BN, false, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(dsh_b))) != cudaSuccess) return err;
    const int64_t tiles_m = (g.M + BM - 1) / BM, tiles_n = (g.N + BN - 1) / BN, nch = g.K / KC;
    // scratch: the decoded blocks of A and B, stream-ordered out of the library's pool and returned to it behind the kernel
    const size_t bytes_a = size_t(tiles_m * nch) * sizeof(Blk64<BM>), bytes_b = size_t(tiles_n * nch) * sizeof(Blk64<BN>);
    cudaMemPool_t pool = nullptr;
    if ((err = scratch_pool(&pool)) != cudaSuccess) return err;
    void* ws = nullptr;
    if ((err = cudaMallocFromPoolAsync(&ws, bytes_a + bytes_b, pool, stream)) != cudaSuccess) return err;
    Blk64<BM>* wa = static_cast<Blk64<BM>*>(ws);
    Blk64<BN>* wb = reinterpret_cast<Blk64<BN>*>(static_cast<unsigned char*>(ws) + bytes_a);
    decode64_kernel<EK, BM, true, 0><<<dim3((unsigned)nch, (unsigned)tiles_m), 256, dsh_a, stream>>>(
        m, static_cast<const unsigned char*>(g.A), g.M, g.lda, wa);
    decode64_kernel<EK, BN, false, 0><<<dim3((unsigned)nch, (unsigned)tiles_n), 256, dsh_b, stream>>>(
        m, static_cast<const unsigned char*>(g.B), g.N, g.ldb, wb);
    dim3 grid((unsigned)tiles_n, (unsigned)tiles_m, 1);
    efdpa64_kernel<EK, L><<<grid, NT, sh, stream>>>(m, g, wa, wb);
    err = cudaGetLastError();
    const cudaError_t err2 = cudaFreeAsync(ws, stream);
    return err != cudaSuccess ? err : err2;
}

}  // namespace

cudaError_t launch_e64(const DevModel& m, const GemmArgs& g, cudaStream_t st) {
    if (m.fmt_a == EF_F16 && m.L == 4) return launch_e_one<EK_F16, 4>(m, g, st);
    if (m.fmt_a == EF_BF16 && m.L == 2) return launch_e_one<EK_BF16, 2>(m, g, st);
    return cudaErrorInvalidValue;
}

}  // namespace fast64

namespace fast {
cudaError_t launch_e(const DevModel& m, const GemmArgs& g, cudaStream_t st) { return fast64::launch_e64(m, g, st); }
}  // namespace fast
}  // namespace mmasim

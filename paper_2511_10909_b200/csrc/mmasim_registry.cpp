// Instruction-to-model registry: Tables 3-7 of the paper expressed through the rules its Section 4.3 states
// (L_max = register bytes / element bytes per generation, F and rho per generation and input class).
#include <cstring>
#include "mmasim_internal.h"

namespace mmasim {

namespace {

struct InFmt {
    int elem;        // ElemFmt
    int cls;         // 0 fp64, 1 fp32, 2 tf32, 3 half (bf16/fp16), 4 fp8, 5 fp6/fp4
    int scaled;      // 0 none, 1 ST (E8M0 / 32), 2 GST MXFP4 (E8M0 / 32), 3 GST NVFP4 (UE4M3 / 16)
    int bytes;       // element size used in the "bytes / element size" rule
};

bool in_fmt_of(int f, InFmt* o) {
    switch (f) {
        case MMASIM_F64: *o = {EF_F64, 0, 0, 8}; return true;
        case MMASIM_F32: *o = {EF_F32, 1, 0, 4}; return true;
        case MMASIM_TF32: *o = {EF_TF32, 2, 0, 4}; return true;
        case MMASIM_BF16: case MMASIM_BF16_1K: *o = {EF_BF16, 3, 0, 2}; return true;
        case MMASIM_F16: *o = {EF_F16, 3, 0, 2}; return true;
        case MMASIM_E4M3: *o = {EF_E4M3, 4, 0, 1}; return true;
        case MMASIM_E5M2: *o = {EF_E5M2, 4, 0, 1}; return true;
        case MMASIM_E3M2: *o = {EF_E3M2, 5, 0, 1}; return true;
        case MMASIM_E2M3: *o = {EF_E2M3, 5, 0, 1}; return true;
        case MMASIM_E2M1: *o = {EF_E2M1, 5, 0, 1}; return true;
        case MMASIM_MXE4M3: *o = {EF_E4M3, 4, 1, 1}; return true;
        case MMASIM_MXE5M2: *o = {EF_E5M2, 4, 1, 1}; return true;
        case MMASIM_MXE3M2: *o = {EF_E3M2, 5, 1, 1}; return true;
        case MMASIM_MXE2M3: *o = {EF_E2M3, 5, 1, 1}; return true;
        case MMASIM_MXE2M1: *o = {EF_E2M1, 5, 1, 1}; return true;
        case MMASIM_MXF4_GST: *o = {EF_E2M1, 5, 2, 1}; return true;
        case MMASIM_NVF4_GST: *o = {EF_E2M1, 5, 3, 1}; return true;
        default: return false;
    }
}

}  // namespace

bool registry_lookup(int arch, int a_fmt, int b_fmt, int acc_fmt, mmasim_model* out, const char** why) {
    InFmt ia, ib;
    *why = "";
    if (arch < 0 || arch >= MMASIM_ARCH_COUNT) { *why = "unknown architecture"; return false; }
    if (!in_fmt_of(a_fmt, &ia) || !in_fmt_of(b_fmt, &ib)) { *why = "unknown input type"; return false; }
    if (acc_fmt < 0 || acc_fmt >= MMASIM_ACC_COUNT) { *why = "unknown accumulator type"; return false; }
    if (a_fmt != b_fmt) {
        // Algorithm 7 allows F_A != F_B inside the FP8 / FP6 / FP4 classes of one instruction family
        const bool narrow = ia.cls >= 4 && ib.cls >= 4 && ia.scaled == ib.scaled && ia.scaled <= 1;
        if (!narrow) { *why = "A and B types cannot be mixed for this model"; return false; }
    }
    DevModel d;
    std::memset(&d, 0, sizeof(d));
    d.fmt_a = ia.elem;
    d.fmt_b = ib.elem;
    d.acc = acc_fmt;
    d.frac = fmt_desc(ia.elem).mbits + fmt_desc(ib.elem).mbits;
    const bool nvidia = arch <= MMASIM_RTX_BLACKWELL;
    const int cls = ia.cls > ib.cls ? ia.cls : ib.cls;
    bool ok = false;

    if (cls == 0) {                       // FP64: chain of FMAs on NVIDIA Ampere and later, CDNA2, CDNA3
        ok = acc_fmt == MMASIM_ACC_F64 &&
             ((nvidia && arch >= MMASIM_AMPERE) || arch == MMASIM_CDNA2 || arch == MMASIM_CDNA3);
        d.family = FAM_FMA;
    } else if (cls == 1) {                // FP32 inputs exist only on AMD: chain of FMAs
        ok = acc_fmt == MMASIM_ACC_F32 && !nvidia;
        d.family = FAM_FMA;
    } else if (nvidia) {
        // register bytes per operand fragment: Volta 8, Turing/Ampere/Ada 16, Hopper and later 32
        const int bytes = arch == MMASIM_VOLTA ? 8 : (arch <= MMASIM_ADA ? 16 : 32);
        const int F_wide = arch == MMASIM_VOLTA ? 23 : (arch <= MMASIM_ADA ? 24 : 25);
        const bool blackwell = arch >= MMASIM_BLACKWELL;
        d.family = FAM_T;
        d.L = bytes / ia.bytes;
        d.F = F_wide;
        d.rho = acc_fmt == MMASIM_ACC_F16 ? RHO_RNE_FP16 : RHO_RZ_FP32;
        if (cls == 2) ok = arch >= MMASIM_AMPERE && acc_fmt == MMASIM_ACC_F32;
        else if (cls == 3) {
            const bool bf16 = ia.elem == EF_BF16;
            ok = a_fmt != MMASIM_BF16_1K && (bf16 ? (arch >= MMASIM_AMPERE && acc_fmt == MMASIM_ACC_F32)
                                                   : acc_fmt != MMASIM_ACC_F64);
        } else if (ia.scaled == 0) {      // FP8 from Ada on, FP6/FP4 from Blackwell on
            ok = acc_fmt != MMASIM_ACC_F64 && (cls == 4 ? arch >= MMASIM_ADA : blackwell);
            if (!blackwell) {             // Ada / Hopper FP8: 13 fractional bits, truncated-FP32 output
                d.F = 13;
                if (acc_fmt == MMASIM_ACC_F32) d.rho = RHO_RZ_E8M13;
            }
        } else if (ia.scaled == 1) {      // MXFP8/6/4: scaled T-FDPA, one E8M0 scale per 32 elements
            ok = blackwell && acc_fmt == MMASIM_ACC_F32;
            d.family = FAM_ST;
            d.k_block = 32;
            d.scale_fmt = EF_E8M0;
        } else {                          // MXFP4 / NVFP4 group-scaled
            ok = blackwell && acc_fmt == MMASIM_ACC_F32;
            d.family = FAM_GST;
            d.L = 64;
            d.G = 16;
            d.F = 35;
            d.k_block = ia.scaled == 2 ? 32 : 16;
            d.scale_fmt = ia.scaled == 2 ? EF_E8M0 : EF_UE4M3;
            d.frac = 2 * fmt_desc(EF_E2M1).mbits + 2 * fmt_desc(d.scale_fmt).mbits;
            d.packed4 = 1;
        }
    } else if (arch == MMASIM_CDNA1) {    // exact FDPA: BF16 L = 2, FP16 L = 4
        ok = cls == 3 && a_fmt != MMASIM_BF16_1K && acc_fmt == MMASIM_ACC_F32;
        d.family = FAM_E;
        d.L = ia.elem == EF_BF16 ? 2 : 4;
        d.rho = RHO_RNE_FP32;
    } else if (arch == MMASIM_CDNA2) {    // FTZ-Add / FTZ-Mul trees: P = 2 for plain BF16, else 4
        ok = cls == 3 && acc_fmt == MMASIM_ACC_F32;
        d.family = FAM_FTZ;
        d.P = a_fmt == MMASIM_BF16 ? 2 : 4;
    } else {                              // CDNA3: 16 bytes / element size, F = 24, F2 = 31, RNE-FP32
        ok = acc_fmt == MMASIM_ACC_F32 && a_fmt != MMASIM_BF16_1K && ia.scaled == 0 && (cls == 2 || cls == 3 || cls == 4);
        d.family = cls == 4 ? FAM_GTR : FAM_TR;
        d.L = 16 / ia.bytes;
        d.F = 24;
        d.F2 = 31;
        d.rho = RHO_RNE_FP32;
    }
    if (!ok) { *why = "no MMA instruction with these types on this architecture (Tables 3-7)"; return false; }

    out->arch = arch;
    out->a_fmt = a_fmt;
    out->b_fmt = b_fmt;
    out->acc_fmt = acc_fmt;
    out->dev = d;
    mmasim_info& i = out->info;
    std::memset(&i, 0, sizeof(i));
    const int fam_pub[] = {MMASIM_FAM_FMA, MMASIM_FAM_FTZ_ADDMUL, MMASIM_FAM_E_FDPA, MMASIM_FAM_T_FDPA,
                           MMASIM_FAM_ST_FDPA, MMASIM_FAM_GST_FDPA, MMASIM_FAM_TR_FDPA, MMASIM_FAM_GTR_FDPA};
    i.family = fam_pub[d.family];
    i.l_max = d.L;
    i.F = d.F;
    i.F2 = d.F2;
    i.rho = (d.family == FAM_FMA || d.family == FAM_FTZ || d.family == FAM_E) ? MMASIM_RHO_NONE : d.rho;
    i.P = d.P;
    i.G = d.G;
    i.k_block = d.k_block;
    i.a_bits = d.packed4 ? 4 : fmt_desc(d.fmt_a).storage_bits;
    i.b_bits = d.packed4 ? 4 : fmt_desc(d.fmt_b).storage_bits;
    i.acc_bytes = acc_fmt == MMASIM_ACC_F64 ? 8 : (acc_fmt == MMASIM_ACC_F16 ? 2 : 4);
    return true;
}

}  // namespace mmasim

// The FlashAttention-2 recurrence: cyc_flash_attention.  See include/cyc.h.
#include "api_internal.h"
#include "fa2_kernel.cuh"

namespace cyc {

// ------------------------------------------------------------------ FlashAttention-2 recurrence
// Scratch of the sliced tail: at most one part per SM, eight warps of row threads per part, sized for the larger head dimension.
constexpr int kFa2MaxSms = 160;
constexpr size_t kFa2TailDataBytes = static_cast<size_t>(kFa2MaxSms) * 8 * fa2_tail_slot_floats(128) * sizeof(float);
constexpr size_t kFa2TailCounterBytes = static_cast<size_t>(kFa2MaxSms / 2) * 8 * sizeof(int);

// How many parts each unit of the grid's last, partial round is cut into (0 = no tail): the parts of that round must
// fit the SMs at once, every part keeps at least two key tiles, at most FA2_TAIL_MAX_PARTS.
static int fa2_tail_parts(long long units, long long key_tiles, int sms) {
    if (sms > kFa2MaxSms) return 0;
    const long long rem = units % sms;
    if (rem == 0) return 0;
    const long long parts = std::min<long long>({sms / rem, key_tiles / 2, FA2_TAIL_MAX_PARTS});
    return parts >= 2 ? static_cast<int>(parts) : 0;
}

template <int D>
static int launch_fa2(long long batch, long long N, long long M, const void* Q, const void* K, const void* V, float* O, cudaStream_t st, int sms) {
    CUtensorMap tmQ, tmK, tmV;
    int rc = make_map(&tmQ, CYC_BF16_F32, Q, D, N, batch, D, N * D, 64, FA2_BM);
    if (rc) return rc;
    rc = make_map(&tmK, CYC_BF16_F32, K, D, M, batch, D, M * D, 64, FA2_BN);
    if (rc) return rc;
    rc = make_map(&tmV, CYC_BF16_F32, V, D, M, batch, D, M * D, 64, FA2_BN);
    if (rc) return rc;
    Fa2Params p;
    p.O = O;
    p.N = static_cast<int>(N); p.M = static_cast<int>(M);
    p.tiles_q = static_cast<int>((N + FA2_ROWS - 1) / FA2_ROWS);
    p.scale_log2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(D)));
    if (int rc_ = status_word(&p.status)) return rc_;
    auto kern = fa2_kernel<D>;
    {
        // the kernel redistributes the registers it was launched with among its warps and counts on 128 per thread
        static std::atomic<int> checked{0};
        if (!checked.load()) {
            cudaFuncAttributes fa;
            CYC_CUDA(cudaFuncGetAttributes(&fa, kern));
            if (fa.numRegs < FA2_REGS_LAUNCH) {
                snprintf(g_err, sizeof g_err, "flash attention kernel compiled to %d registers per thread, %d expected", fa.numRegs, FA2_REGS_LAUNCH);
                return CYC_ERR_CUDA;
            }
            checked.store(1);
        }
    }
    if (int rc_ = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), Fa2Smem<D>::TOTAL)) return rc_;
    const long long units = batch * p.tiles_q;
    long long ctas = units;
    p.full_units = static_cast<int>(units);
    p.tail_parts = 0;
    p.tail_ws = nullptr;
    p.tail_counters = nullptr;
    if (const int parts = fa2_tail_parts(units, (M + FA2_BN - 1) / FA2_BN, sms)) {
        uint8_t* data = nullptr;
        int* counters = nullptr;
        if (int rc_ = kept_scratch_for(st, SCRATCH_ATTENTION_TAIL, kFa2TailDataBytes, kFa2TailCounterBytes, &data, &counters)) return rc_;
        if (data) {
            const long long rem = units % sms;
            p.full_units = static_cast<int>(units - rem);
            p.tail_parts = parts;
            p.tail_ws = reinterpret_cast<float*>(data);
            p.tail_counters = counters;
            ctas = p.full_units + rem * parts;
        }
    }
    if (log_enabled())
        fprintf(stderr, "cyc: attention batch=%lld N=%lld M=%lld d=%d -> fa2 units=%lld tail_units=%lld tail_parts=%d ctas=%lld\n", batch, N, M, D, units,
                units - p.full_units, p.tail_parts, ctas);
    CYC_CUDA(launch_pdl(kern, static_cast<unsigned>(ctas), FA2_THREADS, Fa2Smem<D>::TOTAL, st, tmQ, tmK, tmV, p));
    g_launches.fetch_add(1);
    return CYC_OK;
}
}  // namespace cyc

using namespace cyc;

extern "C" int cyc_flash_attention(int64_t batch, int64_t N, int64_t M, int64_t d, int dtype, const void* Q, const void* K,
                                   const void* V, void* O, void* stream, unsigned flags) {
    if (batch <= 0 || N <= 0 || M <= 0 || d <= 0 || !Q || !K || !V || !O || flags != 0) return CYC_ERR_INVALID_ARG;
    if (dtype != CYC_F32 && dtype != CYC_BF16_F32 && dtype != CYC_I8_I32) return CYC_ERR_INVALID_ARG;
    const uintptr_t q0 = reinterpret_cast<uintptr_t>(Q), k0 = reinterpret_cast<uintptr_t>(K), v0 = reinterpret_cast<uintptr_t>(V),
                    o0 = reinterpret_cast<uintptr_t>(O);
    if ((q0 | k0 | v0) % 2 || o0 % 4) return CYC_ERR_INVALID_ARG;
    const uintptr_t obytes = static_cast<uintptr_t>(batch) * N * d * 4, qbytes = static_cast<uintptr_t>(batch) * N * d * 2,
                    kbytes = static_cast<uintptr_t>(batch) * M * d * 2;
    if ((o0 < q0 + qbytes && q0 < o0 + obytes) || (o0 < k0 + kbytes && k0 < o0 + obytes) || (o0 < v0 + kbytes && v0 < o0 + obytes))
        return CYC_ERR_INVALID_ARG;  // O over an input
    if (dtype != CYC_BF16_F32 || (d != 64 && d != 128)) {
        snprintf(g_err, sizeof g_err, "flash attention: bf16 inputs with head dimension 64 or 128 only");
        return CYC_ERR_UNSUPPORTED;
    }
    if ((q0 | k0 | v0 | o0) % 16) {
        snprintf(g_err, sizeof g_err, "flash attention: Q, K, V and O must be 16-byte aligned");
        return CYC_ERR_UNSUPPORTED;
    }
    const long long tiles_q = (N + FA2_ROWS - 1) / FA2_ROWS;
    if (N > 0x7fffffffll || M > 0x7fffffffll || batch * tiles_q > 0x7fffffffll) return CYC_ERR_UNSUPPORTED;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    if (di.cc_major != 10) {
        snprintf(g_err, sizeof g_err, "tensor-core kernels need an sm_100 device");
        return CYC_ERR_UNSUPPORTED;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return d == 64 ? launch_fa2<64>(batch, N, M, Q, K, V, static_cast<float*>(O), st, di.sms)
                   : launch_fa2<128>(batch, N, M, Q, K, V, static_cast<float*>(O), st, di.sms);
}

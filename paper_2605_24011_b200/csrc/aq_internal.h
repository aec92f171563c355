// Host-side internals shared by the .cu files of libaq (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/aq.h"
#include "aq_per_device.h"

#define AQ_HANDLE_MAGIC 0x41514831u   /* "AQH1" */

struct aq_handle_s {
    uint32_t magic;
    int bits;
    int device;
    int64_t N, K;
    int NT;            // row tiles of 16
    int KP;            // pair slabs of 256 k
    int64_t n_frags;   // NT * KP * 2
    size_t dev_bytes;  // n_frags * frag_bytes
    uint8_t* frags;    // DEVICE: fragment layout
    float* acc;        // DEVICE: [AQ_DECODE_MAX_M][NT*16] accumulation scratch, zero between calls
    uint8_t* sb;       // DEVICE: super-block parameters (32 bytes per row and super-block) of a handle made by aq_pack_sb /
                       // aq_import_sb, else null
    uint8_t* big;      // DEVICE: scratch of aq_linear with M > AQ_DECODE_MAX_M (float32 sums, binary16 copy of bfloat16
                       // activations, row scales), allocated when the handle first sees such a call and grown on demand
    size_t big_bytes;
    int* flags;        // DEVICE: bit 0 = range error seen while packing
    cudaStream_t last_stream;
};

namespace aq {

// status helpers (aq_api.cu)
aq_status_t cuda_fail(cudaError_t e);
bool handle_ok(aq_handle_t h);

// launchers (each checks nothing: arguments are validated by the API layer)
cudaError_t launch_pack(const aq_handle_s* h, const float* W, cudaStream_t s);
cudaError_t launch_pack_opt(const aq_handle_s* h, const float* W, const float* F, int rounds, cudaStream_t s);
cudaError_t launch_import(const aq_handle_s* h, const uint8_t* canon_dev, cudaStream_t s);
cudaError_t launch_export(const aq_handle_s* h, uint8_t* canon_dev, cudaStream_t s);
cudaError_t launch_dequant(const aq_handle_s* h, void* out, aq_dtype_t dt, cudaStream_t s);
// super-block format (aq_superblock.cu): quantise into fragments + side entries; canonical super-block bytes <-> plain
// canonical records carrying the decoded block parameters (to_plain also fills the side entries)
cudaError_t launch_pack_sb(const aq_handle_s* h, const float* W, cudaStream_t s);
cudaError_t launch_sb_records(const aq_handle_s* h, uint8_t* sbcanon_dev, uint8_t* plain_dev, bool to_plain, cudaStream_t s);

// decode path: accumulate x W^T into acc (fp32 [M][ldacc]); x is [M][K] of xdt.  With y_fused the kernel's last CTA
// also writes y[m][n] = cast(acc[m][n]) (row-major [M][N] of ydt) and leaves acc zero again: acc must be the handle's own
cudaError_t launch_gemv(const aq_handle_s* h, const void* x, aq_dtype_t xdt, int M, float* acc,
                        int64_t ldacc, cudaStream_t s, void* y_fused = nullptr, aq_dtype_t ydt = AQ_F32);
// y[m][n] = cast(acc[m][n]) for n < N, then acc = 0
cudaError_t launch_finalize(const float* acc_in, float* acc_zero, int64_t ldacc, void* y, aq_dtype_t ydt,
                            int M, int64_t N, cudaStream_t s);

// prefill path: out[m][n] = (res ? res[m][n] : 0) + tok_scale[m] sum_k x16[m][k] w[n][k]; x16 binary16 [M][K];
// tok_scale (with its flag, see launch_rows_to_f16) or null; out, res fp32 [M][ldo];
// out need not be initialised (the launcher zeroes it when tiles are split over CTAs)
cudaError_t launch_gemm(const aq_handle_s* h, const void* x16, const float* tok_scale, const int* scaled_flag, int M, float* out,
                        int64_t ldo, const float* res, cudaStream_t s);
// bfloat16 rows -> the binary16 operand of the GEMM, the per-row power of two they were divided by (1 unless a row
// leaves binary16's range) and a flag that says whether any row has one
cudaError_t launch_rows_to_f16(const void* x_bf16, void* x16, float* scale, int* flag, int M, int64_t K, cudaStream_t s);
// the same for up to AQ_GEMM_MAX_GROUP matrices of one K that read the same x, as one launch
#define AQ_GEMM_MAX_GROUP 4
cudaError_t launch_gemm_group(const aq_handle_s* const* hs, int n, const void* x16, const float* tok_scale, const int* scaled_flag,
                              int M, float* const* outs, const int64_t* ldos, const float* const* ress, bool outs_ready,
                              cudaStream_t s);
bool gemm_outputs_can_be_preset(float* const* outs, const int64_t* ldos, int n);
bool gemm_stores_first(const aq_handle_s* const* hs, int n, int M, cudaStream_t s);   // then only residuals need presetting

// CTAs the whole-program decode kernel may have when it exchanges row norms through the workspace (one per SM).
constexpr int AQ_NORM_MAX_CTAS = 192;

// Where a program's buffers and staged inputs sit in the caller's workspace (aq_stack.cu).
struct StackPlan {
    std::vector<size_t> buf_off;    // per buffer: float32 [M][width]
    std::vector<size_t> in_off;     // per op: its phase's staged input [M][K] (activation dtype)
    std::vector<int> phase_first;   // first op of each phase (ops that share one input vector)
    std::vector<char> external;     // per buffer: no op writes it and it is not buffer 0 (somebody else fills it)
    std::vector<size_t> pk_off;     // per buffer (M <= AQ_DECODE_MAX_M only): its packed 64-bit sums [M][width]
    size_t pk_begin = 0, pk_end = 0;   // the packed sums' region: zero at the start of a decode pass
    std::vector<size_t> nm_off;     // per op that opens an RMS-normalised phase (3 <= M <= AQ_DECODE_MAX_M): the CTAs'
                                    // partial sums of squares [AQ_NORM_MAX_CTAS][M] of 8 bytes, inside the region above; else 0
    std::vector<size_t> x16_off;    // per op (bfloat16, M > AQ_DECODE_MAX_M only): its phase's binary16 operand [M][K] ...
    std::vector<size_t> rs_off;     // ... the row scales [M] float32 ...
    std::vector<size_t> flag_off;   // ... and the phase's "some row is scaled" flag (int), inside [flags_begin, flags_end)
    size_t flags_begin = 0, flags_end = 0;
    size_t stage_off = 0;           // end of the float32 buffers
    size_t total = 0;
};

// whole-program decode (M <= AQ_DECODE_MAX_M) in one persistent kernel: 0 = launched,
// 1 = the program does not fit that kernel (nothing launched), -1 = CUDA error in *err
// (out: the caller's rounded copy of buffer out_buf, or null; *wrote_out: the kernel itself writes it; op_first, op_end:
// the ops of the program this launch runs, whole phases; clear: the packed sums are zeroed first)
int launch_decode_stack(const aq_stack_t* p, const StackPlan& plan, int M, aq_dtype_t dt, uint8_t* ws, cudaStream_t s,
                        cudaError_t* err, void* out, int out_buf, bool* wrote_out, int op_first = 0, int op_end = -1, bool clear = true,
                        const std::vector<uint8_t>* program_key = nullptr);
void decode_program_key(const aq_stack_t* p, std::vector<uint8_t>& key);   // the program's share of a plan's key
void decode_stack_forget(aq_handle_t h);   // drops cached device tables that name h
int read_decode_status(bool clear);        // nonzero: a bounded wait in the decode-stack kernel ran out
void set_decode_wait_ns(unsigned long long ns);   // limit of every wait in that kernel (0: the default, two seconds)
void set_decode_hold(bool on);             // testing: tables built while on expect a contribution that never comes

// Programmatic dependent launch, used along the prefill path: a kernel launched with launch_pdl may become
// resident while its predecessor on the stream still runs; it must execute pdl_wait() before it touches anything the
// predecessor wrote, and a kernel lets its successor in early with pdl_launch_dependents().
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg;
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}
#endif

// inter-tensor stage (aq_stage1.cu)
cudaError_t launch_rbf_gram(const void* A, aq_dtype_t dt, int64_t K, int64_t d, float sigma, float* out, int64_t ld,
                            cudaStream_t s);
// combine: 0 = out[0] receives Eq. 2; 1, 2 = out[combine] receives it, and with 2 also out[0] = -alpha out[1] + beta out[2]
cudaError_t launch_hsic(const float* KA, const float* KB, int64_t K, int64_t lda, int64_t ldb, double* out, int combine,
                        double alpha, double beta, cudaStream_t s);
int allocate_bits_host(const double* S, const int64_t* numel, const int32_t* layer_of, int64_t n, const int32_t* types,
                       int n_types, double budget, int32_t* bits_out, double* objective_out);   // 0 ok, 1 malformed, 2 budget
int read_stage1_status(bool clear);

// single-token attention over a key/value cache (aq_attn.cu); head dimension 128
size_t attn_scratch_bytes(int n_kv);
cudaError_t launch_attn_decode(const void* q, const void* kc, const void* vc, void* out, int M, int n_heads, int n_kv, int64_t L,
                               int64_t Lmax, float scale, aq_dtype_t dt, aq_dtype_t out_dt, void* scratch, cudaStream_t s);
cudaError_t launch_rope(void* x, int n_heads, int D, int64_t pos, float theta, aq_dtype_t dt, cudaStream_t s);
cudaError_t launch_attn_prepare(const float* q, const float* k, const float* v, void* q16, void* kc, void* vc, int M, int H, int Hkv,
                                int64_t pos, int64_t Lmax, float theta, aq_dtype_t dt, cudaStream_t s);
cudaError_t launch_kv_append(void* kc, void* vc, const void* k, const void* v, int n_kv, int D, int64_t pos, int64_t Lmax, cudaStream_t s);

int current_device();               // cudaGetDevice, or -1
int sm_count();                     // of the current device
void count_launch(int n = 1);       // process-wide count of this library's kernel launches
int read_gemm_status(bool clear);   // nonzero: a bounded wait in the GEMM kernel ran out

}  // namespace aq

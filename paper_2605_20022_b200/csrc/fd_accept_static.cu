// fd_verify_accept_static: the greedy verification of fd_verify_accept for callers that may not
// allocate device memory.  Its scratch (one 64-bit running maximum per candidate row and the
// finished-CTA counter) lives in a fixed array inside the library image instead of in an fd_ctx.
#include <mutex>

#include "fd_internal.cuh"


namespace {

// [0, FD_STATIC_MAX_ROWS) row keys, then 8 spare words: [MAX_ROWS] the CTA ticket, [MAX_ROWS + 1] a
// sink for the status bits of callers that pass no status pointer.  32 KB + 64 B per GPU that
// loads the library, held until the process exits.
static __device__ __align__(256) unsigned long long fd_static_scratch[FD_STATIC_MAX_ROWS + 8];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned long long* g_scratch_addr[kMaxDevices];  // device address of fd_static_scratch, per device
bool g_ready[kMaxDevices];

// In host code `fd_static_scratch` names a host-side shadow of the symbol, not device memory;
// the address a kernel may use has to be asked for, once per device, with that device current.
fd_status scratch_for_current_device(unsigned long long** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FD_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_ready[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, fd_static_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return FD_ERR_CUDA;
        }
        g_scratch_addr[dev] = static_cast<unsigned long long*>(ptr);
        g_ready[dev] = true;
    }
    *out = g_scratch_addr[dev];
    return FD_OK;
}

}  // namespace

extern "C" fd_status fd_verify_accept_static(int vocab, int batch, int total_cand_rows, const float* logits,
                                             const int32_t* draft_tokens, const int32_t* q_lens,
                                             const int32_t* n_mask, int32_t* accepted_len, int32_t* bonus_token,
                                             int32_t* device_status, void* stream) {
    if (vocab <= 0 || batch < 0 || total_cand_rows < 0) return FD_ERR_INVALID_ARG;
    if (total_cand_rows > FD_STATIC_MAX_ROWS || batch > FD_STATIC_MAX_BATCH) return FD_ERR_STATIC_LIMIT;
    if (batch == 0) return total_cand_rows == 0 ? FD_OK : FD_ERR_INVALID_ARG;
    if (!q_lens || !n_mask || !accepted_len || !bonus_token) return FD_ERR_INVALID_ARG;
    if (total_cand_rows > 0 && (!logits || !draft_tokens)) return FD_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(logits) % 4 != 0) return FD_ERR_INVALID_ARG;
    const long long ctas = (long long)total_cand_rows * ((vocab + fd::kAcceptChunk - 1) / fd::kAcceptChunk);
    if (ctas > 0x7fffffffLL) return FD_ERR_UNSUPPORTED;

    unsigned long long* scratch = nullptr;
    const fd_status st = scratch_for_current_device(&scratch);
    if (st != FD_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The array keeps whatever the previous call (of anyone in this process) left behind: the keys of
    // this call's rows, the ticket and the status sink must start at zero.
    if (cudaMemsetAsync(scratch, 0, sizeof(unsigned long long) * (size_t)total_cand_rows, s) != cudaSuccess ||
        cudaMemsetAsync(scratch + FD_STATIC_MAX_ROWS, 0, sizeof(unsigned long long) * 8, s) != cudaSuccess) {
        cudaGetLastError();
        return FD_ERR_CUDA;
    }
    fd::AcceptParams p;
    p.batch = batch; p.total_rows = total_cand_rows; p.vocab = vocab;
    p.logits = logits; p.drafts = draft_tokens; p.q_lens = q_lens; p.n_mask = n_mask;
    p.accepted = accepted_len; p.bonus = bonus_token;
    p.chained = 0;
    p.keys = scratch;
    p.ticket = reinterpret_cast<unsigned int*>(scratch + FD_STATIC_MAX_ROWS);
    p.status = device_status ? device_status : reinterpret_cast<int*>(scratch + FD_STATIC_MAX_ROWS + 1);
    fd::launch_accept(p, s);
    return cudaGetLastError() == cudaSuccess ? FD_OK : FD_ERR_CUDA;
}

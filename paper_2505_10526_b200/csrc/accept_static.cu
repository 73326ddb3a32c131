// massv_accept_static: the acceptance call for callers that cannot allocate.
//
// Some hosts of this library have no way to obtain device memory at the point
// where they verify a block: a serving loop whose memory pool was carved up at
// start-up and is full, a plug-in that runs inside someone else's CUDA context
// under a "no allocation after initialisation" rule, or code on a latency path
// where cudaMalloc (which synchronises the device) is forbidden.  For them the
// scratch that massv_accept takes from the caller's workspace lives here, in a
// fixed array that is part of the library image on every GPU that loads it.
#include <mutex>

#include "kernels.cuh"

using namespace massv;

namespace {

// Limits of the built-in scratch.
constexpr int kStaticMaxRows = 64;          // B * (gamma + 1)
constexpr int kStaticMaxBatch = 64;
constexpr int kStaticMaxVocab = 524288;
constexpr int kStaticMaxParts = 192;        // lm_head_num_partials() never exceeds this (one slot per CTA, at most 192 CTAs)
constexpr int kStaticMaxChunks = kStaticMaxVocab / kResidualChunk;

constexpr size_t kA = 256;
constexpr size_t up(size_t x) { return (x + kA - 1) / kA * kA; }
constexpr size_t kOffMax = 0;
constexpr size_t kOffSum = kOffMax + up((size_t)kStaticMaxParts * kStaticMaxRows * sizeof(float));
constexpr size_t kOffIdx = kOffSum + up((size_t)kStaticMaxParts * kStaticMaxRows * sizeof(float));
constexpr size_t kOffState = kOffIdx + up((size_t)kStaticMaxParts * kStaticMaxRows * sizeof(int32_t));
constexpr size_t kOffChunks = kOffState + up((size_t)kStaticMaxBatch * sizeof(SeqState));
constexpr size_t kOffCounters = kOffChunks + up((size_t)kStaticMaxBatch * kStaticMaxChunks * sizeof(double));
constexpr size_t kScratchBytes = kOffCounters + up((size_t)kStaticMaxBatch * sizeof(unsigned int));   // about 210 KiB

// The scratch itself.  In host code this name is only a handle for
// cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_accept_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch on the current device, resolved once per device.
int scratch_address(char** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MASSV_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_accept_scratch) != cudaSuccess || ptr == nullptr) return MASSV_ERR_CUDA;
        g_scratch_addr[dev] = ptr;
    }
    *out = static_cast<char*>(g_scratch_addr[dev]);
    return MASSV_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" int massv_accept_static(const massv_accept_desc* desc, const void* hidden, const void* lm_head,
                                   const int32_t* draft_tokens, const float* draft_probs, const float* u_accept,
                                   const float* u_sample, int32_t* out_tokens, int32_t* accept_len, float* logits_out,
                                   float* probs_out, int32_t* dev_status, massv_stream_t stream) {
    if (!desc) return MASSV_ERR_INVALID_ARG;
    if (desc->batch < 1 || desc->gamma < 0 || desc->hidden < 1 || desc->vocab < 1 || !(desc->temperature >= 0.f))
        return MASSV_ERR_INVALID_ARG;
    if (desc->gamma > kMaxRows - 1 || desc->hidden % 64 != 0 || desc->vocab % 8 != 0 || desc->flags != 0)
        return MASSV_ERR_UNSUPPORTED;
    const long M = (long)desc->batch * (desc->gamma + 1);
    const int n_part = lm_head_num_partials((int)M, desc->vocab);
    const int n_chunks = (desc->vocab + kResidualChunk - 1) / kResidualChunk;
    // the built-in scratch is fixed: refuse what does not fit instead of overrunning it
    if (M > kStaticMaxRows || desc->batch > kStaticMaxBatch || desc->vocab > kStaticMaxVocab ||
        n_part > kStaticMaxParts || n_chunks > kStaticMaxChunks)
        return MASSV_ERR_WORKSPACE;
    const bool sampling = desc->temperature > 0.f;
    if (!hidden || !lm_head || !out_tokens || !accept_len) return MASSV_ERR_INVALID_ARG;
    if (desc->gamma > 0 && !draft_tokens) return MASSV_ERR_INVALID_ARG;
    if (sampling && (!logits_out || !u_sample || (desc->gamma > 0 && (!draft_probs || !u_accept))))
        return MASSV_ERR_INVALID_ARG;
    if (!sampling && probs_out) return MASSV_ERR_INVALID_ARG;
    if (!aligned16(hidden) || !aligned16(lm_head) || (draft_probs && !aligned16(draft_probs)) ||
        (logits_out && !aligned16(logits_out)) || (probs_out && !aligned16(probs_out)))
        return MASSV_ERR_INVALID_ARG;

    char* ws = nullptr;
    const int rc = scratch_address(&ws);
    if (rc != MASSV_OK) return rc;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    // The array keeps whatever the previous call left.  Nothing in it has to be cleared from the host:
    // every part is written by a kernel of this call before a later kernel reads it (the arrival
    // counters of the residual draw are zeroed by the scan kernel that runs before it).

    LmHeadParams g;
    g.M = (int)M; g.K = desc->hidden; g.V = desc->vocab;
    g.greedy = sampling ? 0 : 1;
    g.inv_T_log2e = sampling ? 1.4426950408889634f / desc->temperature : 0.f;
    g.hidden = static_cast<const __nv_bfloat16*>(hidden);
    g.lm_head = static_cast<const __nv_bfloat16*>(lm_head);
    g.logits = logits_out;
    g.n_part = n_part;
    g.part_max = reinterpret_cast<float*>(ws + kOffMax);
    g.part_sum = reinterpret_cast<float*>(ws + kOffSum);
    g.part_idx = reinterpret_cast<int32_t*>(ws + kOffIdx);
    g.dev_status = dev_status;
    int n_part_used = 0;
    if (launch_lm_head(g, s, &n_part_used) != cudaSuccess) return MASSV_ERR_CUDA;

    AcceptParams a;
    a.B = desc->batch; a.gamma = desc->gamma; a.V = desc->vocab; a.T = desc->temperature;
    a.n_part = n_part_used; a.part_max = g.part_max; a.part_sum = g.part_sum; a.part_idx = g.part_idx;
    a.logits = logits_out;
    a.draft_tokens = draft_tokens; a.draft_probs = draft_probs; a.u_accept = u_accept; a.u_sample = u_sample;
    a.out_tokens = out_tokens; a.accept_len = accept_len; a.probs_out = probs_out;
    a.seq_state = reinterpret_cast<SeqState*>(ws + kOffState);
    a.chunk_sums = reinterpret_cast<double*>(ws + kOffChunks);
    a.counters = reinterpret_cast<unsigned int*>(ws + kOffCounters);
    a.n_chunks = n_chunks;
    a.dev_status = dev_status;
    return launch_accept(a, s) == cudaSuccess ? MASSV_OK : MASSV_ERR_CUDA;
}

// C-ABI entry points of the whole-stack W4A16 decode launch: the host-side plan (how every
// problem's quanta are dealt to the CTAs) and the launch itself.
#include <cuda_fp16.h>

#include <cstring>

#include "common.h"
#include "stack.h"

namespace mnnllm {
namespace {

constexpr size_t kSmemBudget = 227 * 1024;
constexpr long long kStageBudget = 40 * 1024;   // staged activations per CTA at most

int mp_of(int M) { return M <= 1 ? 1 : (M <= 2 ? 2 : (M <= 4 ? 4 : 8)); }

// most quanta a CTA receives when U runs of `gran` quanta are dealt evenly to n CTAs
long long max_share(long long U, int gran, int n) {
    if (U < n) return gran;
    return ((U + n - 1) / n) * gran;
}

}  // namespace
}  // namespace mnnllm

using namespace mnnllm;

extern "C" {

size_t mnnllm_stack_plan_size(int count) {
    if (count < 1 || count > MNNLLM_STACK_MAX_PROBLEMS) return 0;
    return sizeof(StackHeader) + (size_t)count * sizeof(StackProblem);
}

int mnnllm_stack_plan_w4a16(const mnnllm_stack_problem* problems, int count, int M, int group, int n_sms,
                            void* plan_out) {
    if (!problems || !plan_out || count < 1 || count > MNNLLM_STACK_MAX_PROBLEMS || M < 1) return MNNLLM_ERR_INVALID_ARG;
    if (M > 8 || (group != 64 && group != 128)) return MNNLLM_ERR_UNSUPPORTED;
    if (n_sms == 0) {
        if (!device_is_supported()) return MNNLLM_ERR_UNSUPPORTED;
        n_sms = device_sm_count();
    }
    if (n_sms < 1) return MNNLLM_ERR_INVALID_ARG;
    const int MP = mp_of(M);
    const int W = kStackConsumerWarps;

    for (int p = 0; p < count; ++p) {
        const mnnllm_stack_problem& q = problems[p];
        if (!q.x || !q.packed || !q.y || q.N < 1 || q.K < 1) return MNNLLM_ERR_INVALID_ARG;
        if (q.K % group != 0) return MNNLLM_ERR_UNSUPPORTED;
        if (q.y_dtype != MNNLLM_F16 && q.y_dtype != MNNLLM_BF16 && q.y_dtype != MNNLLM_F32) return MNNLLM_ERR_UNSUPPORTED;
        if (((uintptr_t)q.x & 15) || ((uintptr_t)q.y & 15) || ((uintptr_t)q.packed & 127)) return MNNLLM_ERR_ALIGNMENT;
        if (q.n_deps < 0 || q.n_deps > MNNLLM_STACK_MAX_DEPS) return MNNLLM_ERR_INVALID_ARG;
        for (int d = 0; d < q.n_deps; ++d)
            if (q.deps[d] < 0 || q.deps[d] >= p) return MNNLLM_ERR_INVALID_ARG;   // only earlier problems
    }

    StackHeader H;
    std::memset(&H, 0, sizeof(H));
    StackProblem* out = reinterpret_cast<StackProblem*>((uint8_t*)plan_out + sizeof(StackHeader));
    std::memset(out, 0, (size_t)count * sizeof(StackProblem));
    int fused_of[MNNLLM_STACK_MAX_PROBLEMS];   // caller's problem -> problem of the plan
    int n_plan = 0;
    auto same_deps = [&](const mnnllm_stack_problem& a, const mnnllm_stack_problem& b) {
        if (a.n_deps != b.n_deps) return false;
        for (int i = 0; i < a.n_deps; ++i) {
            bool found = false;
            for (int j = 0; j < b.n_deps; ++j) found |= a.deps[i] == b.deps[j];
            if (!found) return false;
        }
        return true;
    };
    // Neighbours in the list that read the same activations and wait for the same predecessors
    // (q, k, v; gate, up) become ONE problem of the plan: their row blocks are dealt to the CTAs
    // together, so they cost one pass of the problem loop instead of one each.
    for (int p = 0; p < count;) {
        int e = p + 1;
        while (e < count && e - p < kStackMaxSub && problems[e].x == problems[p].x && problems[e].K == problems[p].K &&
               same_deps(problems[e], problems[p]))
            ++e;
        StackProblem& D = out[n_plan];
        const W4Geometry g0 = w4_geometry(problems[p].N, problems[p].K, group);
        D.x = problems[p].x;
        D.K = problems[p].K;
        D.row_block_bytes = g0.row_block_bytes;
        D.NC = g0.n_chunks; D.NS = g0.n_slabs;
        int nb = 0;
        for (int i = p; i < e; ++i) {
            const W4Geometry g = w4_geometry(problems[i].N, problems[i].K, group);
            nb += g.n_row_blocks;
            D.packed[i - p] = (const uint8_t*)problems[i].packed;
            D.y[i - p] = problems[i].y;
            D.N[i - p] = problems[i].N;
            D.nb_end[i - p] = nb;
            D.y_dtypes |= problems[i].y_dtype << (8 * (i - p));
            fused_of[i] = n_plan;
        }
        for (int i = e - p; i < kStackMaxSub; ++i) D.nb_end[i] = nb;
        D.NB = nb;
        for (int d = 0; d < problems[p].n_deps; ++d) {      // predecessors in the plan's numbering, once each
            const int f = fused_of[problems[p].deps[d]];
            bool have = false;
            for (int j = 0; j < D.n_deps; ++j) have |= D.deps[j] == f;
            if (!have) {
                D.deps[D.n_deps] = f;
                D.deps_nb[D.n_deps] = out[f].NB;
                ++D.n_deps;
            }
        }
        ++n_plan;
        p = e;
    }

    long long max_quanta = 1, xs_bytes = 0;
    int rot = 0;
    for (int p = 0; p < n_plan; ++p) {
        StackProblem& D = out[p];
        D.weff = D.NC <= W ? (W / D.NC) * D.NC : W;
        // Whole 16-row blocks per CTA (no exchange between CTAs) or runs of single quanta (even
        // shares, blocks shared between neighbours): whichever needs fewer rounds of the CTA's
        // warps, an exchange counting as half a round.
        const long long Q = (long long)D.NB * D.NC;
        if (Q * n_sms >= (1ll << 31)) return MNNLLM_ERR_UNSUPPORTED;   // the kernel deals quanta in 32-bit arithmetic
        const long long whole = max_share(D.NB, D.NC, n_sms), single = max_share(Q, 1, n_sms);
        const double cost_whole = (double)((whole + D.weff - 1) / D.weff);
        const double cost_single = (double)((single + D.weff - 1) / D.weff) + 0.5;
        D.gran = (D.NC > 1 && cost_single < cost_whole) ? 1 : D.NC;
        const long long U = Q / D.gran;
        const long long share = D.gran == 1 ? single : whole;
        max_quanta = share > max_quanta ? share : max_quanta;
        // activations go through shared memory when the chunks one CTA needs are small enough
        const long long x_need = (share < D.NC ? share : D.NC) * (long long)M * kChunkK * 2;
        D.stage_x = x_need <= kStageBudget ? 1 : 0;
        if (D.stage_x && x_need > xs_bytes) xs_bytes = x_need;
        // consecutive small problems start on different SMs
        D.rot = rot;
        rot = (int)((rot + (U < n_sms ? U : 0)) % n_sms);
    }
    // the ring takes what the partial sums leave of the CTA's shared memory
    // the ring takes what is left of the CTA's shared memory: the same number of slots for each consumer warp
    int slots = 0;
    for (int r = 1; r <= 8; ++r)
        if (stack_w4a16_smem(group, MP, n_plan, r * W, (int)max_quanta, (int)xs_bytes) <= kSmemBudget) slots = r * W;
    if (slots < W) return MNNLLM_ERR_UNSUPPORTED;   // a problem too large for M <= 8 at this shape
    H.magic = kStackMagic; H.version = 1;
    H.count = n_plan; H.M = M; H.group = group; H.MP = MP;
    H.n_ctas = n_sms;
    H.ring_slots = slots;
    H.max_quanta = (int32_t)max_quanta;
    H.xs_bytes = (uint32_t)xs_bytes;
    H.smem_bytes = (uint32_t)stack_w4a16_smem(group, MP, n_plan, slots, (int)max_quanta, (int)xs_bytes);
    std::memcpy(plan_out, &H, sizeof(H));
    return MNNLLM_OK;
}

size_t mnnllm_stack_workspace_size(const void* plan_host) {
    if (!plan_host) return 0;
    StackHeader H;
    std::memcpy(&H, plan_host, sizeof(H));
    if (H.magic != kStackMagic) return 0;
    return stack_ws_bytes(H.count, H.n_ctas, H.MP);
}

int mnnllm_stack_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    if (!workspace || workspace_bytes == 0) return MNNLLM_ERR_INVALID_ARG;
    if (cudaMemsetAsync(workspace, 0, workspace_bytes, (cudaStream_t)stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return MNNLLM_ERR_CUDA;
    }
    return MNNLLM_OK;
}

int mnnllm_linear_w4a16_stack(const void* plan_host, const void* plan_dev, void* workspace, size_t workspace_bytes,
                              void* stream) {
    if (!plan_host || !plan_dev) return MNNLLM_ERR_INVALID_ARG;
    StackHeader H;
    std::memcpy(&H, plan_host, sizeof(H));
    if (H.magic != kStackMagic || H.version != 1 || H.count < 1) return MNNLLM_ERR_INVALID_ARG;
    if ((uintptr_t)plan_dev & 15) return MNNLLM_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < stack_ws_bytes(H.count, H.n_ctas, H.MP)) return MNNLLM_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 255) return MNNLLM_ERR_ALIGNMENT;
    if (!device_is_supported()) return MNNLLM_ERR_UNSUPPORTED;
    if (H.n_ctas > device_sm_count()) return MNNLLM_ERR_UNSUPPORTED;   // all CTAs must be resident
    uint32_t* status = status_word_ptr();
    if (!status) return MNNLLM_ERR_CUDA;
    StackWorkspace ws;
    uint8_t* base = (uint8_t*)workspace;
    ws.epoch = (uint32_t*)base;
    ws.done = (uint32_t*)(base + 4);
    ws.flags = (uint32_t*)(base + stack_ws_flags_offset());
    ws.parts = (unsigned long long*)(base + stack_ws_parts_offset(H.count));
    const void* problems_dev = (const uint8_t*)plan_dev + sizeof(StackHeader);
    if (stack_w4a16_launch(H, problems_dev, ws, status, (cudaStream_t)stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return MNNLLM_ERR_CUDA;
    }
    return MNNLLM_OK;
}

}  // extern "C"

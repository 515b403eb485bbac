// C-ABI entry points of the weight-only (W4A16 / W8A16) decode path: argument checks, the launch
// plan (how rows and k-chunks are spread over warps, CTAs and clusters) and the kernel launches.
#include <cuda_fp16.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "common.h"
#include "gemv.h"
#include "ptx.cuh"

namespace mnnllm {

__device__ uint32_t g_status_word = 0;

namespace {
struct DeviceFacts {
    bool known;
    int cc_major, sm_count;
    uint32_t* status_ptr;
};
PerDevice<DeviceFacts> g_facts;

// the current device's facts, asked of the runtime on first use
cudaError_t device_facts(DeviceFacts& out) {
    return g_facts.with([&](DeviceFacts& f) {
        if (!f.known) {
            const int dev = current_device();
            void* p = nullptr;
            cudaError_t e = cudaDeviceGetAttribute(&f.cc_major, cudaDevAttrComputeCapabilityMajor, dev);
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&f.sm_count, cudaDevAttrMultiProcessorCount, dev);
            if (e == cudaSuccess) e = cudaGetSymbolAddress(&p, g_status_word);
            if (e != cudaSuccess) return e;
            f.status_ptr = (uint32_t*)p;
            f.known = true;
        }
        out = f;
        return cudaSuccess;
    });
}
}  // namespace

int device_is_supported() {
    DeviceFacts f;
    if (device_facts(f) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    return f.cc_major == 10;
}

int device_sm_count() {
    DeviceFacts f;
    if (device_facts(f) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    return f.sm_count;
}

uint32_t* status_word_ptr() {
    DeviceFacts f;
    if (device_facts(f) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    return f.status_ptr;
}

// One warp waits on a barrier that nobody will ever arrive at, with the same bounded wait the
// kernels use; when the wait runs out it records a code in the status word and returns normally.
__global__ void wait_timeout_kernel(uint32_t max_polls, uint32_t* status) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        ptx::fence_mbar_init();
    }
    __syncwarp();
    if (!ptx::mbar_wait_bounded_compact(&bar, 0, max_polls) && threadIdx.x == 0)
        atomicOr(status, MNNLLM_DEBUG_TIMEOUT_DETAIL);
}

namespace {

struct Plan {
    int CS, WC, SR, RBI, stages;
    int clusters;  // total clusters of the launch (persistent: about one resident set)
};

// Resident CTAs per SM, asked of the runtime once per configuration and device, and cached.
int cached_occupancy(int bits, int group, int MP, int W, int SR, int S) {
    struct Entry { int key[6]; int occ; };
    struct Table { Entry e[64]; int n; };
    static PerDevice<Table> tables;
    const int key[6] = {bits, group, MP, W, SR, S};
    int occ = 0;
    (void)tables.with([&](Table& t) {
        for (int i = 0; i < t.n; ++i)
            if (!std::memcmp(t.e[i].key, key, sizeof(key))) { occ = t.e[i].occ; return cudaSuccess; }
        return cudaSuccess;
    });
    if (occ) return occ;
    // asked outside the table's lock: the query itself takes the kernels' own per-device locks
    occ = bits == 4 ? gemv_w4a16_occupancy(group, MP, W, SR, S) : gemv_w8a16_occupancy(W, SR, S);
    if (occ < 1) occ = 1;
    (void)tables.with([&](Table& t) {
        if (t.n < 64) {
            std::memcpy(t.e[t.n].key, key, sizeof(key));
            t.e[t.n++].occ = occ;
        }
        return cudaSuccess;
    });
    return occ;
}

// How the quanta (16 rows x 512 k) of a launch are spread: WC warps of a CTA take different
// k-chunks, SR groups of warps take different row blocks, a cluster of CS CTAs splits K further
// when there are too few row blocks to occupy the GPU.  The grid is persistent: about as many
// CTAs as fit on the GPU at once, each walking an even share of the row blocks in rounds of
// SR * RBI blocks, so that the activation fragments a warp builds are reused RBI times.
Plan make_plan(int nb_total, int nc_max, int group, int MP, int bits = 4) {
    Plan p;
    p.CS = 1;
    while (p.CS < 8 && p.CS * 2 <= nc_max && nc_max >= 4 &&
           (nb_total * p.CS < 120 || (nb_total * p.CS < 400 && p.CS * kGemvMaxWarps < nc_max)))
        p.CS *= 2;
    p.WC = (nc_max + p.CS - 1) / p.CS;
    if (p.WC > kGemvMaxWarps) p.WC = kGemvMaxWarps;
    p.SR = kGemvMaxWarps / p.WC;
    const int n_sms = device_sm_count() > 0 ? device_sm_count() : 148;
    while (p.SR > 1 && nb_total * p.CS < n_sms * p.SR) --p.SR;
    p.stages = 3;
    p.RBI = 0;
    int forced_clusters = 0;
    bool stages_forced = false;
    if (const char* env = std::getenv("MNNLLM_GEMV_PLAN")) {  // tuning override: "CS,WC,SR,RBI,stages[,clusters]"
        int v[6] = {0, 0, 0, 0, 0, 0};
        if (std::sscanf(env, "%d,%d,%d,%d,%d,%d", &v[0], &v[1], &v[2], &v[3], &v[4], &v[5]) >= 5) {
            if (v[0] >= 1 && v[0] <= 8) p.CS = v[0];
            if (v[1] >= 1 && v[1] <= kGemvMaxWarps) p.WC = v[1];
            if (v[2] >= 1 && v[1] * v[2] <= kGemvMaxWarps) p.SR = v[2];
            if (v[3] >= 1 && v[3] <= kGemvMaxRBI) p.RBI = v[3];
            if (v[4] >= 1 && v[4] <= kGemvMaxStages) { p.stages = v[4]; stages_forced = true; }
            if (v[5] >= 1) forced_clusters = v[5];
        }
    }
    auto smem = [&](int st) {
        return bits == 4 ? gemv_w4a16_smem(group, MP, p.WC * p.SR, p.SR, st) : gemv_w8a16_smem(p.WC * p.SR, p.SR, st);
    };
    while (p.stages > 1 && smem(p.stages) > 220 * 1024) --p.stages;
    // Ring depth: a warp with only a few quanta wants them all in flight before the activations
    // arrive (three slots); long streams ran 3 % faster with two (measured on the 7B stack and the LM
    // head).  The shallower ring can also let one more CTA fit an SM, so the grid is sized again
    // after the depth has been chosen.
    for (int pass = 0; pass < 2; ++pass) {
        const int occ = cached_occupancy(bits, group, MP, p.WC * p.SR, p.SR, p.stages);
        int clusters = n_sms * occ / p.CS;
        const int max_useful = (nb_total + p.SR - 1) / p.SR;  // at least SR row blocks per cluster
        if (clusters > max_useful) clusters = max_useful;
        if (forced_clusters) clusters = forced_clusters;
        if (clusters < 1) clusters = 1;
        p.clusters = clusters;
        if (stages_forced || pass == 1) break;
        const long long warps = (long long)clusters * p.CS * p.WC * p.SR;
        const long long quanta = (long long)nb_total * nc_max;
        if (quanta > 4 * warps && p.stages > 2) p.stages = 2; else break;
    }
    if (p.RBI == 0) {
        p.RBI = (nb_total + p.clusters * p.SR - 1) / (p.clusters * p.SR);
        p.RBI = p.RBI < 1 ? 1 : (p.RBI > kGemvMaxRBI ? kGemvMaxRBI : p.RBI);
    }
    return p;
}

// Splits the launch's clusters over the problems in proportion to their row blocks (at least one each).
void share_clusters(const int* nb, int count, int total, int SR, int* out) {
    int nb_total = 0;
    for (int i = 0; i < count; ++i) nb_total += nb[i];
    for (int i = 0; i < count; ++i) {
        long long want = ((long long)total * nb[i] + nb_total / 2) / nb_total;
        const int cap = (nb[i] + SR - 1) / SR;
        if (want > cap) want = cap;
        if (want < 1) want = 1;
        out[i] = (int)want;
    }
}

int check_problem(const mnnllm_w4a16_problem& q, int M) {
    if (!q.x || !q.packed || !q.y || M < 1 || q.N < 1 || q.K < 1) return MNNLLM_ERR_INVALID_ARG;
    if ((q.group != 64 && q.group != 128) || q.K % q.group != 0) return MNNLLM_ERR_UNSUPPORTED;
    if (q.y_dtype != MNNLLM_F16 && q.y_dtype != MNNLLM_BF16 && q.y_dtype != MNNLLM_F32) return MNNLLM_ERR_UNSUPPORTED;
    if (((uintptr_t)q.x & 15) || ((uintptr_t)q.y & 15) || ((uintptr_t)q.packed & 127)) return MNNLLM_ERR_ALIGNMENT;
    return MNNLLM_OK;
}

struct LoraArgs {   // bypass of one problem of a batch (r == 0: none)
    const __half* A;     // [N, r]
    const __half* B;     // [r, K]
    float* t;            // [M, r] scratch
    unsigned int* sync;  // two counters, zero between launches
    int r;
};

int run_batch(const mnnllm_w4a16_problem* problems, int count, int M, int x_dtype, cudaStream_t stream,
              const LoraArgs* lora = nullptr) {
    if (!problems || count < 1 || count > MNNLLM_MAX_BATCH) return MNNLLM_ERR_INVALID_ARG;
    const int group = problems[0].group;
    for (int i = 0; i < count; ++i) {
        const int st = check_problem(problems[i], M);
        if (st != MNNLLM_OK) return st;
        if (problems[i].group != group) return MNNLLM_ERR_UNSUPPORTED;
    }
    if (!device_is_supported()) return MNNLLM_ERR_UNSUPPORTED;
    uint32_t* status = status_word_ptr();
    if (!status) return MNNLLM_ERR_CUDA;

    int nb_total = 0, nc_max = 0;
    for (int i = 0; i < count; ++i) {
        const W4Geometry g = w4_geometry(problems[i].N, problems[i].K, group);
        nb_total += g.n_row_blocks;
        nc_max = g.n_chunks > nc_max ? g.n_chunks : nc_max;
    }
    // tokens are processed in passes of at most 8 (one pass over the weights each)
    for (int m0 = 0; m0 < M; m0 += 8) {
        const int m = (M - m0) < 8 ? (M - m0) : 8;
        const int MP = m <= 1 ? 1 : (m <= 2 ? 2 : (m <= 4 ? 4 : 8));
        const Plan plan = make_plan(nb_total, nc_max, group, MP);
        GemvLaunch L;
        std::memset(&L, 0, sizeof(L));
        L.count = count; L.M = m; L.WC = plan.WC; L.SR = plan.SR; L.RBI = plan.RBI; L.stages = plan.stages;
        int clusters = 0, nbs[MNNLLM_MAX_BATCH], ncl[MNNLLM_MAX_BATCH];
        for (int i = 0; i < count; ++i) nbs[i] = w4_geometry(problems[i].N, problems[i].K, group).n_row_blocks;
        share_clusters(nbs, count, plan.clusters, plan.SR, ncl);
        for (int i = 0; i < count; ++i) {
            const mnnllm_w4a16_problem& q = problems[i];
            const W4Geometry g = w4_geometry(q.N, q.K, group);
            GemvProblem& P = L.prob[i];
            const size_t ybytes = q.y_dtype == MNNLLM_F32 ? 4 : 2;
            P.packed = (const uint8_t*)q.packed;
            P.x = (const __half*)q.x + (size_t)m0 * q.K;
            P.y = (uint8_t*)q.y + (size_t)m0 * q.N * ybytes;
            P.N = q.N; P.K = q.K;
            P.NB = g.n_row_blocks; P.NC = g.n_chunks; P.NS = g.n_slabs;
            P.cluster_begin = clusters;
            P.n_clusters = ncl[i];
            P.y_dtype = q.y_dtype;
            P.x_dtype = x_dtype;
            P.row_block_bytes = g.row_block_bytes;
            if (lora && lora[i].r > 0) {
                P.lora_A = lora[i].A;
                P.lora_B = lora[i].B;
                P.lora_t = lora[i].t;   // every pass of eight tokens reuses the scratch from its start
                P.lora_sync = lora[i].sync;
                P.lora_r = lora[i].r;
            }
            clusters += ncl[i];
        }
        if (gemv_w4a16_launch(L, group, MP, clusters, plan.CS, status, stream) != cudaSuccess) {
            (void)cudaGetLastError();
            return MNNLLM_ERR_CUDA;
        }
    }
    return MNNLLM_OK;
}

}  // namespace
}  // namespace mnnllm

using namespace mnnllm;

extern "C" {

int mnnllm_device_supported(void) { return device_is_supported(); }

int mnnllm_read_status(void* stream, uint32_t* detail) {
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return MNNLLM_ERR_CUDA;
    uint32_t* p = status_word_ptr();
    if (!p) return MNNLLM_ERR_CUDA;
    uint32_t v = 0, zero = 0;
    if (cudaMemcpy(&v, p, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return MNNLLM_ERR_CUDA;
    if (v && cudaMemcpy(p, &zero, 4, cudaMemcpyHostToDevice) != cudaSuccess) return MNNLLM_ERR_CUDA;
    if (detail) *detail = v;
    return v ? MNNLLM_ERR_TIMEOUT : MNNLLM_OK;
}

int mnnllm_debug_wait_timeout(int max_polls, void* stream) {
    if (max_polls < 1 || max_polls > 1000) return MNNLLM_ERR_INVALID_ARG;
    if (!device_is_supported()) return MNNLLM_ERR_UNSUPPORTED;
    uint32_t* status = status_word_ptr();
    if (!status) return MNNLLM_ERR_CUDA;
    wait_timeout_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((uint32_t)max_polls, status);
    if (cudaGetLastError() != cudaSuccess) return MNNLLM_ERR_CUDA;
    return MNNLLM_OK;
}

int mnnllm_linear_w4a16_batch(const mnnllm_w4a16_problem* problems, int count, int M, void* stream) {
    return run_batch(problems, count, M, MNNLLM_F16, (cudaStream_t)stream);
}

size_t mnnllm_workspace_size_lora(int M, int rank) {
    if (M < 1 || rank < 1 || rank > MNNLLM_LORA_MAX_RANK) return 0;
    return 256 + 8 * (size_t)rank * 8;   // epoch and counter | tagged t of one pass of at most eight tokens
}

int mnnllm_lora_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    if (!workspace || workspace_bytes < 256) return MNNLLM_ERR_INVALID_ARG;
    if (cudaMemsetAsync(workspace, 0, workspace_bytes, (cudaStream_t)stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return MNNLLM_ERR_CUDA;
    }
    return MNNLLM_OK;
}

int mnnllm_linear_w4a16_lora(const void* x, const void* packed, const void* lora_A, const void* lora_B, void* y, int M,
                             int N, int K, int group, int rank, int x_dtype, int y_dtype, void* workspace,
                             size_t workspace_bytes, void* stream) {
    if (!lora_A || !lora_B || rank < 1 || rank > MNNLLM_LORA_MAX_RANK) return MNNLLM_ERR_INVALID_ARG;
    if (x_dtype != MNNLLM_F16 && x_dtype != MNNLLM_BF16) return MNNLLM_ERR_UNSUPPORTED;
    mnnllm_w4a16_problem q;
    q.x = x; q.packed = packed; q.y = y; q.N = N; q.K = K; q.group = group; q.y_dtype = y_dtype;
    const int st = check_problem(q, M);
    if (st != MNNLLM_OK) return st;
    if (((uintptr_t)lora_B & 15) || ((uintptr_t)lora_A & 1)) return MNNLLM_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < mnnllm_workspace_size_lora(M, rank)) return MNNLLM_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 15) return MNNLLM_ERR_ALIGNMENT;
    LoraArgs l;
    l.A = (const __half*)lora_A; l.B = (const __half*)lora_B;
    l.sync = (unsigned int*)workspace;
    l.t = (float*)((uint8_t*)workspace + 256);
    l.r = rank;
    return run_batch(&q, 1, M, x_dtype, (cudaStream_t)stream, &l);
}

int mnnllm_linear_w8a16(const void* x, const void* packed, void* y, int M, int N, int K, int y_dtype, void* stream) {
    if (!x || !packed || !y || M < 1 || N < 1 || K < 1) return MNNLLM_ERR_INVALID_ARG;
    if (K % kSlabK8 != 0) return MNNLLM_ERR_UNSUPPORTED;
    if (y_dtype != MNNLLM_F16 && y_dtype != MNNLLM_BF16 && y_dtype != MNNLLM_F32) return MNNLLM_ERR_UNSUPPORTED;
    if (((uintptr_t)x & 15) || ((uintptr_t)y & 15) || ((uintptr_t)packed & 127)) return MNNLLM_ERR_ALIGNMENT;
    if (!device_is_supported()) return MNNLLM_ERR_UNSUPPORTED;
    uint32_t* status = status_word_ptr();
    if (!status) return MNNLLM_ERR_CUDA;
    const W8Geometry g = w8_geometry(N, K);
    const Plan plan = make_plan(g.n_row_blocks, g.n_chunks, 0, 8, 8);
    const size_t ybytes = y_dtype == MNNLLM_F32 ? 4 : 2;
    for (int m0 = 0; m0 < M; m0 += 8) {
        GemvLaunch L;
        std::memset(&L, 0, sizeof(L));
        L.count = 1; L.M = (M - m0) < 8 ? (M - m0) : 8; L.WC = plan.WC; L.SR = plan.SR; L.RBI = plan.RBI;
        L.stages = plan.stages;
        GemvProblem& P = L.prob[0];
        P.packed = (const uint8_t*)packed;
        P.x = (const __half*)x + (size_t)m0 * K;
        P.y = (uint8_t*)y + (size_t)m0 * N * ybytes;
        P.N = N; P.K = K; P.NB = g.n_row_blocks; P.NC = g.n_chunks; P.NS = g.n_slabs;
        P.cluster_begin = 0; P.n_clusters = plan.clusters; P.y_dtype = y_dtype;
        P.row_block_bytes = g.row_block_bytes; P.table_offset = g.table_offset;
        const int clusters = plan.clusters;
        if (gemv_w8a16_launch(L, clusters, plan.CS, status, (cudaStream_t)stream) != cudaSuccess) {
            (void)cudaGetLastError();
            return MNNLLM_ERR_CUDA;
        }
    }
    return MNNLLM_OK;
}

int mnnllm_linear_w4a16_ex(const void* x, const void* packed, void* y, int M, int N, int K, int group, int x_dtype,
                           int y_dtype, void* stream) {
    if (x_dtype != MNNLLM_F16 && x_dtype != MNNLLM_BF16)
        return x_dtype == MNNLLM_F32 ? MNNLLM_ERR_UNSUPPORTED : MNNLLM_ERR_INVALID_ARG;
    mnnllm_w4a16_problem p;
    p.x = x; p.packed = packed; p.y = y; p.N = N; p.K = K; p.group = group; p.y_dtype = y_dtype;
    return run_batch(&p, 1, M, x_dtype, (cudaStream_t)stream);
}

int mnnllm_linear_w4a16(const void* x, const void* packed, void* y, int M, int N, int K, int group, void* stream) {
    return mnnllm_linear_w4a16_ex(x, packed, y, M, N, K, group, MNNLLM_F16, MNNLLM_F16, stream);
}

}  // extern "C"

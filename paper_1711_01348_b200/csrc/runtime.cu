// Device side of the C ABI: the interpreter kernel, the zero-fill kernel and the launchers
// behind tad_forward / tad_backward / tad_step_host.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <mutex>
#include <new>
#include <string>

#include "plan.h"
#include "program.h"
#include "vm_shapes.h"

namespace tad {
void set_error(const std::string &m);
}

// One build of the interpreter per vector shape, each in an object file of its own (vm_inst.cu).
#define TAD_DECLARE_VM(TA, UB) bool tad_launch_vm_##TA##_##UB(const TadpProgram &prog, const TadpPointers &ptrs, bool debug, unsigned items, unsigned sms, cudaStream_t stream);
TAD_VM_SHAPES(TAD_DECLARE_VM)
bool tad_launch_vm_16_1_rich(const TadpProgram &prog, const TadpPointers &ptrs, bool debug, unsigned items, unsigned sms, cudaStream_t stream);
cudaError_t tad_launch_contract(const TadcProgram &P, const TadpPointers &ptrs, unsigned sms, cudaStream_t stream);
cudaError_t tad_launch_ew(const TadeProgram &P, const TadpPointers &ptrs, unsigned sms, cudaStream_t stream);
cudaError_t tad_launch_line(const TadlProgram &P, const TadpPointers &ptrs, unsigned sms, cudaStream_t stream);

namespace {


// Adds the zsplit planes of partial sums up and writes the gradient elements: compact index
// c -> outer variables -> output offset.  A block takes 32 consecutive cells (one per lane,
// so that every plane is read in full sectors); its warp w adds planes w, w + W, ... in that
// order and the warps' subtotals are added in warp order: the same association every run.
// W = 8 warps per block for up to 128 planes (many small blocks, all resident at once), 32 beyond.
// Masked gradients write only outputs whose flag says that some term was accumulated.
template <int REDUCE_WARPS>
__global__ void __launch_bounds__(REDUCE_WARPS * 32)
tad_reduce_partials(const __grid_constant__ TadpProgram P, float *out, const float *part)
{
    __shared__ float sub[REDUCE_WARPS][32];
    const unsigned n = (unsigned)P.part_limit;
    const int planes = P.zsplit;
    const unsigned lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    for (unsigned c0 = blockIdx.x * 32u; c0 < n; c0 += gridDim.x * 32u) {
        const unsigned c = c0 + lane;
        float sum = 0.f;
        if (c < n) {
#pragma unroll 4
            for (int s = (int)warp; s < planes; s += REDUCE_WARPS) sum += part[(size_t)s * n + c];
        }
        sub[warp][lane] = sum;
        __syncthreads();
        if (warp == 0 && c < n && !(P.write_only_live && part[(size_t)planes * n + c] == 0.f)) {
            unsigned rem = c, off = (unsigned)P.out_base;
            for (int v = P.n_outer - 1; v >= 0; --v) {
                const unsigned ext = (unsigned)P.outer_ext[v];
                const unsigned digit = rem % ext; rem /= ext;
                off += (unsigned)P.out_coef[v] * (unsigned)(P.outer_lo[v] + (int)digit);
            }
            if (off < (unsigned)P.out_limit) {
                float total = P.accumulate ? out[off] : 0.f;
                const int used = planes < REDUCE_WARPS ? planes : REDUCE_WARPS;
                for (int w = 0; w < used; ++w) total += sub[w][lane];
                out[off] = total;
            }
        }
        __syncthreads();
    }
}

void launch_reduce_partials(const TadpProgram &P, const TadpPointers &ptrs, unsigned blocks, cudaStream_t stream)
{
    if (P.zsplit > 128) tad_reduce_partials<32><<<blocks, 32 * 32, 0, stream>>>(P, ptrs.out, ptrs.part);
    else tad_reduce_partials<8><<<blocks, 8 * 32, 0, stream>>>(P, ptrs.out, ptrs.part);
}

// Sixteen independent multiply-add chains per thread, operands in registers only: the rate at which this GPU
// retires FP32 multiply-adds under its own clocks (the denominator of the ALU-bound roofline fractions).
__global__ void __launch_bounds__(256)
tad_fma_rate_kernel(float *sink, int iters, float m)
{
    float a[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) a[i] = (float)(threadIdx.x + i) * 1e-3f;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 16; ++i) a[i] = fmaf(a[i], m, 1e-7f);
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) s += a[i];
    if (s == 12345.678f) *sink = s;             // never true: keeps the chains alive
}

__global__ void tad_fill_zero(float *out, unsigned n)
{
    const unsigned stride = gridDim.x * blockDim.x;
    for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) out[i] = 0.f;
}

int sm_count()
{
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    return n;
}

unsigned long long item_count(const TadpProgram &P, int ta, int ub)
{
    unsigned long long n = 1;
    for (int v = 0; v < P.n_outer; ++v) {
        unsigned long long e = (unsigned long long)P.outer_ext[v];
        if (v == P.lane_var) e = (e + 32ull * ta - 1) / (32ull * ta);
        else if (ub > 1 && P.unroll_kind == 1 && v == P.unroll_var) e = (e + ub - 1) / ub;
        n *= e;
    }
    return n;
}

tad_status zero_fill(float *out, int64_t n, cudaStream_t stream);

// A second stream per plan.  Passes that only stream a tensor through memory (row and column sums, the zero fill of
// a gradient) are independent of the contraction they accompany and bound by another unit: they run beside it,
// forked from and joined to the caller's stream with events (which also works inside a stream capture).
struct Side {
    cudaStream_t s = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr, filled = nullptr;
    void release()
    {
        if (fork) cudaEventDestroy(fork);
        if (join) cudaEventDestroy(join);
        if (filled) cudaEventDestroy(filled);
        if (s) cudaStreamDestroy(s);
        s = nullptr; fork = join = filled = nullptr;
    }
};

// contraction kernels: one launch of the tile kernel per program
tad_status launch_contractions(const tad::Kernel &k, const TadpPointers &ptrs, cudaStream_t stream, Side *side)
{
    bool forked = false;
    for (size_t i = 0; i < k.contract.size(); ++i) {
        TadcProgram P = k.contract[i];
        if (P.ksplit > 1 && !ptrs.part) { tad::set_error("internal: partial-sum buffer missing"); return TAD_ERR_WORKSPACE; }
        // 16-byte copies and stores need 16-byte aligned tensors: fall back to 4-byte accesses otherwise
        auto misaligned = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
        if (P.modeA == TG_ROW16 && misaligned(ptrs.in[P.ptrA])) P.modeA = TG_ROW;
        if (P.ptrB >= 0 && P.modeB == TG_ROW16 && misaligned(ptrs.in[P.ptrB])) P.modeB = TG_ROW;
        if (P.out_vec4 && misaligned(ptrs.out)) P.out_vec4 = 0;
        // the streaming kernel copies B in 16-byte pieces
        if (P.shape == 5 && misaligned(ptrs.in[P.ptrB])) P.shape = 3;
        // single-column passes beside the tile kernel: no planes of partial sums, outputs of their own
        const bool beside = side && k.contract.size() > 1 && i > 0 && P.ksplit == 1 && !P.accumulate && (P.shape == 4 || P.shape == 6);
        cudaStream_t on = stream;
        if (beside) {
            if (!forked) {
                if (cudaEventRecord(side->fork, stream) != cudaSuccess || cudaStreamWaitEvent(side->s, side->fork, 0) != cudaSuccess) {
                    tad::set_error("event record / wait failed"); return TAD_ERR_CUDA;
                }
                forked = true;
            }
            on = side->s;
        }
        const cudaError_t e = tad_launch_contract(P, ptrs, (unsigned)sm_count(), on);
        if (e != cudaSuccess) { tad::set_error(std::string("contraction launch failed: ") + cudaGetErrorString(e)); return TAD_ERR_CUDA; }
    }
    if (forked && (cudaEventRecord(side->join, side->s) != cudaSuccess || cudaStreamWaitEvent(stream, side->join, 0) != cudaSuccess)) {
        tad::set_error("event record / wait failed"); return TAD_ERR_CUDA;
    }
    return TAD_OK;
}

// does the kernel (or one of the kernels that prepare its tensors) read through this pointer slot?
bool reads_slot(const tad::Kernel &k, int slot)
{
    for (const tad::Kernel &pk : k.pre) if (reads_slot(pk, slot)) return true;
    if (!k.contract.empty()) {
        for (const TadcProgram &P : k.contract) {
            if (P.ptrA == slot || P.ptrB == slot) return true;
            for (int e = 0; e < P.n_epi; ++e) if ((P.epi_op[e] == TE_MUL_LOAD || P.epi_op[e] == TE_ADD_LOAD) && P.epi_ptr[e] == slot) return true;
        }
        return false;
    }
    if (!k.ew.empty()) {
        for (int i = 0; i < k.ew[0].n_loads; ++i) if (k.ew[0].loads[i].ptr == slot) return true;
        return false;
    }
    if (!k.line.empty()) {
        for (int i = 0; i < k.line[0].n_loads; ++i) if (k.line[0].loads[i].ptr == slot) return true;
        for (int i = 0; i < k.line[0].n_scale; ++i) if (k.line[0].scale[i].ptr == slot) return true;
        return false;
    }
    for (int i = 0; i < k.prog.n_loads; ++i) if (k.prog.loads[i].ptr == slot) return true;
    return false;
}

// a kernel that only streams one tensor through memory into a tensor of its own: a single row- or column-sum pass
bool streams_only(const tad::Kernel &k)
{
    return k.pre.empty() && k.contract.size() == 1 && k.contract[0].ksplit == 1 && !k.contract[0].accumulate &&
           (k.contract[0].shape == 4 || k.contract[0].shape == 6);
}

// pending: an event the kernel that writes the output must wait for (the zero fill of its tensor on the second stream)
tad_status launch(const tad::Kernel &k, TadpPointers ptrs, bool debug, cudaStream_t stream, char *aux_base = nullptr,
                  Side *side = nullptr, cudaEvent_t pending = nullptr)
{
    if (!k.aux.empty()) {
        // auxiliary tensors of this kernel, then the kernels that fill them, in order
        if (!aux_base) { tad::set_error("this plan needs a workspace (auxiliary tensors): pass one of tad_workspace_bytes() bytes"); return TAD_ERR_WORKSPACE; }
        for (const tad::Kernel::Aux &a : k.aux) ptrs.in[a.slot] = reinterpret_cast<const float *>(aux_base + a.offset);
        // kernels that only stream a tensor run on the second stream, beside the kernels that do not read their result
        std::vector<int> beside;                       // slots of tensors being written on the second stream
        auto join = [&]() {
            if (beside.empty()) return true;
            beside.clear();
            return cudaEventRecord(side->join, side->s) == cudaSuccess && cudaStreamWaitEvent(stream, side->join, 0) == cudaSuccess;
        };
        // Launch order: the streaming passes move up to right behind the last kernel whose result they read, so that
        // they are issued before the long kernels they run beside (every tensor has one writer: moving a kernel up
        // past kernels that neither feed it nor read it changes nothing)
        const bool use_side = side && k.pre.size() > 1;
        std::vector<int> order;
        for (int i = 0; i < (int)k.pre.size(); ++i) {
            if (!(use_side && streams_only(k.pre[i]))) { order.push_back(i); continue; }
            size_t at = order.size();
            while (at > 0 && !reads_slot(k.pre[i], k.aux[k.pre[order[at - 1]].out_aux].slot)) --at;
            order.insert(order.begin() + at, i);
        }
        for (int i : order) {
            const tad::Kernel &pk = k.pre[i];
            TadpPointers pp = ptrs;
            pp.out = reinterpret_cast<float *>(aux_base + k.aux[pk.out_aux].offset);
            const bool on_side = use_side && streams_only(pk);
            bool wait = false;
            for (int slot : beside) wait = wait || reads_slot(pk, slot);
            if (wait && !on_side && !join()) { tad::set_error("event record / wait failed"); return TAD_ERR_CUDA; }
            if (on_side) {
                if (cudaEventRecord(side->fork, stream) != cudaSuccess || cudaStreamWaitEvent(side->s, side->fork, 0) != cudaSuccess) {
                    tad::set_error("event record / wait failed"); return TAD_ERR_CUDA;
                }
                beside.push_back(k.aux[pk.out_aux].slot);
            }
            const tad_status st = launch(pk, pp, debug, on_side ? side->s : stream, nullptr, on_side ? nullptr : side);
            if (st != TAD_OK) return st;
        }
        if (!join()) { tad::set_error("event record / wait failed"); return TAD_ERR_CUDA; }
    }
    if (pending && cudaStreamWaitEvent(stream, pending, 0) != cudaSuccess) { tad::set_error("event wait failed"); return TAD_ERR_CUDA; }
    if (!k.contract.empty()) return launch_contractions(k, ptrs, stream, side);
    if (!k.ew.empty()) {
        const cudaError_t e = tad_launch_ew(k.ew[0], ptrs, (unsigned)sm_count(), stream);
        if (e != cudaSuccess) { tad::set_error(std::string("element-wise launch failed: ") + cudaGetErrorString(e)); return TAD_ERR_CUDA; }
        return TAD_OK;
    }
    if (!k.line.empty()) {
        const TadlProgram &L = k.line[0];
        if (L.zsplit > 1 && !ptrs.part) { tad::set_error("internal: partial-sum buffer missing"); return TAD_ERR_WORKSPACE; }
        cudaError_t e = tad_launch_line(L, ptrs, (unsigned)sm_count(), stream);
        if (e == cudaSuccess && L.zsplit > 1) {
            const unsigned n = (unsigned)k.prog.part_limit;
            const unsigned rblocks = std::min((n + 31u) / 32u, (unsigned)sm_count() * 8u);
            launch_reduce_partials(k.prog, ptrs, rblocks, stream);
            e = cudaGetLastError();
        }
        if (e != cudaSuccess) { tad::set_error(std::string("line-sum launch failed: ") + cudaGetErrorString(e)); return TAD_ERR_CUDA; }
        return TAD_OK;
    }
    const int zsplit = k.prog.zsplit > 1 ? k.prog.zsplit : 1;
    if (zsplit > 1) {
        if (!ptrs.part) { tad::set_error("internal: partial-sum buffer missing"); return TAD_ERR_WORKSPACE; }
        if (k.prog.write_only_live) {
            // masked gradients: the flag plane must start at zero
            tad_status st = zero_fill(ptrs.part + (size_t)zsplit * k.prog.part_limit, k.prog.part_limit, stream);
            if (st != TAD_OK) return st;
        }
    }
    const unsigned long long items64 = item_count(k.prog, k.vec, k.vec_u) * (unsigned long long)zsplit;
    if (items64 == 0) return TAD_OK;
    if (items64 >= (1ull << 32)) { tad::set_error("too many work items"); return TAD_ERR_UNSUPPORTED; }
    const unsigned items = (unsigned)items64;
    bool launched = true;
    if (k.rich && !debug && k.vec == 16 && k.vec_u == 1) launched = tad_launch_vm_16_1_rich(k.prog, ptrs, debug, items, (unsigned)sm_count(), stream);
    else switch (k.vec * 100 + k.vec_u) {
#define TAD_CASE_VM(TA, UB) case TA * 100 + UB: launched = tad_launch_vm_##TA##_##UB(k.prog, ptrs, debug, items, (unsigned)sm_count(), stream); break;
    TAD_VM_SHAPES(TAD_CASE_VM)
    default: tad::set_error("internal: no kernel for this vector shape"); return TAD_ERR_UNSUPPORTED;
    }
    if (!launched) { tad::set_error("internal: this vector shape has no kernel build for the program (bounds checks or a relative loop)"); return TAD_ERR_UNSUPPORTED; }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { tad::set_error(std::string("kernel launch failed: ") + cudaGetErrorString(e)); return TAD_ERR_CUDA; }
    if (zsplit > 1) {
        const unsigned n = (unsigned)k.prog.part_limit;
        const unsigned rblocks = std::min((n + 31u) / 32u, (unsigned)sm_count() * 8u);
        launch_reduce_partials(k.prog, ptrs, rblocks, stream);
        e = cudaGetLastError();
        if (e != cudaSuccess) { tad::set_error(std::string("reduce launch failed: ") + cudaGetErrorString(e)); return TAD_ERR_CUDA; }
    }
    return TAD_OK;
}

tad_status zero_fill(float *out, int64_t n, cudaStream_t stream)
{
    const unsigned blocks = (unsigned)std::min<int64_t>((n + 255) / 256, (int64_t)sm_count() * 16);
    tad_fill_zero<<<blocks, 256, 0, stream>>>(out, (unsigned)n);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { tad::set_error(std::string("zero fill launch failed: ") + cudaGetErrorString(e)); return TAD_ERR_CUDA; }
    return TAD_OK;
}

}  // namespace

// streams and events of tad_step_host, owned by a plan
struct HostStep {
    static constexpr int N_EVENTS = 4 + TADP_MAX_PTRS;
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t ev[N_EVENTS] = {};
    void release()
    {
        for (cudaEvent_t &e : ev) if (e) { cudaEventDestroy(e); e = nullptr; }
        if (in) cudaStreamDestroy(in);
        if (out) cudaStreamDestroy(out);
        in = out = nullptr;
    }
};

// Scratch of tad_backward_noalloc: lives in the library image, one copy per GPU that loads it.
static __device__ __align__(256) unsigned char tad_noalloc_scratch[TAD_NOALLOC_SCRATCH_BYTES];

namespace {

constexpr int NOALLOC_MAX_DEVICES = 64;
void *g_noalloc_ptr[NOALLOC_MAX_DEVICES] = {};
std::mutex g_noalloc_mutex;

size_t pad256(size_t b) { return (b + 255) & ~size_t(255); }

// workspace layout: [256 B debug word, debug_bounds plans only][stage 0][stage 1]...
size_t stage_offset(const tad_plan *plan, int s)
{
    return (plan->opt.debug_bounds ? 256 : 0) + size_t(s) * pad256(size_t(plan->out_elems) * 4);
}

// workspace layout: ... [planes of partial sums][auxiliary tensors]
size_t aux_offset(const tad_plan *plan)
{
    return stage_offset(plan, (int)plan->stages.size()) + pad256(plan->partial_bytes);
}

// some kernel of the forward pass divides a summation among blocks (planes of partial sums in the workspace)
bool forward_splits(const tad::Kernel &k)
{
    for (const TadcProgram &cp : k.contract) if (cp.ksplit > 1) return true;
    for (const tad::Kernel &pk : k.pre) if (forward_splits(pk) || (pk.contract.empty() && pk.prog.zsplit > 1)) return true;
    return false;
}

bool check_workspace(const tad_plan *plan, void *workspace, size_t workspace_bytes)
{
    const size_t need = tad_workspace_bytes(plan);
    if (need && (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u))) {
        tad::set_error("workspace missing, smaller than tad_workspace_bytes() or not 256-byte aligned");
        return false;
    }
    return true;
}

bool fill_inputs(const tad_plan *plan, const float *const *args, const float *df, void *workspace, TadpPointers &ptrs)
{
    for (int a = 0; a < plan->n_args; ++a) {
        if (!args[a]) { tad::set_error("NULL argument tensor"); return false; }
        ptrs.in[a] = args[a];
    }
    ptrs.in[plan->n_args] = df;
    if (plan->opt.saved_forward) {
        if (!args[plan->n_args]) { tad::set_error("this plan was compiled with saved_forward: args[n_args] must be the forward output f"); return false; }
        ptrs.in[TADP_F_SLOT] = args[plan->n_args];
    }
    for (int s = 0; s < (int)plan->stages.size(); ++s)
        ptrs.in[plan->n_args + 1 + s] = reinterpret_cast<const float *>(static_cast<char *>(workspace) + stage_offset(plan, s));
    ptrs.debug = plan->opt.debug_bounds ? static_cast<int32_t *>(workspace) : nullptr;
    ptrs.part = plan->partial_bytes
        ? reinterpret_cast<float *>(static_cast<char *>(workspace) + stage_offset(plan, (int)plan->stages.size())) : nullptr;
    return true;
}

}  // namespace

namespace {
std::mutex g_side_mutex;
thread_local bool t_create_nothing = false;       // set while tad_backward_noalloc runs

// the plan's second stream, created by the first call that can use it (nullptr: run everything on the caller's stream)
Side *side_of(const tad_plan *plan)
{
    std::lock_guard<std::mutex> lock(g_side_mutex);
    if (plan->side) return static_cast<Side *>(plan->side);
    if (t_create_nothing) return nullptr;
    Side *sd = new (std::nothrow) Side();
    if (!sd) return nullptr;
    bool ok = cudaStreamCreateWithFlags(&sd->s, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&sd->fork, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&sd->join, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&sd->filled, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { sd->release(); delete sd; cudaGetLastError(); return nullptr; }
    plan->side = sd;
    return sd;
}
}  // namespace

void tad_release_host_step(const tad_plan *plan)
{
    if (plan && plan->side) {
        Side *sd = static_cast<Side *>(plan->side);
        sd->release();
        delete sd;
        plan->side = nullptr;
    }
    if (!plan || !plan->host_step) return;
    HostStep *hs = static_cast<HostStep *>(plan->host_step);
    hs->release();
    delete hs;
    plan->host_step = nullptr;
}

extern "C" {

size_t tad_workspace_bytes(const tad_plan *plan)
{
    if (!plan) return 0;
    return aux_offset(plan) + pad256(plan->aux_bytes);
}

tad_status tad_forward(const tad_plan *plan, const float *const *args, float *f,
                       void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!plan || !f || (plan->n_args && !args)) { tad::set_error("NULL argument"); return TAD_ERR_INVALID_ARG; }
    const bool needs_ws = !plan->forward.aux.empty() || forward_splits(plan->forward);
    if (needs_ws && !check_workspace(plan, workspace, workspace_bytes)) return TAD_ERR_WORKSPACE;
    TadpPointers ptrs{};
    for (int a = 0; a < plan->n_args; ++a) {
        if (!args[a]) { tad::set_error("NULL argument tensor"); return TAD_ERR_INVALID_ARG; }
        ptrs.in[a] = args[a];
    }
    ptrs.out = f;
    ptrs.debug = nullptr;
    char *aux_base = nullptr;
    if (needs_ws) {
        ptrs.part = plan->partial_bytes
            ? reinterpret_cast<float *>(static_cast<char *>(workspace) + stage_offset(plan, (int)plan->stages.size())) : nullptr;
        aux_base = static_cast<char *>(workspace) + aux_offset(plan);
    }
    return launch(plan->forward, ptrs, false, (cudaStream_t)cuda_stream, aux_base, side_of(plan));
}

tad_status tad_backward_stage(const tad_plan *plan, const float *const *args, const float *df,
                              void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!plan || !df || (plan->n_args && !args)) { tad::set_error("NULL argument"); return TAD_ERR_INVALID_ARG; }
    if (!check_workspace(plan, workspace, workspace_bytes)) return TAD_ERR_WORKSPACE;
    TadpPointers ptrs{};
    if (!fill_inputs(plan, args, df, workspace, ptrs)) return TAD_ERR_INVALID_ARG;
    for (int s = 0; s < (int)plan->stages.size(); ++s) {
        ptrs.out = reinterpret_cast<float *>(static_cast<char *>(workspace) + stage_offset(plan, s));
        tad_status st = launch(plan->stages[s], ptrs, plan->opt.debug_bounds != 0, (cudaStream_t)cuda_stream,
                               workspace ? static_cast<char *>(workspace) + aux_offset(plan) : nullptr, side_of(plan));
        if (st != TAD_OK) return st;
    }
    return TAD_OK;
}

tad_status tad_backward_arg(const tad_plan *plan, const float *const *args, const float *df,
                            int32_t arg, float *darg, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!plan || !df || !darg || (plan->n_args && !args)) { tad::set_error("NULL argument"); return TAD_ERR_INVALID_ARG; }
    if (arg < 0 || arg >= plan->n_args) { tad::set_error("no such argument"); return TAD_ERR_INVALID_ARG; }
    if (!check_workspace(plan, workspace, workspace_bytes)) return TAD_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    TadpPointers ptrs{};
    if (!fill_inputs(plan, args, df, workspace, ptrs)) return TAD_ERR_INVALID_ARG;
    Side *side = side_of(plan);
    cudaEvent_t pending = nullptr;
    if (plan->arg_kernels[arg].empty() || plan->arg_zero_fill[arg]) {
        // the fill of a gradient whose first kernel prepares auxiliary tensors runs beside that preparation
        const bool beside = side && !plan->arg_kernels[arg].empty() && !plan->backward[plan->arg_kernels[arg][0]].pre.empty();
        if (beside) {
            if (cudaEventRecord(side->fork, stream) != cudaSuccess || cudaStreamWaitEvent(side->s, side->fork, 0) != cudaSuccess) {
                tad::set_error("event record / wait failed"); return TAD_ERR_CUDA;
            }
        }
        tad_status st = zero_fill(darg, plan->arg_elems[arg], beside ? side->s : stream);
        if (st != TAD_OK) return st;
        if (beside) {
            if (cudaEventRecord(side->filled, side->s) != cudaSuccess) { tad::set_error("event record failed"); return TAD_ERR_CUDA; }
            pending = side->filled;
        }
    }
    ptrs.out = darg;
    for (int ki : plan->arg_kernels[arg]) {
        tad_status st = launch(plan->backward[ki], ptrs, plan->opt.debug_bounds != 0, stream,
                               workspace ? static_cast<char *>(workspace) + aux_offset(plan) : nullptr, side, pending);
        pending = nullptr;
        if (st != TAD_OK) return st;
    }
    return TAD_OK;
}

tad_status tad_backward(const tad_plan *plan, const float *const *args, const float *df,
                        float *const *dargs, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!plan || !df || !dargs || (plan->n_args && !args)) { tad::set_error("NULL argument"); return TAD_ERR_INVALID_ARG; }
    bool need_stage = false;
    for (int a = 0; a < plan->n_args; ++a)
        if (dargs[a])
            for (int ki : plan->arg_kernels[a]) if (!plan->backward[ki].stages_used.empty()) need_stage = true;
    if (need_stage) {
        tad_status st = tad_backward_stage(plan, args, df, workspace, workspace_bytes, cuda_stream);
        if (st != TAD_OK) return st;
    }
    for (int a = 0; a < plan->n_args; ++a) {
        if (!dargs[a]) continue;
        tad_status st = tad_backward_arg(plan, args, df, a, dargs[a], workspace, workspace_bytes, cuda_stream);
        if (st != TAD_OK) return st;
    }
    return TAD_OK;
}

size_t tad_staging_bytes(const tad_plan *plan)
{
    if (!plan) return 0;
    auto pad = [](size_t b) { return (b + 255) & ~size_t(255); };
    size_t total = pad(tad_workspace_bytes(plan));
    for (int a = 0; a < plan->n_args; ++a) total += 2 * pad(size_t(plan->arg_elems[a]) * 4);   // x^p and dx^p
    total += 2 * pad(size_t(plan->out_elems) * 4);                                            // f and df
    return total;
}

tad_status tad_step_host(const tad_plan *plan, const float *const *h_args, const float *h_df,
                         float *h_f, float *const *h_dargs, void *staging, size_t staging_bytes, void *cuda_stream)
{
    if (!plan || !h_args || !h_df || !h_dargs || !staging) { tad::set_error("NULL argument"); return TAD_ERR_INVALID_ARG; }
    if (staging_bytes < tad_staging_bytes(plan) || (reinterpret_cast<uintptr_t>(staging) & 255u)) {
        tad::set_error("staging buffer too small or not 256-byte aligned");
        return TAD_ERR_WORKSPACE;
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    auto pad = [](size_t b) { return (b + 255) & ~size_t(255); };
    char *cur = static_cast<char *>(staging);
    void *ws = cur; cur += pad(tad_workspace_bytes(plan));
    const float *d_args[TADP_MAX_PTRS]; float *d_dargs[TADP_MAX_PTRS];
    auto check = [](cudaError_t e, const char *what) {
        if (e != cudaSuccess) { tad::set_error(std::string(what) + ": " + cudaGetErrorString(e)); return false; }
        return true;
    };
    for (int a = 0; a < plan->n_args; ++a) cur += 2 * pad(size_t(plan->arg_elems[a]) * 4);   // x^p and dx^p, filled below
    const size_t fbytes = size_t(plan->out_elems) * 4;
    float *d_f = reinterpret_cast<float *>(cur); cur += pad(fbytes);
    float *d_df = reinterpret_cast<float *>(cur); cur += pad(fbytes);

    // Copies run on two streams of their own so that they overlap the kernels: df goes up while the
    // forward pass runs, f and every gradient come down while the next kernels run.  The streams and
    // events belong to the plan: made by the first call, reused by every later one.
    if (!plan->host_step) {
        HostStep *hs = new (std::nothrow) HostStep();
        if (!hs) { tad::set_error("out of host memory"); return TAD_ERR_NOMEM; }
        bool ok = cudaStreamCreateWithFlags(&hs->in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&hs->out, cudaStreamNonBlocking) == cudaSuccess;
        for (int i = 0; ok && i < HostStep::N_EVENTS; ++i) ok = cudaEventCreateWithFlags(&hs->ev[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) { hs->release(); delete hs; tad::set_error("creating the copy streams and events failed"); return TAD_ERR_CUDA; }
        plan->host_step = hs;
    }
    struct Side {
        HostStep *hs; int used = 0;
        cudaStream_t in, out;
        cudaEvent_t event() { return used < HostStep::N_EVENTS ? hs->ev[used++] : nullptr; }
    } side{static_cast<HostStep *>(plan->host_step)};
    side.in = side.hs->in; side.out = side.hs->out;
    cudaEvent_t ev_start = side.event(), ev_args = side.event(), ev_df = side.event(), ev_f = side.event();
    if (!ev_start || !ev_args || !ev_df || !ev_f) { tad::set_error("event creation failed"); return TAD_ERR_CUDA; }
    // whatever the caller queued on its stream comes first
    if (!check(cudaEventRecord(ev_start, stream), "event record") || !check(cudaStreamWaitEvent(side.in, ev_start, 0), "stream wait") ||
        !check(cudaStreamWaitEvent(side.out, ev_start, 0), "stream wait")) return TAD_ERR_CUDA;
    cur = static_cast<char *>(staging) + pad(tad_workspace_bytes(plan));
    for (int a = 0; a < plan->n_args; ++a) {
        const size_t bytes = size_t(plan->arg_elems[a]) * 4;
        float *dx = reinterpret_cast<float *>(cur); cur += pad(bytes);
        float *dg = reinterpret_cast<float *>(cur); cur += pad(bytes);
        if (!h_args[a]) { tad::set_error("NULL host argument"); return TAD_ERR_INVALID_ARG; }
        if (!check(cudaMemcpyAsync(dx, h_args[a], bytes, cudaMemcpyHostToDevice, side.in), "copy of an argument")) return TAD_ERR_CUDA;
        d_args[a] = dx; d_dargs[a] = h_dargs[a] ? dg : nullptr;
    }
    if (!check(cudaEventRecord(ev_args, side.in), "event record")) return TAD_ERR_CUDA;
    if (!check(cudaMemcpyAsync(d_df, h_df, fbytes, cudaMemcpyHostToDevice, side.in), "copy of df")) return TAD_ERR_CUDA;
    if (!check(cudaEventRecord(ev_df, side.in), "event record")) return TAD_ERR_CUDA;

    tad_status st = TAD_OK;
    if (!check(cudaStreamWaitEvent(stream, ev_args, 0), "stream wait")) return TAD_ERR_CUDA;
    if (h_f || plan->opt.saved_forward) {
        st = tad_forward(plan, d_args, d_f, ws, tad_workspace_bytes(plan), stream);
        if (st != TAD_OK) return st;
        if (h_f) {
            if (!check(cudaEventRecord(ev_f, stream), "event record") || !check(cudaStreamWaitEvent(side.out, ev_f, 0), "stream wait") ||
                !check(cudaMemcpyAsync(h_f, d_f, fbytes, cudaMemcpyDeviceToHost, side.out), "copy of f")) return TAD_ERR_CUDA;
        }
    }
    if (plan->opt.saved_forward) d_args[plan->n_args] = d_f;      // the backward pass reads f
    if (!check(cudaStreamWaitEvent(stream, ev_df, 0), "stream wait")) return TAD_ERR_CUDA;
    if (plan->opt.debug_bounds && !check(cudaMemsetAsync(ws, 0, 256, stream), "clearing the debug word")) return TAD_ERR_CUDA;
    bool need_stage = false;
    for (int a = 0; a < plan->n_args; ++a)
        if (d_dargs[a])
            for (int ki : plan->arg_kernels[a]) if (!plan->backward[ki].stages_used.empty()) need_stage = true;
    if (need_stage) {
        st = tad_backward_stage(plan, d_args, d_df, ws, tad_workspace_bytes(plan), stream);
        if (st != TAD_OK) return st;
    }
    // largest gradient first: its copy to the host runs while the kernels of the others do
    int order[TADP_MAX_PTRS];
    for (int a = 0; a < plan->n_args; ++a) order[a] = a;
    std::stable_sort(order, order + plan->n_args, [&](int x, int y) { return plan->arg_elems[x] > plan->arg_elems[y]; });
    for (int oi = 0; oi < plan->n_args; ++oi) {
        const int a = order[oi];
        if (!d_dargs[a]) continue;
        st = tad_backward_arg(plan, d_args, d_df, a, d_dargs[a], ws, tad_workspace_bytes(plan), stream);
        if (st != TAD_OK) return st;
        cudaEvent_t ev_g = side.event();
        if (!ev_g) { tad::set_error("event creation failed"); return TAD_ERR_CUDA; }
        if (!check(cudaEventRecord(ev_g, stream), "event record") || !check(cudaStreamWaitEvent(side.out, ev_g, 0), "stream wait") ||
            !check(cudaMemcpyAsync(h_dargs[a], d_dargs[a], size_t(plan->arg_elems[a]) * 4, cudaMemcpyDeviceToHost, side.out), "copy of a gradient"))
            return TAD_ERR_CUDA;
    }
    if (!check(cudaStreamSynchronize(stream), "stream synchronise") || !check(cudaStreamSynchronize(side.out), "stream synchronise") ||
        !check(cudaStreamSynchronize(side.in), "stream synchronise")) return TAD_ERR_CUDA;
    return TAD_OK;
}

tad_status tad_backward_noalloc(const tad_plan *plan, const float *const *args, const float *df,
                                float *const *dargs, void *cuda_stream)
{
    if (!plan) { tad::set_error("NULL plan"); return TAD_ERR_INVALID_ARG; }
    const size_t need = tad_workspace_bytes(plan);
    if (need > TAD_NOALLOC_SCRATCH_BYTES) {
        char msg[160];
        snprintf(msg, sizeof msg, "this plan needs %zu bytes of scratch, tad_backward_noalloc holds at most %zu; "
                                  "use tad_backward with a caller-provided workspace", need, (size_t)TAD_NOALLOC_SCRATCH_BYTES);
        tad::set_error(msg);
        return TAD_ERR_WORKSPACE;
    }
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) {
        tad::set_error(e != cudaSuccess ? std::string("cudaGetDevice: ") + cudaGetErrorString(e) : "device ordinal out of range");
        return TAD_ERR_CUDA;
    }
    void *scratch = nullptr;
    {
        // once per device, with that device current: the array's name is only a host-side handle,
        // the device address has to be asked for
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!g_noalloc_ptr[dev]) {
            void *p = nullptr;
            e = cudaGetSymbolAddress(&p, tad_noalloc_scratch);
            if (e != cudaSuccess || !p) {
                tad::set_error(std::string("cudaGetSymbolAddress: ") + cudaGetErrorString(e));
                return TAD_ERR_CUDA;
            }
            g_noalloc_ptr[dev] = p;
        }
        scratch = g_noalloc_ptr[dev];
    }
    if (plan->opt.debug_bounds) {
        // the array keeps what the last call left: the debug word has to start at zero
        e = cudaMemsetAsync(scratch, 0, 256, (cudaStream_t)cuda_stream);
        if (e != cudaSuccess) { tad::set_error(std::string("clearing the debug word: ") + cudaGetErrorString(e)); return TAD_ERR_CUDA; }
    }
    // (this entry point creates nothing: the second stream is used only if an earlier call of another entry point made it)
    t_create_nothing = true;
    const tad_status st = tad_backward(plan, args, df, dargs, scratch, TAD_NOALLOC_SCRATCH_BYTES, cuda_stream);
    t_create_nothing = false;
    return st;
}

tad_status tad_measure_fp32_rate(void *cuda_stream, double *tflops)
{
    if (!tflops) { tad::set_error("NULL argument"); return TAD_ERR_INVALID_ARG; }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    float *sink = nullptr;
    const unsigned blocks = (unsigned)sm_count() * 8u, threads = 256u;
    const int iters = 4096;
    cudaError_t e = cudaMalloc(&sink, sizeof(float));
    if (e == cudaSuccess) e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    float ms = 0.f;
    if (e == cudaSuccess) {
        tad_fma_rate_kernel<<<blocks, threads, 0, stream>>>(sink, iters, 1.0001f);           // warm-up
        e = cudaEventRecord(e0, stream);
        if (e == cudaSuccess) { tad_fma_rate_kernel<<<blocks, threads, 0, stream>>>(sink, iters, 1.0001f); e = cudaGetLastError(); }
        if (e == cudaSuccess) e = cudaEventRecord(e1, stream);
        if (e == cudaSuccess) e = cudaEventSynchronize(e1);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (sink) cudaFree(sink);
    if (e != cudaSuccess || ms <= 0.f) { tad::set_error(std::string("measuring the multiply-add rate: ") + cudaGetErrorString(e)); return TAD_ERR_CUDA; }
    const double flops = 2.0 * 16.0 * (double)iters * (double)blocks * (double)threads;
    *tflops = flops / (ms * 1e-3) / 1e12;
    return TAD_OK;
}

tad_status tad_debug_status(const tad_plan *plan, void *workspace, void *cuda_stream)
{
    if (!plan) { tad::set_error("NULL plan"); return TAD_ERR_INVALID_ARG; }
    if (!plan->opt.debug_bounds) return TAD_OK;
    if (!workspace) {
        // the scratch of tad_backward_noalloc on the current device, if that entry point has run here
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) { tad::set_error("no current device"); return TAD_ERR_CUDA; }
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        workspace = g_noalloc_ptr[dev];
        if (!workspace) { tad::set_error("NULL workspace (and tad_backward_noalloc has not run on this device)"); return TAD_ERR_INVALID_ARG; }
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    int32_t word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, workspace, sizeof word, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e == cudaSuccess && word != 0) e = cudaMemsetAsync(workspace, 0, sizeof word, stream);
    if (e != cudaSuccess) { tad::set_error(std::string("reading the debug word: ") + cudaGetErrorString(e)); return TAD_ERR_CUDA; }
    if (word != 0) {
        char msg[96];
        snprintf(msg, sizeof msg, "a kernel skipped an out-of-range access (code 0x%x)", word);
        tad::set_error(msg);
        return TAD_ERR_OUT_OF_RANGE;
    }
    return TAD_OK;
}

}  // extern "C"

// A stack of fully-connected block-circulant layers run as one call (the paper evaluates whole networks, e.g.
// the three FC layers of AlexNet, and its hardware keeps activations on chip between layers).
//
// Between two staged layers with the same block size the activation is only ever transformed again, so the
// inverse-transform kernel of layer l and the input-transform kernel of layer l + 1 are replaced by one relay
// kernel (circ_staged.cu): Y operand of l -> inverse transform, bias, activation, forward transform -> X operand
// of l + 1.  A stack of D layers is then 2 D + 1 launches instead of 3 D and the D - 1 intermediate activations
// never reach memory.  Boundaries that cannot be relayed (small batches on the single-launch kernel, different
// block sizes, bfloat16 activations between the layers) fall back to the ordinary per-layer forward through an
// intermediate buffer the stack owns.
#include <new>
#include <vector>

#include "circ_common.cuh"

namespace circ {

struct Stack {
    std::vector<Layer*> layers;   // borrowed: the caller keeps ownership of the layer handles
    void* act[2];                 // ping-pong activation buffers for boundaries that are not relayed
    size_t act_bytes;
    int relayed;                  // boundaries relayed by the last forward
};

static int variant_for(const Layer* L, int batch) {
    if (L->variant != CIRC_VARIANT_AUTO) return L->variant;
    if (fused_fc_preferred(L, batch, tensor_supported(L))) return CIRC_VARIANT_FUSED;
    return tensor_supported(L) ? CIRC_VARIANT_TENSOR : CIRC_VARIANT_STAGED;
}

// the per-layer workspace of the ordinary forward: all problems of X and of Y (the slack covers the alignment gap)
static size_t stack_workspace(const Layer* L, const Extent& e) {
    return ((size_t)2 * e.Bh * padded_q(L->geo.q) * L->geo.k + (size_t)2 * e.Bho * L->geo.p * L->geo.k) * sizeof(float) + 512;
}

static int grow_activations(Stack* S, size_t need) {
    if (need <= S->act_bytes) return CIRC_OK;
    cudaFree(S->act[0]);
    cudaFree(S->act[1]);
    S->act[0] = S->act[1] = nullptr;
    S->act_bytes = 0;
    if (dev_alloc(&S->act[0], need) != cudaSuccess || dev_alloc(&S->act[1], need) != cudaSuccess) {
        cudaGetLastError();
        set_error(CIRC_ERR_ALLOC, "allocation of the intermediate activations (2 x %zu bytes) failed", need);
        return CIRC_ERR_ALLOC;
    }
    S->act_bytes = need;
    return CIRC_OK;
}

static bool staged(int variant) { return variant == CIRC_VARIANT_TENSOR || variant == CIRC_VARIANT_STAGED; }

}  // namespace circ

using namespace circ;

extern "C" {

circ_stack_handle circ_stack_create(const circ_handle* layers, int count) {
    if (!layers || count < 1 || count > 64) {
        set_error(CIRC_ERR_ARG, "layers is NULL or count=%d not in [1, 64]", count);
        return nullptr;
    }
    for (int l = 0; l < count; ++l) {
        const Layer* L = reinterpret_cast<const Layer*>(layers[l]);
        if (!L || L->kind != 0) {
            set_error(CIRC_ERR_ARG, "layer %d is NULL or not a fully-connected handle", l);
            return nullptr;
        }
        if (l > 0) {
            const Layer* P = reinterpret_cast<const Layer*>(layers[l - 1]);
            if (P->m != L->n || P->device != L->device) {
                set_error(CIRC_ERR_SHAPE, "layer %d takes %d inputs but layer %d produces %d (or they live on different devices)", l,
                          L->n, l - 1, P->m);
                return nullptr;
            }
        }
    }
    // stacked layers hand their operands to one another in the embedded layout: keep every layer on it
    for (int l = 0; l < count; ++l) reinterpret_cast<Layer*>(layers[l])->no_twin = 1;   // (its kernels are called directly here)
    Stack* S = new (std::nothrow) Stack();
    if (!S) {
        set_error(CIRC_ERR_ALLOC, "host allocation failed");
        return nullptr;
    }
    for (int l = 0; l < count; ++l) S->layers.push_back(reinterpret_cast<Layer*>(layers[l]));
    S->act[0] = S->act[1] = nullptr;
    S->act_bytes = 0;
    S->relayed = 0;
    return reinterpret_cast<circ_stack_handle>(S);
}

void circ_stack_destroy(circ_stack_handle s) {
    Stack* S = reinterpret_cast<Stack*>(s);
    if (!S) return;
    cudaFree(S->act[0]);
    cudaFree(S->act[1]);
    delete S;
}

int circ_stack_reserve(circ_stack_handle s, long max_batch) {
    Stack* S = reinterpret_cast<Stack*>(s);
    if (!S || max_batch < 1 || max_batch > (1L << 30)) {
        set_error(CIRC_ERR_ARG, "bad stack handle or max_batch %ld", max_batch);
        return CIRC_ERR_ARG;
    }
    size_t act = 0;
    for (Layer* L : S->layers) {
        int rc = circ_reserve(reinterpret_cast<circ_handle>(L), max_batch);
        if (rc != CIRC_OK) return rc;
        const size_t bytes = (size_t)max_batch * L->m * 4;
        if (bytes > act) act = bytes;
    }
    return S->layers.size() > 1 ? grow_activations(S, act) : CIRC_OK;
}

int circ_stack_relayed(circ_stack_handle s) {
    const Stack* S = reinterpret_cast<const Stack*>(s);
    return S ? S->relayed : 0;
}

int circ_stack_forward(circ_stack_handle s, const void* x, void* y, int batch, void* stream) {
    Stack* S = reinterpret_cast<Stack*>(s);
    if (!S || !x || !y || x == y || (reinterpret_cast<uintptr_t>(x) & 15u) || (reinterpret_cast<uintptr_t>(y) & 15u)) {
        set_error(CIRC_ERR_ARG, "bad stack handle, or x / y NULL, equal or not 16-byte aligned");
        return CIRC_ERR_ARG;
    }
    if (batch < 1) {
        set_error(CIRC_ERR_SHAPE, "batch=%d must be >= 1", batch);
        return CIRC_ERR_SHAPE;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int D = (int)S->layers.size();
    Extent e;
    e.B = e.Bo = batch;
    e.Bh = e.Bho = (batch + 1) / 2;
    e.H = e.Ho = 1;
    e.W = e.Wo = batch;
    e.Nh = e.Bh;

    // which boundaries are relayed: both sides staged, same block size, float32 activations between them
    std::vector<int> variant(D);
    std::vector<char> relay(D, 0);   // relay[l]: boundary between l and l + 1
    size_t act_need = 0;
    for (int l = 0; l < D; ++l) {
        Layer* L = S->layers[l];
        variant[l] = variant_for(L, batch);
        if (variant[l] == CIRC_VARIANT_FUSED && !fused_fc_supported(L, batch)) {
            set_error(CIRC_ERR_UNSUPPORTED, "layer %d: the fused kernel does not serve batch=%d", l, batch);
            return CIRC_ERR_UNSUPPORTED;
        }
        if (variant[l] == CIRC_VARIANT_TENSOR && !tensor_supported(L)) {
            set_error(CIRC_ERR_UNSUPPORTED, "layer %d: the tensor-core contraction needs q %% 4 == 0", l);
            return CIRC_ERR_UNSUPPORTED;
        }
    }
    for (int l = 0; l + 1 < D; ++l) {
        const Layer* A = S->layers[l];
        const Layer* Bn = S->layers[l + 1];
        relay[l] = staged(variant[l]) && staged(variant[l + 1]) && A->geo.k == Bn->geo.k && !embedded(A->geo) && !embedded(Bn->geo) && A->y_dtype == CIRC_F32 &&
                   Bn->x_dtype == CIRC_F32;
        if (!relay[l]) {
            const size_t bytes = (size_t)batch * A->m * (A->y_dtype == CIRC_BF16 ? 2 : 4);
            if (bytes > act_need) act_need = bytes;
            if (A->y_dtype != Bn->x_dtype) {
                set_error(CIRC_ERR_ARG, "layer %d writes a different element type than layer %d reads", l, l + 1);
                return CIRC_ERR_ARG;
            }
        }
    }
    int rc;
    if ((rc = grow_activations(S, act_need)) != CIRC_OK) return rc;

    int relayed = 0, pong = 0;
    const void* in = x;          // activation entering layer l, when it is not handed over as an operand
    bool operand_ready = false;  // layer l's X operand was written by the relay of the boundary before it
    for (int l = 0; l < D; ++l) {
        Layer* L = S->layers[l];
        const bool last = l + 1 == D;
        if (!staged(variant[l])) {   // single-launch kernel: plain forward into the next buffer (never relayed)
            void* out = last ? y : S->act[pong];
            if ((rc = launch_fused_fc(L, in, out, batch, st)) != CIRC_OK) return rc;
            L->last_variant = CIRC_VARIANT_FUSED;
            in = out;
            pong ^= 1;
            continue;
        }
        const bool tensor = variant[l] == CIRC_VARIANT_TENSOR;
        if ((rc = ensure_workspace(L, stack_workspace(L, e))) != CIRC_OK) return rc;
        if ((rc = ensure_forms(L, tensor ? FORM_A_BF16 : FORM_A_F32, st)) != CIRC_OK) return rc;   // stacks use the embedded weights
        float* xop = static_cast<float*>(L->ws);
        float* yop = xop + (((size_t)2 * e.Bh * padded_q(L->geo.q) * L->geo.k + 63) & ~(size_t)63);   // (bfloat16 runs may be padded)
        if (!operand_ready) {
            const int xmode = !tensor ? 0 : (L->x_dtype == CIRC_BF16 ? 2 : 1);
            if ((rc = launch_input_fft(L, in, xop, xmode, e, st)) != CIRC_OK) return rc;
        }
        if (tensor)
            rc = launch_contract_tc(L, reinterpret_cast<const __nv_bfloat16*>(xop), yop, e, L->x_dtype == CIRC_BF16 ? 1 : 2, st);
        else
            rc = launch_contract_fma(L, xop, yop, e, st);
        if (rc != CIRC_OK) return rc;
        L->last_variant = variant[l];
        if (!last && relay[l]) {
            Layer* Nx = S->layers[l + 1];
            if ((rc = ensure_workspace(Nx, stack_workspace(Nx, e))) != CIRC_OK) return rc;
            const int xmode_next = variant[l + 1] == CIRC_VARIANT_TENSOR ? 1 : 0;
            if ((rc = launch_relay(L, yop, Nx->ws, xmode_next, e, st)) != CIRC_OK) return rc;
            operand_ready = true;
            ++relayed;
        } else {
            void* out = last ? y : S->act[pong];
            if ((rc = launch_output_ifft(L, yop, out, e, st)) != CIRC_OK) return rc;
            in = out;
            pong ^= 1;
            operand_ready = false;
        }
    }
    S->relayed = relayed;
    return CIRC_OK;
}

}  // extern "C"

// Prompt classifier, MLP variant (embedding, two fully connected layers, softmax -> argmax):
// routes each prompt to one of the heterogeneous draft models.  One block per sequence.
#include "kernels.h"

namespace sd {

template <typename T>
__global__ void __launch_bounds__(256) k_classifier(SeqState S, SeqList list, SeqList forced, const T* __restrict__ embed, int d, int vocab,
                                                    const float* __restrict__ w1, const float* __restrict__ b1, int dh,
                                                    const float* __restrict__ w2, const float* __restrict__ b2, int nc) {
    extern __shared__ float sm[];
    float* e = sm;             // [d] mean-pooled prompt embedding
    float* z = sm + d;         // [dh] hidden activations
    float* o = z + dh;         // [nc] class scores
    const int i = blockIdx.x, slot = list.ids[i];
    if (forced.ids[i] >= 0) {  // task type given with the request: no classification
        if (threadIdx.x == 0) S.draft_id[slot] = min(forced.ids[i], nc - 1);
        return;
    }
    const int n = S.n_prompt[slot];
    const int32_t* toks = S.tokens + (size_t)slot * S.tok_stride;
    for (int k = threadIdx.x; k < d; k += blockDim.x) {
        float acc = 0.f;
        for (int t = 0; t < n; ++t) {
            int tok = toks[t];
            tok = (tok < 0 || tok >= vocab) ? 0 : tok;
            acc += to_f32<T>(embed[(size_t)tok * d + k]);
        }
        e[k] = acc / (float)n;
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    for (int j = warp; j < dh; j += nw) {
        float acc = 0.f;
        for (int k = lane; k < d; k += 32) acc = fmaf(w1[(size_t)j * d + k], e[k], acc);
        acc = warp_sum(acc);
        if (lane == 0) z[j] = fmaxf(acc + b1[j], 0.f);
    }
    __syncthreads();
    for (int c = warp; c < nc; c += nw) {
        float acc = 0.f;
        for (int j = lane; j < dh; j += 32) acc = fmaf(w2[(size_t)c * dh + j], z[j], acc);
        acc = warp_sum(acc);
        if (lane == 0) o[c] = acc + b2[c];
    }
    __syncthreads();
    if (threadIdx.x == 0) {    // softmax is monotone: its argmax is the argmax of the scores
        int best = 0;
        for (int c = 1; c < nc; ++c) if (o[c] > o[best]) best = c;
        S.draft_id[slot] = best;
    }
}

cudaError_t launch_classifier(const SeqState& S, const SeqList& list, const SeqList& forced,
                              const void* embed, int dtype, int d, int vocab,
                              const float* w1, const float* b1, int d_hidden, const float* w2, const float* b2,
                              int n_classes, cudaStream_t st) {
    if (list.n <= 0) return cudaSuccess;
    size_t smem = sizeof(float) * (size_t)(d + d_hidden + n_classes);
    if (dtype == SD_BF16) k_classifier<bf16><<<list.n, 256, smem, st>>>(S, list, forced, (const bf16*)embed, d, vocab, w1, b1, d_hidden, w2, b2, n_classes);
    else k_classifier<float><<<list.n, 256, smem, st>>>(S, list, forced, (const float*)embed, d, vocab, w1, b1, d_hidden, w2, b2, n_classes);
    return cudaGetLastError();
}

}  // namespace sd

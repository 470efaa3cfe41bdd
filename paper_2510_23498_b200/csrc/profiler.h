// Measurement hook: CUDA-event brackets around contraction launches, summed per class after a synchronise.
#pragma once
#include <cuda_runtime.h>

#include <vector>

namespace mpode {

struct Profiler {
    static constexpr int kClasses = 4;   // 0 forward layers, 1 input-gradient layers, 2 weight-gradient layers,
                                         // 3 fused backward launches (input- and weight-gradient phases together)
    bool enabled = false;
    struct Rec { cudaEvent_t a, b; int klass; double flops; };
    std::vector<Rec> recs;
    std::vector<cudaEvent_t> pool;
    cudaEvent_t get() {
        if (!pool.empty()) { cudaEvent_t e = pool.back(); pool.pop_back(); return e; }
        cudaEvent_t e;
        cudaEventCreate(&e);
        return e;
    }
    void begin(int klass, double flops, cudaStream_t st) {
        Rec r{get(), get(), klass, flops};
        cudaEventRecord(r.a, st);
        recs.push_back(r);
    }
    void end(cudaStream_t st) { cudaEventRecord(recs.back().b, st); }
    // sums and clears the records; the stream must be idle
    void collect(double* ms, long long* launches, double* flops) {
        for (int k = 0; k < kClasses; ++k) { ms[k] = 0; launches[k] = 0; flops[k] = 0; }
        for (auto& r : recs) {
            float t = 0.f;
            if (cudaEventElapsedTime(&t, r.a, r.b) == cudaSuccess) ms[r.klass] += t;
            launches[r.klass] += 1;
            flops[r.klass] += r.flops;
            pool.push_back(r.a);
            pool.push_back(r.b);
        }
        recs.clear();
    }
    ~Profiler() {
        for (auto& r : recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
        for (auto e : pool) cudaEventDestroy(e);
    }
};

extern thread_local Profiler* tl_profiler;

// Which kernels the contractions of the last forward / backward pair went to.
struct PathCounters {
    long long tc = 0;      // layer-by-layer contractions on the tensor-core kernels
    long long simt = 0;    // layer-by-layer contractions on the CUDA-core kernel
    long long fused = 0;   // launches of the fused Runge-Kutta kernel
    long long whole = 0;   // launches of the whole-solve kernels for very small networks
};
extern thread_local PathCounters* tl_counters;

}  // namespace mpode

// Optional event profiler: one cudaEvent pair around every launch site, summed per stage.
#include <new>
#include <vector>

#include "dc_common.cuh"

struct dc_prof {
    bool on = false;
    std::vector<cudaEvent_t> pool;          // recycled events
    struct Pair { cudaEvent_t a, b; int stage; };
    std::vector<Pair> pairs;                // recorded since the last read-out
    cudaEvent_t open_start = nullptr;
    cudaEvent_t get()
    {
        if (!pool.empty()) { cudaEvent_t e = pool.back(); pool.pop_back(); return e; }
        cudaEvent_t e = nullptr;
        if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        return e;
    }
};

dc_prof_scope::dc_prof_scope(dc_cache* cache, int st) : c(cache), stage(st)
{
    dc_prof* p = c->prof;
    if (!p || !p->on) return;
    p->open_start = p->get();
    if (p->open_start) cudaEventRecord(p->open_start, c->stream);
}

// The event lists grow with push_back; a failed allocation must not leave through the C ABI: the pair is
// dropped (its events destroyed) and that launch goes untimed.
static bool keep_event(std::vector<cudaEvent_t>& v, cudaEvent_t e)
{
    try { v.push_back(e); return true; } catch (...) { cudaEventDestroy(e); return false; }
}

dc_prof_scope::~dc_prof_scope()
{
    dc_prof* p = c->prof;
    if (!p || !p->on || !p->open_start) return;
    cudaEvent_t b = p->get();
    if (!b) { keep_event(p->pool, p->open_start); p->open_start = nullptr; return; }
    cudaEventRecord(b, c->stream);
    try { p->pairs.push_back({p->open_start, b, stage}); }
    catch (...) { cudaEventDestroy(p->open_start); cudaEventDestroy(b); }
    p->open_start = nullptr;
}

void dc_prof_release(dc_cache* c)
{
    if (!c->prof) return;
    for (auto& pr : c->prof->pairs) { cudaEventDestroy(pr.a); cudaEventDestroy(pr.b); }
    for (auto e : c->prof->pool) cudaEventDestroy(e);
    delete c->prof;
    c->prof = nullptr;
}

extern "C" int dc_cache_set_profiling(dc_cache* c, int enable)
{
    if (!c) return DC_ERR_ARG;
    if (!c->prof) c->prof = new (std::nothrow) dc_prof();
    if (!c->prof) return DC_ERR_ALLOC;
    c->prof->on = enable != 0;
    return DC_OK;
}

extern "C" int dc_cache_profile(dc_cache* c, float* ms_host, int64_t* launches_host)
{
    if (!c || !ms_host) return DC_ERR_ARG;
    for (int i = 0; i < DC_PROFILE_STAGES; ++i) { ms_host[i] = 0.f; if (launches_host) launches_host[i] = 0; }
    if (!c->prof) return DC_OK;
    DC_CUDA(cudaStreamSynchronize(c->stream));
    for (auto& pr : c->prof->pairs) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, pr.a, pr.b) == cudaSuccess) {
            ms_host[pr.stage] += ms;
            if (launches_host) launches_host[pr.stage] += 1;
        }
        keep_event(c->prof->pool, pr.a); keep_event(c->prof->pool, pr.b);
    }
    cudaGetLastError();
    c->prof->pairs.clear();
    return DC_OK;
}

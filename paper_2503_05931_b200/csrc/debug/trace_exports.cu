// Debug build only (-DAED_TRACE): the whole library plus one entry point that copies out the device-side timeline
// (ids with the low bits of the cycle counter, and %globaltimer stamps where taken) and clears it.  The product library is built from aed_dec.cu alone and has neither.
#ifndef AED_TRACE
#error "trace_exports.cu is for -DAED_TRACE builds"
#endif
#include "../aed_dec.cu"

extern "C" int32_t aed_dec_trace_read(aed_dec_t *dec, int32_t max_events, uint32_t *ids, unsigned long long *t_ns)
{
    if (!dec) return AED_ERR_INVALID_ARG;
    if (cudaStreamSynchronize(dec->stream) != cudaSuccess) return AED_ERR_CUDA;
    static TraceBuf host;
    char *src = dec->ws + dec->lay.state + 256;
    if (cudaMemcpy(&host, src, sizeof host, cudaMemcpyDeviceToHost) != cudaSuccess) return AED_ERR_CUDA;
    cudaMemset(src, 0, 8);
    int n = host.count < (1u << 16) ? (int)host.count : (1 << 16);
    if (n > max_events) n = max_events;
    for (int i = 0; i < n; ++i) {
        ids[i] = (host.ev[i].id & 0xffu) | (host.ev[i].pad << 8);      // id | low 24 bits of the SM's cycle counter
        t_ns[i] = host.ev[i].t_ns;
    }
    return n;
}

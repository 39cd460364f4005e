// Stand-alone probe (not part of the library): how fast can 1, 8, 32 or all SMs pull bytes from HBM,
// with bulk async copies through a ring of NS stages of SB bytes, and with plain 16-byte loads?
// Built and run by `python -m paper_2203_16487_b200.diagnostics --ingest-probe`.
#include <cuda_runtime.h>
#include <cstdio>
#include <cstdint>
#include <cstdlib>
__device__ __forceinline__ uint32_t s32(const void* p){return (uint32_t)__cvta_generic_to_shared(p);}
__device__ __forceinline__ void mbar_init(uint32_t b, uint32_t c){asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;"::"r"(b),"r"(c):"memory");}
__device__ __forceinline__ void expect(uint32_t b, uint32_t n){asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"::"r"(b),"r"(n):"memory");}
__device__ __forceinline__ uint32_t tryw(uint32_t b, uint32_t p){uint32_t ok;asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0,1,0,p;\n}":"=r"(ok):"r"(b),"r"(p):"memory");return ok;}
__device__ __forceinline__ void bulk(uint32_t d, const void* s, uint32_t n, uint32_t b){asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"::"r"(d),"l"(s),"r"(n),"r"(b):"memory");}
template<int NS>
__global__ void k_bulk(const unsigned char* src, size_t per_cta, int SB, int* sink){
  extern __shared__ __align__(128) unsigned char sm[];
  __shared__ __align__(8) uint64_t full[NS];
  const unsigned char* p = src + (size_t)blockIdx.x*per_cta;
  int nst = per_cta / SB;
  if(threadIdx.x==0){ for(int i=0;i<NS;i++) mbar_init(s32(&full[i]),1); asm volatile("fence.mbarrier_init.release.cluster;":::"memory"); }
  __syncthreads();
  if(threadIdx.x==0){
    for(int i=0;i<NS && i<nst;i++){ expect(s32(&full[i]),SB); bulk(s32(sm)+i*SB, p+(size_t)i*SB, SB, s32(&full[i])); }
    int acc=0;
    for(int i=0;i<nst;i++){
      int s=i%NS; long long t0=clock64();
      while(!tryw(s32(&full[s]),(i/NS)&1)){ if(clock64()-t0>2000000000LL) break; }
      acc += sm[s*SB];
      int n=i+NS; if(n<nst){ expect(s32(&full[s]),SB); bulk(s32(sm)+s*SB, p+(size_t)n*SB, SB, s32(&full[s])); }
    }
    if(acc==12345) *sink=acc;
  }
}
__global__ void k_ldg(const uint4* src, size_t per_cta_u4, int* sink){
  const uint4* p = src + (size_t)blockIdx.x*per_cta_u4;
  uint32_t acc=0;
  for(size_t i=threadIdx.x;i<per_cta_u4;i+=blockDim.x*8){
    uint4 v[8];
    #pragma unroll
    for(int u=0;u<8;u++){ size_t j=i+(size_t)u*blockDim.x; v[u]= j<per_cta_u4? __ldcg(p+j): make_uint4(0,0,0,0);}
    #pragma unroll
    for(int u=0;u<8;u++) acc+=v[u].x^v[u].w;
  }
  if(acc==12345) *sink=acc;
}
int main(int argc,char**argv){
  size_t total=(size_t)1<<30; unsigned char* buf; cudaMalloc(&buf,total); cudaMemset(buf,1,total); int* sink; cudaMalloc(&sink,4);
  cudaEvent_t e0,e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
  int ctas[]={1,8,32,148};
  for(int SB: {16384,32768}) for(int NS: {4,6}) for(int c: ctas){
    size_t per=(size_t)8<<20; if (per*c>total) per=total/c; per = per/SB*SB;
    size_t smem=(size_t)NS*SB; float ms;
    if(NS==4){ cudaFuncSetAttribute(k_bulk<4>,cudaFuncAttributeMaxDynamicSharedMemorySize,(int)smem); k_bulk<4><<<c,32,smem>>>(buf,per,SB,sink); cudaDeviceSynchronize(); cudaEventRecord(e0); k_bulk<4><<<c,32,smem>>>(buf,per,SB,sink); cudaEventRecord(e1);} 
    else { cudaFuncSetAttribute(k_bulk<6>,cudaFuncAttributeMaxDynamicSharedMemorySize,(int)smem); k_bulk<6><<<c,32,smem>>>(buf,per,SB,sink); cudaDeviceSynchronize(); cudaEventRecord(e0); k_bulk<6><<<c,32,smem>>>(buf,per,SB,sink); cudaEventRecord(e1);} 
    cudaEventSynchronize(e1); cudaEventElapsedTime(&ms,e0,e1);
    printf("bulk SB=%d NS=%d ctas=%d: %.1f GB/s per CTA, %.1f GB/s total (%s)\n",SB,NS,c,per/ms/1e6,per*c/ms/1e6,cudaGetErrorString(cudaGetLastError()));
  }
  for(int c: ctas) for(int th: {256,1024}){
    size_t per=(size_t)8<<20; if (per*c>total) per=total/c/4096*4096; float ms;   // stay inside the buffer
    k_ldg<<<c,th>>>((const uint4*)buf,per/16,sink); cudaDeviceSynchronize(); cudaEventRecord(e0); k_ldg<<<c,th>>>((const uint4*)buf,per/16,sink); cudaEventRecord(e1); cudaEventSynchronize(e1); cudaEventElapsedTime(&ms,e0,e1);
    printf("ldg threads=%d ctas=%d: %.1f GB/s per CTA, %.1f GB/s total\n",th,c,per/ms/1e6,per*c/ms/1e6);
  }
  // One-shot short stream: every SM pulls 224 KB once (33 MB in all, the size of the vocabulary matrix), after the
  // L2 was filled with (a) clean lines by a read sweep, (b) dirty lines by a write sweep.  "empty" is the
  // event-to-event time of a kernel that does nothing.
  {
    unsigned char* big; cudaMalloc(&big,(size_t)512<<20); cudaMemset(big,2,(size_t)512<<20);
    const int SB=32768; const size_t per=(size_t)7*SB; size_t smem=(size_t)7*SB; float ms;
    cudaFuncSetAttribute(k_bulk<7>,cudaFuncAttributeMaxDynamicSharedMemorySize,(int)smem);
    for(int mode=0; mode<3; mode++) for(int rep=0; rep<3; rep++){
      if(mode==0) k_ldg<<<592,1024>>>((const uint4*)big,((size_t)512<<20)/16/592,sink);
      if(mode==1) cudaMemsetAsync(big,rep,(size_t)512<<20);
      cudaDeviceSynchronize();
      cudaEventRecord(e0);
      if(mode==2) k_bulk<7><<<148,32,smem>>>(buf,0,SB,sink); else k_bulk<7><<<148,32,smem>>>(buf,per,SB,sink);
      cudaEventRecord(e1); cudaEventSynchronize(e1); cudaEventElapsedTime(&ms,e0,e1);
      printf("one-shot 148 x 224 KB after %s: %.2f us  (%.0f GB/s incl. launch)  (%s)\n", mode==0?"clean read sweep":mode==1?"dirty write sweep":"nothing (empty kernel)", ms*1e3, mode==2?0.0:per*148/ms/1e6, cudaGetErrorString(cudaGetLastError()));
    }
  }
  return 0;
}

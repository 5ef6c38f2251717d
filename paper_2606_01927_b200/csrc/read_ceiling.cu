// Measurement tool (not part of the library): how fast can a kernel that does nothing but read
// the metric workload's logits (256 rows x 152064 bf16 = 78 MB, rotating over 8 buffers so L2
// never helps) go on this GPU, in the row-per-CTA shape the sampler uses and as a flat
// grid-stride read?  The answer bounds what the sampler's roofline fraction can reach at this
// size, where launch ramp and tail are a few microseconds of a ~12 microsecond transfer.
// Build: nvcc -O3 -gencode arch=compute_100a,code=sm_100a -o read_ceiling read_ceiling.cu
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#define CK(x) do{cudaError_t e=(x); if(e!=cudaSuccess){printf("err %s line %d\n",cudaGetErrorString(e),__LINE__); return 1;}}while(0)

template<int NT,int U>
__global__ void __launch_bounds__(NT) k_ldg(const uint4* __restrict__ p, int nvec_row, int rows_per_cta_split, unsigned* out){
  // CTA handles row = blockIdx.x / split, segment = blockIdx.x % split
  int split = rows_per_cta_split;
  int row = blockIdx.x / split, seg = blockIdx.x % split;
  int nv = nvec_row / split;
  const uint4* rp = p + (size_t)row*nvec_row + (size_t)seg*nv;
  unsigned acc=0;
  int ntiles = (nv + NT*U-1)/(NT*U);
  uint4 cur[U], nxt[U];
  #pragma unroll
  for(int u=0;u<U;u++){int v=u*NT+threadIdx.x; cur[u]= v<nv? __ldg(rp+v): make_uint4(0,0,0,0);}
  for(int t=0;t<ntiles;t++){
    if(t+1<ntiles){
      #pragma unroll
      for(int u=0;u<U;u++){int v=(t+1)*NT*U+u*NT+threadIdx.x; nxt[u]= v<nv? __ldg(rp+v): make_uint4(0,0,0,0);}
    }
    #pragma unroll
    for(int u=0;u<U;u++){ acc = max(acc, max(max(cur[u].x,cur[u].y),max(cur[u].z,cur[u].w))); }
    #pragma unroll
    for(int u=0;u<U;u++) cur[u]=nxt[u];
  }
  if(acc==0x12345678u) out[0]=acc;
}
// simple grid-stride, no row structure
__global__ void k_flat(const uint4* __restrict__ p, size_t n, unsigned* out){
  unsigned acc=0;
  size_t stride=(size_t)gridDim.x*blockDim.x;
  for(size_t i=(size_t)blockIdx.x*blockDim.x+threadIdx.x;i<n;i+=stride*4){
    uint4 a=__ldg(p+i); uint4 b= i+stride<n? __ldg(p+i+stride):a; uint4 c= i+2*stride<n? __ldg(p+i+2*stride):a; uint4 d= i+3*stride<n? __ldg(p+i+3*stride):a;
    acc=max(acc,max(max(a.x,b.y),max(c.z,d.w)));
  }
  if(acc==0x12345678u) out[0]=acc;
}
int main(){
  const int B=256, V=152064; const int nvec_row=V/8; size_t bytes=(size_t)B*V*2;
  const int NB=8; void* bufs[NB]; for(int i=0;i<NB;i++){CK(cudaMalloc(&bufs[i],bytes)); CK(cudaMemset(bufs[i],i+1,bytes));}
  unsigned* out; CK(cudaMalloc(&out,4));
  cudaEvent_t e0,e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
  auto timeit=[&](auto launch,const char* name){
    for(int i=0;i<5;i++) launch(i%NB);
    cudaDeviceSynchronize();
    cudaEventRecord(e0); int K=100; for(int i=0;i<K;i++) launch(i%NB); cudaEventRecord(e1); cudaEventSynchronize(e1);
    float ms; cudaEventElapsedTime(&ms,e0,e1); double us=ms*1e3/K; printf("%-40s %8.2f us  %7.1f GB/s\n",name,us,bytes/us/1e3);
  };
  timeit([&](int i){k_ldg<512,4><<<256,512>>>((const uint4*)bufs[i],nvec_row,1,out);},"ldg NT512 U4 256 CTAs (row/CTA)");
  timeit([&](int i){k_ldg<512,2><<<256,512>>>((const uint4*)bufs[i],nvec_row,1,out);},"ldg NT512 U2 256 CTAs");
  timeit([&](int i){k_ldg<512,4><<<512,512>>>((const uint4*)bufs[i],nvec_row,2,out);},"ldg NT512 U4 512 CTAs (half row)");
  timeit([&](int i){k_ldg<512,4><<<1024,512>>>((const uint4*)bufs[i],nvec_row,4,out);},"ldg NT512 U4 1024 CTAs (quarter row)");
  timeit([&](int i){k_ldg<256,4><<<1024,256>>>((const uint4*)bufs[i],nvec_row,4,out);},"ldg NT256 U4 1024 CTAs (quarter row)");
  timeit([&](int i){k_ldg<1024,2><<<256,1024>>>((const uint4*)bufs[i],nvec_row,1,out);},"ldg NT1024 U2 256 CTAs");
  timeit([&](int i){k_ldg<256,8><<<256,256>>>((const uint4*)bufs[i],nvec_row,1,out);},"ldg NT256 U8 256 CTAs");
  timeit([&](int i){k_flat<<<148*4,512>>>((const uint4*)bufs[i],bytes/16,out);},"flat grid-stride 592x512");
  timeit([&](int i){k_flat<<<148*8,256>>>((const uint4*)bufs[i],bytes/16,out);},"flat grid-stride 1184x256");
  timeit([&](int i){k_flat<<<148*2,1024>>>((const uint4*)bufs[i],bytes/16,out);},"flat grid-stride 296x1024");
  timeit([&](int i){cudaMemcpyAsync(bufs[(i+1)%NB],bufs[i],bytes,cudaMemcpyDeviceToDevice);},"cudaMemcpy D2D (bytes counted once)");
  return 0;
}

import sys, torch
sys.path.insert(0,'.')
from paper_2401_11504_b200 import binding as b
dev="cuda"
T=4096
g=[torch.randn(T,11008,device=dev,dtype=torch.bfloat16) for _ in range(2)]
u=[torch.randn(T,11008,device=dev,dtype=torch.bfloat16) for _ in range(2)]
dh=[torch.randn(T,11008,device=dev,dtype=torch.bfloat16) for _ in range(2)]
o0=torch.empty_like(g[0]); o1=torch.empty_like(g[0])
x=[torch.randn(4*T,4096,device=dev,dtype=torch.bfloat16) for _ in range(2)]
dy=[torch.randn(4*T,4096,device=dev,dtype=torch.bfloat16) for _ in range(2)]
y=torch.empty_like(x[0]); w=torch.rand(4096,device=dev,dtype=torch.bfloat16)
for i in range(2):
    b.templora_swiglu_fwd(g[i],u[i],o0); b.templora_swiglu_bwd(g[i],u[i],dh[i],o0,o1)
    b.templora_rmsnorm_fwd(x[i],w,1e-5,y); b.templora_rmsnorm_bwd(x[i],w,dy[i],1e-5,y)
torch.cuda.synchronize()
print("ok")

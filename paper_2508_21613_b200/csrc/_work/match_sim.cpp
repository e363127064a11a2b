// host emulation of warp_match<NC> with bounds checks (lanes simulated in lock-step)
#include <cstdio>
#include <cstdlib>
#include <cstdint>
#include <climits>
#include <vector>
#include <algorithm>
#include <cassert>
using namespace std;
const int MAXM=256;
struct Work{ long long u[MAXM]; short match[MAXM], prev[MAXM]; int row_col[MAXM]; uint8_t olo[MAXM],ohi[MAXM],nlo[MAXM],nhi[MAXM];};
long long PW[129];
static long long rc(long long need,int a,int b,int x,int y){int lo=max(a,x),hi=min(b,y); assert(hi<=128&&lo>=0); return need-(hi>lo?PW[hi]-PW[lo]:0);}
#define CHK(i,n) do{ if((i)<0||(i)>=(n)){printf("OOB %s=%d n=%d line %d\n",#i,(int)(i),(int)(n),__LINE__); exit(1);} }while(0)
long long sim(Work&w,int n,int NC){
  const long long INF=LLONG_MAX/4;
  vector<vector<long long>> v(32,vector<long long>(NC)),slack=v,need=v; vector<vector<int>> nlo(32,vector<int>(NC)),nhi=nlo;
  for(int lane=0;lane<32;lane++)for(int c=0;c<NC;c++){int j=c*32+lane; nlo[lane][c]=j<n?w.nlo[j]:0; nhi[lane][c]=j<n?w.nhi[j]:0; need[lane][c]=nhi[lane][c]>nlo[lane][c]?PW[nhi[lane][c]]-PW[nlo[lane][c]]:0; v[lane][c]=INF; if(j<n){w.u[j]=0;w.match[j]=-1;w.row_col[j]=-1;}}
  for(int lane=0;lane<32;lane++)for(int i=0;i<n;i++)for(int c=0;c<NC;c++){long long cost=rc(need[lane][c],w.olo[i],w.ohi[i],nlo[lane][c],nhi[lane][c]); v[lane][c]=min(v[lane][c],cost);}
  for(int lane=0;lane<32;lane++)for(int c=0;c<NC;c++){int j=c*32+lane; if(j>=n)continue; for(int i=0;i<n;i++){ if(rc(need[lane][c],w.olo[i],w.ohi[i],nlo[lane][c],nhi[lane][c])!=v[lane][c])continue; if(w.row_col[i]==-1){w.row_col[i]=j;w.match[j]=i;break;}}}
  int matched0=0; for(int i=0;i<n;i++) matched0+=w.row_col[i]>=0;
  for(int r=0;r<n;r++){
    if(w.row_col[r]>=0)continue;
    for(int lane=0;lane<32;lane++)for(int c=0;c<NC;c++){slack[lane][c]=INF; if(c*32+lane<n)w.prev[c*32+lane]=n;}
    vector<uint32_t> tree(32,0); int col=n,row=r; bool done=false;
    for(int step=0;step<=n;step++){
      CHK(row,n);
      int a=w.olo[row],b=w.ohi[row]; long long ur=w.u[row];
      long long delta=INF; int next=n;
      for(int lane=0;lane<32;lane++){ long long d=INF;int nx=n; for(int c=0;c<NC;c++){int j=c*32+lane; if(j>=n||((tree[lane]>>c)&1))continue; long long red=rc(need[lane][c],a,b,nlo[lane][c],nhi[lane][c])-ur-v[lane][c]; if(red<0){printf("negative reduced cost %lld\n",red);exit(1);} if(red<slack[lane][c]){slack[lane][c]=red;w.prev[j]=col;} if(slack[lane][c]<d){d=slack[lane][c];nx=j;}} if(d<delta||(d==delta&&nx<next)){delta=d;next=nx;} }
      if(next>=n){printf("broken\n");return -1;}
      for(int lane=0;lane<32;lane++)for(int c=0;c<NC;c++){int j=c*32+lane;if(j>=n)continue; if((tree[lane]>>c)&1){CHK(w.match[j],n); w.u[w.match[j]]+=delta; v[lane][c]-=delta;} else slack[lane][c]-=delta;}
      w.u[r]+=delta;
      col=next; tree[col&31]|=1u<<(col>>5); row=w.match[col]; if(row<0){done=true;break;}
    }
    if(!done){printf("step bound\n");return -1;}
    int c=col; for(int step=0;step<=n&&c!=n;step++){CHK(c,n); int p=w.prev[c]; if(p!=n)CHK(p,n); w.match[c]=p==n?r:w.match[p]; c=p;}
  }
  long long total=0; for(int j=0;j<n;j++){CHK(w.match[j],n); int lane=j&31,c=j>>5; total+=rc(need[lane][c],w.olo[w.match[j]],w.ohi[w.match[j]],nlo[lane][c],nhi[lane][c]);}
  printf("n=%d NC=%d matched by start-up %d total %lld\n",n,NC,matched0,total);
  return total;
}
int main(){ srand(1); PW[0]=0; for(int l=0;l<96;l++)PW[l+1]=PW[l]+1000+rand()%10;
  int L=96; int ns[]={1,2,3,7,31,32,33,64,65,100,200,255,256};
  for(int n:ns)for(int kind=0;kind<2;kind++){ Work w; for(int j=0;j<n;j++){ for(int t=0;t<2;t++){int a=rand()%(L+1); int b=a+rand()%(L+1-a); if(kind==0){int S=1+rand()%12; int i=rand()%S; a=i*L/S; b=(i+1)*L/S;} if(t){w.olo[j]=a;w.ohi[j]=b;}else{w.nlo[j]=a;w.nhi[j]=b;}}}
    int NC=n<=32?1:n<=64?2:n<=128?4:8; sim(w,n,NC);}
}

"""Mutation check of the oracle pins (run by hand: python tests/oracle_mutation_check.py).
Applies one plausible mistake at a time to the oracle source (restored afterwards),
runs the CPU oracle tests and expects at least one of them to fail: a mutation that
survives means a pin is missing.  28 of 28 mutations are killed.  Indices on the command line run only those."""
import subprocess, shutil, sys, os
ROOT=os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
muts=[
 ('oracle/protocol.py','return np.asarray(G, np.float64) @ np.asarray(U, np.float64)','return np.asarray(G, np.float64) @ np.asarray(U, np.float64).T'),
 ('oracle/protocol.py','C[i] = x[(i - 1) % N].copy()   # receive','C[i] = x[(i + 1) % N].copy()   # receive'),
 ('oracle/protocol.py','if k <= c:\n                C[i] = C[i] + D[i][k - 1]','if k < c:\n                C[i] = C[i] + D[i][k - 1]'),
 ('oracle/protocol.py','j = k - N + 1\n                C[i] = C[i] - D[i][j - 1]','j = k - N + 1\n                C[i] = C[i] + D[i][j - 1]'),
 ('oracle/protocol.py','j = k - N + 1\n','j = k - N + 2\n'),
 ('oracle/protocol.py','if k <= N - 1:\n                B[i][k - 1]','if k <= N:\n                B[i][min(k - 1, N - 2)]'),
 ('oracle/protocol.py','M[r * c:(r + 1) * c, N - 1 - r:N - 1 - r + c] = U[(i + r) % N]','M[r * c:(r + 1) * c, r:r + c] = U[(i + r) % N]'),
 ('oracle/protocol.py','M[r * c:(r + 1) * c, N - 1 - r:N - 1 - r + c] = U[(i + r) % N]','M[r * c:(r + 1) * c, N - 1 - r:N - 1 - r + c] = U[(i - r) % N]'),
 ('oracle/protocol.py','return scale * (np.asarray(Y, np.float64) @ np.asarray(R, np.float64))','return scale * (np.asarray(Y, np.float64) @ np.asarray(R, np.float64)[::-1])'),
 ('oracle/protocol.py','return g.reshape(c, p).T.copy()','return g.reshape(p, c).copy()'),
 ('oracle/protocol.py','return c + N - 2','return c + N - 1'),
 ('oracle/designs.py','U_mp[N - 1 - k] = mp.inverse(A_k)','U_mp[k] = mp.inverse(A_k)'),
 ('oracle/designs.py','R_mp = [_stack(rows, -i, L + 1, c) for i in range(N)]','R_mp = [_stack(rows, i, L + 1, c) for i in range(N)]'),
 ('oracle/designs.py','m, r = divmod(l, N)            # floor division: r in [0, N)\n                rows[l] = mp.matrix([[Bm[r, j] * dv[j] ** m','m, r = divmod(l, N)            # floor division: r in [0, N)\n                rows[l] = mp.matrix([[Bm[r, j] * dv[j] ** (m + 1)'),
 ('oracle/designs.py','Dv = [zj ** N for zj in z]','Dv = [zj ** (N - 1) for zj in z]'),
 ('oracle/designs.py','B[l, j] = z[j] ** l','B[l, j] = z[j] ** (l + 1)'),
 ('oracle/designs.py','Dv = [1 + mp.mpf(eps) * mp.mpf(x) for x in h]\n        des = mpc(Bm, Dv, N, c, dps, "epsilon")','Dv = [1 - mp.mpf(eps) * mp.mpf(x) * mp.mpf(x) for x in h]\n        des = mpc(Bm, Dv, N, c, dps, "epsilon")'),
 ('oracle/designs.py','F[j, k] = (-1) ** (j - k) * comb(j, k)','F[j, k] = (-1) ** (j + k + 1) * comb(j, k)'),
 ('oracle/designs.py','(i - 1 - k) % N, c) for i in range(N)], axis=1)','(i - k) % N, c) for i in range(N)], axis=1)'),
 ('oracle/designs.py','b0 = a0 * kappa_max / np.sqrt(N)','b0 = a0 * kappa_max'),
 ('oracle/designs.py','blocks = [B * h ** j for j in range(beta)]','blocks = [B * h ** (j + 1) for j in range(beta)]'),
 ('oracle/designs.py','E = [(l + t) % N for t in range(s)]','E = [(l - t) % N for t in range(s)]'),
 ('oracle/designs.py','blocks.append((B * h ** beta)[E, :])','blocks.append((B * h ** (beta - 1))[E, :])'),
 ('oracle/designs.py','compute_uv=False)[-1]) for l in range(N))','compute_uv=False)[0]) for l in range(N))'),
 ('oracle/designs.py','U.append(Uk_T.T)','U.append(Uk_T)'),
 ('oracle/designs.py','out.append((X * np.clip(s, a0, b0)) @ Zt)','out.append((X * np.clip(s, a0, b0)) @ Zt.T)'),
 ('oracle/designs.py','return [np.linalg.lstsq(protocol.m_matrix(U, i), T, rcond=None)[0] for i in range(N)]','return [np.linalg.lstsq(protocol.m_matrix(U, (i + 1) % N), T, rcond=None)[0] for i in range(N)]'),
 ('oracle/designs.py','Tk = np.concatenate([np.eye(c)] * N, axis=1)','Tk = np.concatenate([np.eye(c)] * (N - 1) + [np.zeros((c, c))], axis=1)'),
]
def main():
    survived=[]
    only=[int(a) for a in sys.argv[1:]]
    for idx,(f,old,new) in enumerate(muts):
        if only and idx not in only: continue
        path=os.path.join(ROOT,f); src=open(path).read()
        if old not in src:
            print(idx,'PATTERN NOT FOUND',f,old[:40]); continue
        open(path,'w').write(src.replace(old,new,1))
        try:
            r=subprocess.run([sys.executable,'-m','pytest','tests/test_oracle_protocol.py','tests/test_oracle_designs.py','-x','-q','-p','no:cacheprovider'],cwd=ROOT,capture_output=True,text=True,timeout=600)
            failed = r.returncode!=0
            last=[l for l in r.stdout.splitlines() if 'FAILED' in l or 'passed' in l or 'failed' in l or 'Error' in l][-2:]
            print(idx,'KILLED' if failed else 'SURVIVED',f,'|',old[:50].replace('\n',' '),'|',last[:1])
            if not failed: survived.append(idx)
        finally:
            open(path,'w').write(src)
    print('survived:',survived)


if __name__ == "__main__":
    main()

"""Exhaustive certification of the fp32-storage forward kernels (not collected by pytest: run by hand).

    python tests/certify_fp32_exhaustive.py [kind,kind,...] [--strict] [--out=FILE.json]

Every fp32 bit pattern with |x| <= 130 (2 x 1.12e9 values per kind; beyond that every kind is
saturated) goes through nfad_act_forward on cuda:0 and is compared with the fp64 oracle in the
metrics of tests/parity.py.  Prints, per kind, the worst value error in ulp, the worst
derivative error in the gate's metric (strict for x >= 0, scaled by |h| + |x h'| for x < 0),
the worst subnormal-result errors in units of 2^-149 and the count of non-finite outputs; with
--out=FILE.json the same numbers are also written to that file.  About three minutes per kind on a
16-core host.  With --strict the inputs go through nfad_act_forward_strict instead and the derivative
is measured in strict ulp of f' itself for every x (no scaling).
"""
import json
import os
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, 'tests'))
import oracle, ulp
from paper_2209_10778_b200 import binding as nfad
oracle.set_threads(oracle.max_threads())
STRICT = '--strict' in sys.argv
OUT = next((a.split('=', 1)[1] for a in sys.argv[1:] if a.startswith('--out=')), None)
args = [a for a in sys.argv[1:] if not a.startswith('--')]
kinds = args[0].split(',') if args else ['gelu_erf','gelu_tanh','swish','mish']
hi_bits = int(np.float32(130.0).view(np.uint32))
CH = 1 << 25
res = {}
for kind in kinds:
    t0 = time.time()
    worst = dict(y=0.0, y_x=0.0, d_gate=0.0, d_x=0.0, d_strict_p999=[], sub_y=0.0, sub_d=0.0, bad=0)
    for sign in (0, 0x80000000):
        for start in range(0, hi_bits + 1, CH):
            stop = min(start + CH, hi_bits + 1)
            bits = torch.arange(start, stop, dtype=torch.int64, device='cuda') + sign
            x = (bits & 0xFFFFFFFF).to(torch.int64)
            x = torch.where(x >= 2**31, x - 2**32, x).to(torch.int32).view(torch.float32).contiguous()
            y = torch.empty_like(x); d = torch.empty_like(x)
            (nfad.nfad_act_forward_strict if STRICT else nfad.nfad_act_forward)(kind, x, y, d)
            torch.cuda.synchronize()
            xh, yh, dh = x.cpu().numpy(), y.cpu().numpy(), d.cpu().numpy()
            f, fp, T = oracle.forward(kind, 'f32', xh, want_cond=True)
            def u32(v):
                return np.maximum(np.spacing(np.abs(v).astype(np.float32)).astype(np.float64), 2.0**-149)
            ey = np.abs(yh.astype(np.float64) - f) / u32(f)
            es = np.abs(dh.astype(np.float64) - fp) / u32(fp)
            ec = np.abs(dh.astype(np.float64) - fp) / u32(np.maximum(T, np.abs(fp)))
            gate = es if STRICT else np.where(xh >= 0, es, ec)
            suby = np.abs(f) < 2.0**-126; subd = (np.abs(fp) < 2.0**-126) & ((T < 2.0**-100) | STRICT)
            ny = np.where(suby, 0, ey); nd = np.where(subd, 0, gate)
            i = int(ny.argmax()); j = int(nd.argmax())
            if ny[i] > worst['y']: worst['y'] = float(ny[i]); worst['y_x'] = float(xh[i])
            if nd[j] > worst['d_gate']: worst['d_gate'] = float(nd[j]); worst['d_x'] = float(xh[j])
            if suby.any(): worst['sub_y'] = max(worst['sub_y'], float((np.abs(yh.astype(np.float64)-f)[suby]/2.0**-149).max()))
            if subd.any(): worst['sub_d'] = max(worst['sub_d'], float((np.abs(dh.astype(np.float64)-fp)[subd]/2.0**-149).max()))
            worst['bad'] += int((~np.isfinite(yh)).sum() + (~np.isfinite(dh)).sum())
    worst.pop('d_strict_p999')
    worst['seconds'] = time.time() - t0
    res[kind] = worst
    print(kind, json.dumps(worst), flush=True)
if OUT:
    os.makedirs(os.path.dirname(os.path.abspath(OUT)), exist_ok=True)
    json.dump(res, open(OUT, 'w'))

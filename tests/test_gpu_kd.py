"""cast_kd_loss (Eq. 13: eta KL(P_t || P_s) + (1 - eta) CE, per token, with its gradient) against the CPU oracle.

Tolerances, from the arithmetic (fp32 sums of up to 32768 exponentials formed by 512 threads and a tree, ex2-based
exponentials with relative error ~2e-7 |x|, against an fp64 oracle):
    loss   |cuda - oracle| <= 2e-5 + 1e-5 |oracle|
    grad   |cuda - oracle| <= 2^-8 |oracle| + 4e-6 grad_scale (P_s + P_t)     (one bf16 ulp of the value, plus the
           absolute error of the two probabilities, which matters where they nearly cancel)"""
import numpy as np
import pytest
import torch

import paper_2509_25996_b200 as cast
from paper_2509_25996_b200 import binding as B
from paper_2509_25996_b200 import workloads
from oracle import adams_oracle as orc
import gpu_util as U

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def logits(tokens, vocab, seed, spread):
    gen = torch.Generator().manual_seed(seed)
    return (torch.randn((tokens, vocab), generator=gen) * spread).to(torch.bfloat16)


def run(student, teacher, labels, eta, grad_scale, want_grad=True, offset=0):
    tokens, vocab = student.shape
    n = tokens * vocab
    # `offset` shifts the buffers off a 16-byte boundary (scalar path)
    ds = U.Guarded(n + offset, torch.bfloat16, DEV); ds.view[offset:].copy_(student.reshape(-1))
    dt = U.Guarded(n + offset, torch.bfloat16, DEV); dt.view[offset:].copy_(teacher.reshape(-1))
    dg = U.Guarded(n + offset, torch.bfloat16, DEV)
    dl = torch.full((tokens,), float("nan"), device=DEV)
    dy = torch.from_numpy(labels).to(DEV)
    before = cast.cast_kernel_launch_count()
    cast.check(cast.cast_kd_loss(ds.view[offset:], dt.view[offset:], dy, dl, dg.view[offset:] if want_grad else None,
                                 tokens, vocab, eta, grad_scale, torch.cuda.current_stream()))
    torch.cuda.synchronize()
    assert cast.cast_kernel_launch_count() == before + 1
    assert ds.intact() and dt.intact() and dg.intact()
    return dl.cpu().numpy().astype(np.float64), dg.view[offset:].float().cpu().numpy().reshape(tokens, vocab).astype(np.float64)


def check(student, teacher, labels, eta, grad_scale, label, **kw):
    loss, grad = run(student, teacher, labels, eta, grad_scale, **kw)
    ref_loss, ref_grad = orc.kd_loss(workloads.bf16_bits(student), workloads.bf16_bits(teacher), labels, eta, grad_scale)
    assert np.all(np.abs(loss - ref_loss) <= 2e-5 + 1e-5 * np.abs(ref_loss)), f"{label}: loss off by {np.max(np.abs(loss - ref_loss)):.3g}"
    ps = torch.softmax(student.double(), -1).numpy()
    pt = torch.softmax(teacher.double(), -1).numpy()
    bound = 2.0 ** -8 * np.abs(ref_grad) + 4e-6 * abs(float(np.float32(grad_scale))) * (ps + pt) + 1e-38
    worst = np.max(np.abs(grad - ref_grad) / bound)
    assert worst <= 1.0, f"{label}: gradient off by {worst:.3g} x the bound"


@pytest.mark.parametrize("tokens,vocab", [(3, 8), (5, 256), (4, 4104), (3, 32000), (2, 32768), (2, 50272), (2, 128256)])
@pytest.mark.parametrize("eta", [0.0, 1.0 / 3.0, 1.0])
def test_kd_loss_vector_paths(tokens, vocab, eta):
    """Rows from one vector per row to 128256 logits: the register-resident path (up to 32768) and the re-reading path."""
    s, t = logits(tokens, vocab, 1, 3.0), logits(tokens, vocab, 2, 4.0)
    labels = np.array([(7 * i + 3) % vocab for i in range(tokens)], dtype=np.int32)
    labels[-1] = -100
    check(s, t, labels, eta, 1.0 / tokens, f"{tokens}x{vocab} eta {eta}")


@pytest.mark.parametrize("vocab,offset", [(50257, 0), (257, 0), (1000, 1), (7, 0)])
def test_kd_loss_scalar_path(vocab, offset):
    """Vocabularies that are not a multiple of 8 (GPT-2's 50257) and buffers off a 16-byte boundary."""
    tokens = 3
    s, t = logits(tokens, vocab, 3, 2.0), logits(tokens, vocab, 4, 2.0)
    labels = np.array([0, vocab - 1, -1], dtype=np.int32)
    check(s, t, labels, 0.5, 2.0, f"scalar {vocab}+{offset}", offset=offset)


def test_kd_loss_special_rows_and_loss_only():
    tokens, vocab = 4, 512
    s, t = logits(tokens, vocab, 5, 3.0), logits(tokens, vocab, 6, 3.0)
    t[0] = s[0]                      # teacher == student: KL = 0
    s[1] = 0.0                       # uniform student: CE = log V
    s[2, 5] = 60.0                   # one dominant logit: probabilities underflow elsewhere
    t[3, 9] = -80.0                  # a teacher probability that underflows to zero
    labels = np.array([1, 2, 5, 700], dtype=np.int32)       # the last one is out of range: no target
    loss, grad = run(s, t, labels, 1.0 / 3.0, 1.0)
    lab2 = labels.copy(); lab2[3] = -1
    ref_loss, ref_grad = orc.kd_loss(workloads.bf16_bits(s), workloads.bf16_bits(t), lab2, 1.0 / 3.0, 1.0)
    assert np.all(np.abs(loss - ref_loss) <= 2e-5 + 1e-5 * np.abs(ref_loss))
    assert np.all(np.isfinite(grad))
    assert abs(loss[0] - (2.0 / 3.0) * (-np.log(torch.softmax(s[0].double(), -1)[1].item()))) < 1e-4
    # loss alone: same losses, gradient buffer untouched
    only, _ = run(s, t, labels, 1.0 / 3.0, 1.0, want_grad=False)
    assert np.array_equal(only, loss)


def test_kd_loss_rejections():
    s = torch.zeros((2, 16), dtype=torch.bfloat16, device=DEV)
    y = torch.zeros(2, dtype=torch.int32, device=DEV)
    l = torch.zeros(2, device=DEV)
    before = cast.cast_kernel_launch_count()
    assert cast.cast_kd_loss(None, s, y, l, None, 2, 16, 0.5) == B.CAST_ERR_NULL
    assert cast.cast_kd_loss(s, s, y, l, None, 0, 16, 0.5) == B.CAST_ERR_SHAPE
    assert cast.cast_kd_loss(s, s, y, l, None, 2, 16, 1.5) == B.CAST_ERR_HYPER
    assert cast.cast_kd_loss(s, s, y, l, s, 2, 16, 0.5) == B.CAST_ERR_ALIAS
    assert cast.cast_kd_loss(s, s, y.cpu(), l, None, 2, 16, 0.5) == B.CAST_ERR_MEMORY
    assert cast.cast_kernel_launch_count() == before

"""The evaluation pass through the C ABI (alexnet_eval_batch) against the fp64 oracle: centre crop without flip,
dropout replaced by its expectation, logits within rel-L2 2e-2, and the top-1 / top-5 counts exact for the logits the
GPU produced (integer work) and equal to the oracle's wherever the oracle's ranking is not a near-tie."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_1412_2302_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 2e-2


def rel(a, b):
    a, b = np.asarray(a, np.float64).ravel(), np.asarray(b, np.float64).ravel()
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


@pytest.mark.parametrize("inverted", [False, True])
def test_eval_batch_against_oracle(inverted):
    from paper_1412_2302_b200 import alexnet as A
    seed, B = synth.BASE_SEED + 31, 12
    mean = synth.mean_image(seed)
    net = A.AlexNet(batch=B, seed=seed, mean_image=mean, flags=A.FLAG_INVERTED_DROPOUT if inverted else 0)
    w = synth.init_params(seed, variance_preserving=True, bias=0.1)
    net.set_params(w)
    img = synth.images(seed, 0, 0, B)
    onet = O.OracleNet(O.OracleConfig(seed=seed, inverted_dropout=inverted), w.astype(np.float64))
    E = O.evaluate(onet, img, np.zeros(B, np.int32), mean)
    # labels at chosen oracle ranks: 0 (top-1), 2 and 4 (top-5 only), 5 and 40 (neither)
    order = np.argsort(-E["z"], axis=1, kind="stable")
    ranks = np.array([0, 2, 4, 5, 40, 0, 1, 4, 5, 7, 0, 3])
    lab = order[np.arange(B), ranks].astype(np.int32)
    E = O.evaluate(onet, img, lab, mean)
    assert E["top1"].sum() == 3 and E["top5"].sum() == 8
    t1, t5, loss = net.eval_batch(0, torch.from_numpy(img).pin_memory(), torch.from_numpy(lab).pin_memory())
    assert np.array_equal(net.get_tensor("CROPFLIP").reshape(B, 3), np.tile([14, 14, 0], (B, 1)))
    for k in ("x0", "f6", "f7", "z"):
        assert rel(net.get_tensor(k.upper()), E[k]) < TOL, k
    assert abs(loss - E["loss"]) < 2e-2 * max(1.0, abs(E["loss"]))
    zg = net.get_tensor("Z").reshape(B, 1000)
    # integer work: exact for the GPU's own logits
    assert t1 == int(O.topk_correct(zg, lab, 1).sum()) and t5 == int(O.topk_correct(zg, lab, 5).sum())
    # and the oracle's verdict wherever its ranking is not a near-tie at the cut
    noise = 2.0 * np.abs(zg - E["z"]).max()
    zs = -np.sort(-E["z"], axis=1)
    zl = E["z"][np.arange(B), lab]
    for k, got in ((1, O.topk_correct(zg, lab, 1)), (5, O.topk_correct(zg, lab, 5))):
        want = O.topk_correct(E["z"], lab, k)
        clear = np.minimum(np.abs(zl - zs[:, k - 1]), np.abs(zl - zs[:, k])) > noise     # label far from the k-th / (k+1)-th logit
        clear |= (np.abs(zs[:, k - 1] - zs[:, k]) > noise) & (zl != zs[:, k - 1]) & (zl != zs[:, k])
        assert np.array_equal(got[clear], want[clear]), k
    assert np.array_equal(net.get_params(0, 0), w)           # evaluation leaves the parameters alone
    # a loaded training batch must be consumed first
    net.load_batch_async(0, torch.from_numpy(img).pin_memory(), torch.from_numpy(lab).pin_memory(), 0)
    with pytest.raises(A.AlexNetError) as e:
        net.eval_batch(0, torch.from_numpy(img).pin_memory(), torch.from_numpy(lab).pin_memory())
    assert e.value.code == A.ERR_STATE
    net.train_step(0)
    t1b, t5b, _ = net.eval_batch(0, torch.from_numpy(img).pin_memory(), torch.from_numpy(lab).pin_memory())
    assert 0 <= t1b <= t5b <= B
    net.close()

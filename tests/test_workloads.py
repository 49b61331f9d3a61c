"""The seeded input generators: determinism, chunking independence, value grid."""

import numpy as np
import torch

import workloads as W


def test_hidden_states_do_not_depend_on_chunking_and_are_bf16_values():
    w = W.get_workload("c2_llama_32k")
    a = W.hidden_states(w, 0, 3072)
    b = np.concatenate([W.hidden_states(w, 0, 1000), W.hidden_states(w, 1000, 2072)])
    assert np.array_equal(a, b)
    assert np.array_equal(a, W.hidden_states(w, 0, 3072))
    assert np.array_equal(a, torch.from_numpy(a).to(torch.bfloat16).float().numpy())
    assert not np.array_equal(a[:1024], W.hidden_states(w, 1024, 1024))


def test_outlier_rows_are_rare_and_twenty_times_larger():
    w = W.get_workload("c3_llama_128k")
    x = W.hidden_states(w, 0, 16384)
    norms = np.linalg.norm(x, axis=1) / np.sqrt(x.shape[1])
    out = norms > 10
    assert 2 <= out.sum() <= 40
    assert np.allclose(norms[out], 20, rtol=0.1) and np.allclose(norms[~out], 1, rtol=0.1)


def test_topic_mixture_is_clustered():
    w = W.get_workload("c4_phi3_128k")
    x = W.hidden_states(w, 0, 2048)
    xc = x / np.linalg.norm(x, axis=1, keepdims=True)
    adjacent = np.mean(np.sum(xc[1:] * xc[:-1], axis=1))
    assert 0.3 < adjacent < 0.6          # neighbours mostly share a topic mean (cos ~ 0.5)
    assert abs(np.var(x) - 1.0) < 0.1


def test_weights_scale_and_seed():
    sh = W.get_workload("c1_small_gqa").shape
    wqkv, w1, w2 = W.layer_weights(sh, 0)
    assert wqkv.shape == (512, 768) and w1.shape == (768, 256) and w2.shape == (256, 2)
    assert abs(wqkv.std() * np.sqrt(512) - 1) < 0.02
    assert abs(w1.std() * np.sqrt(768) - 1) < 0.02
    assert not np.array_equal(wqkv, W.layer_weights(sh, 1)[0])
    assert np.array_equal(wqkv, W.layer_weights(sh, 0)[0])


def test_chunk_sizes():
    assert W.get_workload("c3_llama_128k").chunk_sizes() == [3072] * 42 + [2048]
    assert W.get_workload("c5_llama_stream_int4").chunk_sizes()[-1] == 1600
    assert len(W.get_workload("c4_phi3_128k").chunk_sizes()) == 128

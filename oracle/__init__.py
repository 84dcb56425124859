"""Plain CPU oracle of the binarised-DNN forward pass.  Test infrastructure only."""
